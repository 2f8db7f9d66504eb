#!/usr/bin/env python
"""Benchmark of the cascade-stage hot path (letterbox -> decode -> NMS -> assemble + crop).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload sweep] [--batch 256]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

A step is one pass of the whole stage over one batch of synthetic frames and detector
heads.  `value` is frames/s with the inputs resident in device memory; `e2e` is the same
pass driven from pinned host buffers with the host<->device copies inside the timed region.
With N > 1 (torchrun) every rank runs the same stage on its own frames (replicas, no
collective on the data path); the time is the maximum over ranks.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import re
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "stage_frames_per_s"
UNIT = "frames/s"

# DRAM traffic from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum) per unit of
# work, so that it can be scaled to the benchmarked launch, with the hash of the kernel
# source the capture was taken from.  An entry whose hash no longer matches the source is
# reported as null.
NCU_TRAFFIC = {
    # kernel: (source files, sha256[:16] of their code (comments and layout stripped) at capture time, bytes per unit, unit)
    # captured on the sweep workload at B = 64; decode_planes on the anchor_free workload at B = 64
    "crop": (("paper_2502_01277_b200/csrc/octo_crop.cu", "paper_2502_01277_b200/csrc/octo_common.cuh"),
             "cb3b58cf225f647f", 487791.2, "crop"),
    "letterbox": (("paper_2502_01277_b200/csrc/octo_letterbox.cu", "paper_2502_01277_b200/csrc/octo_common.cuh"),
                  "82ba43ca31895b9a", 3706404.0, "frame"),
    "decode": (("paper_2502_01277_b200/csrc/octo_decode.cu", "paper_2502_01277_b200/csrc/octo_common.cuh"),
               "5ec9cd6b248b8101", 1740516.0, "frame"),
    "decode_planes": (("paper_2502_01277_b200/csrc/octo_decode.cu", "paper_2502_01277_b200/csrc/octo_common.cuh"),
                      "5ec9cd6b248b8101", 2810668.0, "frame"),
}
# Warp instructions the crop kernel executes per crop (ncu smsp__inst_executed.sum of the same capture):
# the kernel is bound by instruction issue, so its issue rate is reported beside the byte rates.
NCU_CROP_WARP_INST = 84255.7


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=30)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--workload", default="sweep", choices=sorted(workloads.WORKLOADS) + ["two_level", "queue"])
    p.add_argument("--bz", type=int, default=64, help="downstream batch size of the queue workload")
    p.add_argument("--nms-cluster", type=int, default=0, choices=[0, 1, 2, 4, 8],
                   help="CTAs per image of the NMS launches (0: the stage chooses)")
    p.add_argument("--batch", type=int, default=None, help="frames per GPU per step")
    p.add_argument("--impl", default="octo", choices=["octo", "reference"])
    p.add_argument("--e2e-steps", type=int, default=None)
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--interleave", action="store_true",
                   help="also time two stage instances interleaved on two streams (extra JSON field)")
    p.add_argument("--fork-preprocess", action="store_true",
                   help="enqueue the letterbox of a step on a second stream, beside decode / NMS / crop of the "
                        "same batch (they share no data); joins the main stream at the end of the step")
    p.add_argument("--graph", action="store_true",
                   help="replay each step from a captured CUDA graph (small batches are launch-bound)")
    return p.parse_args()


def default_batch(name: str) -> int:
    if name == "two_level":
        return 64
    if name == "queue":
        return 2  # the detector batch size the paper gives its baselines; about 44 items per step
    return 256 if name == "sweep" else workloads.WORKLOADS[name].batch


# ---- algorithmic bytes (what the method must move; numerators of the roofline) --------------

def letterbox_bytes(sizes, s: int) -> int:
    """Source rows that carry weight (as 16-byte-granular row copies) + the fp16 output."""
    total = 0
    cache = {}
    for (w, h) in sizes:
        if (w, h) not in cache:
            nh = max(1, (2 * h * s + w) // (2 * w)) if w >= h else s
            rows = 0
            for dy in range(nh):
                num = (2 * dy + 1) * h - nh
                if num <= 0 or num // (2 * nh) >= h - 1:
                    rows += 1
                else:
                    rows += 1 if num % (2 * nh) == 0 else 2
            cache[(w, h)] = rows * ((3 * w + 15) // 16 * 16) + 3 * s * s * 2
        total += cache[(w, h)]
    return total


def crop_bytes(items: np.ndarray, ow: int, oh: int) -> int:
    """fp16 output of every packed crop + its source rectangle, each counted once."""
    cw = (items["rx1"] - items["rx0"]).astype(np.int64)
    ch = (items["ry1"] - items["ry0"]).astype(np.int64)
    return int(len(items) * 3 * ow * oh * 2 + int((cw * ch * 3).sum()))


def crop_compulsory_bytes(items: np.ndarray, sizes, ow: int, oh: int) -> int:
    """What a crop launch cannot avoid moving through DRAM: the fp16 output of every packed crop +
    every source byte that at least one rectangle covers, counted once per frame (rectangles of a
    frame overlap; the second reader of a byte is served by L2)."""
    total = int(len(items)) * 3 * ow * oh * 2
    order = np.argsort(items["frame"], kind="stable")
    it = items[order]
    bounds = np.flatnonzero(np.diff(it["frame"])) + 1
    for grp in np.split(it, bounds):
        if len(grp) == 0:
            continue
        w, h = sizes[int(grp["frame"][0])]
        mask = np.zeros((h, w), dtype=bool)
        for r in grp:
            mask[r["ry0"]:r["ry1"], r["rx0"]:r["rx1"]] = True
        total += 3 * int(mask.sum())
    return total


def decode_bytes(n: int, a: int, c: int, candidates: int, logits: bool, layout: str = "rows") -> int:
    """Rows layout: one 32-byte sector per head row for the obj scan (logit heads) or the whole
    row (probability heads), plus the full row and the 8-byte key of each candidate.  Planes
    layout: every class plane (the maximum over classes needs all of them), plus four box
    values and the key of each candidate."""
    if layout == "planes":
        return int(4 * c * a * n + candidates * (4 * 32 + 8))
    row = 4 * (5 + c)
    scan = 32 * a * n if logits else row * a * n
    return int(scan + candidates * (row + 8))


def code_only(text: str) -> str:
    """A CUDA source without its comments and without whitespace: what the compiler sees of it, up to
    tokens.  (String literals of these sources contain neither comment markers nor blanks that matter.)"""
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    return re.sub(r"\s+", "", text)


def files_hash(paths) -> str:
    """Hash of the code of the given sources (comments and layout do not count: editing a comment does
    not invalidate counters that were taken from the same kernel)."""
    h = hashlib.sha256()
    for p in paths:
        h.update(code_only(open(os.path.join(ROOT, p), "r", encoding="utf-8").read()).encode())
    return h.hexdigest()[:16]


def traffic_for(kernel: str, units: float):
    ent = NCU_TRAFFIC.get(kernel)
    if not ent:
        return None
    srcs, digest, per_unit, _unit = ent
    if files_hash(srcs) != digest:
        return None
    return per_unit * units


# ---- clocks ---------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm), reasons=sorted(reasons))
        return out


# ---- the reference arm: the CPU oracle ------------------------------------------------------

def oracle_pass(batch, frames_used: int, threads: int) -> float:
    """Seconds the oracle needs for the whole stage on the first `frames_used` frames."""
    import oracle
    wl = batch.workload
    t0 = time.perf_counter()
    oracle.run_stage(batch.frames[:frames_used], batch.sizes[:frames_used], batch.head[:frames_used],
                     wl.net_size, wl.branches, logits=wl.logits, conf=wl.conf_thresh, iou_thr=wl.iou_thresh,
                     max_det=wl.max_det, threads=threads, layout=wl.head_layout, multi_label=wl.multi_label)
    return time.perf_counter() - t0


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_sample_frames(batch_n: int, cores: int) -> int:
    # about 0.25 s of single-core work per 1080p frame -> roughly 5-20 s of wall time
    return max(1, min(batch_n, 64 * cores))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    if name in ("two_level", "queue"):
        print(json.dumps({"impl": "reference", "unavailable": "the reference arm covers the single-stage workloads"}))
        return
    bsz = args.batch or default_batch(name)
    cores = len(os.sched_getaffinity(0))
    sample = cpu_sample_frames(bsz, cores)
    batch = workloads.make_batch(name, batch=sample)
    warm = min(args.warmup, 1)
    for _ in range(warm):
        oracle_pass(batch, min(sample, cores), cores)
    steps = max(1, min(args.steps, 3))
    times = [oracle_pass(batch, sample, cores) for _ in range(steps)]
    t = sum(times) / len(times)
    value = sample / t
    wl = batch.workload
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * t, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{name} B={bsz}", "frames_per_step": sample, "net_size": wl.net_size,
                   "note": "CPU oracle; each step is a bounded sample of the batch"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} of {bsz} frames, whole stage, {cores} threads"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- the CUDA arm ---------------------------------------------------------------------------

def run_octo(args):
    import torch
    import torch.distributed as dist

    import paper_2502_01277_b200 as octo

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    name = args.workload
    bsz = args.batch or default_batch(name)
    batch = workloads.make_batch(name, batch=bsz, first_frame=rank * bsz)
    wl = batch.workload
    n, s = batch.n, wl.net_size
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"

    stage = octo.Stage(device=local_rank, net_size=s, max_batch=n, num_anchors=wl.num_anchors,
                       num_classes=wl.num_classes, head_is_logits=wl.logits, conf_thresh=wl.conf_thresh,
                       iou_thresh=wl.iou_thresh, max_det=wl.max_det, branches=wl.branches,
                       head_layout=wl.head_layout, multi_label=wl.multi_label)
    stage.set_nms_cluster(args.nms_cluster)
    stream = torch.cuda.Stream(dev)
    cap = n * wl.items_per_frame

    # Input sets: a single set once it exceeds 512 MB, else enough rotating copies that the
    # working set is larger than L2 several times over.
    h_frames = [torch.from_numpy(f).pin_memory() for f in batch.frames]
    h_head = torch.from_numpy(batch.head).pin_memory()
    in_bytes = sum(f.numel() for f in h_frames) + h_head.numel() * 4
    out_bytes = n * 3 * s * s * 2 + sum(cap * 3 * ow * oh * 2 for ow, oh in wl.branches)
    n_sets = max(1, min(64, -(-(512 << 20) // (in_bytes + n * 3 * s * s * 2))))

    class Set:
        pass

    sets = []
    with torch.cuda.stream(stream):
        for _ in range(n_sets):
            z = Set()
            z.frames = [f.to(dev, non_blocking=True) for f in h_frames]
            z.head = h_head.to(dev, non_blocking=True)
            z.det_in = torch.empty((n, 3, s, s), dtype=torch.float16, device=dev)
            z.dets = torch.zeros((n, wl.max_det, 32), dtype=torch.uint8, device=dev)
            z.counts = torch.zeros((n,), dtype=torch.int32, device=dev)
            z.crops = [torch.empty((cap, 3, oh, ow), dtype=torch.float16, device=dev) for ow, oh in wl.branches]
            z.offsets = [torch.zeros((n + 1,), dtype=torch.int32, device=dev) for _ in wl.branches]
            z.n_items = [torch.zeros((2,), dtype=torch.int32, device=dev) for _ in wl.branches]
            z.desc = stage.frame_array(z.frames, batch.sizes)
            sets.append(z)
    stream.synchronize()

    side = torch.cuda.Stream(device=dev) if args.fork_preprocess else None
    ev_fork = torch.cuda.Event() if side is not None else None
    ev_join = torch.cuda.Event() if side is not None else None

    def step(z):
        if side is not None:
            # the letterbox reads the frames and writes the detector batch; decode, NMS and crop read the
            # head and the frames: nothing of one is an input of the other within a batch
            ev_fork.record(stream)
            side.wait_event(ev_fork)
            stage.preprocess_array(z.desc, n, z.det_in, stream=side, keepalive=z.frames)
        else:
            stage.preprocess_array(z.desc, n, z.det_in, stream=stream, keepalive=z.frames)
        stage.postprocess(z.head, dets=z.dets, counts=z.counts, stream=stream)
        for b in range(len(wl.branches)):
            stage.crop(b, cap, out=z.crops[b], offsets=z.offsets[b], n_items=z.n_items[b], stream=stream)
        if side is not None:
            ev_join.record(side)
            stream.wait_event(ev_join)

    def barrier():
        if world > 1:
            dist.barrier()

    def timed(nsteps, fn, per_step=None):
        """Device time of nsteps steps (max over ranks).  With per_step (a list), an event is also
        recorded after every step and the step-to-step times (ms, this rank) are appended to it."""
        barrier()
        torch.cuda.synchronize(dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(nsteps + 1 if per_step is not None else 2)]
        ev[0].record(stream)
        for i in range(nsteps):
            fn(i)
            if per_step is not None:
                ev[i + 1].record(stream)
        if per_step is None:
            ev[1].record(stream)
        torch.cuda.synchronize(dev)
        barrier()
        ms = ev[0].elapsed_time(ev[-1])
        if per_step is not None:
            per_step.extend(ev[i].elapsed_time(ev[i + 1]) for i in range(nsteps))
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    # ---- resident-input throughput ----
    warm = max(args.warmup, 3)
    for i in range(warm):
        step(sets[i % n_sets])
    torch.cuda.synchronize(dev)
    launches0 = stage.launch_count
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches_per_step = (stage.launch_count - launches0) // max(warm, 1) if warm else 0
    launches0 = stage.launch_count
    if args.graph:
        # one graph per input/output set: the stage calls only enqueue kernels, so a step can be
        # captured once and replayed; the frame table travels in the kernel parameters
        graphs = []
        for z in sets:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(z)
            graphs.append(g)
        torch.cuda.synchronize(dev)

        def replay(i):
            with torch.cuda.stream(stream):
                graphs[i % n_sets].replay()

        for i in range(3):
            replay(i)
        launches0 = stage.launch_count
        run_step = replay
        ms_total = timed(args.steps, replay)
        gpu_launches = launches_per_step * args.steps  # kernels run from the graph, not counted by the stage
    else:
        run_step = lambda i: step(sets[i % n_sets])  # noqa: E731
        ms_total = timed(args.steps, run_step)
        gpu_launches = stage.launch_count - launches0
    ms_per_step = ms_total / args.steps
    value = world * n / (ms_per_step * 1e-3)

    # ---- distribution over single steps: >= 50 steps, an event after each one ----
    # (informational: `value` above is the plain K-step figure; a per-step event keeps the next
    # launch from overlapping the end of the step, which costs small batches a few microseconds)
    dist_steps = max(50, args.steps)
    per = []
    timed(dist_steps, run_step, per_step=per)
    step_stats = {"steps": dist_steps, "ms_median": statistics.median(per), "ms_min": min(per),
                  "us_per_pass_median": 1e3 * statistics.median(per), "us_per_pass_min": 1e3 * min(per)}
    # the L2-warm figure of small batches: one input/output set over and over (it fits L2)
    l2_warm = None
    if n <= 16 and n_sets > 1:
        warm_fn = (lambda i: replay(0)) if args.graph else (lambda i: step(sets[0]))
        for i in range(3):
            warm_fn(i)
        perw = []
        timed(dist_steps, warm_fn, per_step=perw)
        l2_warm = {"steps": dist_steps, "ms_median": statistics.median(perw), "ms_min": min(perw),
                   "frames_per_s_median": world * n / (statistics.median(perw) * 1e-3),
                   "note": "one input/output set reused every step: the working set stays in L2"}

    # ---- two stage instances interleaved on two streams (informational) ----
    # Co-located instances fill each other's gaps: the latency-bound decode and NMS kernels of one
    # pass run beside the bandwidth-bound letterbox and crop kernels of the other.
    interleaved = None
    if args.interleave:
        stage2 = octo.Stage(device=local_rank, net_size=s, max_batch=n, num_anchors=wl.num_anchors,
                            num_classes=wl.num_classes, head_is_logits=wl.logits, conf_thresh=wl.conf_thresh,
                            iou_thresh=wl.iou_thresh, max_det=wl.max_det, branches=wl.branches,
                            head_layout=wl.head_layout, multi_label=wl.multi_label)
        stream2 = torch.cuda.Stream(dev)
        z1 = sets[0]
        z2 = Set()
        with torch.cuda.stream(stream2):
            z2.frames, z2.head, z2.desc = z1.frames, z1.head, z1.desc  # inputs are only read
            z2.det_in = torch.empty_like(z1.det_in)
            z2.dets, z2.counts = torch.zeros_like(z1.dets), torch.zeros_like(z1.counts)
            z2.crops = [torch.empty_like(c_) for c_ in z1.crops]
            z2.offsets = [torch.zeros_like(o_) for o_ in z1.offsets]
            z2.n_items = [torch.zeros_like(o_) for o_ in z1.n_items]
        lanes2 = [(stage, stream, z1), (stage2, stream2, z2)]

        def step2(i):
            st_, sm_, z_ = lanes2[i % 2]
            st_.preprocess_array(z_.desc, n, z_.det_in, stream=sm_, keepalive=z_.frames)
            st_.postprocess(z_.head, dets=z_.dets, counts=z_.counts, stream=sm_)
            for b in range(len(wl.branches)):
                st_.crop(b, cap, out=z_.crops[b], offsets=z_.offsets[b], n_items=z_.n_items[b], stream=sm_)

        for i in range(4):
            step2(i)
        torch.cuda.synchronize(dev)
        k2 = 2 * ((args.steps + 1) // 2)
        e0, e1, ej = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        stream2.wait_event(e0)
        for i in range(k2):
            step2(i)
        ej.record(stream2)
        stream.wait_event(ej)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        ms2 = e0.elapsed_time(e1) / k2
        interleaved = {"value": world * n / (ms2 * 1e-3), "unit": UNIT, "ms_per_step": ms2, "steps": k2,
                       "mode": "two stage instances on two streams, passes alternating"}
        stage2.close()

    # sanity of the run + sizes for the byte accounting (outside the timed region)
    z0 = sets[0]
    totals = [tuple(int(v) for v in t.cpu()) for t in z0.n_items]
    for b, (packed, total) in enumerate(totals):
        if packed != total:
            raise SystemExit(f"branch {b}: provisioned {cap} crop slots but the batch holds {total} items")
    stage.stats(stream)
    status = stage.status(stream)
    if status & ~0x8:
        raise SystemExit(f"device status word {status:#x}")
    items = [stage.item_table(b, totals[b][0]) for b in range(len(wl.branches))]

    # ---- per-kernel device times: the same steps with an event pair around every launch ----
    stage.set_timing(True)
    for i in range(warm):  # the first event pairs are created here, outside the measured pass
        step(sets[i % n_sets])
    stage.kernel_times(stream)
    ms_ev_total = timed(args.steps, lambda i: step(sets[i % n_sets]))
    kt = stage.kernel_times(stream)
    stage.set_timing(False)
    clocks = sampler.stop() if rank == 0 else {}
    stats = stage.stats(stream)
    cand_per_step = stats["candidates"] / args.steps
    kern = {}
    alg = {
        "letterbox": letterbox_bytes(batch.sizes, s),
        "decode": decode_bytes(n, wl.num_anchors, wl.num_classes, int(cand_per_step), wl.logits, wl.head_layout),
        "crop": sum(crop_bytes(items[b], *wl.branches[b]) for b in range(len(wl.branches))) / len(wl.branches),
    }
    names = octo.binding.KERNEL_NAMES
    for k in names:
        ms_sum, cnt = kt[k]
        if cnt == 0:
            continue
        avg = ms_sum / cnt
        kern[k] = {"launches_per_step": cnt / args.steps, "ms_per_launch": avg, "share": None}
        if k in alg:
            kern[k]["alg_bytes_per_launch"] = alg[k]
            kern[k]["gbs"] = alg[k] / (avg * 1e-3) / 1e9
            kern[k]["frac_of_hbm_peak"] = kern[k]["gbs"] / hbm_peak
    tot_ms = sum(kt[k][0] for k in names)
    for k in kern:
        kern[k]["share"] = kt[k][0] / tot_ms if tot_ms > 0 else None
    dominant = max((k for k in kern if k in alg), key=lambda k: kt[k][0])
    units = {"letterbox": n, "decode": n, "crop": len(items[0])}[dominant]
    # the per-unit ncu figures were taken on 1080p frames and 224x224 crops: other shapes get none
    traffic = (traffic_for("decode_planes" if dominant == "decode" and wl.head_layout == "planes" else dominant, units)
               if name in ("sweep", "anchor_free") else None)
    dom_ms = kern[dominant]["ms_per_launch"]
    roofline = {
        "kernel": dominant, "bound": "hbm", "achieved": kern[dominant]["gbs"], "peak": hbm_peak,
        "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({peak_kind})", "unit": "GB/s",
        "frac": kern[dominant]["gbs"] / hbm_peak, "frac_of_nominal_8TBs": kern[dominant]["gbs"] / 8000.0,
        "basis": "algorithmic bytes per launch / CUDA-event time"
                 + (": fp16 output + the source rectangle of every crop, each rectangle counted once per crop "
                    "although rectangles of a frame overlap and repeats are served by L2" if dominant == "crop" else ""),
        "alg_bytes_per_launch": alg[dominant], "ms_per_launch": dom_ms,
        "traffic": traffic,
        # the same launch on the bytes that reach DRAM (ncu dram__bytes, scaled by the units processed)
        "frac_dram": (traffic / (dom_ms * 1e-3) / 1e9 / hbm_peak) if traffic else None,
    }
    if dominant == "crop":
        # What limits the kernel in practice: instruction issue (ncu: issue slots about 70 % busy, no
        # memory pipe above 60 %).  Issue rate = executed warp instructions / time against one
        # instruction per scheduler and clock (4 schedulers per SM) at the clock seen during the run.
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = clocks.get("sm_mhz") or peaks.get("sm_max_mhz") or 1965.0
        inst = NCU_CROP_WARP_INST * units if traffic else None
        roofline["issue"] = {
            "limits_the_kernel": True, "warp_inst_per_launch": inst,
            "achieved_ginst_s": inst / (dom_ms * 1e-3) / 1e9 if inst else None,
            "peak_ginst_s": sm_count * 4 * mhz * 1e6 / 1e9,
            "frac": (inst / (dom_ms * 1e-3)) / (sm_count * 4 * mhz * 1e6) if inst else None,
            "peak_source": f"{sm_count} SMs x 4 schedulers x {mhz:.0f} MHz (clock sampled during the run)",
        }
        comp = sum(crop_compulsory_bytes(items[b], batch.sizes, *wl.branches[b]) for b in range(len(wl.branches))) \
            / len(wl.branches)
        roofline["compulsory_bytes"] = comp  # output + every covered source byte once per frame
        roofline["frac_compulsory"] = comp / (dom_ms * 1e-3) / 1e9 / hbm_peak

    # ---- end to end from pinned host buffers ----
    # The batch is streamed as sub-batches of up to 32 frames over two lanes (stage + stream +
    # device buffers each), so the H2D copies of one sub-batch overlap the kernels and the D2H
    # copies of the other.  Every sub-batch is a complete stage pass; all results reach the host.
    e2e = None
    if not args.no_e2e:
        e2e_steps = args.e2e_steps or max(3, min(args.steps, 10))
        c = min(n, 32)
        chunks = [(i, min(i + c, n)) for i in range(0, n, c)]
        ccap = c * wl.items_per_frame

        class Lane:
            pass

        lanes = []
        for _ in range(2 if len(chunks) > 1 else 1):
            ln = Lane()
            ln.stage = octo.Stage(device=local_rank, net_size=s, max_batch=c, num_anchors=wl.num_anchors,
                                  num_classes=wl.num_classes, head_is_logits=wl.logits,
                                  conf_thresh=wl.conf_thresh, iou_thresh=wl.iou_thresh, max_det=wl.max_det,
                                  branches=wl.branches, head_layout=wl.head_layout, multi_label=wl.multi_label)
            ln.stream = torch.cuda.Stream(dev)
            ln.small = torch.cuda.Event()
            ln.head = torch.empty((c,) + tuple(h_head.shape[1:]), dtype=torch.float32, device=dev)
            ln.det_in = torch.empty((c, 3, s, s), dtype=torch.float16, device=dev)
            ln.dets = torch.zeros((c, wl.max_det, 32), dtype=torch.uint8, device=dev)
            ln.counts = torch.zeros((c,), dtype=torch.int32, device=dev)
            ln.crops = [torch.empty((ccap, 3, oh, ow), dtype=torch.float16, device=dev) for ow, oh in wl.branches]
            ln.off = [torch.zeros((c + 1,), dtype=torch.int32, device=dev) for _ in wl.branches]
            ln.ni = [torch.zeros((2,), dtype=torch.int32, device=dev) for _ in wl.branches]
            ln.h_ni = [torch.zeros((2,), dtype=torch.int32).pin_memory() for _ in wl.branches]
            ln.frames = {}
            lanes.append(ln)
        # device frame buffers per (lane, shape): sub-batches may mix frame sizes
        h_dets = torch.empty((n, wl.max_det, 32), dtype=torch.uint8).pin_memory()
        h_counts = torch.empty((n,), dtype=torch.int32).pin_memory()
        h_off = [torch.empty((len(chunks), c + 1), dtype=torch.int32).pin_memory() for _ in wl.branches]
        h_crops = [torch.empty((max(totals[b][1], 1) + len(chunks), 3, oh, ow), dtype=torch.float16).pin_memory()
                   for b, (ow, oh) in enumerate(wl.branches)]
        for ln in lanes:
            ln.dev_block = torch.empty((c,) + tuple(h_frames[0].shape), dtype=torch.uint8, device=dev)
            ln.dev_frames = [ln.dev_block[k] for k in range(c)]
        same_shape = all(f.shape == h_frames[0].shape for f in h_frames)
        # frames of one shape travel as one pinned block per sub-batch (one copy instead of one per frame)
        h_block = torch.stack(h_frames).pin_memory() if same_shape else None
        d2h = [0]
        read_crops = [True]  # False: the downstream batches stay on the device, where their model runs

        def enqueue(ci):
            lo, hi = chunks[ci]
            ln = lanes[ci % len(lanes)]
            m = hi - lo
            with torch.cuda.stream(ln.stream):
                if same_shape:
                    fr = ln.dev_frames[:m]
                else:
                    fr = [torch.empty_like(h_frames[lo + k], device=dev) for k in range(m)]
                if same_shape:
                    ln.dev_block[:m].copy_(h_block[lo:hi], non_blocking=True)
                else:
                    for k in range(m):
                        fr[k].copy_(h_frames[lo + k], non_blocking=True)
                ln.head[:m].copy_(h_head[lo:hi], non_blocking=True)
                ln.stage.preprocess(fr, batch.sizes[lo:hi], out=ln.det_in[:m], stream=ln.stream)
                ln.stage.postprocess(ln.head[:m], dets=ln.dets[:m], counts=ln.counts[:m], stream=ln.stream)
                for b in range(len(wl.branches)):
                    ln.stage.crop(b, ccap, out=ln.crops[b], offsets=ln.off[b][:m + 1], n_items=ln.ni[b],
                                  stream=ln.stream)
                h_dets[lo:hi].copy_(ln.dets[:m], non_blocking=True)
                h_counts[lo:hi].copy_(ln.counts[:m], non_blocking=True)
                for b in range(len(wl.branches)):
                    h_off[b][ci, :m + 1].copy_(ln.off[b][:m + 1], non_blocking=True)
                    ln.h_ni[b].copy_(ln.ni[b], non_blocking=True)
                ln.small.record(ln.stream)

        def drain(ci, cursor):
            ln = lanes[ci % len(lanes)]
            ln.small.synchronize()  # the packed counts size the crop read-back
            with torch.cuda.stream(ln.stream):
                for b in range(len(wl.branches)):
                    packed = min(int(ln.h_ni[b][0]), ccap, h_crops[b].shape[0] - cursor[b])
                    if read_crops[0]:
                        h_crops[b][cursor[b]:cursor[b] + packed].copy_(ln.crops[b][:packed], non_blocking=True)
                    cursor[b] += packed

        def e2e_step(_i):
            cursor = [0] * len(wl.branches)
            for ci in range(len(chunks) + 1):
                if ci < len(chunks):
                    enqueue(ci)  # stream order protects the lane's buffers from the previous use
                if ci >= 1:
                    drain(ci - 1, cursor)
            for ln in lanes:
                ln.stream.synchronize()
            d2h[0] = (h_dets.numel() + h_counts.numel() * 4 +
                      sum((cursor[b] * h_crops[b][0].numel() * 2 if read_crops[0] else 0) + (n + len(chunks)) * 4 +
                          8 * len(chunks) for b in range(len(wl.branches))))

        for i in range(3):
            e2e_step(i)
        ms_e2e = timed(e2e_steps, e2e_step) / e2e_steps
        e2e = {"value": world * n / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e, "steps": e2e_steps,
               "h2d_bytes_per_step": int(in_bytes), "d2h_bytes_per_step": int(d2h[0]),
               "mode": f"{len(chunks)} sub-batches of <= {c} frames over {len(lanes)} streams; every result read back, "
                       "the packed crops included"}
        # the same with the downstream batches left on the device (where the downstream model would
        # consume them): inputs in, detections / counts / offsets / item counts out
        read_crops[0] = False
        e2e_step(0)
        ms_keep = timed(e2e_steps, e2e_step) / e2e_steps
        e2e["crops_stay_on_device"] = {"value": world * n / (ms_keep * 1e-3), "unit": UNIT, "ms_per_step": ms_keep,
                                       "h2d_bytes_per_step": int(in_bytes), "d2h_bytes_per_step": int(d2h[0])}
        for ln in lanes:
            ln.stage.close()

    # ---- CPU baseline (rank 0, single-GPU runs only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        sample = cpu_sample_frames(n, cores)
        t = oracle_pass(batch, sample, cores)
        one = min(n, 8)
        t1 = oracle_pass(batch, one, 1)
        cpu = {"value": sample / t, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {sample} of {n} frames, whole stage, {cores} threads, {t:.1f} s",
               "single_thread": {"value": one / t1, "unit": UNIT, "sample": f"first {one} frames, {t1:.1f} s"},
               "cpu_model": cpu_model()}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": f"{name} B={n}" + (" per GPU" if world > 1 else ""),
                "frames": "x".join(str(v) for v in batch.sizes[0]) + (" (mixed)" if len(set(batch.sizes)) > 1 else ""),
                "net_size": s, "head": list(batch.head.shape),
                "crops": [list(b) for b in wl.branches], "items_per_step": [t[1] for t in totals],
                "candidates_per_step": cand_per_step, "parallelism": f"replicas x{world}",
                "launch": ("CUDA graph replay" if args.graph else "stream launches")
                + (", letterbox on a second stream" if args.fork_preprocess else ""),
                "nms_ctas_per_image": stage.last_nms_cluster(),
                "l2": (f"{n_sets} rotating input/output sets, {n_sets * (in_bytes + out_bytes) / 2**20:.0f} MiB working set"
                       if n_sets > 1 else f"one set of {(in_bytes + out_bytes) / 2**20:.0f} MiB per step, larger than L2"),
            },
            "e2e": e2e,
            "interleaved": interleaved,
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
            "roofline": roofline,
            "kernels": kern,
            "ms_per_step_with_kernel_events": ms_ev_total / args.steps,
            "step_times": step_stats,
            "l2_warm": l2_warm,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    stage.close()
    if world > 1:
        dist.destroy_process_group()


def run_two_level(args):
    """Two-level cascade (frames -> detector stage -> 256x256 crops -> chained detector stage ->
    64x32 crops).  One step = level-1 pass, hand-off of the item table, level-2 passes.  Timed with
    the hand-off on the device (the reported value) and through the host (stream synchronised and
    item table read back, as between two serving containers).  Single GPU."""
    import torch
    from dataclasses import replace

    import paper_2502_01277_b200 as octo

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n = args.batch or default_batch("two_level")
    wl = replace(workloads.WORKLOADS["traffic_1080p"], branches=((256, 256),))
    batch = workloads.make_batch(wl, batch=n, seed=5)
    s2, c2, max_det2 = 256, 8, 16
    a2 = workloads.num_anchors(s2)
    st1 = octo.Stage(net_size=wl.net_size, max_batch=n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                     max_det=wl.max_det, branches=wl.branches)
    stream = torch.cuda.Stream(dev)
    cap1 = n * wl.items_per_frame
    with torch.cuda.stream(stream):
        frames = [torch.from_numpy(f).to(dev) for f in batch.frames]
        head1 = torch.from_numpy(batch.head).to(dev)
        det_in = torch.empty((n, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev)
        dets1 = torch.zeros((n, wl.max_det, 32), dtype=torch.uint8, device=dev)
        counts1 = torch.zeros((n,), dtype=torch.int32, device=dev)
        crops1 = torch.empty((cap1, 3, 256, 256), dtype=torch.float16, device=dev)
        off1 = torch.zeros((n + 1,), dtype=torch.int32, device=dev)
        ni1 = torch.zeros((2,), dtype=torch.int32, device=dev)
        desc = st1.frame_array(frames, batch.sizes)
        # one dry pass to learn the number of level-1 items, which sizes level 2
        st1.preprocess_array(desc, n, det_in, stream=stream, keepalive=frames)
        st1.postprocess(head1, dets=dets1, counts=counts1, stream=stream)
        st1.crop(0, cap1, out=crops1, offsets=off1, n_items=ni1, stream=stream)
    stream.synchronize()
    n1 = int(ni1[0])
    head2_h = workloads.make_heads(9, n1, s2, num_classes=c2, n_raised=12, n_groups=3)
    st2 = octo.Stage(net_size=s2, max_batch=min(n1, 512), num_anchors=a2, num_classes=c2, max_det=max_det2,
                     branches=((64, 32),))
    c2n = min(n1, 512)  # level-2 batches of at most 512 upstream items
    with torch.cuda.stream(stream):
        head2 = torch.from_numpy(head2_h).to(dev)
        dets2 = torch.zeros((c2n, max_det2, 32), dtype=torch.uint8, device=dev)
        counts2 = torch.zeros((c2n,), dtype=torch.int32, device=dev)
        crops2 = torch.empty((c2n * max_det2, 3, 32, 64), dtype=torch.float16, device=dev)
        off2 = torch.zeros((c2n + 1,), dtype=torch.int32, device=dev)
        ni2 = torch.zeros((2,), dtype=torch.int32, device=dev)

    def level1():
        st1.preprocess_array(desc, n, det_in, stream=stream, keepalive=frames)
        st1.postprocess(head1, dets=dets1, counts=counts1, stream=stream)
        st1.crop(0, cap1, out=crops1, offsets=off1, n_items=ni1, stream=stream)

    def level2(lo, hi):
        st2.postprocess(head2[lo:hi], dets=dets2[: hi - lo], counts=counts2[: hi - lo], stream=stream)
        st2.crop(0, (hi - lo) * max_det2, out=crops2, offsets=off2[: hi - lo + 1], n_items=ni2, stream=stream)

    def step_host(_i):
        level1()
        stream.synchronize()  # hand-off: the downstream stage learns its inputs from the host
        m = int(ni1[0])
        items = st1.item_table(0, m)
        for lo in range(0, m, c2n):
            hi = min(lo + c2n, m)
            st2.adopt_regions(frames, batch.sizes, items[lo:hi], stream=stream)
            level2(lo, hi)

    def step_device(_i):
        level1()
        # hand-off on the device: the chained stage reads the upstream item table where it lies;
        # the level-2 batches are provisioned for the n1 items a pass of this workload yields
        for lo in range(0, n1, c2n):
            hi = min(lo + c2n, n1)
            st2.adopt_items_device(st1, 0, hi - lo, first=lo, stream=stream)
            level2(lo, hi)

    def measure(step):
        for i in range(max(args.warmup, 3)):
            step(i)
        torch.cuda.synchronize(dev)
        l0 = st1.launch_count + st2.launch_count
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / args.steps, st1.launch_count + st2.launch_count - l0

    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    ms_host, _ = measure(step_host)
    ms, launches = measure(step_device)
    clocks = sampler.stop()
    for st in (st1, st2):
        if st.status(stream) & ~0xA:
            raise SystemExit(f"device status word {st.status(stream):#x}")
    line = {
        "metric": METRIC, "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"two_level B={n}", "level1": "1920x1080 -> 640, crops 256x256",
                   "level1_items": n1, "level2": f"head [{n1}, {a2}, {5 + c2}], crops 64x32",
                   "level2_items_last_batch": int(ni2[1]),
                   "handoff": "device (octo_adopt_items_device: no host synchronisation between the levels)",
                   "l2": f"working set {(sum(f.numel() for f in frames) + head1.numel() * 4 + crops1.numel() * 2) / 2**20:.0f} MiB"},
        "host_handoff": {"value": n / (ms_host * 1e-3), "unit": UNIT, "ms_per_step": ms_host,
                         "mode": "item table read back, stream synchronised, octo_adopt_regions"},
        "e2e": None, "gpu_launches": int(launches), "clocks": clocks, "roofline": None, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)
    st1.close()
    st2.close()


def run_queue(args):
    """Serving loop of one downstream model at a fixed batch size bz: per step one detector batch
    (letterbox, decode + NMS), octo_queue_push of its items and octo_queue_pop_due of one batch of bz
    crops (released when full, or when its first item has waited one push).  Timed with stream
    launches and replayed from ONE CUDA graph per bz.  Single GPU."""
    import torch

    import paper_2502_01277_b200 as octo

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, bz = args.batch or default_batch("queue"), args.bz
    wl = workloads.WORKLOADS["traffic_1080p"]
    batch = workloads.make_batch(wl, batch=n)
    ow, oh = wl.branches[0]
    st = octo.Stage(net_size=wl.net_size, max_batch=n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                    max_det=wl.max_det, branches=wl.branches)
    stream = torch.cuda.Stream(dev)
    n_sets = 8  # rotating detector inputs and crop outputs, larger than L2 together
    with torch.cuda.stream(stream):
        frames = [torch.from_numpy(f).to(dev) for f in batch.frames]
        heads = [torch.from_numpy(batch.head).to(dev) for _ in range(n_sets)]
        det_in = [torch.empty((n, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev) for _ in range(n_sets)]
        dets = torch.zeros((n, wl.max_det, 32), dtype=torch.uint8, device=dev)
        counts = torch.zeros((n,), dtype=torch.int32, device=dev)
        crops = [torch.empty((bz, 3, oh, ow), dtype=torch.float16, device=dev) for _ in range(n_sets)]
        items = torch.zeros((bz, octo.QITEM_DTYPE.itemsize), dtype=torch.uint8, device=dev)
        info = torch.zeros((4,), dtype=torch.int32, device=dev)
    stream.synchronize()

    def serve(q, k):
        st.preprocess(frames, batch.sizes, out=det_in[k], stream=stream)
        st.postprocess(heads[k], dets=dets, counts=counts, stream=stream)
        q.push(st, 0, stream=stream)
        q.pop(bz, out=crops[k], items=items, info=info, stream=stream, max_wait=1)

    def measure(fn):
        for i in range(max(args.warmup, 3)):
            fn(i)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / args.steps

    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    q1 = octo.Queue(64 * bz, ow, oh, max_bz=bz)
    ms_stream = measure(lambda i: serve(q1, i % n_sets))
    q1.close()
    q2 = octo.Queue(64 * bz, ow, oh, max_bz=bz)
    serve(q2, 0)  # first launches outside the capture
    stream.synchronize()
    graphs = []
    for k in range(n_sets):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            serve(q2, k)
        graphs.append(g)

    def replay(i):
        with torch.cuda.stream(stream):
            graphs[i % n_sets].replay()

    ms_graph = measure(replay)
    clocks = sampler.stop()
    popped, pending, dropped, _ = (int(v) for v in info.cpu())
    q2.close()
    ms = ms_graph if args.graph else ms_stream
    line = {
        "metric": METRIC, "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"queue B={n} bz={bz}", "frames": "1920x1080", "crops": [ow, oh],
                   "launch": "CUDA graph replay (one graph per bz)" if args.graph else "stream launches",
                   "last_pop": {"popped": popped, "pending": pending, "dropped": dropped},
                   "l2": f"{n_sets} rotating input/output sets"},
        "us_per_step": {"stream_launches": 1e3 * ms_stream, "graph_replay": 1e3 * ms_graph},
        "e2e": None, "gpu_launches": 5 * args.steps, "clocks": clocks, "roofline": None, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)
    st.close()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "queue":
        run_queue(args)
    elif args.workload == "two_level":
        run_two_level(args)
    else:
        run_octo(args)


if __name__ == "__main__":
    main()
