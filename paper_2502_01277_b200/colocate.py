"""Stream executor for co-located stages: recorded stage passes (CUDA graphs) run on the CUDA
streams that octo_coral_schedule assigned them, every stream working through its portions in
start order, cycle after cycle (the paper's inference streams, Section III-C).

This is a demonstrator of the placement routine on real kernels, not a real-time runtime: the
order of the portions on a stream is kept, their absolute start times are not enforced (a stream
runs its next portion as soon as the previous one ends), and the per-model profiles (run time,
memory, width) are whatever the caller measured or assumed.

    python -m paper_2502_01277_b200.colocate        # small demo on cuda:0
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

from .binding import octo_coral_schedule


class StreamExecutor:
    """placements: result of octo_coral_schedule for `instances`; record[i] enqueues instance i's
    work on the stream it is given (it is called once, under graph capture)."""

    def __init__(self, device, placements: Sequence[Optional[Tuple[int, int, int, int, int]]],
                 record: Sequence[Callable], gpu: int = 0):
        import torch
        self._torch = torch
        self.device = torch.device(device)
        lanes: Dict[int, List[Tuple[int, int]]] = {}
        for i, pl in enumerate(placements):
            if pl is not None and pl[0] == gpu:
                lanes.setdefault(pl[1], []).append((pl[2], i))
        self.streams = {s: torch.cuda.Stream(self.device) for s in lanes}
        self.order = {s: [i for _, i in sorted(v)] for s, v in lanes.items()}
        self.graphs: Dict[int, "torch.cuda.CUDAGraph"] = {}
        for s, members in self.order.items():
            for i in members:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.streams[s]):
                    record[i](self.streams[s])
                self.graphs[i] = g
        torch.cuda.synchronize(self.device)

    def run_cycle(self) -> None:
        """One duty cycle: every stream replays its portions in order; streams run side by side."""
        t = self._torch
        for s, members in self.order.items():
            with t.cuda.stream(self.streams[s]):
                for i in members:
                    self.graphs[i].replay()

    def synchronize(self) -> None:
        for st in self.streams.values():
            st.synchronize()


def demo(n_pipelines: int = 6, batch: int = 2, cycles: int = 200, streams: int = 4) -> dict:
    """n_pipelines copies of a small detector stage (one pass = letterbox + decode/NMS + crop of
    `batch` frames) placed on `streams` streams of one GPU; returns passes per second with the
    placement and with everything on one stream."""
    import time

    import torch

    import workloads
    from . import Stage

    dev = torch.device("cuda", 0)
    wl = workloads.WORKLOADS["traffic_1080p"]
    b = workloads.make_batch(wl, batch=batch)
    frames = [torch.from_numpy(f).to(dev) for f in b.frames]
    head = torch.from_numpy(b.head).to(dev)
    stages, bufs = [], []
    for _ in range(n_pipelines):
        st = Stage(device=0, net_size=wl.net_size, max_batch=batch, num_anchors=wl.num_anchors,
                   num_classes=wl.num_classes, max_det=wl.max_det, branches=wl.branches)
        z = dict(det_in=torch.empty((batch, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev),
                 dets=torch.zeros((batch, wl.max_det, 32), dtype=torch.uint8, device=dev),
                 counts=torch.zeros((batch,), dtype=torch.int32, device=dev),
                 crops=torch.empty((batch * 64, 3, wl.branches[0][1], wl.branches[0][0]), dtype=torch.float16, device=dev),
                 off=torch.zeros((batch + 1,), dtype=torch.int32, device=dev),
                 ni=torch.zeros((2,), dtype=torch.int32, device=dev))
        stages.append(st)
        bufs.append(z)

    def one_pass(k, stream):
        st, z = stages[k], bufs[k]
        st.preprocess(frames, b.sizes, out=z["det_in"], stream=stream)
        st.postprocess(head, dets=z["dets"], counts=z["counts"], stream=stream)
        st.crop(0, batch * 64, out=z["crops"], offsets=z["off"], n_items=z["ni"], stream=stream)

    # profile: run time of one pass alone (the paper's batch inference profile)
    s0 = torch.cuda.Stream(dev)
    for k in range(n_pipelines):
        one_pass(k, s0)
    s0.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s0)
    for _ in range(20):
        one_pass(0, s0)
    e1.record(s0)
    s0.synchronize()
    pass_us = max(1, int(1000.0 * e0.elapsed_time(e1) / 20))

    # every pipeline wants the window [0, pass_us) of a cycle long enough for all of them in a row;
    # a small-batch pass is latency-bound and leaves most of the GPU idle: width 250 of 1000
    duty = pass_us * n_pipelines
    mem = sum(st.workspace_bytes for st in stages) // n_pipelines
    instances = [dict(pipeline=k, model=0, instance=0, util_permille=250, start_us=(k % 2) * pass_us,
                      end_us=(k % 2 + 1) * pass_us, duty_cycle_us=duty, weight_bytes=mem, inter_bytes=mem // 4)
                 for k in range(n_pipelines)]
    gpus = [dict(mem_bytes=64 << 30, util_max_permille=1000, num_streams=streams)]
    placed = octo_coral_schedule(instances, gpus)
    record = [lambda stream, k=k: one_pass(k, stream) for k in range(n_pipelines)]
    ex = StreamExecutor(dev, placed, record)
    single = StreamExecutor(dev, [None if p is None else (0, 0, 10 * k, 10 * k + 1, duty) for k, p in enumerate(placed)], record)

    def rate(executor) -> float:
        for _ in range(10):
            executor.run_cycle()
        executor.synchronize()
        t0 = time.perf_counter()
        for _ in range(cycles):
            executor.run_cycle()
        executor.synchronize()
        return cycles * sum(len(v) for v in executor.order.values()) / (time.perf_counter() - t0)

    out = {"pass_us_alone": pass_us, "placed": placed, "streams_used": len(ex.streams),
           "passes_per_s_colocated": rate(ex), "passes_per_s_one_stream": rate(single), "batch": batch}
    out["colocation_gain"] = out["passes_per_s_colocated"] / out["passes_per_s_one_stream"]  # > 1: co-location paid
    for st in stages:
        st.close()
    return out


if __name__ == "__main__":
    import json
    print(json.dumps(demo()))
