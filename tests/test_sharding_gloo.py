"""The multi-GPU form of the stage is replicas: frames are independent, each rank packs its
own downstream batches, and nothing crosses ranks on the data path.  This checks the host
logic of that form with two CPU ranks over gloo: disjoint contiguous shards, per-rank
results equal to the matching slice of the single-process result, and the max-over-ranks
timing reduction the benchmark uses."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import workloads
from workloads.synth import shard_range


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, total, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = shard_range(total, rank, world)
    b = workloads.make_batch("traffic_1080p", batch=hi - lo, first_frame=lo, threads=1)
    wl = b.workload
    r = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                         do_letterbox=False, do_crops=False)
    t = torch.tensor([0.5 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    frames = torch.tensor([hi - lo], dtype=torch.int64)
    dist.all_reduce(frames, op=dist.ReduceOp.SUM)
    q.put((rank, lo, hi, r.counts.tolist(), r.dets["anchor"][:, :8].tolist(), float(t.item()), int(frames.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replicas_match_single_process():
    total, world = 5, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, total, q)) for r in range(world)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    b = workloads.make_batch("traffic_1080p", batch=total, threads=1)
    wl = b.workload
    ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                           do_letterbox=False, do_crops=False)
    covered = []
    for rank, lo, hi, counts, anchors, tmax, frames in out:
        covered += list(range(lo, hi))
        assert counts == ref.counts[lo:hi].tolist()
        assert anchors == ref.dets["anchor"][lo:hi, :8].tolist()
        assert tmax == 0.5 + (world - 1) and frames == total
    assert covered == list(range(total))


def test_shard_range_partitions():
    for total in (0, 1, 7, 64, 255):
        for world in (1, 2, 3, 8):
            spans = [shard_range(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
