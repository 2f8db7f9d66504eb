"""The stream executor runs recorded stage passes on the streams the placement routine chose; the
results of every co-located pass must equal those of a direct call."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_01277_b200 as octo
import workloads
from gpu_harness import make_stage
from paper_2502_01277_b200.colocate import StreamExecutor, demo

pytestmark = pytest.mark.gpu


def test_colocated_passes_give_the_direct_results():
    wl = workloads.WORKLOADS["traffic_1080p"]
    dev = torch.device("cuda", 0)
    n_pipe, n = 5, 2
    batches = [workloads.make_batch(wl, batch=n, seed=50 + k) for k in range(n_pipe)]
    stages = [make_stage(wl, n) for _ in range(n_pipe)]
    try:
        bufs = []
        for b in batches:
            bufs.append(dict(frames=[torch.from_numpy(f).to(dev) for f in b.frames], head=torch.from_numpy(b.head).to(dev),
                             det_in=torch.empty((n, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev),
                             dets=torch.zeros((n, wl.max_det, 32), dtype=torch.uint8, device=dev),
                             counts=torch.zeros((n,), dtype=torch.int32, device=dev)))

        def one_pass(k, stream):
            z = bufs[k]
            stages[k].preprocess(z["frames"], batches[k].sizes, out=z["det_in"], stream=stream)
            stages[k].postprocess(z["head"], dets=z["dets"], counts=z["counts"], stream=stream)

        s0 = torch.cuda.Stream(dev)
        for k in range(n_pipe):
            one_pass(k, s0)  # set-up outside any capture
        s0.synchronize()
        inst = [dict(pipeline=k, model=0, instance=0, util_permille=300, start_us=0, end_us=100, duty_cycle_us=1000,
                     weight_bytes=1 << 20, inter_bytes=1 << 20) for k in range(n_pipe)]
        placed = octo.octo_coral_schedule(inst, [dict(mem_bytes=1 << 30, util_max_permille=1000, num_streams=4)])
        # three streams of width 300 fit under 1000; the window 0..100 is free once per stream
        assert [p is not None for p in placed] == [True, True, True, False, False]
        assert sorted(p[1] for p in placed[:3]) == [0, 1, 2]
        for z in bufs:
            z["counts"].fill_(-1)
        ex = StreamExecutor(dev, placed, [lambda stream, k=k: one_pass(k, stream) for k in range(n_pipe)])
        for _ in range(3):
            ex.run_cycle()
        ex.synchronize()
        for k in range(n_pipe):
            d, c = octo.dets_to_numpy(bufs[k]["dets"], bufs[k]["counts"])
            if placed[k] is None:
                assert c.tolist() == [-1] * n  # never ran
                continue
            b = batches[k]
            ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                                   do_letterbox=False, do_crops=False)
            assert np.array_equal(c, ref.counts)
            for i, m in enumerate(c):
                assert np.array_equal(d[i, :m]["anchor"], ref.dets[i, :m]["anchor"])
    finally:
        for st in stages:
            st.close()


def test_demo_runs_and_reports_both_rates():
    """The demonstrator places, runs and reports; which rate is higher is a measurement that its
    output states (python -m paper_2502_01277_b200.colocate), not something a test asserts."""
    out = demo(n_pipelines=4, batch=1, cycles=50, streams=4)
    assert all(p is not None for p in out["placed"]) and out["streams_used"] >= 2
    assert out["passes_per_s_colocated"] > 0 and out["passes_per_s_one_stream"] > 0
