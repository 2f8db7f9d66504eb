"""A stage pass only enqueues kernels on the caller's stream, so it can be recorded once into a
CUDA graph and replayed on new data in the same buffers (one graph per downstream batch size is
how a serving loop avoids launch overhead on small batches).  The replayed results must meet the
same parity bar as direct calls."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2502_01277_b200 as octo
import workloads
from gpu_harness import half_absdiff, make_stage
from test_gpu_parity import PIX_TOL

pytestmark = pytest.mark.gpu


def test_stage_pass_replayed_from_a_cuda_graph():
    wl = replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((640, 360),), branches=((64, 64), (96, 32)),
                 n_raised=80, n_groups=10)
    n, cap = 3, 128
    batches = [workloads.make_batch(wl, batch=n, seed=40 + k) for k in range(3)]
    dev = torch.device("cuda", 0)
    st = make_stage(wl, n)
    stream = torch.cuda.Stream(dev)
    try:
        with torch.cuda.stream(stream):
            frames = [torch.empty_like(torch.from_numpy(f), device=dev) for f in batches[0].frames]
            head = torch.empty(batches[0].head.shape, dtype=torch.float32, device=dev)
            det_in = torch.empty((n, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev)
            dets = torch.zeros((n, wl.max_det, 32), dtype=torch.uint8, device=dev)
            counts = torch.zeros((n,), dtype=torch.int32, device=dev)
            crops = [torch.zeros((cap, 3, oh, ow), dtype=torch.float16, device=dev) for ow, oh in wl.branches]
            offs = [torch.zeros((n + 1,), dtype=torch.int32, device=dev) for _ in wl.branches]
            nis = [torch.zeros((2,), dtype=torch.int32, device=dev) for _ in wl.branches]

        def one_pass():
            st.preprocess(frames, batches[0].sizes, out=det_in, stream=stream)
            st.postprocess(head, dets=dets, counts=counts, stream=stream)
            for b in range(len(wl.branches)):
                st.crop(b, cap, out=crops[b], offsets=offs[b], n_items=nis[b], stream=stream)

        def load(bt):
            with torch.cuda.stream(stream):
                for d, f in zip(frames, bt.frames):
                    d.copy_(torch.from_numpy(f), non_blocking=False)
                head.copy_(torch.from_numpy(bt.head))

        load(batches[0])
        one_pass()  # a direct pass first: the library's one-time set-up stays outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_pass()
        for bt in batches[1:] + batches[:1]:
            load(bt)
            with torch.cuda.stream(stream):
                for c in crops:
                    c.fill_(0)
                graph.replay()
            stream.synchronize()
            ref = oracle.run_stage(bt.frames, bt.sizes, bt.head, wl.net_size, wl.branches, max_det=wl.max_det)
            d, c = octo.dets_to_numpy(dets, counts)
            assert np.array_equal(c, ref.counts)
            for i, k in enumerate(c):
                assert np.array_equal(d[i, :k]["anchor"], ref.dets[i, :k]["anchor"])
                assert np.array_equal(d[i, :k]["x1"].view(np.uint32), ref.dets[i, :k]["x1"].view(np.uint32))
            got_in = det_in.view(torch.int16).cpu().numpy().view(np.uint16)
            assert half_absdiff(got_in, ref.det_in) <= PIX_TOL
            for b in range(len(wl.branches)):
                packed, total = (int(v) for v in nis[b].cpu())
                assert total == len(ref.items[b]) and packed == min(total, cap)
                assert np.array_equal(offs[b].cpu().numpy(), ref.offsets[b])
                got = crops[b][:packed].view(torch.int16).cpu().numpy().view(np.uint16)
                assert half_absdiff(got, ref.crops[b][:packed]) <= PIX_TOL
            assert st.status(stream) == 0
    finally:
        st.close()
