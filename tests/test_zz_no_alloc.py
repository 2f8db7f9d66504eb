"""The allocation-free entry point against the stage-based one.

octo_postprocess_frame_static exists for programs that cannot allocate GPU memory while
they run (a real-time loop with a fixed memory budget, a plug-in living in a host
application's pool): it decodes one frame's head and runs NMS on a workspace compiled into
the library instead of one obtained from cudaMalloc.  It must return exactly what
octo_postprocess_batch returns for the same frame.  The workspace is shared by all calls and
keeps old contents, so the check is made on two calls in a row, the second with far fewer
candidates than the first, then on the first input again.

This file is named so that pytest collects it after every other test file.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import paper_2502_01277_b200 as octo
import workloads
from paper_2502_01277_b200 import binding as B

pytestmark = pytest.mark.gpu

W, H, S = 1280, 720, 640


def _heads():
    base = replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((W, H),))
    dense = workloads.make_batch(replace(base, n_raised=3000, n_groups=200, max_det=300), batch=1, seed=21)
    sparse = workloads.make_batch(replace(base, n_raised=120, n_groups=15, max_det=300), batch=1, seed=22)
    return dense, sparse


def _via_stage(stage, batch):
    frame = torch.from_numpy(batch.frames[0]).cuda()
    stage.preprocess([frame], [(W, H)])
    dets, counts = stage.postprocess(torch.from_numpy(batch.head).cuda())
    torch.cuda.synchronize()
    d, c = octo.dets_to_numpy(dets, counts)
    return d[0, : c[0]].copy(), int(c[0])


def _via_static(batch, max_det=300):
    wl = batch.workload
    head = torch.from_numpy(batch.head[0]).cuda()
    dets = torch.full((max_det, 32), 0xAB, dtype=torch.uint8, device="cuda")
    count = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    octo.octo_postprocess_frame_static(0, head.data_ptr(), wl.num_anchors, wl.num_classes, True, wl.conf_thresh,
                                       wl.iou_thresh, max_det, S, W, H, dets.data_ptr(), count.data_ptr(),
                                       int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    c = int(count.item())
    d = dets.cpu().numpy().view(B.DET_DTYPE).reshape(-1)
    return d[:c].copy(), c


def test_static_workspace_entry_matches_stage_entry_on_consecutive_calls():
    dense, sparse = _heads()
    wl = dense.workload
    stage = octo.Stage(net_size=S, max_batch=1, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                       max_det=300, branches=((64, 64),))
    try:
        want_dense, n_dense = _via_stage(stage, dense)
        want_sparse, n_sparse = _via_stage(stage, sparse)
    finally:
        stage.close()
    assert n_dense > n_sparse > 5
    # two calls in a row on the shared workspace, then the first input once more
    for batch, want, n in ((dense, want_dense, n_dense), (sparse, want_sparse, n_sparse),
                           (dense, want_dense, n_dense)):
        got, c = _via_static(batch)
        assert c == n
        assert got.tobytes() == want.tobytes()  # same bit-exact bar as the other detection tests


def test_static_workspace_entry_rejects_sizes_beyond_its_limits():
    head = torch.zeros((8, 85), dtype=torch.float32, device="cuda")
    dets = torch.zeros((4, 32), dtype=torch.uint8, device="cuda")
    count = torch.zeros((1,), dtype=torch.int32, device="cuda")
    args = dict(device=0, d_head=head.data_ptr(), num_anchors=8, num_classes=80, head_is_logits=True,
                conf_thresh=0.25, iou_thresh=0.45, max_det=4, net_size=S, frame_w=W, frame_h=H,
                d_dets=dets.data_ptr(), d_count=count.data_ptr())
    for over in (dict(num_anchors=32769), dict(max_det=1025)):
        with pytest.raises(octo.OctoError) as ei:
            octo.octo_postprocess_frame_static(**{**args, **over})
        assert ei.value.code == B.OCTO_E_CAPACITY
    with pytest.raises(octo.OctoError) as ei:
        octo.octo_postprocess_frame_static(**{**args, "d_dets": 0})
    assert ei.value.code == B.OCTO_E_INVALID_ARG
    # an all-background head is a valid input and yields no detections
    head.fill_(-9.0)
    octo.octo_postprocess_frame_static(**args)
    torch.cuda.synchronize()
    assert int(count.item()) == 0
