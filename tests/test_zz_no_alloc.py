"""The allocation-free entry point against the stage-based one.

octo_postprocess_frame_static exists for programs that cannot allocate GPU memory while
they run (a real-time loop with a fixed memory budget, a plug-in living in a host
application's pool): it decodes one frame's head and runs NMS on a workspace compiled into
the library instead of one obtained from cudaMalloc.  It must return exactly what
octo_postprocess_batch returns for the same frame, which in turn is what the CPU oracle computes.
The workspace is shared by all calls and keeps old contents, so the check is made on calls in a
row whose candidate counts go up and down: a dense head, a head with more candidates than the
NMS kernel holds on chip (the part of the workspace that only the global-memory path uses), a
sparse head, and the first two again.  The status word of each call is read back as well.

This file is named so that pytest collects it after every other test file.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2502_01277_b200 as octo
import workloads
from paper_2502_01277_b200 import binding as B

pytestmark = pytest.mark.gpu

W, H, S = 1280, 720, 640


def _heads():
    base = replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((W, H),))
    dense = workloads.make_batch(replace(base, n_raised=3000, n_groups=200, max_det=300), batch=1, seed=21)
    sparse = workloads.make_batch(replace(base, n_raised=120, n_groups=15, max_det=300), batch=1, seed=22)
    huge = workloads.make_batch(replace(base, n_raised=9500, n_groups=700, max_det=300), batch=1, seed=23)
    return dense, sparse, huge


def _via_oracle(batch, max_det=300):
    wl = batch.workload
    d, ncand = oracle.postprocess_image(batch.head[0], W, H, S, True, wl.conf_thresh, wl.iou_thresh, max_det)
    return d, int(ncand)


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
    status = octo.octo_static_status(0, int(torch.cuda.current_stream().cuda_stream))  # synchronises
    c = int(count.item())
    d = dets.cpu().numpy().view(B.DET_DTYPE).reshape(-1)
    return d[:c].copy(), c, status


def test_static_workspace_entry_matches_stage_entry_on_consecutive_calls():
    dense, sparse, huge = _heads()
    wl = dense.workload
    stage = octo.Stage(net_size=S, max_batch=1, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                       max_det=300, branches=((64, 64),))
    try:
        via_stage = {id(b): _via_stage(stage, b) for b in (dense, sparse, huge)}
    finally:
        stage.close()
    via_oracle = {id(b): _via_oracle(b) for b in (dense, sparse, huge)}
    assert via_oracle[id(huge)][1] > 8192 > via_oracle[id(dense)][1] > 256 > via_oracle[id(sparse)][1]
    assert via_stage[id(dense)][1] > via_stage[id(sparse)][1] > 5
    # calls in a row on the shared workspace; the candidate count goes up and down between them
    for batch in (dense, huge, sparse, huge, dense, sparse):
        got, c, status = _via_static(batch)
        want, n = via_stage[id(batch)]
        assert c == n
        assert got.tobytes() == want.tobytes()  # same bit-exact bar as the other detection tests
        ref, _ = via_oracle[id(batch)]
        assert c == len(ref) and got.tobytes() == ref[:c].tobytes()  # and the oracle itself
        # more candidates than fit on chip take the global-memory path and say so; nothing else is set
        assert status == (B.OCTO_STATUS_BIG_NMS if batch is huge else 0)


def test_static_workspace_entry_reports_dropped_rows():
    """A head row with a non-finite value is dropped, as by a stage, and the status word of the call
    says so; the next call starts from a clean word."""
    _, sparse, _ = _heads()
    bad = sparse.head[0].copy()
    raised = np.nonzero(bad[:, 4] > 0)[0]
    bad[raised[0], 0] = np.nan
    bad[raised[1], 5 + 3] = np.inf
    wl = sparse.workload
    want, _ = oracle.postprocess_image(bad, W, H, S, True, wl.conf_thresh, wl.iou_thresh, 300)
    broken = replace(sparse, head=bad[None])
    got, c, status = _via_static(broken)
    assert c == len(want) and got.tobytes() == want[:c].tobytes()
    assert status == B.OCTO_STATUS_NONFINITE
    _, _, status = _via_static(sparse)
    assert status == 0


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
