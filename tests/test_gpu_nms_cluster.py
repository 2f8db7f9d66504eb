"""NMS with a thread-block cluster per image: every cluster size gives the oracle's detections, and the
automatic choice switches clusters on after crowded images and off again after sparse ones."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import workloads
from gpu_harness import make_stage, run_stage_gpu
from paper_2502_01277_b200 import binding as B

pytestmark = pytest.mark.gpu


def _batch(n_raised, n_groups, batch, seed=5, max_det=300):
    wl = replace(workloads.WORKLOADS["traffic_1080p"], n_raised=n_raised, n_groups=n_groups,
                 frame_sizes=((640, 360),), max_det=max_det)
    return workloads.make_batch(wl, batch=batch, seed=seed)


def _oracle_dets(b):
    wl = b.workload
    return oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, logits=wl.logits,
                            conf=wl.conf_thresh, iou_thr=wl.iou_thresh, max_det=wl.max_det, do_letterbox=False,
                            do_crops=False, threads=8)


@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
@pytest.mark.parametrize("n_raised,n_groups,batch", [(5000, 250, 3), (2500, 90, 2), (700, 60, 1), (150, 20, 2)])
def test_every_cluster_size_gives_the_same_detections(cluster, n_raised, n_groups, batch):
    """Crowded images (general path, classes dealt to the warps of all CTAs), a mid-sized one and sparse
    ones (short path, first CTA alone) under a forced cluster size."""
    from test_gpu_parity import _check_dets
    b = _batch(n_raised, n_groups, batch, max_det=1000 if n_raised > 1000 else 300)
    st = make_stage(b.workload, b.n)
    try:
        st.set_nms_cluster(cluster)
        ref = _oracle_dets(b)
        for _ in range(2):  # twice: the candidate counters must be left clean for the next pass
            res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[8])
            assert st.last_nms_cluster() == cluster
            _check_dets(res, ref)
            assert res.status & ~(B.OCTO_STATUS_BIG_NMS | 0x2) == 0
    finally:
        st.close()


def test_more_candidates_than_fit_on_chip_under_a_cluster():
    """The global-memory path belongs to the first CTA of a cluster alone."""
    from test_gpu_parity import _check_dets
    b = _batch(9000, 600, 1, seed=3)
    st = make_stage(b.workload, b.n)
    try:
        st.set_nms_cluster(4)
        ref = _oracle_dets(b)
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[8])
        assert res.status & B.OCTO_STATUS_BIG_NMS
        _check_dets(res, ref)
    finally:
        st.close()


def test_automatic_choice_follows_the_candidate_counts():
    from test_gpu_parity import _check_dets
    dense = _batch(5000, 250, 2, max_det=1000)
    sparse = replace(dense, head=_batch(150, 20, 2, max_det=1000).head)
    st = make_stage(dense.workload, dense.n)
    try:
        with pytest.raises(B.OctoError):
            st.set_nms_cluster(3)
        ref_dense, ref_sparse = _oracle_dets(dense), _oracle_dets(sparse)
        res = run_stage_gpu(st, sparse.frames, sparse.sizes, sparse.head, max_items=[8])
        assert st.last_nms_cluster() == 1
        res = run_stage_gpu(st, dense.frames, dense.sizes, dense.head, max_items=[8])  # synchronises
        assert st.last_nms_cluster() == 1  # nothing crowded had been seen when this pass was launched
        _check_dets(res, ref_dense)
        res = run_stage_gpu(st, dense.frames, dense.sizes, dense.head, max_items=[8])
        assert st.last_nms_cluster() > 1  # two images on 148 SMs: the largest cluster the device schedules
        _check_dets(res, ref_dense)
        for i in range(66):  # sparse passes: the crowded one falls out of the stage's latest 64 launches
            res = run_stage_gpu(st, sparse.frames, sparse.sizes, sparse.head, max_items=[8])
            if i < 2 or i > 62:
                _check_dets(res, ref_sparse)
            assert st.last_nms_cluster() == (1 if i >= 64 else st.last_nms_cluster())
        assert st.last_nms_cluster() == 1
    finally:
        st.close()


def test_more_images_than_sms_run_two_half_sized_ctas_per_sm():
    """A batch of more images than the GPU has SMs is launched with two half-sized CTAs per SM while
    no crowded image is known.  Such a CTA holds 4096 candidates on chip: in the first pass an image
    with 5000 goes through the global-memory path and one with 700 through the general on-chip path
    on half the threads; the crowded image is reported, so the second pass is full-sized again, and
    after 64 sparse launches the half-sized form returns.  Every pass gives the oracle's detections."""
    from test_gpu_parity import _check_dets
    n = torch.cuda.get_device_properties(0).multi_processor_count + 2
    sparse = _batch(150, 20, n, max_det=1000)
    mixed = replace(sparse, head=sparse.head.copy())
    mixed.head[3] = _batch(5000, 250, 1, seed=8, max_det=1000).head[0]
    mixed.head[n // 2] = _batch(700, 60, 1, seed=9, max_det=1000).head[0]
    ref_sparse, ref_mixed = _oracle_dets(sparse), _oracle_dets(mixed)
    assert ref_mixed.n_cand[3] > 4096 and 256 < ref_mixed.n_cand[n // 2] <= 4096 and ref_sparse.n_cand.max() <= 256
    st = make_stage(sparse.workload, n)
    try:
        res = run_stage_gpu(st, mixed.frames, mixed.sizes, mixed.head, max_items=[8])
        assert st.last_nms_half_ctas() and st.last_nms_cluster() == 1
        _check_dets(res, ref_mixed)
        assert res.status & ~0x2 == 0  # 5000 candidates fit a full-sized CTA: no BIG_NMS report
        res = run_stage_gpu(st, mixed.frames, mixed.sizes, mixed.head, max_items=[8])
        assert not st.last_nms_half_ctas()
        _check_dets(res, ref_mixed)
        for i in range(66):
            res = run_stage_gpu(st, sparse.frames, sparse.sizes, sparse.head, max_items=[8])
            assert st.last_nms_half_ctas() == (i >= 64)
        _check_dets(res, ref_sparse)
        assert res.status & ~0x2 == 0
    finally:
        st.close()
