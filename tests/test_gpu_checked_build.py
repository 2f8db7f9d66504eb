"""The range-checked build of the library (-DOCTO_BOUNDS_CHECK): every computed shared- and
global-memory index of the kernels is tested against its range; a miss sets OCTO_STATUS_BOUNDS
and skips the access.  It stands in for a memory checker.  The stage is driven through that
library on small, ragged and randomised cases; the results must still equal the oracle's and the
status word must stay clean."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workloads
from paper_2502_01277_b200 import binding as B
from paper_2502_01277_b200 import build as cuda_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked():
    """Swap the checked library in for the duration of the module."""
    path = cuda_build.build(checked=True)
    normal = B._lib
    B._lib = None
    lib = B.load_library(path)
    B._lib = lib
    yield lib
    B._lib = normal


def _compare(res, ref, branches):
    from test_gpu_parity import PIX_TOL, _check_dets
    from gpu_harness import half_absdiff
    assert res.status & B.OCTO_STATUS_BOUNDS == 0, "an index left its range"
    assert res.status & ~0x8 == 0
    assert half_absdiff(res.det_in, ref.det_in) <= PIX_TOL
    _check_dets(res, ref)
    for k in range(len(branches)):
        total = len(ref.items[k])
        assert res.n_items[k] == (total, total)
        it = res.items[k]
        assert np.array_equal(np.stack([it["rx0"], it["ry0"], it["rx1"], it["ry1"]], 1).reshape(-1, 4),
                              ref.rects[k].reshape(-1, 4))
        assert half_absdiff(res.crops[k][:total], ref.crops[k][:total]) <= PIX_TOL


@pytest.mark.parametrize("name,batch", [("tiny", None), ("traffic_1080p", 3), ("two_branch", 5), ("dense_nms", 2)])
def test_workloads_under_the_checked_build(checked, name, batch):
    from gpu_harness import make_stage, run_stage_gpu
    b = workloads.make_batch(name, batch=batch)
    wl = b.workload
    st = make_stage(wl, b.n)
    try:
        assert ctypes.cast(st.handle, ctypes.c_void_p).value  # created by the checked library
        ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, logits=wl.logits,
                               conf=wl.conf_thresh, iou_thr=wl.iou_thresh, max_det=wl.max_det, threads=8)
        cap = [len(ref.items[k]) + 1 for k in range(len(wl.branches))]
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=cap)
        _compare(res, ref, wl.branches)
    finally:
        st.close()


def test_global_memory_nms_path_under_the_checked_build(checked):
    from test_gpu_parity import _small_case, _check_dets
    from gpu_harness import make_stage, run_stage_gpu
    b = _small_case(9000, 600, batch=1)
    wl = b.workload
    st = make_stage(wl, b.n)
    try:
        ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                               do_letterbox=False, do_crops=False)
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[16])
        assert res.status & B.OCTO_STATUS_BIG_NMS and res.status & B.OCTO_STATUS_BOUNDS == 0
        _check_dets(res, ref)
    finally:
        st.close()


@pytest.mark.parametrize("seed,large", [(s, False) for s in range(0, 64, 4)] + [(s, True) for s in (1, 5, 7)])
def test_random_configurations_under_the_checked_build(checked, seed, large):
    from test_gpu_fuzz import _case
    from gpu_harness import make_stage, run_stage_gpu
    b, frames, sizes, cfg = _case(seed, large=large)
    wl = b.workload
    st = make_stage(wl, b.n, **cfg)
    try:
        ref = oracle.run_stage(frames, sizes, b.head, wl.net_size, wl.branches, logits=wl.logits,
                               conf=wl.conf_thresh, iou_thr=wl.iou_thresh, max_det=wl.max_det,
                               pad_value=cfg["pad_value"], swap_rb=cfg["swap_rb"], class_masks=cfg["class_masks"],
                               agnostic=cfg["class_agnostic"], layout=wl.head_layout, multi_label=wl.multi_label,
                               crop_options=cfg["crop_options"], threads=8)
        cap = [len(ref.items[k]) + 1 for k in range(len(wl.branches))]
        res = run_stage_gpu(st, frames, sizes, b.head, max_items=cap)
        _compare(res, ref, wl.branches)
    finally:
        st.close()


def test_very_wide_rectangles_under_the_checked_build(checked):
    """Column tiling of the crop kernel (rectangles wider than a staging buffer)."""
    import paper_2502_01277_b200 as octo
    from gpu_harness import run_stage_gpu
    rng = np.random.default_rng(8)
    w, h, s = 7000, 24, 640
    pitch = (3 * w + 15) // 16 * 16
    img = np.zeros((h, pitch), dtype=np.uint8)
    img[:, :3 * w] = rng.integers(0, 256, size=(h, 3 * w), dtype=np.uint8)
    C, A = 4, 64
    head = np.full((1, A, 5 + C), -9.0, dtype=np.float32)
    nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
    g = w / nw
    for k, (cx, cy, bw, bh) in enumerate([(3500, 12, 7000, 24), (2100, 10, 4100, 8), (6000, 20, 1500, 4)]):
        head[0, k, :4] = [cx / g + pl, cy / g + pt, bw / g, bh / g]
        head[0, k, 4] = 4.0 - 0.1 * k
        head[0, k, 5 + k] = 5.0
    st = octo.Stage(net_size=s, max_batch=1, num_anchors=A, num_classes=C, branches=((224, 16),))
    try:
        res = run_stage_gpu(st, [img], [(w, h)], head)
        ref = oracle.run_stage([img], [(w, h)], head, s, ((224, 16),))
        _compare(res, ref, ((224, 16),))
    finally:
        st.close()


@pytest.mark.parametrize("ow,oh", [(24, 40), (136, 40), (456, 40), (904, 20), (2048, 9)])
def test_output_widths_around_the_unit_layout_under_the_checked_build(checked, ow, oh):
    """Crop work layouts with an odd number of column units, fewer and more units than consumer
    threads: the same cases as in the parity module, with every index range-checked."""
    from test_gpu_parity import test_crop_output_widths_around_the_unit_layout as case
    case(ow, oh)  # asserts parity and a clean status word (OCTO_STATUS_BOUNDS included)


@pytest.mark.parametrize("cluster", [1, 4])
def test_crowded_image_under_the_checked_build(checked, cluster):
    """General NMS path with the sorted merge, alone and on a cluster of CTAs (finished classes written
    into the first CTA's shared memory), with every index range-checked."""
    from test_gpu_nms_cluster import _batch, _oracle_dets
    from test_gpu_parity import _check_dets
    from gpu_harness import make_stage, run_stage_gpu
    b = _batch(5000, 250, 2, max_det=1000)
    st = make_stage(b.workload, b.n)
    try:
        st.set_nms_cluster(cluster)
        ref = _oracle_dets(b)
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[8])
        assert st.last_nms_cluster() == cluster
        assert res.status & B.OCTO_STATUS_BOUNDS == 0, "an index left its range"
        _check_dets(res, ref)
    finally:
        st.close()


def test_half_sized_nms_ctas_under_the_checked_build(checked):
    """More images than SMs: two half-sized NMS CTAs per SM, with an image on the general on-chip path
    and one that exceeds the smaller on-chip capacity, every index range-checked (the case of the
    NMS module; it asserts the launch forms and parity, the status word is checked there too)."""
    from test_gpu_nms_cluster import test_more_images_than_sms_run_two_half_sized_ctas_per_sm as case
    case()
