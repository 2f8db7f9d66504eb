"""GPU parity of the branch options of the crop kernel (aspect-preserving fit, mean/std
normalisation) against the CPU oracle, through the C ABI.

Packing and rectangles are bit-exact as always.  Crops must agree within 2e-3 in value.  The two
sides interpolate in double and in binary32 (difference about 1e-6) and can therefore land on
different sides of a binary16 rounding boundary, i.e. one binary16 step apart; normalised values
stay below 4 in magnitude with the constants used here, where that step is at most 1.95e-3."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import workloads
from gpu_harness import half_absdiff, make_stage, run_stage_gpu
from test_gpu_parity import PIX_TOL, _check_dets

pytestmark = pytest.mark.gpu

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)


def _check(res, ref, b, normalised):
    total = len(ref.items[b])
    assert res.n_items[b] == (total, total) and np.array_equal(res.offsets[b], ref.offsets[b])
    it = res.items[b]
    assert np.array_equal(np.stack([it["frame"], it["det"]], 1), ref.items[b])
    assert np.array_equal(np.stack([it["rx0"], it["ry0"], it["rx1"], it["ry1"]], 1), ref.rects[b])
    got, want = res.crops[b][:total], ref.crops[b][:total]
    assert half_absdiff(got, want) <= PIX_TOL
    if normalised:
        assert np.abs(want.view(np.float16).astype(np.float32)).max() < 4.0
    assert np.all(res.crops[b][total:] == 0x7BFF)


def _run(b, crop_options, **stage_over):
    wl = b.workload
    st = make_stage(wl, b.n, crop_options=crop_options, **stage_over)
    try:
        ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                               do_letterbox=False, crop_options=crop_options, threads=8,
                               pad_value=stage_over.get("pad_value", 114), swap_rb=stage_over.get("swap_rb", True))
        cap = [len(ref.items[k]) + 2 for k in range(len(wl.branches))]
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=cap)
        _check_dets(res, ref)
        assert res.status == 0
        return res, ref
    finally:
        st.close()


def _batch(branches, batch=3, **over):
    wl = replace(workloads.WORKLOADS["traffic_1080p"], branches=branches, n_raised=60, n_groups=12,
                 frame_sizes=((1280, 720),), **over)
    return workloads.make_batch(wl, batch=batch, seed=31)


def test_keep_aspect_crops():
    b = _batch(((224, 224), (96, 160)))
    opts = [{"keep_aspect": True}, {"keep_aspect": True}]
    res, ref = _run(b, opts)
    for k in range(2):
        _check(res, ref, k, normalised=False)
    # the canvas is there and holds the pad value exactly
    assert np.any(res.crops[0][: len(ref.items[0])] == 0x3727)
    rects = ref.rects[0]
    assert len(np.unique((rects[:, 2] - rects[:, 0]) - (rects[:, 3] - rects[:, 1]))) > 5  # wide and tall boxes


def test_normalised_crops_and_mixed_branches():
    """One plain branch, one normalised, one with both options: a stage mixes them freely."""
    b = _batch(((64, 64), (224, 224), (128, 96)))
    opts = [None, {"mean": MEAN, "std": STD}, {"keep_aspect": True, "mean": MEAN, "std": STD}]
    res, ref = _run(b, opts)
    _check(res, ref, 0, normalised=False)
    _check(res, ref, 1, normalised=True)
    _check(res, ref, 2, normalised=True)
    v = res.crops[1][: len(ref.items[1])].view(np.float16).astype(np.float32)
    assert v.min() < -1.0 and v.max() > 1.0


def test_options_without_swap_and_with_another_pad_value():
    b = _batch(((64, 48),), batch=2)
    opts = [{"keep_aspect": True, "mean": (0.1, 0.2, 0.3), "std": (0.5, 0.25, 1.0)}]
    res, ref = _run(b, opts, swap_rb=False, pad_value=7)
    _check(res, ref, 0, normalised=True)


def test_keep_aspect_of_extreme_and_very_wide_rectangles():
    """Hand-placed boxes: a sliver that fits to a single column, a rectangle wider than one
    staging buffer (column tiles, canvas rows above and below), a box of the slot's own shape."""
    import paper_2502_01277_b200 as octo
    rng = np.random.default_rng(9)
    w, h, s = 7000, 40, 640
    pitch = (3 * w + 15) // 16 * 16
    img = np.zeros((h, pitch), dtype=np.uint8)
    img[:, :3 * w] = rng.integers(0, 256, size=(h, 3 * w), dtype=np.uint8)
    C, A = 4, 64
    head = np.full((1, A, 5 + C), -9.0, dtype=np.float32)
    nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
    g = w / nw
    boxes = [(3500, 20, 7000, 40), (2100, 10, 4100, 8), (100, 20, 2, 40), (6000, 20, 64, 32), (5000, 30, 4000, 3)]
    for k, (cx, cy, bw, bh) in enumerate(boxes):
        head[0, k, :4] = [cx / g + pl, cy / g + pt, bw / g, bh / g]
        head[0, k, 4] = 4.0 - 0.1 * k
        head[0, k, 5 + (k % C)] = 5.0
    for (ow, oh) in [(224, 64), (1024, 16), (64, 32)]:
        opts = [{"keep_aspect": True}]
        st = octo.Stage(net_size=s, max_batch=1, num_anchors=A, num_classes=C, branches=((ow, oh),),
                        crop_options=opts)
        try:
            res = run_stage_gpu(st, [img], [(w, h)], head)
            ref = oracle.run_stage([img], [(w, h)], head, s, ((ow, oh),), crop_options=opts)
            assert ref.counts[0] == len(boxes)
            _check_dets(res, ref)
            total = len(ref.items[0])
            assert res.n_items[0] == (total, total)
            assert half_absdiff(res.crops[0][:total], ref.crops[0]) <= PIX_TOL
            assert res.status == 0
        finally:
            st.close()


def test_bad_option_values_are_rejected():
    import paper_2502_01277_b200 as octo
    for bad in ({"std": (0.2, 0.0, 0.2)}, {"std": (0.2, -1.0, 0.2)}, {"mean": (float("nan"), 0, 0)}):
        with pytest.raises(octo.OctoError):
            octo.Stage(crop_options=[bad])
