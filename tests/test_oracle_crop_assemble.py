"""Pins for the oracle's crop rectangle, ROI crop-resize and batch assembler, plus
whole-stage invariants on the synthetic workloads."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from oracle import DET_DTYPE


def _det(x1, y1, x2, y2, cls=0, score=0.9):
    d = np.zeros(1, dtype=DET_DTYPE)
    d["x1"], d["y1"], d["x2"], d["y2"], d["cls"], d["score"] = x1, y1, x2, y2, cls, score
    return d


# ---- crop rectangle ---------------------------------------------------------------------

@pytest.mark.parametrize("box,wh,rect", [
    ((300.0, 180.0, 480.0, 360.0), (1920, 1080), (300, 180, 480, 360)),
    ((300.25, 180.75, 479.5, 359.01), (1920, 1080), (300, 180, 480, 360)),  # floor / ceil outward
    ((0.0, 0.0, 1920.0, 1080.0), (1920, 1080), (0, 0, 1920, 1080)),
    ((1920.0, 1080.0, 1920.0, 1080.0), (1920, 1080), (1919, 1079, 1920, 1080)),  # clamped box at the far corner
    ((0.0, 0.0, 0.0, 0.0), (1920, 1080), (0, 0, 1, 1)),
    ((10.5, 20.5, 10.6, 20.6), (64, 64), (10, 20, 11, 21)),
    ((10.0, 20.0, 10.0, 20.0), (64, 64), (10, 20, 11, 21)),  # empty box still yields one pixel
])
def test_crop_rect_hand_cases(box, wh, rect):
    assert oracle.crop_rect(_det(*box), *wh) == rect


def test_crop_rect_always_inside_frame():
    rng = np.random.default_rng(2)
    for _ in range(3000):
        w, h = int(rng.integers(1, 300)), int(rng.integers(1, 300))
        x = np.sort(rng.uniform(-50, w + 50, 2))
        y = np.sort(rng.uniform(-50, h + 50, 2))
        # detections are clamped to the frame before they reach the crop stage
        x, y = np.clip(x, 0, w), np.clip(y, 0, h)
        r = oracle.crop_rect(_det(x[0], y[0], x[1], y[1]), w, h)
        assert 0 <= r[0] < r[2] <= w and 0 <= r[1] < r[3] <= h
        assert r[0] <= x[0] or r[0] == w - 1
        assert r[2] >= x[1] or r[2] == r[0] + 1


# ---- crop -------------------------------------------------------------------------------

def test_crop_identity_on_integer_box():
    rng = np.random.default_rng(11)
    img = rng.integers(0, 256, size=(90, 120, 3), dtype=np.uint8)
    out = oracle.crop(img, 120, 90, _det(17, 9, 17 + 32, 9 + 24), 32, 24)
    want = (img[9:33, 17:49, ::-1].astype(np.float64) / 255).astype(np.float16).view(np.uint16)
    assert np.array_equal(out, want.transpose(2, 0, 1))


def test_crop_full_frame_equals_resize_of_frame():
    rng = np.random.default_rng(12)
    img = rng.integers(0, 256, size=(45, 80, 3), dtype=np.uint8)
    out = oracle.crop(img, 80, 45, _det(0, 0, 80, 45), 64, 64, swap_rb=False)
    core = oracle.resize_f64(img, (0, 0, 80, 45), 64, 64)
    assert np.array_equal(out, (core / 255).astype(np.float16).view(np.uint16))


def test_crop_matches_library_cut_then_resize():
    rng = np.random.default_rng(13)
    img = rng.integers(0, 256, size=(100, 140, 3), dtype=np.uint8)
    d = _det(20.3, 10.9, 97.2, 71.5)
    rx0, ry0, rx1, ry1 = oracle.crop_rect(d, 140, 100)
    assert (rx0, ry0, rx1, ry1) == (20, 10, 98, 72)
    out = oracle.crop(img, 140, 100, d, 56, 40).view(np.float16).astype(np.float64)
    t = torch.from_numpy(img[ry0:ry1, rx0:rx1, ::-1].astype(np.float64).copy()).permute(2, 0, 1)[None]
    ref = torch.nn.functional.interpolate(t, size=(40, 56), mode="bilinear", align_corners=False)[0].numpy() / 255
    assert np.array_equal(out, ref.astype(np.float16).astype(np.float64))


def test_crop_one_pixel_rectangle_is_constant():
    img = np.zeros((8, 8, 3), dtype=np.uint8)
    img[3, 5] = (10, 20, 30)
    out = oracle.crop(img, 8, 8, _det(5.2, 3.2, 5.3, 3.3), 8, 8).view(np.float16)
    assert np.all(out[0] == np.float16(30 / 255)) and np.all(out[2] == np.float16(10 / 255))


# ---- assembler --------------------------------------------------------------------------

def _dets_with_classes(per_frame, max_det):
    d = np.zeros((len(per_frame), max_det), dtype=DET_DTYPE)
    for n, cl in enumerate(per_frame):
        d["cls"][n, : len(cl)] = cl
        d["cls"][n, len(cl):] = 1  # stale records beyond the count must be ignored
    return d, np.array([len(c) for c in per_frame], dtype=np.int32)


def test_assemble_hand_case():
    d, c = _dets_with_classes([[0, 1, 2], [], [3, 4]], 5)
    off, items, (packed, total) = oracle.assemble(d, c, 5)
    assert list(off) == [0, 3, 3, 5] and (packed, total) == (5, 5)
    assert items.tolist() == [[0, 0], [0, 1], [0, 2], [2, 0], [2, 1]]
    off, items, (packed, total) = oracle.assemble(d, c, 5, first_item=2, max_items=2)
    assert list(off) == [0, 3, 3, 5] and (packed, total) == (2, 5)
    assert items.tolist() == [[0, 2], [2, 0]]
    off, items, (packed, total) = oracle.assemble(d, c, 5, first_item=4, max_items=8)
    assert (packed, total) == (1, 5) and items.tolist() == [[2, 1]]
    off, items, (packed, total) = oracle.assemble(d, c, 5, first_item=9, max_items=8)
    assert (packed, total) == (0, 5)


def test_assemble_class_mask():
    d, c = _dets_with_classes([[0, 33, 2, 33], [33], [2, 2]], 4)
    mask33 = [0, 1 << 1, 0, 0]
    off, items, (packed, total) = oracle.assemble(d, c, 4, class_mask=mask33)
    assert list(off) == [0, 2, 3, 3] and total == 3
    assert items.tolist() == [[0, 1], [0, 3], [1, 0]]
    off, items, (packed, total) = oracle.assemble(d, c, 4, class_mask=[0, 0, 0, 0])
    assert list(off) == [0, 0, 0, 0] and (packed, total) == (0, 0)


def test_assemble_all_zero_counts():
    d, c = _dets_with_classes([[], [], []], 3)
    off, items, n = oracle.assemble(d, c, 3)
    assert list(off) == [0, 0, 0, 0] and n == (0, 0) and len(items) == 0


# ---- whole stage on the synthetic workloads ----------------------------------------------

def test_stage_tiny_invariants():
    b = workloads.make_batch("tiny")
    wl = b.workload
    r = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det)
    k = int(r.counts[0])
    assert 20 <= k <= 40 and r.n_cand[0] >= k
    d = r.dets[0, :k]
    assert np.all(np.diff(d["score"]) <= 0)
    assert np.all((d["x1"] >= 0) & (d["x2"] <= 320) & (d["y1"] >= 0) & (d["y2"] <= 240))
    assert list(r.offsets[0]) == [0, k]
    assert np.all((r.rects[0][:, 0] >= 0) & (r.rects[0][:, 2] <= 320) & (r.rects[0][:, 0] < r.rects[0][:, 2]))
    assert np.all((r.rects[0][:, 1] >= 0) & (r.rects[0][:, 3] <= 240) & (r.rects[0][:, 1] < r.rects[0][:, 3]))
    assert r.crops[0].shape == (k, 3, 64, 64)
    # letterbox of the tiny frame: scale 1 -> interior is an exact copy
    img = b.frames[0][:, :960].reshape(240, 320, 3)
    want = (img[:, :, ::-1].astype(np.float64) / 255).astype(np.float16).view(np.uint16).transpose(2, 0, 1)
    assert np.array_equal(r.det_in[0][:, 40:280], want)


def test_stage_two_branch_packing_consistent():
    b = workloads.make_batch("two_branch", batch=6)
    wl = b.workload
    assert len(set(b.sizes)) == 2  # the batch really mixes 720p and 1080p
    r = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                         do_letterbox=False, do_crops=False, threads=4)
    for br in range(2):
        assert np.array_equal(np.diff(r.offsets[br]), r.counts)
        assert len(r.items[br]) == int(r.counts.sum())
    assert np.array_equal(r.items[0], r.items[1])
    for (f, j), rect in zip(r.items[0], r.rects[0]):
        w, h = b.sizes[f]
        assert 0 <= rect[0] < rect[2] <= w and 0 <= rect[1] < rect[3] <= h


def test_margin_report_on_the_workloads(capsys):
    """How close the synthetic workloads come to a flipped decision (double precision).  Bit
    exactness of the CUDA path rests on the fixed binary32 formulas, not on wide margins: in
    the dense scene neighbouring scores are a few ulps apart."""
    rows = []
    for name in ("tiny", "traffic_1080p", "dense_nms", "sweep"):
        b = workloads.make_batch(name, batch=1)
        r = oracle.margin_report(b.head[0])
        rows.append((name, r))
        assert r["candidates"] > 0 and r["min_abs_score_minus_conf"] > 0 and r["min_score_gap"] >= 0
        assert np.isfinite(r["min_abs_iou_minus_thr"])
    with capsys.disabled():
        for name, r in rows:
            print(f"\n  margins {name}: cand={r['candidates']} |score-conf|>={r['min_abs_score_minus_conf']:.3e} "
                  f"score gap>={r['min_score_gap']:.3e} |IoU-thr|>={r['min_abs_iou_minus_thr']:.3e}", end="")


def test_queue_hand_case():
    """FIFO across pushes, newest dropped at capacity, oldest-pending stamp: worked by hand."""
    q = oracle.OracleQueue(capacity=5)
    q.push([(0, 0), (0, 1), (2, 0)], [(0, 0, 1, 1)] * 3, ["a", "b", "c"])          # seq 0: 3 items
    q.push([(1, 0), (1, 1), (1, 2)], [(0, 0, 2, 2)] * 3, ["d", "e", "f"])          # seq 1: 2 fit, 1 dropped
    recs, info = q.pop(2)
    assert [(r[0], r[1], r[2]) for r in recs] == [(0, 0, 0), (0, 0, 1)] and info == (2, 3, 1, 0)
    q.push([(0, 0)], [(1, 1, 3, 3)], ["g"])                                         # seq 2
    recs, info = q.pop(3)
    assert [(r[0], r[1], r[2], r[4]) for r in recs] == [(0, 2, 0, "c"), (1, 1, 0, "e"), (1, 1, 1, "e")]
    assert info == (3, 1, 1, 2)
    recs, info = q.pop(4)
    assert [(r[0], r[3]) for r in recs] == [(2, (1, 1, 3, 3))] and info == (1, 0, 1, -1)
    assert q.pop(2) == ([], (0, 0, 1, -1))


def test_queue_release_rule_hand_case():
    """A batch is released when full, or when its first item has waited max_wait pushes: by hand."""
    q = oracle.OracleQueue(capacity=16)
    q.push([(0, 0), (0, 1)], [(0, 0, 1, 1)] * 2, ["a"])            # push 0: 2 items, waited 0
    assert q.pop(4, max_wait=2) == ([], (0, 2, 0, 0))               # not full, head waited 0 pushes
    q.push([(0, 0)], [(0, 0, 1, 1)], ["b"])                        # push 1: 3 pending, head waited 1
    assert q.pop(4, max_wait=2)[1] == (0, 3, 0, 0)
    q.push([], [], [])                                             # push 2 (an empty batch): head waited 2
    recs, info = q.pop(4, max_wait=2)
    assert [(r[0], r[2]) for r in recs] == [(0, 0), (0, 1), (1, 0)] and info == (3, 0, 0, -1)
    assert q.pop(4, max_wait=0) == ([], (0, 0, 0, -1))              # nothing pending: nothing due
    q.push([(0, k) for k in range(5)], [(0, 0, 1, 1)] * 5, ["c"])  # push 3: a full batch is due at once
    recs, info = q.pop(4, max_wait=9)
    assert len(recs) == 4 and info == (4, 1, 0, 3)
    assert q.pop(4, max_wait=0)[1] == (1, 0, 0, -1)                 # max_wait 0: any pending item is due
