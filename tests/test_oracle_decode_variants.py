"""Pins of the oracle's decode variants (planes layout, multi-label candidates).  CPU only.

The variants are tied to the already pinned row decode by reductions that hold exactly
(sigma(30) == 1.0f, probability 1.0 as the objectness factor), to hand-worked rows evaluated in
double precision, and to a numpy evaluation of the synthetic heads."""
import numpy as np

import workloads
from oracle import oracle as o


def _sig(x):
    return 1.0 / (1.0 + np.exp(-np.asarray(x, dtype=np.float64)))


def _rows(n, c=6, seed=0):
    rng = np.random.default_rng(seed)
    h = np.empty((n, 5 + c), dtype=np.float32)
    h[:, 0:2] = rng.uniform(0, 320, (n, 2))
    h[:, 2:4] = rng.uniform(8, 120, (n, 2))
    h[:, 4:] = rng.normal(-1.0, 2.0, (n, 1 + c))
    return h


def test_planes_decode_equals_row_decode_with_unit_objectness():
    """sigma(30) is exactly 1.0f, so a row head whose obj logit is 30 scores fl(1 * sigma(c)) =
    sigma(c): the planes rule.  Same for probabilities with obj = 1."""
    assert o.sigmoid(np.float32(30.0)) == np.float32(1.0)
    h = _rows(500, c=7, seed=1)
    for logits in (True, False):
        hr = h.copy()
        if not logits:
            hr[:, 4:] = _sig(hr[:, 4:]).astype(np.float32)
        hr[:, 4] = 30.0 if logits else 1.0
        want = o.decode(hr, logits=logits, conf=0.25)
        got = o.decode(workloads.rows_to_planes(hr), logits=logits, conf=0.25, layout="planes")
        assert len(want) > 20 and np.array_equal(got, want)


def test_planes_layout_indexing_is_value_major():
    """Element e of anchor a sits at [e, a]: a head built by hand, one candidate."""
    a, c = 5, 3
    hp = np.full((4 + c, a), -9.0, dtype=np.float32)
    hp[0:4, :] = [[10.0] * a, [20.0] * a, [4.0] * a, [6.0] * a]
    hp[4 + 2, 3] = 3.0  # class 2 of anchor 3
    got = o.decode(hp, layout="planes")
    assert len(got) == 1
    d = got[0]
    assert (d["anchor"], d["cls"]) == (3, 2)
    assert (d["x1"], d["y1"], d["x2"], d["y2"]) == (8.0, 17.0, 12.0, 23.0)
    assert abs(float(d["score"]) - float(_sig(3.0))) < 1e-6


def test_multi_label_hand_row():
    """obj logit 2, class logits (2, 1, -5): scores .8808*.8808, .8808*.7311, .8808*.0067."""
    h = np.zeros((3, 5 + 3), dtype=np.float32)
    h[:, 0:4] = [50, 60, 10, 20]
    h[:, 4:] = -9.0
    h[1, 4:] = [2.0, 2.0, 1.0, -5.0]
    got = o.decode(h, multi_label=True)
    assert [(int(d["anchor"]), int(d["cls"])) for d in got] == [(1, 0), (1, 1)]
    want = _sig(2.0) * _sig([2.0, 1.0])
    assert np.allclose(got["score"], want, rtol=0, atol=1e-6)
    assert abs(want[0] - 0.7758) < 1e-4 and abs(want[1] - 0.6439) < 1e-4
    for f, v in (("x1", 45.0), ("y1", 50.0), ("x2", 55.0), ("y2", 70.0)):
        assert np.all(got[f] == v)
    # the single-label rule keeps only the best class of that anchor
    one = o.decode(h)
    assert len(one) == 1 and one[0]["cls"] == 0 and one[0]["score"] == got[0]["score"]


def test_multi_label_against_numpy_and_single_label():
    for layout in ("rows", "planes"):
        h = _rows(3000, c=9, seed=3)
        hd = h if layout == "rows" else workloads.rows_to_planes(h)
        cls = _sig(h[:, 5:])
        score = cls * (_sig(h[:, 4:5]) if layout == "rows" else 1.0)
        # values within 1e-6 of the threshold (binary32 rounding could decide either way) are
        # taken out of the head; every remaining decision is clear in double precision
        close = np.abs(score - 0.25) < 1e-6
        h[:, 5:][close] = -9.0
        hd = h if layout == "rows" else workloads.rows_to_planes(h)
        score = np.where(close, 0.0, score)
        want = np.argwhere(score > 0.25)  # (anchor, class) in row-major order
        got = o.decode(hd, conf=0.25, layout=layout, multi_label=True)
        assert len(want) > 100
        assert np.array_equal(np.stack([got["anchor"], got["cls"]], 1), want)
        assert np.allclose(got["score"], score[want[:, 0], want[:, 1]], rtol=0, atol=2e-7)
        # single label = the first best-scoring class of each anchor that has any candidate
        one = o.decode(hd, conf=0.25, layout=layout)
        assert np.array_equal(one["anchor"], np.unique(want[:, 0]))
        for d in one[:200]:
            m = got[got["anchor"] == d["anchor"]]
            assert d["score"] == m["score"].max()


def test_multi_label_degenerate_anchor_drops_all_its_classes():
    h = np.zeros((2, 5 + 2), dtype=np.float32)
    h[:, 0:4] = [50, 60, 10, 20]
    h[:, 4:] = 3.0
    h[1, 6] = np.nan
    got = o.decode(h, multi_label=True)
    assert [(int(d["anchor"]), int(d["cls"])) for d in got] == [(0, 0), (0, 1)]
    hp = workloads.rows_to_planes(h)
    got = o.decode(hp, layout="planes", multi_label=True)
    assert [(int(d["anchor"]), int(d["cls"])) for d in got] == [(0, 0), (0, 1)]
    hp[2, 0] = 0.0  # w = 0
    assert len(o.decode(hp, layout="planes", multi_label=True)) == 0


def test_order_breaks_score_and_anchor_ties_by_class():
    c = np.zeros(3, dtype=o.DET_DTYPE)
    c["score"] = [0.5, 0.5, 0.5]
    c["anchor"] = [4, 4, 2]
    c["cls"] = [7, 3, 9]
    s = o.sort_candidates(c)
    assert [(int(d["anchor"]), int(d["cls"])) for d in s] == [(2, 9), (4, 3), (4, 7)]


def test_multi_label_nms_keeps_both_classes_of_one_anchor():
    """Two classes of one anchor share a box (IoU 1) but never suppress each other under
    class-aware NMS; a weaker same-class neighbour is suppressed by each of them."""
    h = np.full((3, 5 + 2), -9.0, dtype=np.float32)
    h[0, :] = [100, 100, 40, 40, 3.0, 3.0, 2.0]    # classes 0 and 1
    h[1, :] = [102, 100, 40, 40, 2.0, 1.0, -9.0]   # class 0, IoU with row 0 = 38/42 > 0.45
    h[2, :] = [300, 300, 40, 40, 2.0, -9.0, 2.5]   # class 1, far away
    dets, ncand = o.postprocess_image(h, 640, 640, 640, multi_label=True)
    assert ncand == 4
    assert [(int(d["anchor"]), int(d["cls"])) for d in dets] == [(0, 0), (0, 1), (2, 1)]
    assert dets["score"][0] > dets["score"][1] > dets["score"][2]


def test_anchor_free_workload_counts():
    b = workloads.make_batch("anchor_free", batch=2)
    wl = b.workload
    assert b.head.shape == (2, 4 + wl.num_classes, 8400)
    for i in range(2):
        dets, ncand = o.postprocess_image(b.head[i], 1920, 1080, 640, layout="planes")
        assert ncand == wl.n_raised and 15 <= len(dets) <= 60
        assert np.all(np.diff(dets["score"]) <= 0)


def test_chained_stage_with_planes_head_reduces_to_the_row_form():
    """A chained stage's planes head equals the row head with unit objectness (sigma(30) == 1.0f):
    same detections, mapped into the same upstream rectangle."""
    h = workloads.make_heads(77, 2, 256, num_classes=6, n_raised=14, n_groups=4)
    h[:, :, 4] = 30.0
    for i in range(2):
        region = (10 + i, 20, 200, 150 + i)
        want, nw = o.postprocess_region(h[i], region, 256, max_det=12)
        got, ng = o.postprocess_region(workloads.rows_to_planes(h[i]), region, 256, max_det=12, layout="planes")
        assert nw == ng and len(want) > 3 and np.array_equal(got, want)
        assert np.all((want["x1"] >= region[0]) & (want["x2"] <= region[2]))
