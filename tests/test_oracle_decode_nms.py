"""Pins for the oracle's decode / score / ordering / NMS / scale-back rules.

Compared against: the logistic function in double, hand-worked rows and boxes, an exact
rational brute force over all subsets of tiny box sets, and torchvision's CPU batched_nms
on inputs whose IoUs stay clear of the threshold.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torchvision

import oracle
from oracle import DET_DTYPE

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mk(boxes, scores, classes, anchors=None):
    n = len(boxes)
    d = np.zeros(n, dtype=DET_DTYPE)
    b = np.asarray(boxes, dtype=np.float32).reshape(n, 4)
    d["x1"], d["y1"], d["x2"], d["y2"] = b[:, 0], b[:, 1], b[:, 2], b[:, 3]
    d["score"] = np.asarray(scores, dtype=np.float32)
    d["cls"] = np.asarray(classes, dtype=np.int32)
    d["anchor"] = np.arange(n, dtype=np.int32) if anchors is None else np.asarray(anchors, dtype=np.int32)
    return d


def _head_row(C, cx=100.0, cy=100.0, w=20.0, h=30.0, obj=-8.0, cls=None, fill=-8.0):
    r = np.full(5 + C, fill, dtype=np.float32)
    r[:5] = [cx, cy, w, h, obj]
    for k, v in (cls or {}).items():
        r[5 + k] = v
    return r


# ---- logistic function ------------------------------------------------------------------

def _ulp_diff(a32, ref64):
    a = np.asarray(a32, dtype=np.float32)
    ulp = np.spacing(np.abs(ref64).astype(np.float32)).astype(np.float64)
    return np.abs(a.astype(np.float64) - ref64) / ulp


def test_sigmoid_against_double():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 4, 50000), np.linspace(-30, 30, 4001),
                        rng.uniform(-1e-3, 1e-3, 1000)]).astype(np.float32)
    got = oracle.sigmoid(x)
    ref = 1.0 / (1.0 + np.exp(-x.astype(np.float64)))
    assert _ulp_diff(got, ref).max() <= 2.0


def test_sigmoid_special_values():
    s = oracle.sigmoid
    assert float(s(0.0)) == 0.5
    assert float(s(30.0)) == 1.0 and float(s(1e9)) == 1.0 and float(s(np.inf)) == 1.0
    lo = float(s(-30.0))
    assert lo == float(s(-1e9)) and abs(lo - math.exp(-30)) < 1e-6 * math.exp(-30)
    assert lo > 2.0 ** -126  # a normal number: flush-to-zero modes cannot change it
    # monotone on a fine grid around the decision region
    x = np.linspace(-3, 3, 20001).astype(np.float32)
    y = oracle.sigmoid(x)
    assert np.all(np.diff(y) >= 0)
    # symmetric values sum to one within rounding
    assert np.allclose(oracle.sigmoid(x) + oracle.sigmoid(-x), 1.0, atol=3e-7)


# ---- decode -----------------------------------------------------------------------------

def test_decode_hand_row():
    C = 80
    head = np.stack([_head_row(C), _head_row(C, cx=50, cy=60, w=20, h=10, obj=2.0, cls={17: 2.0}),
                     _head_row(C)])
    c = oracle.decode(head)
    assert len(c) == 1
    r = c[0]
    assert (r["anchor"], r["cls"]) == (1, 17)
    assert abs(float(r["score"]) - (1 / (1 + math.exp(-2))) ** 2) < 2e-7  # 0.8808^2 = 0.7758
    assert (r["x1"], r["y1"], r["x2"], r["y2"]) == (40.0, 55.0, 60.0, 65.0)


def test_decode_threshold_is_strict():
    C = 4
    head = _head_row(C, obj=0.0, cls={0: 0.0})[None]  # sigma(0)*sigma(0) = 0.25 exactly
    assert len(oracle.decode(head, conf=0.25)) == 0
    below = float(np.nextafter(np.float32(0.25), np.float32(0)))
    assert len(oracle.decode(head, conf=below)) == 1


def test_decode_argmax_tie_goes_to_lowest_class():
    C = 6
    head = _head_row(C, obj=3.0, cls={4: 2.5, 2: 2.5, 5: 1.0})[None]
    assert int(oracle.decode(head)[0]["cls"]) == 2


def test_decode_best_class_only_one_candidate_per_anchor():
    C = 6
    head = _head_row(C, obj=4.0, cls={1: 3.0, 3: 2.9})[None]
    c = oracle.decode(head)
    assert len(c) == 1 and int(c[0]["cls"]) == 1


def test_decode_probability_mode():
    C = 3
    head = np.array([[10, 10, 4, 4, 0.9, 0.1, 0.8, 0.3], [10, 10, 4, 4, 0.5, 0.5, 0.2, 0.1]], dtype=np.float32)
    c = oracle.decode(head, logits=False, conf=0.25)
    assert len(c) == 1 and int(c[0]["cls"]) == 1
    assert float(c[0]["score"]) == float(np.float32(0.9) * np.float32(0.8))


@pytest.mark.parametrize("col,val", [(0, np.nan), (1, np.inf), (2, 0.0), (2, -3.0), (3, np.nan),
                                     (4, np.nan), (5 + 2, np.nan), (5 + 1, np.inf), (3, 0.0)])
def test_decode_drops_degenerate_rows(col, val):
    C = 4
    row = _head_row(C, obj=3.0, cls={1: 3.0})
    assert len(oracle.decode(row[None])) == 1
    row[col] = val
    assert len(oracle.decode(row[None])) == 0


def test_decode_on_synthetic_head_finds_the_raised_anchors():
    import workloads
    b = workloads.make_batch("tiny")
    c = oracle.decode(b.head[0])
    h = b.head[0].astype(np.float64)
    sig = lambda v: 1 / (1 + np.exp(-v))
    score = sig(h[:, 4]) * sig(h[:, 5:].max(axis=1))
    safe = np.abs(score - 0.25) > 1e-5
    want = np.nonzero((score > 0.25) & safe)[0]
    got = c["anchor"]
    assert set(want) <= set(got) and set(got) <= set(np.nonzero((score > 0.25) | ~safe)[0])
    assert 25 <= len(c) <= 45  # 40 raised anchors, most above threshold
    assert np.allclose(c["score"], score[c["anchor"]], rtol=1e-6)
    assert np.array_equal(c["cls"], h[c["anchor"], 5:].argmax(axis=1))
    assert np.all(np.diff(c["anchor"]) > 0)


# ---- ordering ---------------------------------------------------------------------------

def test_sort_ties_by_lower_anchor():
    d = _mk([[0, 0, 1, 1]] * 4, [0.5, 0.9, 0.5, 0.7], [0, 0, 0, 0], anchors=[7, 11, 3, 5])
    s = oracle.sort_candidates(d)
    assert list(s["anchor"]) == [11, 5, 3, 7]


def test_sort_identical_rows_from_head():
    C = 4
    head = np.stack([_head_row(C) for _ in range(10)])
    head[7] = head[3] = _head_row(C, obj=2.0, cls={1: 2.0})
    head[5] = _head_row(C, obj=3.0, cls={0: 3.0})
    s = oracle.sort_candidates(oracle.decode(head)[::-1])
    assert list(s["anchor"]) == [5, 3, 7]


# ---- IoU and NMS ------------------------------------------------------------------------

@pytest.mark.parametrize("d,num,den", [(1, 81, 119), (2, 64, 136), (3, 49, 151), (5, 25, 175),
                                        (6, 16, 184), (10, 0, 200), (12, 0, 200)])
def test_iou_hand_values(d, num, den):
    a = _mk([[0, 0, 10, 10]], [1], [0])
    b = _mk([[d, d, 10 + d, 10 + d]], [1], [0])
    want = float(np.float32(num) / np.float32(den))
    assert oracle.iou(a, b) == want and oracle.iou(b, a) == want


def test_iou_asymmetric_boxes_and_degenerate():
    a = _mk([[0, 0, 4, 2]], [1], [0])
    b = _mk([[1, 1, 3, 5]], [1], [0])  # inter 2x1 = 2, areas 8 + 8, union 14
    assert oracle.iou(a, b) == float(np.float32(2) / np.float32(14))
    z = _mk([[3, 3, 3, 3]], [1], [0])
    assert oracle.iou(z, z) == 0.0  # zero union -> 0, not NaN


def _load_worked():
    rows = []
    for line in open(os.path.join(GOLDEN, "nms_worked.txt")):
        line = line.split("#")[0].split()
        if line:
            rows.append(line)
    names = [r[0] for r in rows]
    d = _mk([[float(v) for v in r[1:5]] for r in rows], [float(r[5]) for r in rows],
            [int(r[6]) for r in rows])
    return names, d


def test_nms_worked_example():
    names, d = _load_worked()
    perm = np.array([4, 2, 0, 5, 3, 1])  # scrambled input order
    s = oracle.sort_candidates(d[perm])
    keep = oracle.nms(s, 0.45, 300)
    assert [names[a] for a in s["anchor"][keep]] == ["A", "F", "D", "E"]
    assert [names[a] for a in s["anchor"][oracle.nms(s, 0.45, 2)]] == ["A", "F"]  # cap
    assert [names[a] for a in s["anchor"][oracle.nms(s, 0.9, 300)]] == ["A", "B", "F", "C", "D", "E"]


def test_nms_threshold_is_strict():
    a = [0, 0, 10, 10]
    b = [0, 0, 10, 5]  # IoU exactly 0.5
    s = oracle.sort_candidates(_mk([a, b], [0.9, 0.8], [0, 0]))
    assert len(oracle.nms(s, 0.5, 10)) == 2
    assert len(oracle.nms(s, float(np.nextafter(np.float32(0.5), np.float32(0))), 10)) == 1


def _exact_iou(a, b):
    iw = max(0, min(a[2], b[2]) - max(a[0], b[0]))
    ih = max(0, min(a[3], b[3]) - max(a[1], b[1]))
    inter = iw * ih
    uni = (a[2] - a[0]) * (a[3] - a[1]) + (b[2] - b[0]) * (b[3] - b[1]) - inter
    return Fraction(inter, uni) if uni > 0 else Fraction(0)


def _characterised_sets(boxes, classes, thr, max_det):
    """All subsets K of positions (boxes already in score order) such that (i) no member is
    overlapped (> thr, same class) by an earlier member and (ii) every non-member before the
    cap point is overlapped by an earlier member.  Exact rational arithmetic."""
    n = len(boxes)
    over = [[classes[i] == classes[j] and _exact_iou(boxes[i], boxes[j]) > thr for j in range(n)]
            for i in range(n)]
    sols = []
    for bits in range(1 << n):
        K = [i for i in range(n) if bits >> i & 1]
        if len(K) > max_det:
            continue
        ok = all(not any(over[j][i] for j in K if j < i) for i in K)
        if not ok:
            continue
        last = K[-1] if len(K) == max_det and K else n  # positions after the cap are unconstrained
        limit = n if len(K) < max_det else last
        ok = all(any(over[j][i] for j in K if j < i) for i in range(limit) if i not in K)
        if ok:
            sols.append(K)
    return sols


@pytest.mark.parametrize("thr_num,thr_den", [(1, 2), (9, 20), (1, 4)])
def test_nms_brute_force_tiny_sets(thr_num, thr_den):
    rng = np.random.default_rng(thr_den)
    thr = Fraction(thr_num, thr_den)
    thr32 = float(np.float32(thr_num / thr_den))
    done = 0
    while done < 150:
        n = int(rng.integers(1, 9))
        xy = rng.integers(0, 7, size=(n, 2))
        wh = rng.integers(2, 7, size=(n, 2))
        boxes = [(int(x), int(y), int(x + w), int(y + h)) for (x, y), (w, h) in zip(xy, wh)]
        classes = [int(v) for v in rng.integers(0, 2, size=n)]
        # skip sets with a pair so close to the threshold that binary32 rounding decides
        if any(abs(float(_exact_iou(a, b)) - float(thr)) < 1e-6 and _exact_iou(a, b) != thr
               for a, b in itertools.combinations(boxes, 2)):
            continue
        if thr_den == 20 and any(_exact_iou(a, b) == thr for a, b in itertools.combinations(boxes, 2)):
            continue  # 9/20 is not a binary32 number: fl(9/20) == fl(0.45) while 9/20 > fl(0.45)
        max_det = int(rng.integers(1, n + 2))
        scores = np.sort(rng.random(n).astype(np.float32))[::-1]
        sols = _characterised_sets(boxes, classes, thr, max_det)
        assert len(sols) == 1
        order = rng.permutation(n)
        d = _mk([boxes[i] for i in order], scores[order], [classes[i] for i in order], anchors=order)
        s = oracle.sort_candidates(d)
        assert list(s["anchor"]) == list(range(n))
        keep = oracle.nms(s, thr32, max_det)
        assert list(keep) == sols[0]
        done += 1


def test_nms_matches_torchvision_on_margin_safe_inputs():
    rng = np.random.default_rng(5)
    for trial in range(20):
        n = 300
        cxy = rng.uniform(50, 400, size=(n, 2)).astype(np.float32)
        # centres cluster so that overlaps are frequent
        cxy[: n // 2] = cxy[n // 2:][rng.integers(0, n - n // 2, n // 2)] + rng.normal(0, 6, (n // 2, 2))
        wh = rng.uniform(20, 80, size=(n, 2)).astype(np.float32)
        boxes = np.concatenate([cxy - wh / 2, cxy + wh / 2], axis=1).astype(np.float32)
        classes = rng.integers(0, 3, n)
        scores = rng.permutation(n).astype(np.float32) / n + 0.001
        tb = torch.from_numpy(boxes.astype(np.float64))
        ious = torchvision.ops.box_iou(tb, tb).numpy()
        same = classes[:, None] == classes[None, :]
        bad = (np.abs(ious - 0.45) < 1e-4) & same
        np.fill_diagonal(bad, False)
        drop = np.unique(np.nonzero(bad)[0])
        sel = np.setdiff1d(np.arange(n), drop)
        boxes, classes, scores = boxes[sel], classes[sel], scores[sel]
        ref = torchvision.ops.batched_nms(torch.from_numpy(boxes), torch.from_numpy(scores),
                                          torch.from_numpy(classes), 0.45).numpy()
        s = oracle.sort_candidates(_mk(boxes, scores, classes))
        keep = oracle.nms(s, 0.45, 10 ** 6)
        assert list(s["anchor"][keep]) == list(ref)
        assert len(keep) < len(sel)  # the case really suppresses something


def test_nms_invariants_on_dense_synthetic_head():
    import workloads
    b = workloads.make_batch("dense_nms", batch=1)
    w, h = b.sizes[0]
    dets, ncand = oracle.postprocess_image(b.head[0], w, h, 640, max_det=1000)
    assert 4000 <= ncand <= 5200
    assert 200 <= len(dets) <= 1000
    assert np.all(np.diff(dets["score"]) <= 0)
    # no two kept boxes of a class overlap above the threshold (checked in letterbox space,
    # in double, on the un-scaled candidates)
    c = oracle.sort_candidates(oracle.decode(b.head[0]))
    keep = oracle.nms(c, 0.45, 1000)
    k = c[keep]
    tb = torch.from_numpy(np.stack([k["x1"], k["y1"], k["x2"], k["y2"]], 1).astype(np.float64))
    ious = torchvision.ops.box_iou(tb, tb).numpy()
    same = k["cls"][:, None] == k["cls"][None, :]
    np.fill_diagonal(same, False)
    assert ious[same].max() <= 0.45 + 1e-6
    # every dropped candidate ranked before the last kept one is covered by an earlier kept one
    kept_set = set(int(i) for i in keep)
    allb = torch.from_numpy(np.stack([c["x1"], c["y1"], c["x2"], c["y2"]], 1).astype(np.float64))
    cover = torchvision.ops.box_iou(allb, tb).numpy()
    last = int(keep[-1])
    for i in range(last):
        if i in kept_set:
            continue
        earlier = keep < i
        hit = (cover[i] > 0.45 - 1e-6) & earlier & (k["cls"] == c["cls"][i])
        assert hit.any()


# ---- scale-back -------------------------------------------------------------------------

def test_scale_back_hand_case_1080p():
    d = _mk([[100, 200, 160, 260]], [0.9], [0])
    out = oracle.scale_back(d, 1920, 1080, 640)[0]
    assert (out["x1"], out["y1"], out["x2"], out["y2"]) == (300.0, 180.0, 480.0, 360.0)


def test_scale_back_clamps_to_frame():
    d = _mk([[-20, 100, 700, 620]], [0.9], [0])
    out = oracle.scale_back(d, 1920, 1080, 640)[0]
    assert (out["x1"], out["y1"], out["x2"], out["y2"]) == (0.0, 0.0, 1920.0, 1080.0)


def test_scale_back_portrait_and_inexact_gain():
    # 1080x1920 portrait: nw=360, pad_left=140, gain 3 in both axes
    d = _mk([[150, 10, 200, 30]], [0.9], [0])
    out = oracle.scale_back(d, 1080, 1920, 640)[0]
    assert (out["x1"], out["y1"], out["x2"], out["y2"]) == (30.0, 30.0, 180.0, 90.0)
    # 1000x600 -> 640x384, pad_top 128, gain 1.5625 exactly
    d = _mk([[64, 160, 128, 224]], [0.9], [0])
    out = oracle.scale_back(d, 1000, 600, 640)[0]
    assert (out["x1"], out["y1"], out["x2"], out["y2"]) == (100.0, 50.0, 200.0, 150.0)
    # 1366x768 -> gain is not a binary32 number; compare with double within 1e-4 relative
    nw, nh, pl, pt = oracle.letterbox_geometry(1366, 768, 640)
    d = _mk([[101.3, 277.7, 333.1, 401.9]], [0.9], [0])
    out = oracle.scale_back(d, 1366, 768, 640)[0]
    want = [(float(d["x1"][0]) - pl) * 1366 / nw, (float(d["y1"][0]) - pt) * 768 / nh,
            (float(d["x2"][0]) - pl) * 1366 / nw, (float(d["y2"][0]) - pt) * 768 / nh]
    got = [float(out[k]) for k in ("x1", "y1", "x2", "y2")]
    assert np.allclose(got, want, rtol=1e-6)


def test_chained_stage_maps_boxes_into_the_upstream_rectangle():
    """Second-level stage: a 180x180 rectangle at (300, 180) stretched to 256x256; gain 180/256 =
    0.703125 is a binary32 number, so the hand values are exact."""
    C = 4
    head = np.stack([_head_row(C, cx=128, cy=192, w=128, h=128, obj=3.0, cls={2: 3.0}),   # (64,128)-(192,256)
                     _head_row(C, cx=10, cy=250, w=60, h=40, obj=2.0, cls={1: 2.0})])     # pokes out left / bottom
    dets, ncand = oracle.postprocess_region(head, (300, 180, 480, 360), 256)
    assert ncand == 2 and len(dets) == 2
    a, b = dets[0], dets[1]
    assert (a["x1"], a["y1"], a["x2"], a["y2"]) == (345.0, 270.0, 435.0, 360.0)
    # (-20,230)-(40,270) -> x: 300 - 14.06 -> clamped to 300 ; 300 + 28.125 ; y: 180 + 161.71875 ; clamped to 360
    assert (b["x1"], b["x2"], b["y2"]) == (300.0, 328.125, 360.0)
    assert float(b["y1"]) == 180.0 + 230 * 0.703125
    # the region of a first-level stage is the whole frame: same numbers as scale_back
    d1, _ = oracle.postprocess_image(head, 256, 256, 256)
    d2, _ = oracle.postprocess_region(head, (0, 0, 256, 256), 256)
    assert d1.tobytes() == d2.tobytes()


def test_class_agnostic_variant_worked_example_and_library():
    """Decode variant: NMS across classes.  In the worked example D (class 1) has B's box, which
    overlaps A by 0.681, so it dies as soon as classes are ignored: kept A, F, E."""
    names, d = _load_worked()
    s = oracle.sort_candidates(d)
    assert [names[a] for a in s["anchor"][oracle.nms(s, 0.45, 300, agnostic=True)]] == ["A", "F", "E"]
    assert [names[a] for a in s["anchor"][oracle.nms(s, 0.45, 300)]] == ["A", "F", "D", "E"]
    rng = np.random.default_rng(15)
    for trial in range(10):
        n = 250
        cxy = rng.uniform(50, 300, size=(n, 2)).astype(np.float32)
        wh = rng.uniform(20, 80, size=(n, 2)).astype(np.float32)
        boxes = np.concatenate([cxy - wh / 2, cxy + wh / 2], axis=1).astype(np.float32)
        classes = rng.integers(0, 5, n)
        scores = rng.permutation(n).astype(np.float32) / n + 0.001
        tb = torch.from_numpy(boxes.astype(np.float64))
        ious = torchvision.ops.box_iou(tb, tb).numpy()
        bad = np.abs(ious - 0.45) < 1e-4
        np.fill_diagonal(bad, False)
        sel = np.setdiff1d(np.arange(n), np.unique(np.nonzero(bad)[0]))
        boxes, classes, scores = boxes[sel], classes[sel], scores[sel]
        ref = torchvision.ops.nms(torch.from_numpy(boxes), torch.from_numpy(scores), 0.45).numpy()
        c = oracle.sort_candidates(_mk(boxes, scores, classes))
        keep = oracle.nms(c, 0.45, 10 ** 6, agnostic=True)
        assert list(c["anchor"][keep]) == list(ref)
        assert len(keep) < len(oracle.nms(c, 0.45, 10 ** 6))  # fewer survive than with classes
