"""GPU parity of the decode variants (planes-layout heads, multi-label candidates) against the
CPU oracle, through the C ABI.  Same bar as the main parity tests: kept anchors, classes, order,
counts, packing and rectangles bit-exact, scores and corners bit-equal, crops within 2e-3."""
import os
from dataclasses import replace

import numpy as np
import pytest

import oracle
import workloads
from gpu_harness import half_absdiff, make_stage, run_stage_gpu
from test_gpu_parity import PIX_TOL, _check_branch, _check_dets, _oracle

pytestmark = pytest.mark.gpu


def _compare(b, head=None, num_anchors=None, max_items=None, **oracle_kw):
    wl = b.workload
    head = b.head if head is None else head
    over = {} if num_anchors is None else {"num_anchors": num_anchors}
    st = make_stage(wl, b.n, **over)
    try:
        b2 = replace(b, head=head)
        ref = _oracle(b2, do_letterbox=False, **oracle_kw)
        cap = [int(len(ref.items[k])) + 2 for k in range(len(wl.branches))] if max_items is None else max_items
        res = run_stage_gpu(st, b.frames, b.sizes, head, max_items=cap)
        _check_dets(res, ref)
        for k in range(len(wl.branches)):
            _check_branch(res, ref, k, max_items=cap[k])
        return res, ref
    finally:
        st.close()


def _small(layout, multi_label=False, batch=2, seed=21, **over):
    base = workloads.WORKLOADS["anchor_free" if layout == "planes" else "traffic_1080p"]
    wl = replace(base, n_raised=150, n_groups=20, frame_sizes=((640, 360),), branches=((64, 64),),
                 multi_label=multi_label, **over)
    return workloads.make_batch(wl, batch=batch, seed=seed)


def _raise_second_class(b, every=3):
    """Give every `every`-th raised anchor a second (and sometimes third) strong class."""
    h = b.head
    planes = b.workload.head_layout == "planes"
    for i in range(b.n):
        cls = h[i, 4:, :].T if planes else h[i, :, 5:]  # view [A, C]
        raised = np.nonzero(cls.max(axis=1) > 0)[0]
        for j, a in enumerate(raised[::every]):
            k = int(cls[a].argmax())
            cls[a, (k + 1) % cls.shape[1]] = cls[a, k] - 0.25
            if j % 2:
                cls[a, (k + 5) % cls.shape[1]] = cls[a, k] - 0.5
    return b


def test_config_anchor_free():
    """Planes layout [n, 4 + C, A] end to end on the anchor-free workload (vector-load path)."""
    b = workloads.make_batch("anchor_free", batch=4)
    res, ref = _compare(b)
    assert res.status == 0
    assert int(ref.n_cand.min()) == b.workload.n_raised and int(ref.counts.min()) > 10
    assert res.stats["candidates"] == int(ref.n_cand.sum())


def test_planes_scalar_path_and_probabilities():
    """A not a multiple of four takes the scalar-load kernel; probability form of the head."""
    b = _small("planes", logits=False)
    assert 0.0 <= b.head[:, 4:].min() and b.head[:, 4:].max() <= 1.0
    a = b.workload.num_anchors - 3
    head = np.ascontiguousarray(b.head[:, :, :a])
    res, ref = _compare(b, head=head, num_anchors=a)
    assert int(ref.counts.min()) > 5


def test_planes_nonfinite_and_degenerate_anchors():
    b = _small("planes", batch=1)
    h = b.head
    raised = np.nonzero(h[0, 4:].max(axis=0) > 0)[0]
    h[0, 0, raised[0]] = np.nan          # cx
    h[0, 3, raised[1]] = np.inf          # h
    h[0, 2, raised[2]] = 0.0             # w = 0
    h[0, 3, raised[3]] = -4.0            # h < 0
    h[0, 4 + 17, raised[4]] = np.nan     # one class value
    h[0, 4 + 3, 11] = -np.inf            # background anchor with a non-finite class value
    res, ref = _compare(b)
    assert res.status & 0x1
    kept = set(ref.dets[0, :ref.counts[0]]["anchor"].tolist())
    assert not (set(raised[:5].tolist()) & kept) and len(kept) > 5


@pytest.mark.parametrize("layout", ["rows", "planes"])
def test_multi_label_candidates(layout):
    b = _raise_second_class(_small(layout, multi_label=True, batch=3))
    res, ref = _compare(b)
    one = _oracle(replace(b, workload=replace(b.workload, multi_label=False)), do_letterbox=False, do_crops=False)
    assert int(ref.n_cand.sum()) > int(one.n_cand.sum()) + 40
    assert res.stats["candidates"] == int(ref.n_cand.sum())
    # some anchor appears with two classes among the kept detections
    d = ref.dets[0, :ref.counts[0]]
    assert len(set(d["anchor"].tolist())) < len(d)
    assert res.status == 0


def test_multi_label_probability_rows_with_ties():
    """Probability head; two classes of one anchor with the same value tie in score and are
    ordered by class."""
    b = _raise_second_class(_small("rows", multi_label=True, batch=1, logits=False))
    h = b.head
    # anchors that survive NMS under their own best class: their tied second class survives too
    one = _oracle(replace(b, workload=replace(b.workload, multi_label=False)), do_letterbox=False, do_crops=False)
    raised = one.dets[0, :6]["anchor"]
    for a in raised:
        k = int(h[0, a, 5:].argmax())
        h[0, a, 5 + (k + 9) % 80] = h[0, a, 5 + k]
    res, ref = _compare(b)
    d = ref.dets[0, :ref.counts[0]]
    pairs = 0
    for a in raised:
        m = d[d["anchor"] == a]
        same = [x for x in m if x["score"] == m["score"].max()]
        if len(same) >= 2:
            pairs += 1
            assert [int(x["cls"]) for x in same] == sorted(int(x["cls"]) for x in same)
    assert pairs >= 1


def test_multi_label_overflow_sets_the_status_bit():
    """More candidates than the workspace holds (conf 0 makes every class of every anchor one):
    the excess is dropped, the status bit says so, and the call still returns max_det detections."""
    b = _small("rows", multi_label=True, batch=1, conf_thresh=0.0)
    wl = b.workload
    st = make_stage(wl, b.n)
    try:
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[8])
        assert res.status & 0x10
        assert res.counts.tolist() == [wl.max_det]
    finally:
        st.close()


def test_variant_configuration_is_validated():
    import paper_2502_01277_b200 as octo
    with pytest.raises(octo.OctoError):
        octo.Stage(multi_label=True, class_agnostic=True)
    cfg = octo.make_config()
    cfg.head_layout = 7
    with pytest.raises(octo.OctoError):
        octo.binding.octo_stage_create(cfg)
