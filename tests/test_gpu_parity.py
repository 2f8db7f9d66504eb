"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer results (candidate sets, kept anchors and their order, classes,
counts, offsets, item tables, crop rectangles) must be bit-exact, and so must scores and box
coordinates, which are computed in a fixed binary32 sequence on both sides.  fp16 pixels may
differ by at most 2e-3 in value (the oracle interpolates in double, the kernels in fp32)."""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
from gpu_harness import half_absdiff, make_stage, run_stage_gpu

pytestmark = pytest.mark.gpu

PIX_TOL = 2e-3
THREADS = max(1, min(16, os.cpu_count() or 1))


def _check_dets(res, ref):
    assert np.array_equal(res.counts, ref.counts)
    for i, k in enumerate(ref.counts):
        g, o = res.dets[i, :k], ref.dets[i, :k]
        assert np.array_equal(g["anchor"], o["anchor"]), f"frame {i}: kept anchors / order differ"
        assert np.array_equal(g["cls"], o["cls"])
        assert np.array_equal(g["score"].view(np.uint32), o["score"].view(np.uint32)), f"frame {i}: scores not bit-equal"
        for f in ("x1", "y1", "x2", "y2"):
            assert np.array_equal(g[f].view(np.uint32), o[f].view(np.uint32)), f"frame {i}: {f} not bit-equal"


def _check_branch(res, ref, b, first_item=0, max_items=None, crops_checked=None):
    total = len(ref.items[b])
    assert np.array_equal(res.offsets[b], ref.offsets[b])
    cap = total if max_items is None else max_items
    packed = int(np.clip(total - first_item, 0, cap))
    assert res.n_items[b] == (packed, total)
    it = res.items[b]
    want = ref.items[b][first_item:first_item + packed]
    assert np.array_equal(np.stack([it["frame"], it["det"]], 1).reshape(-1, 2), want.reshape(-1, 2))
    rects = np.stack([it["rx0"], it["ry0"], it["rx1"], it["ry1"]], 1).reshape(-1, 4)
    assert np.array_equal(rects, ref.rects[b][first_item:first_item + packed].reshape(-1, 4))
    if ref.crops[b] is not None:
        m = min(packed, len(ref.crops[b]) - first_item) if crops_checked is None else crops_checked
        if m > 0:
            d = half_absdiff(res.crops[b][:m], ref.crops[b][first_item:first_item + m])
            assert d <= PIX_TOL, f"branch {b}: crop max-abs {d}"
    return packed


def _oracle(b, **kw):
    wl = b.workload
    args = dict(logits=wl.logits, conf=wl.conf_thresh, iou_thr=wl.iou_thresh, max_det=wl.max_det, threads=THREADS,
                layout=wl.head_layout, multi_label=wl.multi_label)
    args.update(kw)
    return oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, **args)


def _full_config(name, batch=None):
    """The whole stage on a workload batch: every letterboxed frame and every crop is compared
    with the oracle, beside the detections, the packing and the rectangles."""
    b = workloads.make_batch(name, batch=batch)
    wl = b.workload
    st = make_stage(wl, b.n)
    try:
        ref = _oracle(b)
        cap = [int(len(ref.items[k])) + 3 for k in range(len(wl.branches))]
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=cap)
        assert res.status & ~0x8 == 0
        d = half_absdiff(res.det_in, ref.det_in)
        assert d <= PIX_TOL, f"letterbox max-abs {d}"
        _check_dets(res, ref)
        for k in range(len(wl.branches)):
            assert len(ref.crops[k]) == len(ref.items[k])  # the oracle rendered every crop
            packed = _check_branch(res, ref, k, max_items=cap[k])
            # slots beyond the packed ones are untouched
            assert np.all(res.crops[k][packed:] == 0x7BFF)
        assert res.stats["candidates"] == int(ref.n_cand.sum())
        assert res.stats["kept"] == int(ref.counts.sum())
        return b, res, ref
    finally:
        st.close()


def test_config_tiny():
    b, res, ref = _full_config("tiny")
    # scale 1: the interior of the letterbox is an exact copy, so this config is bit-exact
    assert np.array_equal(res.det_in, ref.det_in)


def test_config_traffic_1080p():
    b, res, ref = _full_config("traffic_1080p")
    # 3:1 reduction is point sampling: bit-exact as well
    assert np.array_equal(res.det_in, ref.det_in)
    assert int(ref.counts.min()) >= 10


def test_config_two_branch():
    b, res, ref = _full_config("two_branch")
    assert len(set(b.sizes)) == 2
    assert np.array_equal(res.items[0][["frame", "det"]], res.items[1][["frame", "det"]])


def test_config_dense_nms():
    b, res, ref = _full_config("dense_nms")
    assert int(ref.n_cand.min()) > 4000 and int(ref.counts.max()) <= 1000


@pytest.mark.parametrize("batch", [1, 4, 16, 64, 256])
def test_config_sweep(batch):
    """Every point of the throughput sweep, the benchmarked B = 256 included, on the whole batch
    (3:1 point sampling makes the letterbox bit-exact)."""
    b, res, ref = _full_config("sweep", batch=batch)
    assert np.array_equal(res.det_in, ref.det_in)
    if batch == 256:
        # the launch shape the benchmark times: whole crops as tiles, the last ones cut into bands
        assert res.n_items[0][0] > 3 * 148 * 4


# ---- letterbox geometry / resize cases --------------------------------------------------

@pytest.mark.parametrize("w,h,s", [(1280, 720, 640), (1080, 1920, 640), (333, 517, 320), (100, 37, 640),
                                   (641, 479, 416), (24, 24, 640), (3840, 2160, 640), (1366, 768, 1280),
                                   (5, 3, 8), (1, 1, 32), (2000, 3, 64)])
def test_letterbox_shapes(w, h, s):
    rng = np.random.default_rng(w * 7 + h)
    pitch = (3 * w + 15) // 16 * 16 + (16 if w % 2 else 0)
    img = np.zeros((h, pitch), dtype=np.uint8)
    img[:, :3 * w] = rng.integers(0, 256, size=(h, 3 * w), dtype=np.uint8)
    img[:, 3 * w:] = 255  # row padding must never leak into the result
    wl = workloads.WORKLOADS["tiny"]
    import paper_2502_01277_b200 as octo
    st = octo.Stage(net_size=s, max_batch=2, num_anchors=64, num_classes=4, branches=((8, 8),))
    try:
        d = torch.from_numpy(img).cuda()
        out = st.preprocess([d, d], [(w, h), (w, h)])
        torch.cuda.synchronize()
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        want = oracle.letterbox(img, w, h, s)
        assert half_absdiff(got[0], want) <= PIX_TOL
        assert np.array_equal(got[0], got[1])
        nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
        mask = np.ones((s, s), dtype=bool)
        mask[pt:pt + nh, pl:pl + nw] = False
        assert np.all(got[0][:, mask] == 0x3727)
        assert st.status() == 0
    finally:
        st.close()


def test_letterbox_no_swap_and_pad_value():
    import paper_2502_01277_b200 as octo
    rng = np.random.default_rng(5)
    img = rng.integers(0, 256, size=(90, 160 * 3), dtype=np.uint8)
    st = octo.Stage(net_size=96, max_batch=1, num_anchors=64, num_classes=4, branches=((8, 8),),
                    swap_rb=False, pad_value=7)
    try:
        out = st.preprocess([torch.from_numpy(img).cuda()], [(160, 90)])
        torch.cuda.synchronize()
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)[0]
        want = oracle.letterbox(img, 160, 90, 96, pad_value=7, swap_rb=False)
        assert half_absdiff(got, want) <= PIX_TOL
        assert got[0, 0, 0] == int(oracle.f64_to_half(7 / 255))
    finally:
        st.close()


# ---- decode / NMS edge cases ------------------------------------------------------------

def _small_case(n_raised, n_groups, batch=2, seed=11, **wl_over):
    from dataclasses import replace
    wl = replace(workloads.WORKLOADS["traffic_1080p"], n_raised=n_raised, n_groups=n_groups,
                 frame_sizes=((640, 360),), **wl_over)
    return workloads.make_batch(wl, batch=batch, seed=seed)


def _run_and_compare(b, stage_over=None, **run_kw):
    wl = b.workload
    st = make_stage(wl, b.n, **(stage_over or {}))
    try:
        ref = _oracle(b, **{k: v for k, v in (stage_over or {}).items() if k in ("max_det",)})
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, **run_kw)
        _check_dets(res, ref)
        return res, ref
    finally:
        st.close()


def test_no_detections_at_all():
    b = _small_case(0, 1, conf_thresh=0.9)
    res, ref = _run_and_compare(b)
    assert res.counts.tolist() == [0, 0]
    assert res.n_items[0] == (0, 0) and res.offsets[0].tolist() == [0, 0, 0]
    assert np.all(res.crops[0] == 0x7BFF)


def test_more_candidates_than_fit_on_chip():
    """> 8192 candidates in one image: the global-memory NMS path must give the same answer."""
    b = _small_case(9000, 600, batch=2)
    res, ref = _run_and_compare(b, max_items=[64])
    assert int(ref.n_cand.max()) > 8192
    assert res.status & 0x8
    assert np.array_equal(res.offsets[0], ref.offsets[0])


def test_max_det_cap_is_hit():
    from dataclasses import replace
    b = _small_case(600, 600, batch=2, max_det=37)
    res, ref = _run_and_compare(b)
    assert res.counts.tolist() == [37, 37]


def test_max_det_cap_is_hit_with_few_candidates():
    """The cap inside the short path (at most 256 candidates per image)."""
    b = _small_case(200, 200, batch=3, max_det=11)
    res, ref = _run_and_compare(b)
    assert int(ref.n_cand.max()) <= 256 and res.counts.tolist() == [11, 11, 11]


@pytest.mark.parametrize("n_raised", [255, 256, 257, 300])
def test_candidate_counts_around_the_short_path_limit(n_raised):
    b = _small_case(n_raised, 30, batch=2)
    res, ref = _run_and_compare(b)
    assert abs(int(ref.n_cand.max()) - n_raised) <= 3


def test_class_agnostic_with_few_candidates():
    """One class of up to 256 candidates in the short path (survivor set wider than one word)."""
    b = _small_case(180, 25, batch=2)
    wl = b.workload
    st = make_stage(wl, b.n, class_agnostic=True)
    try:
        ref = _oracle(b, agnostic=True, do_letterbox=False, do_crops=False)
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[8])
        assert 100 < int(ref.n_cand.max()) <= 256
        _check_dets(res, ref)
    finally:
        st.close()


def test_score_ties_break_by_anchor():
    b = _small_case(40, 40, batch=1)
    h = b.head
    rows = np.nonzero(h[0, :, 4] > 0)[0][:12]
    for r in rows[1:]:
        h[0, r, 4:] = h[0, rows[0], 4:]  # identical obj and class values -> identical scores
    # spread the boxes so that none suppresses another
    for k, r in enumerate(rows):
        h[0, r, 0:4] = [30 + 50 * k, 200, 20, 20]
    res, ref = _run_and_compare(b)
    tied = [a for a in ref.dets[0, :ref.counts[0]]["anchor"] if a in set(rows)]
    assert tied == sorted(tied) and len(tied) == len(rows)


def test_nonfinite_and_degenerate_rows_are_dropped():
    b = _small_case(60, 10, batch=1)
    h = b.head
    raised = np.nonzero(h[0, :, 4] > 0)[0]
    h[0, raised[0], 0] = np.nan
    h[0, raised[1], 3] = np.inf
    h[0, raised[2], 2] = 0.0
    h[0, raised[3], 3] = -5.0
    h[0, raised[4], 5 + 79] = np.nan
    h[0, raised[5], 4] = np.inf  # obj = +inf is non-finite: dropped, not sigma = 1
    h[0, 7, 4] = np.nan          # background row with NaN obj
    res, ref = _run_and_compare(b)
    assert res.status & 0x1
    kept = set(ref.dets[0, :ref.counts[0]]["anchor"].tolist())
    assert not (set(raised[:6].tolist()) & kept)


def test_probability_head():
    b = _small_case(80, 12, batch=2, logits=False)
    assert b.head[:, :, 4:].min() >= 0 and b.head[:, :, 4:].max() <= 1
    res, ref = _run_and_compare(b)
    assert int(ref.counts.min()) > 0


def test_class_masks_and_windows():
    b = _small_case(200, 200, batch=3)
    wl = b.workload
    masks = [[0x0000FFFF, 0, 0, 0], [0, 0xFFFF0000, 0x0000FFFF, 0]]
    st = make_stage(wl, b.n, branches=((64, 64), (32, 48)), class_masks=masks)
    try:
        ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, ((64, 64), (32, 48)),
                               max_det=wl.max_det, class_masks=masks, threads=THREADS)
        total0 = len(ref.items[0])
        assert total0 > 10 and len(ref.items[1]) > 10
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[7, 1000], first_item=5)
        _check_dets(res, ref)
        _check_branch(res, ref, 0, first_item=5, max_items=7)
        _check_branch(res, ref, 1, first_item=5, max_items=1000)
        assert res.status & 0x2  # the 7-slot window truncated branch 0
        assert np.all(res.crops[0][7:] == 0x7BFF) if len(res.crops[0]) > 7 else True
    finally:
        st.close()


def test_stage_reuse_across_batches_and_streams():
    """Two different batches through one stage, the second on a side stream; then the first
    again.  Results must not depend on what ran before."""
    wl = workloads.WORKLOADS["traffic_1080p"]
    b1 = workloads.make_batch("traffic_1080p", batch=3)
    b2 = workloads.make_batch("traffic_1080p", batch=2, first_frame=100)
    st = make_stage(wl, 4)
    try:
        r1 = run_stage_gpu(st, b1.frames, b1.sizes, b1.head, max_items=[200])
        side = torch.cuda.Stream()
        r2 = run_stage_gpu(st, b2.frames, b2.sizes, b2.head, max_items=[200], stream=side)
        r1b = run_stage_gpu(st, b1.frames, b1.sizes, b1.head, max_items=[200])
        ref2 = _oracle(b2)
        _check_dets(r2, ref2)
        _check_branch(r2, ref2, 0, max_items=200)
        assert np.array_equal(r1.dets, r1b.dets) and np.array_equal(r1.counts, r1b.counts)
        assert np.array_equal(r1.crops[0], r1b.crops[0]) and np.array_equal(r1.det_in, r1b.det_in)
    finally:
        st.close()


def test_letterbox_on_a_second_stream_beside_the_rest_of_the_pass():
    """The letterbox kernel shares no device data with decode, NMS and crop of the same batch (it
    reads the frames and writes the detector input; they read the head and the frames), so a caller
    may enqueue it on a second stream.  Alternating batches, every pass against the oracle."""
    wl = workloads.WORKLOADS["traffic_1080p"]
    batches = [workloads.make_batch("traffic_1080p", batch=3), workloads.make_batch("traffic_1080p", batch=2, first_frame=50)]
    refs = [_oracle(b) for b in batches]
    st = make_stage(wl, 4)
    side = torch.cuda.Stream()
    try:
        for i in range(8):
            b, ref = batches[i % 2], refs[i % 2]
            r = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[200], preprocess_stream=side)
            assert r.status == 0
            assert half_absdiff(r.det_in, ref.det_in) <= PIX_TOL
            _check_dets(r, ref)
            _check_branch(r, ref, 0, max_items=200)
    finally:
        st.close()


def test_crop_shapes_and_degenerate_boxes():
    """Crops of hand-placed boxes: tiny, frame-sized, clipped at the border, 1-pixel."""
    import paper_2502_01277_b200 as octo
    from oracle import DET_DTYPE
    rng = np.random.default_rng(3)
    w, h, s = 200, 120, 320
    img = rng.integers(0, 256, size=(h, 3 * w + 8), dtype=np.uint8)
    C, A = 4, 64
    head = np.full((1, A, 5 + C), -9.0, dtype=np.float32)
    nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
    g = w / nw
    boxes = [(10, 10, 8, 8), (100, 60, 200, 120), (198, 118, 10, 10), (50.3, 40.7, 0.2, 0.2), (0.5, 60, 3, 100),
             (120, 3, 60, 9)]
    for k, (cx, cy, bw, bh) in enumerate(boxes):
        head[0, k, :4] = [cx / g + pl, cy / g + pt, bw / g, bh / g]
        head[0, k, 4] = 4.0 - 0.1 * k
        head[0, k, 5 + (k % C)] = 5.0
    for (ow, oh) in [(64, 64), (8, 200), (256, 24)]:
        st = octo.Stage(net_size=s, max_batch=1, num_anchors=A, num_classes=C, branches=((ow, oh),))
        try:
            res = run_stage_gpu(st, [img], [(w, h)], head)
            ref = oracle.run_stage([img], [(w, h)], head, s, ((ow, oh),))
            assert ref.counts[0] == len(boxes)
            _check_dets(res, ref)
            _check_branch(res, ref, 0)
        finally:
            st.close()


@pytest.mark.parametrize("ow,oh", [(24, 40), (40, 33), (72, 40), (120, 37), (136, 40), (448, 24), (456, 40),
                                   (896, 12), (904, 20), (2048, 9)])
def test_crop_output_widths_around_the_unit_layout(ow, oh):
    """Output widths at which the crop kernel's work layout changes: an odd number of column units per
    row, fewer / exactly as many / more units than consumer threads, rows of one pass dealt to 1 .. 32
    runs; heights that leave a ragged last pass."""
    import paper_2502_01277_b200 as octo
    rng = np.random.default_rng(100 + ow)
    w, h, s = 416, 240, 320
    img = rng.integers(0, 256, size=(h, (3 * w + 15) // 16 * 16), dtype=np.uint8)
    C, A = 4, 64
    head = np.full((1, A, 5 + C), -9.0, dtype=np.float32)
    nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
    g = w / nw
    boxes = [(208, 120, 416, 240), (100, 60, 37, 21), (300, 200, 150, 60), (50.3, 40.7, 9, 130), (400, 30, 30, 55)]
    for k, (cx, cy, bw, bh) in enumerate(boxes):
        head[0, k, :4] = [cx / g + pl, cy / g + pt, bw / g, bh / g]
        head[0, k, 4] = 4.0 - 0.1 * k
        head[0, k, 5 + (k % C)] = 5.0
    st = octo.Stage(net_size=s, max_batch=1, num_anchors=A, num_classes=C, branches=((ow, oh),))
    try:
        res = run_stage_gpu(st, [img], [(w, h)], head)
        ref = oracle.run_stage([img], [(w, h)], head, s, ((ow, oh),))
        assert ref.counts[0] == len(boxes)
        _check_dets(res, ref)
        _check_branch(res, ref, 0)
        assert res.status == 0
    finally:
        st.close()


def test_crop_of_very_wide_rectangles_is_tiled_by_columns():
    """Rectangles wider than one staging buffer (about 4000 source pixels) are processed in
    column tiles; results must not show the seams."""
    import paper_2502_01277_b200 as octo
    rng = np.random.default_rng(8)
    w, h, s = 7000, 24, 640
    pitch = (3 * w + 15) // 16 * 16
    img = np.zeros((h, pitch), dtype=np.uint8)
    img[:, :3 * w] = rng.integers(0, 256, size=(h, 3 * w), dtype=np.uint8)
    C, A = 4, 64
    head = np.full((1, A, 5 + C), -9.0, dtype=np.float32)
    nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
    g = w / nw
    boxes = [(3500, 12, 7000, 24), (2100, 10, 4100, 8), (5000, 5, 3990, 6), (6000, 20, 1500, 4)]
    for k, (cx, cy, bw, bh) in enumerate(boxes):
        head[0, k, :4] = [cx / g + pl, cy / g + pt, bw / g, bh / g]
        head[0, k, 4] = 4.0 - 0.1 * k
        head[0, k, 5 + k] = 5.0
    for (ow, oh) in [(224, 16), (1024, 8), (8, 8)]:
        st = octo.Stage(net_size=s, max_batch=1, num_anchors=A, num_classes=C, branches=((ow, oh),))
        try:
            res = run_stage_gpu(st, [img], [(w, h)], head)
            ref = oracle.run_stage([img], [(w, h)], head, s, ((ow, oh),))
            assert ref.counts[0] == len(boxes)
            assert (ref.rects[0][:, 2] - ref.rects[0][:, 0]).max() > 6000
            _check_dets(res, ref)
            _check_branch(res, ref, 0)
            assert res.status == 0
        finally:
            st.close()


def test_class_agnostic_nms_variant():
    """Decode variant: suppression across classes; the survivors keep their own class."""
    b = _small_case(400, 60, batch=3)
    wl = b.workload
    st = make_stage(wl, b.n, class_agnostic=True)
    try:
        ref = _oracle(b, agnostic=True)
        ref_aware = _oracle(b, do_letterbox=False, do_crops=False)
        res = run_stage_gpu(st, b.frames, b.sizes, b.head, max_items=[400])
        _check_dets(res, ref)
        _check_branch(res, ref, 0, max_items=400)
        assert int(ref.counts.sum()) < int(ref_aware.counts.sum())
        assert len(set(ref.dets[0, : ref.counts[0]]["cls"].tolist())) > 3
    finally:
        st.close()
