"""Randomised configurations of the whole stage on the GPU against the oracle: frame shapes from
slivers to wide, small and odd crop sizes, both head layouts, logits and probabilities, the NMS
and crop options in random combinations.  Every case is seeded; the bar is the usual one (integers,
scores and corners bit-exact, pixels within 2e-3 of value)."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import workloads
from gpu_harness import half_absdiff, make_stage, run_stage_gpu
from test_gpu_parity import PIX_TOL, _check_dets

pytestmark = pytest.mark.gpu


def _case(seed, large=False):
    """large: frames up to 4K, crops up to 512 x 512 and hundreds of detections, so that the crop
    kernel runs many passes per crop, cuts crops into row bands and ends on its finer tail tiles."""
    rng = np.random.default_rng((5000 if large else 1000) + seed)
    s = int(rng.choice([320, 640])) if large else int(rng.choice([64, 96, 160, 320, 640]))
    n = int(rng.integers(1, 7)) if large else int(rng.integers(1, 5))
    layout = "planes" if rng.random() < 0.4 else "rows"
    logits = bool(rng.random() < 0.7)
    multi = bool(rng.random() < 0.3)
    agnostic = bool(not multi and rng.random() < 0.25)
    nb = int(rng.integers(1, 4))
    branches, opts, masks = [], [], []
    for _ in range(nb):
        if large:
            branches.append((8 * int(rng.integers(8, 65)), int(rng.integers(32, 513))))
        else:
            branches.append((8 * int(rng.integers(1, 9)), int(rng.integers(1, 70))))
        o = {}
        if rng.random() < 0.4:
            o["keep_aspect"] = True
        if rng.random() < 0.4:
            o["mean"] = tuple(float(v) for v in rng.uniform(0.2, 0.6, 3))
            o["std"] = tuple(float(v) for v in rng.uniform(0.3, 1.0, 3))
        opts.append(o or None)
        masks.append(tuple(int(v) for v in rng.integers(0, 1 << 32, 4, dtype=np.uint64)) if rng.random() < 0.3
                     else (0xFFFFFFFF,) * 4)
    sizes = []
    for _ in range(n):
        kind = rng.random()
        if large:
            sizes.append((int(rng.integers(640, 3841)), int(rng.integers(360, 2161))))
        elif kind < 0.2:
            sizes.append((int(rng.integers(1, 8)), int(rng.integers(40, 300))))      # sliver
        elif kind < 0.4:
            sizes.append((int(rng.integers(300, 900)), int(rng.integers(1, 12))))    # strip
        else:
            sizes.append((int(rng.integers(8, 700)), int(rng.integers(8, 500))))
    wl = replace(workloads.WORKLOADS["anchor_free" if layout == "planes" else "traffic_1080p"], net_size=s,
                 n_raised=int(rng.integers(100, 400)) if large else int(rng.integers(0, 60)),
                 n_groups=int(rng.integers(10, 60)) if large else int(rng.integers(1, 12)), size_range=(0.05 * s, 0.5 * s),
                 box_rows=(0.0, float(s)), logits=logits, multi_label=multi, max_det=int(rng.choice([3, 20, 300])),
                 branches=tuple(branches), conf_thresh=float(rng.choice([0.25, 0.5])),
                 iou_thresh=float(rng.choice([0.3, 0.45, 0.6])))
    b = workloads.make_batch(wl, batch=n, seed=2000 + seed)
    frames = []
    for (w, h) in sizes:
        pitch = (3 * w + 15) // 16 * 16 + 16 * int(rng.integers(0, 3))
        f = np.zeros((h, pitch), dtype=np.uint8)
        f[:, :3 * w] = rng.integers(0, 256, (h, 3 * w), dtype=np.uint8)
        frames.append(f)
    cfg = dict(class_agnostic=agnostic, crop_options=opts, class_masks=masks, swap_rb=bool(rng.random() < 0.7),
               pad_value=int(rng.integers(0, 256)))
    return b, frames, sizes, cfg


@pytest.mark.parametrize("seed", range(64))
def test_random_configuration(seed):
    _run_case(*_case(seed))


@pytest.mark.parametrize("seed", range(10))
def test_random_configuration_with_large_frames_and_crops(seed):
    _run_case(*_case(seed, large=True))


def _run_case(b, frames, sizes, cfg):
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
        assert res.status & ~0x8 == 0
        assert half_absdiff(res.det_in, ref.det_in) <= PIX_TOL
        _check_dets(res, ref)
        for k in range(len(wl.branches)):
            total = len(ref.items[k])
            assert res.n_items[k] == (total, total) and np.array_equal(res.offsets[k], ref.offsets[k])
            it = res.items[k]
            assert np.array_equal(np.stack([it["frame"], it["det"]], 1).reshape(-1, 2), ref.items[k].reshape(-1, 2))
            assert np.array_equal(np.stack([it["rx0"], it["ry0"], it["rx1"], it["ry1"]], 1).reshape(-1, 4),
                                  ref.rects[k].reshape(-1, 4))
            got, want = res.crops[k][:total], ref.crops[k][:total]
            # normalised values stay below 4 in magnitude, where one binary16 step is 2^-9 < 2e-3
            assert float(np.abs(want.view(np.float16).astype(np.float32)).max(initial=0.0)) < 4.0
            assert half_absdiff(got, want) <= PIX_TOL
            assert np.all(res.crops[k][total:] == 0x7BFF)
    finally:
        st.close()
