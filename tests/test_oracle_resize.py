"""Pins for the oracle's letterbox geometry, bilinear resize core and half rounding.

Each test compares the oracle with something that is not the oracle: hand-worked values,
closed forms of the sampling rule, or a library routine that implements the same textbook
definition (torch's bilinear interpolation with half-pixel centres, numpy's float16 cast).
"""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    out = []
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            out.append(line.split())
    return out


# ---- geometry ---------------------------------------------------------------------------

@pytest.mark.parametrize("w,h,s,expect", [
    (1920, 1080, 640, (640, 360, 0, 140)),
    (1280, 720, 640, (640, 360, 0, 140)),
    (320, 240, 320, (320, 240, 0, 40)),
    (1080, 1920, 640, (360, 640, 140, 0)),
    (4, 2, 8, (8, 4, 0, 2)),
    (640, 640, 640, (640, 640, 0, 0)),
    (3, 2, 5, (5, 3, 0, 1)),      # 2*5/3 = 3.33 -> 3 ; pad 2 -> top 1, bottom 1
    (5, 3, 8, (8, 5, 0, 1)),      # 3*8/5 = 4.8 -> 5 ; pad 3 -> top 1, bottom 2 (extra at bottom)
    (2, 1, 5, (5, 3, 0, 1)),      # 1*5/2 = 2.5 -> rounds half UP to 3
    (10000, 1, 640, (640, 1, 0, 319)),  # never collapses below one row
])
def test_geometry_hand_cases(w, h, s, expect):
    assert oracle.letterbox_geometry(w, h, s) == expect


def test_geometry_properties():
    rng = np.random.default_rng(7)
    for _ in range(2000):
        w, h = int(rng.integers(1, 5000)), int(rng.integers(1, 5000))
        s = int(rng.choice([32, 320, 416, 640, 1280]))
        nw, nh, pl, pt = oracle.letterbox_geometry(w, h, s)
        assert 1 <= nw <= s and 1 <= nh <= s
        assert max(nw, nh) == s
        assert 0 <= pl and 0 <= pt
        assert pl <= s - nw - pl <= pl + 1 and pt <= s - nh - pt <= pt + 1
        # the short side is the exact ratio rounded to nearest (half up)
        if w >= h:
            assert abs(nh - h * s / w) <= 0.5 + 1e-12 or nh == 1
        else:
            assert abs(nw - w * s / h) <= 0.5 + 1e-12 or nw == 1


# ---- half rounding ----------------------------------------------------------------------

def test_half_rounding_matches_numpy_cast():
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.random(20000), rng.random(2000) * 1e-4, rng.random(2000) * 7e-8,
                        np.arange(256) / 255.0, [0.0, 1.0, 65504.0, 65519.9, 65520.0, 1e-8,
                                                 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25]])
    # exact ties between two neighbouring halves must go to the even one
    h = np.arange(0x3400, 0x3420, dtype=np.uint16).view(np.float16).astype(np.float64)
    ties = (h[:-1] + h[1:]) / 2
    v = np.concatenate([v, ties])
    got = oracle.f64_to_half(v)
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, want)


def test_pad_value_bit_pattern():
    assert int(oracle.f64_to_half(114 / 255.0)) == 0x3727


# ---- resize core ------------------------------------------------------------------------

def test_worked_4x2_letterbox():
    want = np.array(_rows(os.path.join(GOLDEN, "letterbox_4x2.txt")), dtype=np.float64)
    img = np.zeros((2, 4, 3), dtype=np.uint8)
    img[0, :, :] = np.array([0, 40, 80, 120])[:, None]
    img[1, :, :] = np.array([80, 120, 160, 200])[:, None]
    core = oracle.resize_f64(img, (0, 0, 4, 2), 8, 4)
    for c in range(3):
        assert np.array_equal(core[c], want[2:6])
    out = oracle.letterbox(img, 4, 2, 8)
    assert np.array_equal(out, np.broadcast_to((want / 255.0).astype(np.float16).view(np.uint16), (3, 8, 8)))


def test_identity_scale_is_exact_copy():
    rng = np.random.default_rng(0)
    img = rng.integers(0, 256, size=(240, 320, 3), dtype=np.uint8)
    out = oracle.letterbox(img, 320, 240, 320)
    want_rgb = (img[:, :, ::-1].astype(np.float64) / 255.0).astype(np.float16).view(np.uint16)
    assert np.array_equal(out[:, 40:280, :], want_rgb.transpose(2, 0, 1))
    assert np.all(out[:, :40, :] == 0x3727) and np.all(out[:, 280:, :] == 0x3727)
    # without the swap plane p is input channel p
    out2 = oracle.letterbox(img, 320, 240, 320, swap_rb=False)
    assert np.array_equal(out2[0], out[2]) and np.array_equal(out2[1], out[1])


def test_three_to_one_is_point_sampling():
    """1920 -> 640: sx = 3*dx + 1 exactly, so the result is the source pixel (3dx+1, 3dy+1)."""
    rng = np.random.default_rng(3)
    img = rng.integers(0, 256, size=(27, 48, 3), dtype=np.uint8)
    core = oracle.resize_f64(img, (0, 0, 48, 27), 16, 9)
    assert np.array_equal(core, img[1::3, 1::3, :].astype(np.float64).transpose(2, 0, 1))


def test_two_to_one_is_block_mean():
    rng = np.random.default_rng(4)
    img = rng.integers(0, 256, size=(18, 32, 3), dtype=np.uint8)
    core = oracle.resize_f64(img, (0, 0, 32, 18), 16, 9)
    blk = img.astype(np.float64).reshape(9, 2, 16, 2, 3).mean(axis=(1, 3)).transpose(2, 0, 1)
    assert np.array_equal(core, blk)


@pytest.mark.parametrize("cw,ch,nw,nh", [(31, 17, 64, 40), (64, 40, 23, 9), (50, 50, 75, 20)])
def test_affine_image_is_reproduced_away_from_borders(cw, ch, nw, nh):
    """Bilinear interpolation is exact on affine images wherever no tap is clamped.  The
    image is affine on an integer lattice so uint8 storage loses nothing."""
    y, x = np.mgrid[0:ch, 0:cw]
    img = np.stack([2 * x + y, x + 2 * y + 5, 3 * x + 7], axis=-1).astype(np.uint8)
    assert img.max() < 255
    core = oracle.resize_f64(img, (0, 0, cw, ch), nw, nh)
    sx = (np.arange(nw) + 0.5) * cw / nw - 0.5
    sy = (np.arange(nh) + 0.5) * ch / nh - 0.5
    okx = (sx >= 0) & (sx <= cw - 1)
    oky = (sy >= 0) & (sy <= ch - 1)
    SX, SY = np.meshgrid(sx, sy)
    want = np.stack([2 * SX + SY, SX + 2 * SY + 5, 3 * SX + 7])
    sel = np.ix_(range(3), np.nonzero(oky)[0], np.nonzero(okx)[0])
    assert np.allclose(core[sel], want[sel], rtol=0, atol=1e-9)


@pytest.mark.parametrize("cw,ch,nw,nh", [(37, 23, 64, 64), (120, 67, 40, 31), (19, 19, 19, 19),
                                          (200, 113, 224, 224), (7, 5, 3, 2), (1, 1, 4, 4)])
def test_resize_matches_library_bilinear(cw, ch, nw, nh):
    """torch's CPU bilinear interpolation (half-pixel centres, no antialias) in float64 is
    the same textbook definition."""
    rng = np.random.default_rng(cw * 1000 + nw)
    img = rng.integers(0, 256, size=(ch, cw, 3), dtype=np.uint8)
    core = oracle.resize_f64(img, (0, 0, cw, ch), nw, nh)
    t = torch.from_numpy(img.astype(np.float64)).permute(2, 0, 1)[None]
    ref = torch.nn.functional.interpolate(t, size=(nh, nw), mode="bilinear", align_corners=False,
                                          antialias=False)[0].numpy()
    assert np.allclose(core, ref, rtol=0, atol=1e-10)


def test_resize_of_sub_rectangle_equals_cut_then_resize():
    rng = np.random.default_rng(9)
    img = rng.integers(0, 256, size=(60, 80, 3), dtype=np.uint8)
    a = oracle.resize_f64(img, (13, 7, 40, 29), 32, 48)
    b = oracle.resize_f64(np.ascontiguousarray(img[7:36, 13:53]), (0, 0, 40, 29), 32, 48)
    assert np.array_equal(a, b)


def test_row_pitch_is_honoured():
    rng = np.random.default_rng(10)
    img = rng.integers(0, 256, size=(9, 10, 3), dtype=np.uint8)
    padded = np.full((9, 48), 255, dtype=np.uint8)
    padded[:, :30] = img.reshape(9, 30)
    assert np.array_equal(oracle.letterbox(img, 10, 9, 16), oracle.letterbox(padded, 10, 9, 16))
