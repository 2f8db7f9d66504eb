"""Pins of the oracle's crop options (aspect-preserving fit, mean/std normalisation).  CPU only.

Geometry is pinned by hand-worked cases and properties; pixel content by the already pinned
resize core (the fitted image must be exactly that resize at the fitted size, placed at the
computed offset) and by closed forms on constant and affine images."""
import numpy as np
import pytest

from oracle import oracle as o

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)


def _half(v):
    return o.f64_to_half(np.asarray(v, dtype=np.float64))


def _img(w, h, seed=0):
    rng = np.random.default_rng(seed)
    return rng.integers(0, 256, (h, w, 3), dtype=np.uint8)


def _det(x1, y1, x2, y2):
    d = np.zeros(1, dtype=o.DET_DTYPE)
    d["x1"], d["y1"], d["x2"], d["y2"] = x1, y1, x2, y2
    return d


@pytest.mark.parametrize("cw,ch,ow,oh,want", [
    (200, 100, 64, 64, (64, 32, 0, 16)),     # wide: width fills, 100*64/200 = 32
    (100, 200, 64, 64, (32, 64, 16, 0)),     # tall: height fills
    (50, 50, 64, 32, (32, 32, 16, 0)),       # square into a wide slot
    (300, 200, 224, 224, (224, 149, 0, 37)),  # 200*224/300 = 149.33 -> 149; pads 37 / 38
    (3, 2, 8, 8, (8, 5, 0, 1)),              # 2*8/3 = 5.33 -> 5; pads 1 / 2
    (2, 3, 8, 8, (5, 8, 1, 0)),
    (8, 3, 16, 16, (16, 6, 0, 5)),           # exactly 6
    (16, 5, 8, 8, (8, 3, 0, 2)),             # 2.5 rounds half-up to 3; pads 2 / 3
    (3, 1000, 64, 64, (1, 64, 31, 0)),       # never below one pixel
])
def test_fit_geometry_hand_cases(cw, ch, ow, oh, want):
    assert o.fit_geometry(cw, ch, ow, oh) == want


def test_fit_geometry_properties():
    rng = np.random.default_rng(5)
    for _ in range(3000):
        cw, ch = int(rng.integers(1, 3000)), int(rng.integers(1, 3000))
        ow, oh = int(rng.integers(1, 40)) * 8, int(rng.integers(1, 300))
        nw, nh, pl, pt = o.fit_geometry(cw, ch, ow, oh)
        assert 1 <= nw <= ow and 1 <= nh <= oh and (nw == ow or nh == oh)
        assert 0 <= pl <= ow - nw - pl <= pl + 1 and 0 <= pt <= oh - nh - pt <= pt + 1
        # the free side is the exact quotient rounded to nearest (ties up), unless clamped to 1
        if ow * ch <= oh * cw:  # the width fills the slot
            assert nw == ow and (nh == 1 or abs(nh - ch * ow / cw) <= 0.5)
        else:
            assert nh == oh and (nw == 1 or abs(nw - cw * oh / ch) <= 0.5)


def test_keep_aspect_is_the_pinned_resize_placed_on_a_pad_canvas():
    img = _img(90, 70, seed=1)
    d = _det(10.0, 5.0, 70.0, 35.0)  # rectangle 60 x 30
    assert o.crop_rect(d, 90, 70) == (10, 5, 70, 35)
    got = o.crop(img, 90, 70, d, 32, 32, keep_aspect=True, pad_value=114)
    nw, nh, pl, pt = o.fit_geometry(60, 30, 32, 32)
    assert (nw, nh, pl, pt) == (32, 16, 0, 8)
    inner = o.resize_f64(img, (10, 5, 60, 30), nw, nh)[::-1]  # planes R, G, B
    want = np.full((3, 32, 32), _half(114 / 255), dtype=np.uint16)
    want[:, pt:pt + nh, pl:pl + nw] = _half(inner / 255.0)
    assert np.array_equal(got, want)
    assert got[0, 0, 0] == 0x3727
    # a rectangle with the slot's own aspect ratio needs no canvas: identical to the plain crop
    d2 = _det(8.0, 8.0, 72.0, 40.0)  # 64 x 32 into 32 x 16
    assert np.array_equal(o.crop(img, 90, 70, d2, 32, 16, keep_aspect=True), o.crop(img, 90, 70, d2, 32, 16))


def test_normalize_closed_forms():
    const = np.full((40, 50, 3), 128, dtype=np.uint8)
    const[..., 0], const[..., 2] = 10, 250  # B = 10, G = 128, R = 250
    d = _det(5.0, 5.0, 45.0, 35.0)
    got = o.crop(const, 50, 40, d, 16, 8, mean=MEAN, std=STD)
    for p, raw in enumerate((250, 128, 10)):  # planes R, G, B after the swap
        want = _half((raw / 255.0 - np.float32(MEAN[p]).astype(np.float64)) / np.float32(STD[p]).astype(np.float64))
        assert np.all(got[p] == want)
    # without the swap the planes follow the image's own channel order, the constants do not move
    got = o.crop(const, 50, 40, d, 16, 8, swap_rb=False, mean=MEAN, std=STD)
    want0 = _half((10 / 255.0 - np.float64(np.float32(MEAN[0]))) / np.float64(np.float32(STD[0])))
    assert np.all(got[0] == want0)
    # mean 0, std 1 is the plain crop
    img = _img(50, 40, seed=2)
    assert np.array_equal(o.crop(img, 50, 40, d, 16, 8, mean=(0, 0, 0), std=(1, 1, 1)), o.crop(img, 50, 40, d, 16, 8))


def test_normalize_is_affine_in_the_pinned_resize():
    img = _img(64, 48, seed=3)
    d = _det(3.2, 4.7, 50.1, 40.0)
    rx0, ry0, rx1, ry1 = o.crop_rect(d, 64, 48)
    base = o.resize_f64(img, (rx0, ry0, rx1 - rx0, ry1 - ry0), 24, 16)[::-1] / 255.0
    m = np.asarray(MEAN, dtype=np.float32).astype(np.float64)[:, None, None]
    s = np.asarray(STD, dtype=np.float32).astype(np.float64)[:, None, None]
    assert np.array_equal(o.crop(img, 64, 48, d, 24, 16, mean=MEAN, std=STD), _half((base - m) / s))


def test_keep_aspect_with_normalisation_normalises_the_canvas_too():
    img = _img(64, 48, seed=4)
    d = _det(0.0, 0.0, 64.0, 16.0)  # 64 x 16 into 32 x 32 -> 32 x 8, pads 12 / 12
    got = o.crop(img, 64, 48, d, 32, 32, keep_aspect=True, pad_value=0, mean=MEAN, std=STD)
    for p in range(3):
        want = _half((0.0 - np.float64(np.float32(MEAN[p]))) / np.float64(np.float32(STD[p])))
        assert np.all(got[p, :12] == want) and np.all(got[p, 20:] == want)
    assert len(np.unique(got[:, 12:20])) > 50
