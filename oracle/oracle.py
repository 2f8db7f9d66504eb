"""ctypes front end of the CPU oracle (octo_oracle.c).  Test infrastructure only: used by
tests/, the smoke check and the benchmark's CPU-baseline leg, never by the product path."""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "octo_oracle.c")
_LIB = os.path.join(_HERE, "liboctooracle.so")
_lib = None

DET_DTYPE = np.dtype([("x1", "<f4"), ("y1", "<f4"), ("x2", "<f4"), ("y2", "<f4"),
                      ("score", "<f4"), ("cls", "<i4"), ("anchor", "<i4"), ("pad", "<i4")])
assert DET_DTYPE.itemsize == 32


def build(force: bool = False) -> str:
    """Compile the oracle with gcc.  -ffp-contract=off keeps every binary32 operation
    individually rounded, which the index-deciding formulas rely on."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math",
                               "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    i32, f32, vp = ctypes.c_int32, ctypes.c_float, ctypes.c_void_p
    lib.orc_letterbox_geometry.argtypes = [i32, i32, i32, vp, vp, vp, vp]
    lib.orc_letterbox_geometry.restype = None
    lib.orc_resize_f64.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.orc_resize_f64.restype = None
    lib.orc_f64_to_half.argtypes = [ctypes.c_double]
    lib.orc_f64_to_half.restype = ctypes.c_uint16
    lib.orc_letterbox.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp]
    lib.orc_letterbox.restype = None
    lib.orc_sigmoid.argtypes = [f32]
    lib.orc_sigmoid.restype = f32
    lib.orc_decode.argtypes = [vp, i32, i32, i32, f32, vp]
    lib.orc_decode.restype = i32
    lib.orc_decode_ex.argtypes = [vp, i32, i32, i32, f32, i32, i32, vp, i32]
    lib.orc_decode_ex.restype = i32
    lib.orc_postprocess_image_v2.argtypes = [vp, i32, i32, i32, f32, f32, i32, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.orc_postprocess_image_v2.restype = i32
    lib.orc_sort.argtypes = [vp, i32]
    lib.orc_sort.restype = None
    lib.orc_iou.argtypes = [vp, vp]
    lib.orc_iou.restype = f32
    lib.orc_nms.argtypes = [vp, i32, f32, i32, vp]
    lib.orc_nms.restype = i32
    lib.orc_nms_ex.argtypes = [vp, i32, f32, i32, i32, vp]
    lib.orc_nms_ex.restype = i32
    lib.orc_postprocess_image_ex.argtypes = [vp, i32, i32, i32, f32, f32, i32, i32, i32, i32, i32, vp, vp]
    lib.orc_postprocess_image_ex.restype = i32
    lib.orc_scale_back.argtypes = [vp, i32, i32, i32]
    lib.orc_scale_back.restype = None
    lib.orc_postprocess_image.argtypes = [vp, i32, i32, i32, f32, f32, i32, i32, i32, i32, vp, vp]
    lib.orc_postprocess_image.restype = i32
    lib.orc_postprocess_region.argtypes = [vp, i32, i32, i32, f32, f32, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.orc_postprocess_region.restype = i32
    lib.orc_postprocess_region_v2.argtypes = [vp, i32, i32, i32, f32, f32, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.orc_postprocess_region_v2.restype = i32
    lib.orc_crop_rect.argtypes = [vp, i32, i32, vp]
    lib.orc_crop_rect.restype = None
    lib.orc_crop.argtypes = [vp, i32, i32, i32, vp, i32, i32, i32, vp]
    lib.orc_crop.restype = None
    lib.orc_fit_geometry.argtypes = [i32, i32, i32, i32, vp]
    lib.orc_fit_geometry.restype = None
    lib.orc_crop_ex.argtypes = [vp, i32, i32, i32, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp]
    lib.orc_crop_ex.restype = None
    lib.orc_assemble.argtypes = [vp, vp, i32, i32, vp, i32, i32, vp, vp, vp]
    lib.orc_assemble.restype = None
    _lib = lib
    return lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _frame2d(img: np.ndarray) -> np.ndarray:
    """Accept [h, pitch] uint8 rows or [h, w, 3]; return C-contiguous [h, pitch]."""
    a = np.ascontiguousarray(img, dtype=np.uint8)
    if a.ndim == 3:
        a = a.reshape(a.shape[0], a.shape[1] * a.shape[2])
    return a


def letterbox_geometry(w: int, h: int, s: int) -> Tuple[int, int, int, int]:
    """(nw, nh, pad_left, pad_top) of a w x h frame on an s x s canvas."""
    out = np.zeros(4, dtype=np.int32)
    p = _ptr(out)
    _load().orc_letterbox_geometry(w, h, s, p, p + 4, p + 8, p + 12)
    return tuple(int(v) for v in out)


def resize_f64(img: np.ndarray, rect: Tuple[int, int, int, int], nw: int, nh: int) -> np.ndarray:
    """Bilinear resize of rect = (rx0, ry0, cw, ch) of an interleaved uint8 image to
    [3, nh, nw] float64, raw 0..255 values, image channel order."""
    a = _frame2d(img)
    out = np.empty((3, nh, nw), dtype=np.float64)
    rx0, ry0, cw, ch = rect
    _load().orc_resize_f64(_ptr(a), a.shape[1], rx0, ry0, cw, ch, nw, nh, _ptr(out))
    return out


def f64_to_half(v) -> np.ndarray:
    """Round doubles to binary16 bit patterns (uint16), nearest even, single rounding."""
    lib = _load()
    arr = np.asarray(v, dtype=np.float64)
    flat = arr.ravel()
    out = np.fromiter((lib.orc_f64_to_half(float(x)) for x in flat), dtype=np.uint16, count=flat.size)
    return out.reshape(arr.shape)


def letterbox(img: np.ndarray, w: int, h: int, s: int, pad_value: int = 114,
              swap_rb: bool = True) -> np.ndarray:
    """One frame -> uint16 [3, s, s] holding binary16 bit patterns."""
    a = _frame2d(img)
    out = np.empty((3, s, s), dtype=np.uint16)
    _load().orc_letterbox(_ptr(a), w, h, a.shape[1], s, pad_value, 1 if swap_rb else 0, _ptr(out))
    return out


def sigmoid(x) -> np.ndarray:
    lib = _load()
    arr = np.asarray(x, dtype=np.float32)
    flat = arr.ravel()
    out = np.fromiter((lib.orc_sigmoid(float(v)) for v in flat), dtype=np.float32, count=flat.size)
    return out.reshape(arr.shape)


LAYOUTS = {"rows": 0, "planes": 1}


def _head_dims(h: np.ndarray, layout: str) -> Tuple[int, int]:
    """(A, C) of one image's head: rows [A, 5 + C] or planes [4 + C, A]."""
    if layout == "rows":
        return h.shape[0], h.shape[1] - 5
    return h.shape[1], h.shape[0] - 4


def decode(head: np.ndarray, logits: bool = True, conf: float = 0.25, layout: str = "rows",
           multi_label: bool = False) -> np.ndarray:
    """One image's head (rows [A, 5 + C] or planes [4 + C, A], float32) -> candidates (DET_DTYPE)
    in (anchor, class) order, letterbox pixels."""
    h = np.ascontiguousarray(head, dtype=np.float32)
    if layout == "rows" and not multi_label:
        a, row = h.shape
        out = np.zeros(max(a, 1), dtype=DET_DTYPE)
        n = _load().orc_decode(_ptr(h), a, row - 5, 1 if logits else 0, np.float32(conf), _ptr(out))
        return out[:n].copy()
    a, c = _head_dims(h, layout)
    cap = max(a * (c if multi_label else 1), 1)
    out = np.zeros(cap, dtype=DET_DTYPE)
    n = _load().orc_decode_ex(_ptr(h), a, c, 1 if logits else 0, np.float32(conf), LAYOUTS[layout],
                              1 if multi_label else 0, _ptr(out), cap)
    return out[:n].copy()


def sort_candidates(cand: np.ndarray) -> np.ndarray:
    c = np.ascontiguousarray(cand, dtype=DET_DTYPE).copy()
    _load().orc_sort(_ptr(c), len(c))
    return c


def iou(a: np.ndarray, b: np.ndarray) -> float:
    """binary32 IoU of two single records (DET_DTYPE arrays of length 1 or scalars)."""
    aa = np.ascontiguousarray(np.atleast_1d(a), dtype=DET_DTYPE)
    bb = np.ascontiguousarray(np.atleast_1d(b), dtype=DET_DTYPE)
    return float(_load().orc_iou(_ptr(aa), _ptr(bb)))


def nms(sorted_cand: np.ndarray, thr: float = 0.45, max_det: int = 300, agnostic: bool = False) -> np.ndarray:
    """Positions (int32) of the kept elements of an already ordered candidate list."""
    c = np.ascontiguousarray(sorted_cand, dtype=DET_DTYPE)
    keep = np.zeros(max(max_det, 1), dtype=np.int32)
    k = _load().orc_nms_ex(_ptr(c), len(c), np.float32(thr), max_det, 1 if agnostic else 0, _ptr(keep))
    return keep[:k].copy()


def scale_back(dets: np.ndarray, w: int, h: int, s: int) -> np.ndarray:
    d = np.ascontiguousarray(dets, dtype=DET_DTYPE).copy()
    lib = _load()
    for i in range(len(d)):
        lib.orc_scale_back(_ptr(d) + 32 * i, w, h, s)
    return d


def postprocess_image(head: np.ndarray, w: int, h: int, s: int, logits: bool = True,
                      conf: float = 0.25, iou_thr: float = 0.45, max_det: int = 300, agnostic: bool = False,
                      layout: str = "rows", multi_label: bool = False):
    """One image's head (rows [A, 5+C] or planes [4+C, A]) -> (dets in frame pixels [kept],
    candidate count)."""
    hd = np.ascontiguousarray(head, dtype=np.float32)
    dets = np.zeros(max(max_det, 1), dtype=DET_DTYPE)
    ncand = np.zeros(1, dtype=np.int32)
    if layout == "rows" and not multi_label:
        a, row = hd.shape
        k = _load().orc_postprocess_image_ex(_ptr(hd), a, row - 5, 1 if logits else 0, np.float32(conf),
                                             np.float32(iou_thr), max_det, w, h, s, 1 if agnostic else 0,
                                             _ptr(dets), _ptr(ncand))
    else:
        a, c = _head_dims(hd, layout)
        k = _load().orc_postprocess_image_v2(_ptr(hd), a, c, 1 if logits else 0, np.float32(conf),
                                             np.float32(iou_thr), max_det, w, h, s, 1 if agnostic else 0,
                                             LAYOUTS[layout], 1 if multi_label else 0, _ptr(dets), _ptr(ncand))
    return dets[:k].copy(), int(ncand[0])


def postprocess_region(head: np.ndarray, region: Tuple[int, int, int, int], s: int, logits: bool = True,
                       conf: float = 0.25, iou_thr: float = 0.45, max_det: int = 300, layout: str = "rows",
                       multi_label: bool = False):
    """Chained stage: head (rows [A, 5+C] or planes [4+C, A]) of one upstream crop (rectangle
    region = (rx0, ry0, rx1, ry1) stretched to s x s) -> (dets in ORIGINAL-frame pixels [kept],
    candidate count)."""
    hd = np.ascontiguousarray(head, dtype=np.float32)
    dets = np.zeros(max(max_det, 1), dtype=DET_DTYPE)
    ncand = np.zeros(1, dtype=np.int32)
    rx0, ry0, rx1, ry1 = (int(v) for v in region)
    if layout == "rows" and not multi_label:
        a, row = hd.shape
        k = _load().orc_postprocess_region(_ptr(hd), a, row - 5, 1 if logits else 0, np.float32(conf),
                                           np.float32(iou_thr), max_det, s, rx0, ry0, rx1 - rx0, ry1 - ry0,
                                           _ptr(dets), _ptr(ncand))
    else:
        a, c = _head_dims(hd, layout)
        k = _load().orc_postprocess_region_v2(_ptr(hd), a, c, 1 if logits else 0, np.float32(conf),
                                              np.float32(iou_thr), max_det, s, rx0, ry0, rx1 - rx0, ry1 - ry0,
                                              LAYOUTS[layout], 1 if multi_label else 0, _ptr(dets), _ptr(ncand))
    return dets[:k].copy(), int(ncand[0])


def crop_rect(det: np.ndarray, w: int, h: int) -> Tuple[int, int, int, int]:
    """(rx0, ry0, rx1, ry1) of one frame-space detection."""
    d = np.ascontiguousarray(np.atleast_1d(det), dtype=DET_DTYPE)
    r = np.zeros(4, dtype=np.int32)
    _load().orc_crop_rect(_ptr(d), w, h, _ptr(r))
    return tuple(int(v) for v in r)


def fit_geometry(cw: int, ch: int, ow: int, oh: int) -> Tuple[int, int, int, int]:
    """(nw, nh, pad_left, pad_top) of a cw x ch rectangle fitted into an ow x oh slot."""
    g = np.zeros(4, dtype=np.int32)
    _load().orc_fit_geometry(cw, ch, ow, oh, _ptr(g))
    return tuple(int(v) for v in g)


def crop(img: np.ndarray, w: int, h: int, det: np.ndarray, ow: int, oh: int,
         swap_rb: bool = True, keep_aspect: bool = False, pad_value: int = 114,
         mean: Optional[Sequence[float]] = None, std: Optional[Sequence[float]] = None) -> np.ndarray:
    """One detection -> uint16 [3, oh, ow] binary16 bit patterns.  keep_aspect fits the rectangle
    into the slot without distortion; mean / std (per output plane) turn normalisation on."""
    a = _frame2d(img)
    d = np.ascontiguousarray(np.atleast_1d(det), dtype=DET_DTYPE)
    out = np.empty((3, oh, ow), dtype=np.uint16)
    norm = mean is not None or std is not None
    if not keep_aspect and not norm:
        _load().orc_crop(_ptr(a), w, h, a.shape[1], _ptr(d), ow, oh, 1 if swap_rb else 0, _ptr(out))
        return out
    m = np.asarray(mean if mean is not None else (0.0, 0.0, 0.0), dtype=np.float32)
    sd = np.asarray(std if std is not None else (1.0, 1.0, 1.0), dtype=np.float32)
    _load().orc_crop_ex(_ptr(a), w, h, a.shape[1], _ptr(d), ow, oh, 1 if swap_rb else 0,
                        1 if keep_aspect else 0, pad_value, 1 if norm else 0, _ptr(m), _ptr(sd), _ptr(out))
    return out


def assemble(dets: np.ndarray, counts: np.ndarray, max_det: int,
             class_mask: Sequence[int] = (0xFFFFFFFF,) * 4, first_item: int = 0,
             max_items: Optional[int] = None):
    """dets [N, max_det] + counts [N] -> (offsets [N+1], items [packed, 2], (packed, total))."""
    d = np.ascontiguousarray(dets, dtype=DET_DTYPE).reshape(-1, max_det)
    c = np.ascontiguousarray(counts, dtype=np.int32)
    n = len(c)
    if max_items is None:
        max_items = int(n * max_det)
    mask = np.asarray(class_mask, dtype=np.uint32)
    offsets = np.zeros(n + 1, dtype=np.int32)
    items = np.zeros((max(max_items, 1), 2), dtype=np.int32)
    n_items = np.zeros(2, dtype=np.int32)
    _load().orc_assemble(_ptr(d), _ptr(c), n, max_det, _ptr(mask), first_item, max_items,
                         _ptr(offsets), _ptr(items), _ptr(n_items))
    return offsets, items[: int(n_items[0])].copy(), (int(n_items[0]), int(n_items[1]))


@dataclass
class StageResult:
    det_in: Optional[np.ndarray]  # uint16 [N, 3, S, S] or None
    dets: np.ndarray  # DET_DTYPE [N, max_det]
    counts: np.ndarray  # int32 [N]
    n_cand: np.ndarray  # int32 [N]
    offsets: List[np.ndarray] = field(default_factory=list)  # per branch [N+1]
    items: List[np.ndarray] = field(default_factory=list)  # per branch [total, 2]
    rects: List[np.ndarray] = field(default_factory=list)  # per branch [total, 4]
    crops: List[Optional[np.ndarray]] = field(default_factory=list)  # per branch uint16 [total,3,oh,ow]


def run_stage(frames: Sequence[np.ndarray], sizes: Sequence[Tuple[int, int]], head: np.ndarray,
              net_size: int, branches: Sequence[Tuple[int, int]], *, logits: bool = True,
              conf: float = 0.25, iou_thr: float = 0.45, max_det: int = 300, pad_value: int = 114,
              swap_rb: bool = True, class_masks: Optional[Sequence[Sequence[int]]] = None,
              do_letterbox: bool = True, do_crops: bool = True, max_crops: Optional[int] = None,
              threads: int = 1, agnostic: bool = False, layout: str = "rows",
              multi_label: bool = False, crop_options: Optional[Sequence[Optional[dict]]] = None) -> StageResult:
    """Whole stage over one batch, frame by frame (optionally a thread per frame; the C
    routines release the GIL).  max_crops bounds the crops rendered per branch."""
    n = len(frames)
    s = net_size
    det_in = np.empty((n, 3, s, s), dtype=np.uint16) if do_letterbox else None
    dets = np.zeros((n, max_det), dtype=DET_DTYPE)
    counts = np.zeros(n, dtype=np.int32)
    ncand = np.zeros(n, dtype=np.int32)

    def per_frame(i: int) -> None:
        w, h = sizes[i]
        if do_letterbox:
            det_in[i] = letterbox(frames[i], w, h, s, pad_value, swap_rb)
        d, nc = postprocess_image(head[i], w, h, s, logits, conf, iou_thr, max_det, agnostic, layout, multi_label)
        dets[i, : len(d)] = d
        counts[i] = len(d)
        ncand[i] = nc

    def pmap(fn, count):
        if threads > 1 and count > 1:
            with ThreadPoolExecutor(max_workers=threads) as ex:
                list(ex.map(fn, range(count)))
        else:
            for i in range(count):
                fn(i)

    pmap(per_frame, n)
    res = StageResult(det_in, dets, counts, ncand)
    for b, (ow, oh) in enumerate(branches):
        mask = class_masks[b] if class_masks is not None else (0xFFFFFFFF,) * 4
        offsets, items, (packed, total) = assemble(dets, counts, max_det, mask)
        rects = np.zeros((len(items), 4), dtype=np.int32)
        for k, (f, j) in enumerate(items):
            rects[k] = crop_rect(dets[f, j], *sizes[f])
        crops = None
        if do_crops:
            m = len(items) if max_crops is None else min(len(items), max_crops)
            crops = np.empty((m, 3, oh, ow), dtype=np.uint16)

            opt = dict((crop_options[b] if crop_options is not None else None) or {})

            def per_item(k: int, _crops=crops, _items=items, _ow=ow, _oh=oh, _opt=opt) -> None:
                f, j = _items[k]
                w, h = sizes[f]
                _crops[k] = crop(frames[f], w, h, dets[f, j], _ow, _oh, swap_rb, pad_value=pad_value, **_opt)

            pmap(per_item, m)
        res.offsets.append(offsets)
        res.items.append(items)
        res.rects.append(rects)
        res.crops.append(crops)
    return res


def margin_report(head: np.ndarray, logits: bool = True, conf: float = 0.25, iou_thr: float = 0.45) -> dict:
    """Margin certificate of one image in double precision: how close any decision of the stage
    comes to flipping.  Returns the smallest |score - conf| over all anchors, the smallest gap
    between neighbouring scores of the ordered candidates, and the smallest |IoU - iou_thr| over
    all same-class candidate pairs (a superset of the pairs the greedy scan tests)."""
    h = np.asarray(head, dtype=np.float64)
    cls_v = h[:, 5:].max(axis=1)
    if logits:
        score = 1.0 / (1.0 + np.exp(-h[:, 4])) / (1.0 + np.exp(-cls_v))
    else:
        score = h[:, 4] * cls_v
    ok = np.isfinite(h).all(axis=1) & (h[:, 2] > 0) & (h[:, 3] > 0)
    cand = np.nonzero(ok & (score > conf))[0]
    s = np.sort(score[cand])[::-1]
    out = {"candidates": int(len(cand)),
           "min_abs_score_minus_conf": float(np.min(np.abs(score[ok] - conf))) if ok.any() else float("inf"),
           "min_score_gap": float(np.min(-np.diff(s))) if len(s) > 1 else float("inf"),
           "min_abs_iou_minus_thr": float("inf")}
    k = h[cand, 5:].argmax(axis=1)
    x1, y1 = h[cand, 0] - 0.5 * h[cand, 2], h[cand, 1] - 0.5 * h[cand, 3]
    x2, y2 = h[cand, 0] + 0.5 * h[cand, 2], h[cand, 1] + 0.5 * h[cand, 3]
    for c in np.unique(k):
        m = np.nonzero(k == c)[0]
        if len(m) < 2:
            continue
        iw = np.clip(np.minimum(x2[m, None], x2[None, m]) - np.maximum(x1[m, None], x1[None, m]), 0, None)
        ih = np.clip(np.minimum(y2[m, None], y2[None, m]) - np.maximum(y1[m, None], y1[None, m]), 0, None)
        inter = iw * ih
        area = (x2[m] - x1[m]) * (y2[m] - y1[m])
        uni = area[:, None] + area[None, :] - inter
        iou = np.where(uni > 0, inter / np.where(uni > 0, uni, 1.0), 0.0)
        iu = np.triu_indices(len(m), 1)
        out["min_abs_iou_minus_thr"] = min(out["min_abs_iou_minus_thr"], float(np.min(np.abs(iou[iu] - iou_thr))))
    return out
