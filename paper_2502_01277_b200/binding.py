"""ctypes binding of the C-ABI library (include/octo.h).  Argument marshalling only: every
step of the stage runs in the CUDA kernels of liboctostage.so.  There is no CPU fallback;
importing the library fails loudly if the shared object has not been built.

Function names match the C ABI: octo_stage_create, octo_preprocess_batch,
octo_postprocess_batch, octo_crop_batch, ...  `Stage` is a thin convenience object over
them for callers that hold torch tensors (torch provides device memory and streams only).
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liboctostage.so")

OCTO_MAX_BRANCHES = 4
OCTO_MAX_BATCH = 512

OCTO_OK = 0
OCTO_E_INVALID_ARG = -1
OCTO_E_CAPACITY = -2
OCTO_E_ALIGNMENT = -3
OCTO_E_NO_PREPROCESS = -4
OCTO_E_CUDA = -5
OCTO_E_DEVICE_TIMEOUT = -6
OCTO_E_NO_POSTPROCESS = -7
OCTO_E_NO_MEMORY = -8

OCTO_STATUS_NONFINITE = 0x1
OCTO_STATUS_TRUNCATED = 0x2
OCTO_STATUS_COPY_TIMEOUT = 0x4
OCTO_STATUS_BIG_NMS = 0x8
OCTO_STATUS_CAND_OVERFLOW = 0x10
OCTO_STATUS_BOUNDS = 0x20

OCTO_HEAD_ROWS = 0
OCTO_HEAD_PLANES = 1
HEAD_LAYOUTS = {"rows": OCTO_HEAD_ROWS, "planes": OCTO_HEAD_PLANES}

EXPORTS = (
    "octo_stage_create", "octo_stage_destroy", "octo_preprocess_batch", "octo_postprocess_batch",
    "octo_crop_batch", "octo_stage_status", "octo_stage_clear_status", "octo_stage_get_stats",
    "octo_stage_item_table", "octo_stage_copy_items", "octo_stage_set_timing", "octo_stage_kernel_times",
    "octo_stage_workspace_bytes", "octo_stage_launch_count",
    "octo_strerror", "octo_last_cuda_error", "octo_version", "octo_postprocess_frame_static",
    "octo_adopt_regions", "octo_queue_create", "octo_queue_destroy", "octo_queue_push", "octo_queue_pop",
    "octo_queue_pop_due", "octo_coral_schedule", "octo_queue_set_options",
    "octo_adopt_items_device", "octo_stage_selftest_wait", "octo_static_status",
    "octo_stage_set_nms_cluster", "octo_stage_last_nms_cluster", "octo_stage_last_nms_half_ctas",
)


class BranchCfg(ctypes.Structure):
    _fields_ = [("out_w", ctypes.c_int32), ("out_h", ctypes.c_int32), ("class_mask", ctypes.c_uint32 * 4),
                ("keep_aspect", ctypes.c_int32), ("normalize", ctypes.c_int32),
                ("mean", ctypes.c_float * 3), ("std", ctypes.c_float * 3)]


class StageConfig(ctypes.Structure):
    _fields_ = [
        ("device", ctypes.c_int32), ("net_size", ctypes.c_int32), ("max_batch", ctypes.c_int32),
        ("num_anchors", ctypes.c_int32), ("num_classes", ctypes.c_int32),
        ("head_is_logits", ctypes.c_int32), ("conf_thresh", ctypes.c_float),
        ("iou_thresh", ctypes.c_float), ("max_det", ctypes.c_int32), ("pad_value", ctypes.c_int32),
        ("swap_rb", ctypes.c_int32), ("num_branches", ctypes.c_int32), ("class_agnostic", ctypes.c_int32),
        ("head_layout", ctypes.c_int32), ("multi_label", ctypes.c_int32),
        ("branch", BranchCfg * OCTO_MAX_BRANCHES),
    ]


class Frame(ctypes.Structure):
    _fields_ = [("d_data", ctypes.c_void_p), ("width", ctypes.c_int32), ("height", ctypes.c_int32),
                ("pitch_bytes", ctypes.c_int32), ("_pad", ctypes.c_int32)]


class Region(ctypes.Structure):
    _fields_ = [("d_data", ctypes.c_void_p), ("width", ctypes.c_int32), ("height", ctypes.c_int32),
                ("pitch_bytes", ctypes.c_int32), ("rx0", ctypes.c_int32), ("ry0", ctypes.c_int32),
                ("rx1", ctypes.c_int32), ("ry1", ctypes.c_int32), ("_pad", ctypes.c_int32)]


class StageStats(ctypes.Structure):
    _fields_ = [("candidates", ctypes.c_int64), ("kept", ctypes.c_int64), ("packed", ctypes.c_int64),
                ("total_items", ctypes.c_int64), ("status_word", ctypes.c_uint32),
                ("max_candidates_per_image", ctypes.c_int32)]


class CoralInstance(ctypes.Structure):
    _fields_ = [("pipeline", ctypes.c_int32), ("model", ctypes.c_int32), ("instance", ctypes.c_int32),
                ("util_permille", ctypes.c_int32), ("start_us", ctypes.c_int64), ("end_us", ctypes.c_int64),
                ("duty_cycle_us", ctypes.c_int64), ("weight_bytes", ctypes.c_int64), ("inter_bytes", ctypes.c_int64)]


class CoralGpu(ctypes.Structure):
    _fields_ = [("mem_bytes", ctypes.c_int64), ("util_max_permille", ctypes.c_int32), ("num_streams", ctypes.c_int32)]


class CoralPlacement(ctypes.Structure):
    _fields_ = [("gpu", ctypes.c_int32), ("stream", ctypes.c_int32), ("start_us", ctypes.c_int64),
                ("end_us", ctypes.c_int64), ("duty_cycle_us", ctypes.c_int64)]


REGION_DTYPE = np.dtype([("d_data", "<u8"), ("width", "<i4"), ("height", "<i4"), ("pitch_bytes", "<i4"),
                         ("rx0", "<i4"), ("ry0", "<i4"), ("rx1", "<i4"), ("ry1", "<i4"), ("pad", "<i4")])

QITEM_DTYPE = np.dtype([("d_data", "<u8"), ("width", "<i4"), ("height", "<i4"), ("pitch_bytes", "<i4"),
                        ("rx0", "<i4"), ("ry0", "<i4"), ("rx1", "<i4"), ("ry1", "<i4"), ("seq", "<i4"),
                        ("frame", "<i4"), ("det", "<i4")])

KERNEL_NAMES = ("letterbox", "decode", "nms", "assemble", "crop")


class KernelTimes(ctypes.Structure):
    _fields_ = [("ms", ctypes.c_double * 5), ("launches", ctypes.c_int64 * 5), ("dropped", ctypes.c_int64)]


DET_DTYPE = np.dtype([("x1", "<f4"), ("y1", "<f4"), ("x2", "<f4"), ("y2", "<f4"), ("score", "<f4"),
                      ("cls", "<i4"), ("anchor", "<i4"), ("pad", "<i4")])
ITEM_DTYPE = np.dtype([("frame", "<i4"), ("det", "<i4"), ("rx0", "<i4"), ("ry0", "<i4"),
                       ("rx1", "<i4"), ("ry1", "<i4"), ("pad0", "<i4"), ("pad1", "<i4")])

_lib = None


class OctoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if _lib is not None:
            detail = _lib.octo_strerror(code).decode()
            if code == OCTO_E_CUDA:
                detail += " (" + _lib.octo_last_cuda_error().decode() + ")"
        super().__init__(f"{where} failed with status {code}: {detail}")


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """dlopen liboctostage.so and declare the prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ImportError(
            f"{p} not found: build the CUDA library first (python -m paper_2502_01277_b200.build). "
            "There is no fallback path.")
    lib = ctypes.CDLL(p)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.octo_stage_create.argtypes = [ctypes.POINTER(StageConfig), ctypes.POINTER(vp)]
    lib.octo_stage_destroy.argtypes = [vp]
    lib.octo_preprocess_batch.argtypes = [vp, ctypes.POINTER(Frame), i32, vp, vp]
    lib.octo_postprocess_batch.argtypes = [vp, vp, i32, vp, vp, vp]
    lib.octo_adopt_regions.argtypes = [vp, ctypes.POINTER(Region), i32, vp]
    lib.octo_adopt_regions.restype = ctypes.c_int
    lib.octo_adopt_items_device.argtypes = [vp, vp, i32, i32, i32, vp]
    lib.octo_adopt_items_device.restype = ctypes.c_int
    lib.octo_stage_selftest_wait.argtypes = [vp, i32, vp]
    lib.octo_stage_selftest_wait.restype = ctypes.c_int
    lib.octo_static_status.argtypes = [i32, ctypes.POINTER(ctypes.c_uint32), vp]
    lib.octo_static_status.restype = ctypes.c_int
    lib.octo_crop_batch.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.octo_stage_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    lib.octo_stage_clear_status.argtypes = [vp, vp]
    lib.octo_stage_get_stats.argtypes = [vp, ctypes.POINTER(StageStats), vp]
    lib.octo_stage_item_table.argtypes = [vp, i32, ctypes.POINTER(vp)]
    lib.octo_stage_copy_items.argtypes = [vp, i32, vp, i32, vp]
    lib.octo_stage_copy_items.restype = ctypes.c_int
    lib.octo_stage_set_timing.argtypes = [vp, i32]
    lib.octo_stage_set_timing.restype = ctypes.c_int
    lib.octo_stage_set_nms_cluster.argtypes = [vp, i32]
    lib.octo_stage_set_nms_cluster.restype = ctypes.c_int
    lib.octo_stage_last_nms_cluster.argtypes = [vp]
    lib.octo_stage_last_nms_cluster.restype = i32
    lib.octo_stage_last_nms_half_ctas.argtypes = [vp]
    lib.octo_stage_last_nms_half_ctas.restype = i32
    lib.octo_stage_kernel_times.argtypes = [vp, ctypes.POINTER(KernelTimes), vp]
    lib.octo_stage_kernel_times.restype = ctypes.c_int
    lib.octo_postprocess_frame_static.argtypes = [i32, vp, i32, i32, i32, ctypes.c_float, ctypes.c_float,
                                                  i32, i32, i32, i32, vp, vp, vp]
    lib.octo_postprocess_frame_static.restype = ctypes.c_int
    lib.octo_queue_create.argtypes = [i32, i32, i32, i32, i32, i32, ctypes.POINTER(vp)]
    lib.octo_queue_destroy.argtypes = [vp]
    lib.octo_queue_push.argtypes = [vp, vp, i32, vp]
    lib.octo_queue_pop.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.octo_queue_set_options.argtypes = [vp, ctypes.POINTER(BranchCfg), i32]
    lib.octo_queue_set_options.restype = ctypes.c_int
    lib.octo_queue_pop_due.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    lib.octo_queue_pop_due.restype = ctypes.c_int
    for name in ("octo_queue_create", "octo_queue_destroy", "octo_queue_push", "octo_queue_pop"):
        getattr(lib, name).restype = ctypes.c_int
    lib.octo_coral_schedule.argtypes = [ctypes.POINTER(CoralInstance), i32, ctypes.POINTER(CoralGpu), i32,
                                        ctypes.POINTER(CoralPlacement)]
    lib.octo_coral_schedule.restype = ctypes.c_int
    lib.octo_stage_workspace_bytes.argtypes = [vp]
    lib.octo_stage_workspace_bytes.restype = ctypes.c_int64
    lib.octo_stage_launch_count.argtypes = [vp]
    lib.octo_stage_launch_count.restype = ctypes.c_int64
    for name in ("octo_strerror", "octo_last_cuda_error", "octo_version"):
        getattr(lib, name).restype = ctypes.c_char_p
    lib.octo_strerror.argtypes = [ctypes.c_int]
    for name in ("octo_stage_create", "octo_stage_destroy", "octo_preprocess_batch",
                 "octo_postprocess_batch", "octo_crop_batch", "octo_stage_status",
                 "octo_stage_clear_status", "octo_stage_get_stats", "octo_stage_item_table"):
        getattr(lib, name).restype = ctypes.c_int
    if path is None:
        _lib = lib
    return lib


def make_config(*, device: int = 0, net_size: int = 640, max_batch: int = 8, num_anchors: int = 25200,
                num_classes: int = 80, head_is_logits: bool = True, conf_thresh: float = 0.25,
                iou_thresh: float = 0.45, max_det: int = 300, pad_value: int = 114, swap_rb: bool = True,
                branches: Sequence[Tuple[int, int]] = ((224, 224),),
                class_masks: Optional[Sequence[Sequence[int]]] = None,
                class_agnostic: bool = False, head_layout: str = "rows",
                multi_label: bool = False, crop_options: Optional[Sequence[Optional[dict]]] = None) -> StageConfig:
    """crop_options: per branch None or a dict with any of keep_aspect (bool), mean and std
    (three floats each, per output plane; giving them turns normalisation on)."""
    cfg = StageConfig()
    cfg.device, cfg.net_size, cfg.max_batch = device, net_size, max_batch
    cfg.num_anchors, cfg.num_classes = num_anchors, num_classes
    cfg.head_is_logits = 1 if head_is_logits else 0
    cfg.conf_thresh, cfg.iou_thresh = conf_thresh, iou_thresh
    cfg.max_det, cfg.pad_value, cfg.swap_rb = max_det, pad_value, 1 if swap_rb else 0
    cfg.num_branches = len(branches)
    cfg.class_agnostic = 1 if class_agnostic else 0
    cfg.head_layout = HEAD_LAYOUTS[head_layout]
    cfg.multi_label = 1 if multi_label else 0
    for b, (ow, oh) in enumerate(branches[:OCTO_MAX_BRANCHES]):
        cfg.branch[b].out_w, cfg.branch[b].out_h = ow, oh
        mask = class_masks[b] if class_masks is not None else (0xFFFFFFFF,) * 4
        for k in range(4):
            cfg.branch[b].class_mask[k] = int(mask[k]) & 0xFFFFFFFF
        opt = (crop_options[b] if crop_options is not None else None) or {}
        cfg.branch[b].keep_aspect = 1 if opt.get("keep_aspect") else 0
        if "mean" in opt or "std" in opt:
            cfg.branch[b].normalize = 1
            for k in range(3):
                cfg.branch[b].mean[k] = float(opt.get("mean", (0.0, 0.0, 0.0))[k])
                cfg.branch[b].std[k] = float(opt.get("std", (1.0, 1.0, 1.0))[k])
    return cfg


# ---- thin functional layer: same names as the C ABI ------------------------------------------

def octo_stage_create(cfg: StageConfig) -> ctypes.c_void_p:
    lib = load_library()
    h = ctypes.c_void_p()
    rc = lib.octo_stage_create(ctypes.byref(cfg), ctypes.byref(h))
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_stage_create")
    return h


def octo_stage_destroy(handle) -> None:
    load_library().octo_stage_destroy(handle)


def octo_preprocess_batch(handle, frames: Sequence[Tuple[int, int, int, int]], d_out: int, stream: int = 0) -> None:
    """frames: (device_ptr, width, height, pitch_bytes) per frame."""
    n = len(frames)
    arr = (Frame * max(n, 1))()
    for i, (ptr, w, h, pitch) in enumerate(frames):
        arr[i].d_data, arr[i].width, arr[i].height, arr[i].pitch_bytes = ptr, w, h, pitch
    rc = load_library().octo_preprocess_batch(handle, arr, n, d_out, stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_preprocess_batch")


def octo_postprocess_batch(handle, d_head: int, n: int, d_dets: int, d_counts: int, stream: int = 0) -> None:
    rc = load_library().octo_postprocess_batch(handle, d_head, n, d_dets, d_counts, stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_postprocess_batch")


def octo_crop_batch(handle, branch: int, first_item: int, max_items: int, d_out: int, d_offsets: int,
                    d_n_items: int, stream: int = 0) -> None:
    rc = load_library().octo_crop_batch(handle, branch, first_item, max_items, d_out, d_offsets, d_n_items, stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_crop_batch")


def octo_postprocess_frame_static(device: int, d_head: int, num_anchors: int, num_classes: int,
                                  head_is_logits: bool, conf_thresh: float, iou_thresh: float, max_det: int,
                                  net_size: int, frame_w: int, frame_h: int, d_dets: int, d_count: int,
                                  stream: int = 0) -> None:
    """Single-frame decode + NMS on the library's built-in workspace, for callers that may
    not allocate device memory (see include/octo.h).  Pointers are raw device addresses."""
    rc = load_library().octo_postprocess_frame_static(
        device, d_head, num_anchors, num_classes, 1 if head_is_logits else 0, conf_thresh, iou_thresh,
        max_det, net_size, frame_w, frame_h, d_dets, d_count, stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_postprocess_frame_static")


def octo_static_status(device: int = 0, stream: int = 0) -> int:
    """Status word of the last octo_postprocess_frame_static call on the device (synchronises)."""
    w = ctypes.c_uint32(0)
    rc = load_library().octo_static_status(device, ctypes.byref(w), stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_static_status")
    return int(w.value)


def octo_stage_status(handle, stream: int = 0) -> int:
    w = ctypes.c_uint32(0)
    rc = load_library().octo_stage_status(handle, ctypes.byref(w), stream)
    if rc not in (OCTO_OK, OCTO_E_DEVICE_TIMEOUT):
        raise OctoError(rc, "octo_stage_status")
    return int(w.value)


def octo_stage_get_stats(handle, stream: int = 0) -> dict:
    s = StageStats()
    rc = load_library().octo_stage_get_stats(handle, ctypes.byref(s), stream)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_stage_get_stats")
    return {k: int(getattr(s, k)) for k, _ in StageStats._fields_}


# ---- convenience object for torch callers ----------------------------------------------------

class Stage:
    """Owns one octo_stage_t and the torch tensors a caller usually wants around it."""

    def __init__(self, **cfg_kwargs):
        import torch  # device memory and streams only
        self._torch = torch
        self.cfg = make_config(**cfg_kwargs)
        self.handle = octo_stage_create(self.cfg)
        self.device = torch.device("cuda", self.cfg.device)
        self.n = 0
        self._frames_keepalive: List = []

    def close(self) -> None:
        if getattr(self, "handle", None):
            octo_stage_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _stream(self, stream) -> int:
        if stream is None:
            stream = self._torch.cuda.current_stream(self.device)
        return int(stream.cuda_stream)

    def preprocess(self, frames, sizes, out=None, stream=None):
        """frames: list of uint8 CUDA tensors [h, pitch]; sizes: (w, h) per frame.
        Returns the fp16 [n, 3, S, S] batch."""
        t = self._torch
        n, s = len(frames), self.cfg.net_size
        if out is None:
            out = t.empty((n, 3, s, s), dtype=t.float16, device=self.device)
        desc = [(f.data_ptr(), w, h, f.stride(0)) for f, (w, h) in zip(frames, sizes)]
        octo_preprocess_batch(self.handle, desc, out.data_ptr(), self._stream(stream))
        self._frames_keepalive = list(frames)
        self.n = n
        return out

    def frame_array(self, frames, sizes):
        """Descriptor array for tensors whose addresses stay fixed; reuse it with
        preprocess_array to skip the per-call marshalling."""
        arr = (Frame * max(len(frames), 1))()
        for i, (f, (w, h)) in enumerate(zip(frames, sizes)):
            arr[i].d_data, arr[i].width, arr[i].height, arr[i].pitch_bytes = f.data_ptr(), w, h, f.stride(0)
        return arr

    def preprocess_array(self, arr, n, out, stream=None, keepalive=None):
        rc = load_library().octo_preprocess_batch(self.handle, arr, n, out.data_ptr(), self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_preprocess_batch")
        if keepalive is not None:
            self._frames_keepalive = keepalive
        self.n = n
        return out

    def adopt_regions(self, frames, sizes, items, stream=None):
        """Chained stage: this batch = the upstream items (ITEM_DTYPE records: frame index +
        rectangle) of the upstream frames (CUDA tensors [h, pitch]) with their (w, h) sizes."""
        n = len(items)
        fr = np.asarray(items["frame"], dtype=np.int64)
        ptrs = np.array([f.data_ptr() for f in frames], dtype=np.uint64)
        pitches = np.array([f.stride(0) for f in frames], dtype=np.int32)
        wh = np.asarray(sizes, dtype=np.int32).reshape(-1, 2)
        reg = np.zeros(max(n, 1), dtype=REGION_DTYPE)
        if n:
            reg["d_data"][:n] = ptrs[fr]
            reg["width"][:n], reg["height"][:n], reg["pitch_bytes"][:n] = wh[fr, 0], wh[fr, 1], pitches[fr]
            for k in ("rx0", "ry0", "rx1", "ry1"):
                reg[k][:n] = items[k]
        arr = reg.ctypes.data_as(ctypes.POINTER(Region))
        rc = load_library().octo_adopt_regions(self.handle, arr, n, self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_adopt_regions")
        self._frames_keepalive = list(frames)
        self.n = n

    def adopt_items_device(self, upstream: "Stage", branch: int, n: int, first: int = 0, stream=None) -> None:
        """Chained stage without a host hand-off: this batch = entries [first, first + n) of the item
        table the upstream stage's last crop call of `branch` built (octo_adopt_items_device)."""
        rc = load_library().octo_adopt_items_device(self.handle, upstream.handle, branch, first, n,
                                                    self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_adopt_items_device")
        self._frames_keepalive = list(upstream._frames_keepalive)
        self._upstream_keepalive = upstream
        self.n = n

    def selftest_wait(self, polls: int = 256, stream=None) -> None:
        rc = load_library().octo_stage_selftest_wait(self.handle, polls, self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_stage_selftest_wait")

    def postprocess(self, head, dets=None, counts=None, stream=None):
        """head: float32 CUDA tensor [n, A, 5+C].  Returns (dets uint8 [n, max_det, 32], counts int32 [n])."""
        t = self._torch
        n = head.shape[0]
        if dets is None:
            dets = t.empty((n, self.cfg.max_det, 32), dtype=t.uint8, device=self.device)
        if counts is None:
            counts = t.empty((n,), dtype=t.int32, device=self.device)
        octo_postprocess_batch(self.handle, head.data_ptr(), n, dets.data_ptr(), counts.data_ptr(),
                               self._stream(stream))
        self._dets_keepalive = dets
        return dets, counts

    def crop(self, branch, max_items, first_item=0, out=None, offsets=None, n_items=None, stream=None):
        """Returns (crops fp16 [max_items, 3, oh, ow], offsets int32 [n+1], n_items int32 [2])."""
        t = self._torch
        ow, oh = self.cfg.branch[branch].out_w, self.cfg.branch[branch].out_h
        if out is None:
            out = t.empty((max(max_items, 1), 3, oh, ow), dtype=t.float16, device=self.device)
        if offsets is None:
            offsets = t.empty((self.n + 1,), dtype=t.int32, device=self.device)
        if n_items is None:
            n_items = t.empty((2,), dtype=t.int32, device=self.device)
        octo_crop_batch(self.handle, branch, first_item, max_items, out.data_ptr(), offsets.data_ptr(),
                        n_items.data_ptr(), self._stream(stream))
        return out, offsets, n_items

    def item_table(self, branch: int, count: int) -> np.ndarray:
        """Host copy of the first `count` entries of the branch's item table (synchronises)."""
        host = np.zeros(max(count, 1), dtype=ITEM_DTYPE)
        rc = load_library().octo_stage_copy_items(self.handle, branch, host.ctypes.data, count, self._stream(None))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_stage_copy_items")
        return host[:count]

    def status(self, stream=None) -> int:
        return octo_stage_status(self.handle, self._stream(stream))

    def clear_status(self, stream=None) -> None:
        load_library().octo_stage_clear_status(self.handle, self._stream(stream))

    def stats(self, stream=None) -> dict:
        return octo_stage_get_stats(self.handle, self._stream(stream))

    def set_nms_cluster(self, cluster: int) -> None:
        """CTAs per image of the NMS launches: 0 automatic, 1 / 2 / 4 / 8 fixed."""
        rc = load_library().octo_stage_set_nms_cluster(self.handle, int(cluster))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_stage_set_nms_cluster")

    def last_nms_cluster(self) -> int:
        return int(load_library().octo_stage_last_nms_cluster(self.handle))

    def last_nms_half_ctas(self) -> bool:
        return bool(load_library().octo_stage_last_nms_half_ctas(self.handle))

    def set_timing(self, enable: bool) -> None:
        rc = load_library().octo_stage_set_timing(self.handle, 1 if enable else 0)
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_stage_set_timing")

    def kernel_times(self, stream=None) -> dict:
        """{kernel: (summed ms, launches)} since the previous call; synchronises the stream."""
        kt = KernelTimes()
        rc = load_library().octo_stage_kernel_times(self.handle, ctypes.byref(kt), self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_stage_kernel_times")
        out = {name: (float(kt.ms[i]), int(kt.launches[i])) for i, name in enumerate(KERNEL_NAMES)}
        out["dropped"] = int(kt.dropped)
        return out

    @property
    def launch_count(self) -> int:
        return int(load_library().octo_stage_launch_count(self.handle))

    @property
    def workspace_bytes(self) -> int:
        return int(load_library().octo_stage_workspace_bytes(self.handle))


class Queue:
    """Device-side dynamic-batch queue of one downstream branch (octo_queue_* in octo.h)."""

    def __init__(self, capacity: int, out_w: int, out_h: int, max_bz: int, device: int = 0, swap_rb: bool = True):
        import torch
        self._torch = torch
        self.out_w, self.out_h, self.max_bz = out_w, out_h, max_bz
        self.device = torch.device("cuda", device)
        h = ctypes.c_void_p()
        rc = load_library().octo_queue_create(device, capacity, out_w, out_h, 1 if swap_rb else 0, max_bz,
                                              ctypes.byref(h))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_queue_create")
        self.handle = h
        self._keepalive = []

    def close(self) -> None:
        if getattr(self, "handle", None):
            load_library().octo_queue_destroy(self.handle)
            self.handle = None

    def _stream(self, stream) -> int:
        if stream is None:
            stream = self._torch.cuda.current_stream(self.device)
        return int(stream.cuda_stream)

    def set_options(self, keep_aspect: bool = False, mean=None, std=None, pad_value: int = 114) -> None:
        """Crop options of the downstream model (see octo_branch_cfg_t)."""
        br = BranchCfg()
        br.keep_aspect = 1 if keep_aspect else 0
        if mean is not None or std is not None:
            br.normalize = 1
            for k in range(3):
                br.mean[k] = float((mean or (0.0, 0.0, 0.0))[k])
                br.std[k] = float((std or (1.0, 1.0, 1.0))[k])
        rc = load_library().octo_queue_set_options(self.handle, ctypes.byref(br), pad_value)
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_queue_set_options")

    def push(self, stage: "Stage", branch: int = 0, stream=None) -> None:
        rc = load_library().octo_queue_push(self.handle, stage.handle, branch, self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_queue_push")
        self._keepalive.append(list(stage._frames_keepalive))  # frames stay alive while queued
        self._keepalive = self._keepalive[-64:]

    def pop(self, bz: int, out=None, items=None, info=None, stream=None, max_wait: int = -1):
        """Returns (crops fp16 [bz, 3, oh, ow], items uint8 [bz, 48], info int32 [4]).  With
        max_wait >= 0 the batch is only released when it is full or its first item has waited
        that many pushes (octo_queue_pop_due)."""
        t = self._torch
        if out is None:
            out = t.empty((bz, 3, self.out_h, self.out_w), dtype=t.float16, device=self.device)
        if items is None:
            items = t.zeros((bz, QITEM_DTYPE.itemsize), dtype=t.uint8, device=self.device)
        if info is None:
            info = t.zeros((4,), dtype=t.int32, device=self.device)
        rc = load_library().octo_queue_pop_due(self.handle, bz, max_wait, out.data_ptr(), items.data_ptr(),
                                               info.data_ptr(), self._stream(stream))
        if rc != OCTO_OK:
            raise OctoError(rc, "octo_queue_pop_due")
        return out, items, info


def octo_coral_schedule(instances: Sequence[dict], gpus: Sequence[dict]) -> List[Optional[Tuple[int, int, int, int, int]]]:
    """instances: dicts with the fields of octo_coral_instance_t; gpus: dicts with the fields of
    octo_coral_gpu_t.  Returns per instance (gpu, stream, start_us, end_us, duty_cycle_us) or None."""
    ia = (CoralInstance * max(len(instances), 1))()
    for k, d in enumerate(instances):
        for name, _ in CoralInstance._fields_:
            setattr(ia[k], name, int(d[name]))
    ga = (CoralGpu * max(len(gpus), 1))()
    for k, d in enumerate(gpus):
        for name, _ in CoralGpu._fields_:
            setattr(ga[k], name, int(d[name]))
    out = (CoralPlacement * max(len(instances), 1))()
    rc = load_library().octo_coral_schedule(ia, len(instances), ga, len(gpus), out)
    if rc != OCTO_OK:
        raise OctoError(rc, "octo_coral_schedule")
    return [None if out[k].gpu < 0 else (out[k].gpu, out[k].stream, out[k].start_us, out[k].end_us, out[k].duty_cycle_us)
            for k in range(len(instances))]


def dets_to_numpy(dets, counts) -> Tuple[np.ndarray, np.ndarray]:
    """Device (dets uint8 [n, max_det, 32], counts) -> host structured array + counts."""
    d = dets.cpu().numpy().view(DET_DTYPE).reshape(dets.shape[0], dets.shape[1])
    return d, counts.cpu().numpy()
