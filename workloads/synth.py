"""Workload recipes and the ctypes front end of the C generator (gen.c).

The five recipes mirror the configurations the stage is evaluated on: a tiny single-frame
case, an 8-frame 1080p traffic batch, a 64-frame mixed 720p/1080p batch feeding two
downstream branches, a dense-scene NMS stress batch and a batch-size sweep.  Frames are
camera-shaped synthetic images; heads are YOLOv5-layout tensors with a controlled number
of above-threshold, clustered candidates.  They replace the paper's recorded camera
streams (Section V-A, "Data"), which cannot be shipped.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libwlgen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libwlgen.so next to it (gcc; a second or two)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u8p = ctypes.POINTER(ctypes.c_uint8)
        f32p = ctypes.POINTER(ctypes.c_float)
        i32, u64, f32 = ctypes.c_int32, ctypes.c_uint64, ctypes.c_float
        for name in ("wl_frame_uniform", "wl_frame_smooth"):
            fn = getattr(lib, name)
            fn.argtypes = [u64, i32, i32, i32, i32, u8p]
            fn.restype = None
        lib.wl_head.argtypes = [u64, i32, i32, i32, i32, i32, i32] + [f32] * 10 + [i32, f32p]
        lib.wl_head.restype = None
        lib.wl_coin.argtypes = [u64, i32]
        lib.wl_coin.restype = i32
        _lib = lib
    return _lib


def num_anchors(net_size: int) -> int:
    """Three anchors per cell on the stride-8, -16 and -32 grids of a square input."""
    return 3 * sum((net_size // s) ** 2 for s in (8, 16, 32))


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    net_size: int
    frame_sizes: Tuple[Tuple[int, int], ...]  # candidate (w, h); >1 entries => mixed by coin
    batch: int
    frame_kind: str  # "uniform" | "smooth"
    n_raised: int
    n_groups: int
    size_range: Tuple[float, float]
    jitter: float
    scale_range: Tuple[float, float]
    max_det: int
    branches: Tuple[Tuple[int, int], ...]  # (out_w, out_h) per downstream branch
    num_classes: int = 80
    conf_thresh: float = 0.25
    iou_thresh: float = 0.45
    logits: bool = True
    # capacity (crops per frame) a caller would provision for the downstream batch
    items_per_frame: int = 64
    # canvas rows [lo, hi) in which raised boxes are placed so that crops land on image
    # content (rows 140..500 hold a 16:9 frame on a 640 canvas); a recipe constant
    box_rows: Tuple[float, float] = (140.0, 500.0)
    # "rows": head [N, A, 5 + C] with an objectness column; "planes": anchor-free head
    # [N, 4 + C, A] (one prediction per grid cell, no objectness column)
    head_layout: str = "rows"
    multi_label: bool = False
    bg_mean: float = -4.0  # mean of the background obj / class logits

    @property
    def num_anchors(self) -> int:
        return num_anchors(self.net_size) // (3 if self.head_layout == "planes" else 1)


WORKLOADS = {
    "tiny": Workload("tiny", 0, 320, ((320, 240),), 1, "uniform", 40, 40, (8.0, 120.0), 0.0,
                     (1.0, 1.0), 300, ((64, 64),), items_per_frame=64, box_rows=(40.0, 280.0)),
    "traffic_1080p": Workload("traffic_1080p", 1, 640, ((1920, 1080),), 8, "smooth", 150, 20,
                              (40.0, 200.0), 0.15, (0.8, 1.25), 300, ((224, 224),)),
    "two_branch": Workload("two_branch", 2, 640, ((1280, 720), (1920, 1080)), 64, "smooth", 150,
                           20, (40.0, 200.0), 0.15, (0.8, 1.25), 300, ((224, 224), (256, 256))),
    "dense_nms": Workload("dense_nms", 3, 640, ((1920, 1080),), 32, "smooth", 5000, 250,
                          (40.0, 200.0), 0.25, (0.7, 1.4), 1000, ((128, 128),),
                          items_per_frame=1000),
    "sweep": Workload("sweep", 4, 640, ((1920, 1080),), 64, "smooth", 200, 25, (40.0, 200.0),
                      0.15, (0.8, 1.25), 300, ((224, 224),)),
    # decode variant: the sweep recipe with an anchor-free head in planes layout.  Without an
    # objectness factor the score is the class value alone, so the background class logits sit
    # lower (-7) to keep background candidates as rare as in the other recipes.
    "anchor_free": Workload("anchor_free", 5, 640, ((1920, 1080),), 64, "smooth", 200, 25, (40.0, 200.0),
                            0.15, (0.8, 1.25), 300, ((224, 224),), head_layout="planes", bg_mean=-7.0),
}


@dataclass
class Batch:
    workload: Workload
    frames: List[np.ndarray]  # each uint8 [h, pitch]; pixel (y, x) = row[3x : 3x+3] in B, G, R
    sizes: List[Tuple[int, int]]  # (w, h) per frame
    head: np.ndarray  # float32 [N, A, 5 + C] (rows layout) or [N, 4 + C, A] (planes layout)
    first_frame: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return len(self.frames)


def _pitch(w: int) -> int:
    return (3 * w + 15) // 16 * 16


def make_batch(name_or_workload, batch: Optional[int] = None, first_frame: int = 0,
               threads: Optional[int] = None, seed: Optional[int] = None) -> Batch:
    """Generate `batch` frames and heads of a workload, starting at global frame index
    `first_frame` (ranks of a multi-GPU run take disjoint index ranges)."""
    wl = WORKLOADS[name_or_workload] if isinstance(name_or_workload, str) else name_or_workload
    if batch is not None:
        wl = replace(wl, batch=int(batch))
    if seed is not None:
        wl = replace(wl, seed=int(seed))
    lib = _load()
    n, s, a, c = wl.batch, wl.net_size, wl.num_anchors, wl.num_classes
    sizes: List[Tuple[int, int]] = []
    for i in range(n):
        gi = first_frame + i
        if len(wl.frame_sizes) == 1:
            sizes.append(wl.frame_sizes[0])
        else:
            sizes.append(wl.frame_sizes[lib.wl_coin(wl.seed, gi) % len(wl.frame_sizes)])
    frames = [np.empty((h, _pitch(w)), dtype=np.uint8) for (w, h) in sizes]
    planes = wl.head_layout == "planes"
    head = np.empty((n, 4 + c, a) if planes else (n, a, 5 + c), dtype=np.float32)
    u8p = ctypes.POINTER(ctypes.c_uint8)
    f32p = ctypes.POINTER(ctypes.c_float)
    fgen = lib.wl_frame_uniform if wl.frame_kind == "uniform" else lib.wl_frame_smooth

    def one(i: int) -> None:
        gi = first_frame + i
        w, h = sizes[i]
        fgen(wl.seed, gi, w, h, frames[i].shape[1], frames[i].ctypes.data_as(u8p))
        y_lo, y_hi = wl.box_rows
        rows = np.empty((a, 5 + c), dtype=np.float32) if planes else head[i]
        lib.wl_head(wl.seed, gi, s, a, c, wl.n_raised, wl.n_groups, y_lo, y_hi,
                    wl.size_range[0], wl.size_range[1], wl.jitter, wl.scale_range[0],
                    wl.scale_range[1], wl.bg_mean, 2.0, 0.5, 1 if wl.logits else 0,
                    rows.ctypes.data_as(f32p))
        if planes:
            head[i] = rows_to_planes(rows)

    nthreads = threads or min(n, os.cpu_count() or 1)
    if nthreads <= 1 or n == 1:
        for i in range(n):
            one(i)
    else:
        with ThreadPoolExecutor(max_workers=nthreads) as ex:
            list(ex.map(one, range(n)))
    return Batch(wl, frames, sizes, head, first_frame)


def rows_to_planes(rows: np.ndarray) -> np.ndarray:
    """Layout change only: rows [A, 5 + C] -> planes [4 + C, A] with the objectness column dropped."""
    return np.ascontiguousarray(np.concatenate([rows[:, :4], rows[:, 5:]], axis=1).T)


def make_heads(seed: int, n: int, net_size: int, num_classes: int = 80, n_raised: int = 10, n_groups: int = 4,
               size_range: Tuple[float, float] = (30.0, 120.0), jitter: float = 0.15,
               scale_range: Tuple[float, float] = (0.8, 1.25), first: int = 0, logits: bool = True) -> np.ndarray:
    """Heads [n, A, 5 + C] of a chained (second-level) detector whose input is an upstream crop
    stretched to net_size x net_size: same recipe as the frame heads, boxes anywhere on the grid."""
    lib = _load()
    a = num_anchors(net_size)
    head = np.empty((n, a, 5 + num_classes), dtype=np.float32)
    f32p = ctypes.POINTER(ctypes.c_float)
    for i in range(n):
        lib.wl_head(seed, first + i, net_size, a, num_classes, n_raised, n_groups, 0.0, float(net_size),
                    size_range[0], size_range[1], jitter, scale_range[0], scale_range[1], -4.0, 2.0, 0.5,
                    1 if logits else 0, head[i].ctypes.data_as(f32p))
    return head


def shard_range(total: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [begin, end) slice of `total` frames owned by `rank` of `world`."""
    base, rem = divmod(total, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
