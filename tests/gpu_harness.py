"""Helpers for the GPU parity tests: run a workload batch through the C-ABI library and
bring every result back to the host."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

import paper_2502_01277_b200 as octo


@dataclass
class GpuResult:
    det_in: np.ndarray  # uint16 [n, 3, S, S]
    dets: np.ndarray  # DET_DTYPE [n, max_det]
    counts: np.ndarray  # int32 [n]
    offsets: List[np.ndarray] = field(default_factory=list)
    n_items: List[Tuple[int, int]] = field(default_factory=list)
    items: List[np.ndarray] = field(default_factory=list)  # ITEM_DTYPE [packed]
    crops: List[np.ndarray] = field(default_factory=list)  # uint16 [max_items, 3, oh, ow]
    status: int = 0
    stats: dict = field(default_factory=dict)


def upload_frames(frames: Sequence[np.ndarray], device="cuda:0") -> List[torch.Tensor]:
    return [torch.from_numpy(np.ascontiguousarray(f)).to(device) for f in frames]


def make_stage(wl, max_batch: int, **over) -> "octo.Stage":
    kw = dict(net_size=wl.net_size, max_batch=max_batch, num_anchors=wl.num_anchors,
              num_classes=wl.num_classes, head_is_logits=wl.logits, conf_thresh=wl.conf_thresh,
              iou_thresh=wl.iou_thresh, max_det=wl.max_det, branches=wl.branches,
              head_layout=wl.head_layout, multi_label=wl.multi_label)
    kw.update(over)
    return octo.Stage(**kw)


def run_stage_gpu(stage, frames: Sequence[np.ndarray], sizes, head: np.ndarray,
                  max_items: Optional[Sequence[int]] = None, first_item: int = 0,
                  stream: Optional[torch.cuda.Stream] = None, sentinel: int = 0x7BFF,
                  preprocess_stream: Optional[torch.cuda.Stream] = None) -> GpuResult:
    """One pass of the whole stage.  Output buffers are pre-filled with a sentinel so that
    untouched slots can be recognised.  With preprocess_stream the letterbox is enqueued there,
    beside the other kernels of the pass, and joined before the results are read."""
    dev = stage.device
    n = len(frames)
    d_frames = upload_frames(frames, dev)
    d_head = torch.from_numpy(head).to(dev)
    s = stage.cfg.net_size
    ctx = torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream(dev))
    with ctx:
        det_in = torch.full((n, 3, s, s), 0, dtype=torch.int16, device=dev)
        det_in.fill_(sentinel)
        if preprocess_stream is not None:
            main = torch.cuda.current_stream(dev)
            preprocess_stream.wait_stream(main)  # the sentinel fill above
            stage.preprocess(d_frames, sizes, out=det_in.view(torch.float16), stream=preprocess_stream)
        else:
            stage.preprocess(d_frames, sizes, out=det_in.view(torch.float16))
        dets = torch.zeros((n, stage.cfg.max_det, 32), dtype=torch.uint8, device=dev)
        counts = torch.full((n,), -1, dtype=torch.int32, device=dev)
        stage.postprocess(d_head, dets=dets, counts=counts)
        res = GpuResult(None, None, None)
        outs = []
        for b in range(stage.cfg.num_branches):
            ow, oh = stage.cfg.branch[b].out_w, stage.cfg.branch[b].out_h
            mi = max_items[b] if max_items is not None else n * stage.cfg.max_det
            buf = torch.full((max(mi, 1), 3, oh, ow), sentinel, dtype=torch.int16, device=dev)
            out, offsets, n_items = stage.crop(b, mi, first_item=first_item, out=buf.view(torch.float16))
            outs.append((buf, offsets, n_items))
    torch.cuda.synchronize(dev)
    res.det_in = det_in.cpu().numpy().view(np.uint16)
    res.dets, res.counts = octo.dets_to_numpy(dets, counts)
    for b, (buf, offsets, n_items) in enumerate(outs):
        ni = n_items.cpu().numpy()
        res.offsets.append(offsets.cpu().numpy())
        res.n_items.append((int(ni[0]), int(ni[1])))
        res.items.append(stage.item_table(b, int(ni[0])))
        res.crops.append(buf.cpu().numpy().view(np.uint16))
    res.status = stage.status()
    res.stats = stage.stats()
    return res


def half_absdiff(a_bits: np.ndarray, b_bits: np.ndarray, chunk: int = 1 << 24) -> float:
    """Largest |a - b| over two arrays of binary16 bit patterns, taken in slices so that a
    whole batch of crops (gigabytes) never exists as float32 at once."""
    assert a_bits.shape == b_bits.shape
    a = np.ascontiguousarray(a_bits).reshape(-1)
    b = np.ascontiguousarray(b_bits).reshape(-1)
    worst = 0.0
    for lo in range(0, a.size, chunk):
        x = a[lo:lo + chunk].view(np.float16).astype(np.float32)
        y = b[lo:lo + chunk].view(np.float16).astype(np.float32)
        worst = max(worst, float(np.max(np.abs(x - y))))
    return worst
