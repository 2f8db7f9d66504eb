"""CPU oracle of the dynamic-batch queue (test infrastructure only).

The paper's batches fill from bursty arrivals and the first request of a batch waits longest
(Section II, discussion of Eq. 1; Section III-B, Observation 1); it gives no data structure.
Reading used here: a bounded first-in-first-out list of items per downstream branch.  A push
appends the branch's items of one detector batch in item order (frame by frame, NMS order
inside a frame) and stamps them with the push number; items that do not fit are dropped,
newest first; a pop removes the oldest min(bz, pending) items.  A pop with a waiting limit
releases only a full batch, or a partial one whose first item has waited for at least max_wait
pushes (an item queued by push number s has waited seq - 1 - s pushes after `seq` pushes).
"""
from __future__ import annotations

from typing import List, Tuple


class OracleQueue:
    def __init__(self, capacity: int):
        self.capacity = capacity
        self.pending: List[Tuple[int, int, int, Tuple[int, int, int, int], object]] = []
        self.dropped = 0
        self.seq = 0

    def push(self, items, rects, frames_of_batch) -> None:
        """items: [(frame, det)], rects: [(rx0, ry0, rx1, ry1)], frames_of_batch: per-frame payload
        (anything the caller needs to crop later, e.g. (pixels, w, h))."""
        for (f, j), r in zip(items, rects):
            if len(self.pending) < self.capacity:
                self.pending.append((self.seq, int(f), int(j), tuple(int(v) for v in r), frames_of_batch[int(f)]))
            else:
                self.dropped += 1
        self.seq += 1

    def pop(self, bz: int, max_wait: int = -1):
        """Returns (popped records, info) with info = (popped, pending after, dropped so far,
        seq of the oldest item still pending or -1)."""
        if max_wait >= 0 and len(self.pending) < bz:
            if not self.pending or self.seq - 1 - self.pending[0][0] < max_wait:
                oldest = self.pending[0][0] if self.pending else -1
                return [], (0, len(self.pending), self.dropped, oldest)
        out = self.pending[:bz]
        self.pending = self.pending[bz:]
        oldest = self.pending[0][0] if self.pending else -1
        return out, (len(out), len(self.pending), self.dropped, oldest)
