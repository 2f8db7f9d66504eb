"""CPU oracle of the stream / portion placement (test infrastructure only).

The paper's co-location scheduler (Section III-C, Algorithm 2) places model instances on the
streams of GPUs: one replica number at a time over all pipelines and their models; each
instance takes, among the free portions that cover its window, keep the GPU within memory and
utilisation and lie on a stream whose duty cycle is not longer than the instance's, the one with
the least empty space.  This oracle is that statement written as an exhaustive search: nothing is
kept between instances except the list of placements made so far; every quantity (the free gap of
a stream around the window, a GPU's memory and utilisation with the newcomer) is recomputed from
that list for every stream of every GPU, and the feasible candidate with the smallest gap wins.
Readings where the paper is silent: ties go to the lower GPU, then the lower stream; a stream
without residents has no duty cycle and counts as an unbounded gap; a GPU's intermediate memory is
the sum over its streams of the largest intermediate memory among the stream's residents, its
utilisation the sum over its streams of the widest resident; times are integer microseconds.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

INF = float("inf")


@dataclass
class Instance:
    pipeline: int
    model: int
    instance: int
    start: int
    end: int
    duty_cycle: int
    W: int        # weight memory
    I: int        # intermediate memory
    U: int        # utilisation (permille)


@dataclass
class Gpu:
    M: int        # memory
    U_max: int    # utilisation limit (permille)
    streams: int


def scheduling_order(instances: Sequence[Instance]) -> List[int]:
    """Indices in the order the instances are placed: replica number, pipeline, model."""
    return sorted(range(len(instances)), key=lambda i: (instances[i].instance, instances[i].pipeline,
                                                        instances[i].model, i))


def candidates(r: Instance, placed: Sequence[Tuple[Instance, int, int]], gpus: Sequence[Gpu]):
    """Every (gap length, gpu, stream) where r could go, given the placements made so far
    (`placed` = [(instance, gpu, stream)]), by exhaustive search."""
    out = []
    for g, gpu in enumerate(gpus):
        on_gpu = [(q, s) for q, gg, s in placed if gg == g]
        for s in range(gpu.streams):
            res = [q for q, ss in on_gpu if ss == s]
            duty = res[0].duty_cycle if res else 0  # the first resident fixed it (placements are in order)
            if duty > r.duty_cycle:
                continue
            if any(q.start < r.end and r.start < q.end for q in res):
                continue  # the window is not free
            if res and r.end > duty:
                continue  # the window does not lie inside the stream's cycle
            lo = max([q.end for q in res if q.end <= r.start], default=0)
            hi = min([q.start for q in res if q.start >= r.end], default=(duty if res else INF))
            streams = {}
            for q, ss in on_gpu + [(r, s)]:
                streams.setdefault(ss, []).append(q)
            mem = sum(q.W for q, _ in on_gpu) + r.W + sum(max(q.I for q in lst) for lst in streams.values())
            util = sum(max(q.U for q in lst) for lst in streams.values())
            if mem > gpu.M or util > gpu.U_max:
                continue
            out.append((hi - lo, g, s))
    return out


def schedule(instances: Sequence[Instance], gpus: Sequence[Gpu]) -> List[Optional[Tuple[int, int, int, int, int]]]:
    """Returns per instance (gpu, stream, start, end, duty cycle of the stream) or None."""
    placed: List[Tuple[Instance, int, int]] = []
    result: List[Optional[Tuple[int, int, int, int, int]]] = [None] * len(instances)
    for i in scheduling_order(instances):
        r = instances[i]
        cands = candidates(r, placed, gpus)
        if not cands:
            continue
        _, g, s = min(cands)
        placed.append((r, g, s))
        duty = next(q.duty_cycle for q, gg, ss in placed if (gg, ss) == (g, s))
        result[i] = (g, s, r.start, r.end, duty)
    return result
