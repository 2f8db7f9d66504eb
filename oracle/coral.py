"""CPU oracle of the stream / portion placement (test infrastructure only).

Follows the paper's co-location scheduler (Section III-C, Algorithm 2) in its own notation:
FreePortions, pt, s = pt_stream, g = s_gpu, W_g / I_g / U_g, w_g / i_g / u_g, duty_cycle_r,
duty_cycle_s, DividePortion, UpdateList.  Where the paper is silent this oracle takes these
readings: FreePortions is ordered by portion length, then gpu, stream, start (so that the first
feasible portion is the best fit, "minimal empty space"); a stream with no duty cycle yet offers
one portion [0, infinity), cut to the duty cycle once the first instance fixes it; I_g is the sum
over the GPU's streams of I_s, the largest intermediate memory among a stream's residents; times
are integer microseconds.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

INF = float("inf")


@dataclass
class Instance:
    pipeline: int
    model: int
    instance: int
    start: int
    end: int
    duty_cycle: int
    W: int        # weight memory W_m
    I: int        # intermediate memory I_m
    U: int        # utilisation U_r (permille)


@dataclass
class Gpu:
    M: int        # memory M_g
    U_max: int    # utilisation limit U_g^max (permille)
    streams: int


def schedule(instances: Sequence[Instance], gpus: Sequence[Gpu]) -> List[Optional[Tuple[int, int, int, int, int]]]:
    """Returns per instance (gpu, stream, start, end, duty cycle of the stream) or None."""
    W = [0] * len(gpus)                                              # W_g
    I_s: Dict[Tuple[int, int], int] = {}                             # per stream
    U_s: Dict[Tuple[int, int], int] = {}                             # widest resident per stream
    duty: Dict[Tuple[int, int], int] = {}                            # duty_cycle_s (0 = unset)
    FreePortions: List[Tuple[int, int, float, float]] = []           # (gpu, stream, start, end)
    for g, gpu in enumerate(gpus):
        for s in range(gpu.streams):
            I_s[(g, s)] = 0
            U_s[(g, s)] = 0
            duty[(g, s)] = 0
            FreePortions.append((g, s, 0, INF))

    def key(pt):
        return (pt[3] - pt[2], pt[0], pt[1], pt[2])

    result: List[Optional[Tuple[int, int, int, int, int]]] = [None] * len(instances)
    # Main: instanceNumber = 0, 1, ...; for p in scheduledPipelines; for m in p
    numbers = sorted({r.instance for r in instances})
    pipelines = sorted({r.pipeline for r in instances})
    for instanceNumber in numbers:
        for p in pipelines:
            members = sorted((r.model, i) for i, r in enumerate(instances)
                             if r.pipeline == p and r.instance == instanceNumber)
            for _, i in members:
                r = instances[i]
                for pt in sorted(FreePortions, key=key):
                    g, s, pt_start, pt_end = pt
                    w_g = W[g] + r.W
                    I_g = sum(I_s[(g, q)] for q in range(gpus[g].streams))
                    i_g = I_g - I_s[(g, s)] + max(I_s[(g, s)], r.I)
                    u_g = sum(max(U_s[(g, q)], r.U) if q == s else U_s[(g, q)] for q in range(gpus[g].streams))
                    fully_available = pt_start <= r.start and pt_end >= r.end
                    sufficient = w_g + i_g <= gpus[g].M and u_g <= gpus[g].U_max
                    if fully_available and sufficient and r.duty_cycle >= duty[(g, s)]:
                        if duty[(g, s)] == 0:
                            duty[(g, s)] = r.duty_cycle
                        W[g] = w_g
                        I_s[(g, s)] = max(I_s[(g, s)], r.I)
                        U_s[(g, s)] = max(U_s[(g, s)], r.U)
                        # DividePortion / UpdateList
                        FreePortions.remove(pt)
                        cycle_end = min(pt_end, duty[(g, s)])
                        if pt_start < r.start:
                            FreePortions.append((g, s, pt_start, r.start))
                        if r.end < cycle_end:
                            FreePortions.append((g, s, r.end, cycle_end))
                        result[i] = (g, s, r.start, r.end, duty[(g, s)])
                        break
    return result
