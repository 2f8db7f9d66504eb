"""Stream / portion placement (the paper's co-location scheduler, Section III-C, Algorithm 2).  The
oracle (an exhaustive search over every stream for every instance) is pinned by hand-worked
placements and by properties that a replay with separate bookkeeping checks: windows on a stream
never overlap, a stream has one duty cycle and no resident with a shorter one, no GPU exceeds its
memory or utilisation at any point of the sequence, every placement took a gap no wider than any
other feasible gap, and an instance left out had nowhere to go.  The library's routine (interval
sets and running totals, a different construction) must agree with the oracle on random problems.
No GPU is involved: the routine makes no CUDA call."""
import numpy as np
import pytest

import paper_2502_01277_b200 as octo
from oracle import coral
from oracle.coral import Gpu, Instance

MB = 1 << 20


def _inst(p, m, k, start, end, duty, W=100 * MB, I=50 * MB, U=300):
    return Instance(p, m, k, start, end, duty, W, I, U)


def _lib(instances, gpus):
    return octo.octo_coral_schedule(
        [dict(pipeline=r.pipeline, model=r.model, instance=r.instance, util_permille=r.U, start_us=r.start,
              end_us=r.end, duty_cycle_us=r.duty_cycle, weight_bytes=r.W, inter_bytes=r.I) for r in instances],
        [dict(mem_bytes=g.M, util_max_permille=g.U_max, num_streams=g.streams) for g in gpus])


def _check_valid(instances, gpus, placed):
    """Replays the placements in scheduling order with bookkeeping of its own (busy intervals per
    stream, totals per GPU) and checks every property a correct schedule has."""
    busy = {}      # (g, s) -> [(start, end)]
    duty = {}      # (g, s) -> duty cycle
    inter = {}     # (g, s) -> largest intermediate memory
    width = {}     # (g, s) -> widest resident
    weights = [0] * len(gpus)

    def feasible_gaps(r):
        gaps = []
        for g, gpu in enumerate(gpus):
            for s in range(gpu.streams):
                k = (g, s)
                if duty.get(k, 0) > r.duty_cycle:
                    continue
                if any(a < r.end and r.start < b for a, b in busy.get(k, [])):
                    continue
                if k in duty and r.end > duty[k]:
                    continue
                mem = weights[g] + r.W + sum(max(v, r.I) if kk == k else v for kk, v in inter.items() if kk[0] == g)
                util = sum(max(v, r.U) if kk == k else v for kk, v in width.items() if kk[0] == g)
                if k not in inter:
                    mem, util = mem + r.I, util + r.U
                if mem > gpu.M or util > gpu.U_max:
                    continue
                lo = max([b for a, b in busy.get(k, []) if b <= r.start], default=0)
                hi = min([a for a, b in busy.get(k, []) if a >= r.end], default=duty.get(k, float("inf")))
                gaps.append((hi - lo, g, s))
        return gaps

    for i in coral.scheduling_order(instances):
        r, pl = instances[i], placed[i]
        gaps = feasible_gaps(r)
        if pl is None:
            assert not gaps, f"instance {i} was left out although a portion fits: {gaps}"
            continue
        g, s, a, b, d = pl
        assert (a, b) == (r.start, r.end)
        mine = [t for t in gaps if t[1:] == (g, s)]
        assert mine, f"instance {i} sits where it does not fit"
        assert mine[0][0] == min(gaps)[0], "a tighter portion was free"       # best fit
        assert mine[0] == min(gaps), "ties go to the lower GPU, then stream"  # the stated tie rule
        k = (g, s)
        duty.setdefault(k, r.duty_cycle)
        assert d == duty[k] <= r.duty_cycle and b <= d
        busy.setdefault(k, []).append((a, b))
        inter[k] = max(inter.get(k, 0), r.I)
        width[k] = max(width.get(k, 0), r.U)
        weights[g] += r.W
    # the final state once more, from the placements alone
    by_stream = {}
    for r, pl in zip(instances, placed):
        if pl is not None:
            by_stream.setdefault(pl[:2], []).append((pl[2], pl[3], pl[4], r))
    for lst in by_stream.values():
        lst.sort(key=lambda t: t[0])
        assert len({d for _, _, d, _ in lst}) == 1                     # one duty cycle per stream
        for (a0, b0, _, _), (a1, b1, _, _) in zip(lst, lst[1:]):
            assert b0 <= a1                                            # portions never overlap
    for g, gpu in enumerate(gpus):
        res = [(k, v) for k, v in by_stream.items() if k[0] == g]
        mem = sum(r.W for _, lst in res for *_, r in lst) + sum(max(r.I for *_, r in lst) for _, lst in res)
        util = sum(max(r.U for *_, r in lst) for _, lst in res)
        assert mem <= gpu.M and util <= gpu.U_max


def test_the_checker_rejects_wrong_schedules():
    """The replay is only worth something if it fails on mistakes: a placement moved to a wider
    gap, a placement dropped, two overlapping windows."""
    inst = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(0, 1, 0, 40_000, 50_000, 50_000),
            _inst(1, 0, 0, 0, 18_000, 50_000), _inst(1, 1, 0, 30_000, 50_000, 50_000),
            _inst(2, 0, 0, 19_000, 29_000, 50_000)]
    gpus = [Gpu(8 << 30, 1000, 2)]
    good = coral.schedule(inst, gpus)
    _check_valid(inst, gpus, good)
    worse = list(good)
    worse[4] = (0, 0, 19_000, 29_000, 50_000)       # fits on stream 0 too, but in the wider gap
    with pytest.raises(AssertionError):
        _check_valid(inst, gpus, worse)
    dropped = list(good)
    dropped[4] = None
    with pytest.raises(AssertionError):
        _check_valid(inst, gpus, dropped)
    clash = list(good)
    clash[2] = (0, 0, 0, 18_000, 50_000)            # overlaps pipeline 0's first window
    with pytest.raises(AssertionError):
        _check_valid(inst, gpus, clash)


def test_pipeline_models_follow_each_other_on_one_stream():
    """A three-model pipeline, windows back to back inside a 100 ms cycle, one GPU with one stream."""
    inst = [_inst(0, 0, 0, 0, 20_000, 100_000), _inst(0, 1, 0, 20_000, 50_000, 100_000),
            _inst(0, 2, 0, 50_000, 60_000, 100_000)]
    got = coral.schedule(inst, [Gpu(8 << 30, 1000, 1)])
    assert got == [(0, 0, 0, 20_000, 100_000), (0, 0, 20_000, 50_000, 100_000), (0, 0, 50_000, 60_000, 100_000)]


def test_best_fit_takes_the_tightest_gap():
    """Two streams hold gaps of 30 ms and 12 ms that both cover the 10 ms window: the 12 ms gap wins,
    although the other stream comes first."""
    inst = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(0, 1, 0, 40_000, 50_000, 50_000),   # stream 0: gap 10..40
            _inst(1, 0, 0, 0, 18_000, 50_000), _inst(1, 1, 0, 30_000, 50_000, 50_000),   # stream 1: gap 18..30
            _inst(2, 0, 0, 19_000, 29_000, 50_000)]
    got = coral.schedule(inst, [Gpu(8 << 30, 1000, 2)])
    assert got[0][:2] == (0, 0) and got[1][:2] == (0, 0)
    # pipeline 1's first model fits nowhere on stream 0 (window 0..18 ms is taken) -> stream 1
    assert got[2][:2] == (0, 1) and got[3][:2] == (0, 1)
    assert got[4] == (0, 1, 19_000, 29_000, 50_000)


def test_resource_limits_and_duty_cycle_rule():
    # memory: W 100 + I 50 per instance, 240 MB per GPU -> the second instance needs the other GPU
    inst = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(1, 0, 0, 20_000, 30_000, 50_000)]
    got = coral.schedule(inst, [Gpu(240 * MB, 1000, 2), Gpu(240 * MB, 1000, 2)])
    assert got[0][0] == 0 and got[1][0] == 1
    # on one stream the intermediate memory is shared (max, not sum): 100 + 100 + 50 = 250 MB fits 260 MB
    got = coral.schedule(inst, [Gpu(260 * MB, 1000, 1)])
    assert got[0][:2] == (0, 0) and got[1][:2] == (0, 0)
    # utilisation: two streams of width 600 exceed 1000, the same stream does not
    wide = [_inst(0, 0, 0, 0, 10_000, 50_000, U=600), _inst(1, 0, 0, 0, 10_000, 50_000, U=600)]
    assert coral.schedule(wide, [Gpu(8 << 30, 1000, 2)]) == [(0, 0, 0, 10_000, 50_000), None]
    # duty cycle: a 50 ms pipeline may not join a stream that cycles every 100 ms, the reverse is fine
    a = [_inst(0, 0, 0, 0, 10_000, 100_000), _inst(1, 0, 0, 20_000, 30_000, 50_000)]
    assert coral.schedule(a, [Gpu(8 << 30, 1000, 1)]) == [(0, 0, 0, 10_000, 100_000), None]
    b = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(1, 0, 0, 20_000, 30_000, 100_000)]
    assert coral.schedule(b, [Gpu(8 << 30, 1000, 1)]) == [(0, 0, 0, 10_000, 50_000), (0, 0, 20_000, 30_000, 50_000)]
    # ... but not with a window that ends after the shorter cycle
    c = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(1, 0, 0, 45_000, 60_000, 100_000)]
    assert coral.schedule(c, [Gpu(8 << 30, 1000, 1)])[1] is None


def test_first_instances_of_all_pipelines_come_before_second_instances():
    """One stream, room for two windows: both pipelines get their first instance, the replicas
    (same windows) find nothing, whatever the order of the input list."""
    inst = [_inst(0, 0, 1, 0, 10_000, 40_000), _inst(0, 0, 0, 0, 10_000, 40_000),
            _inst(1, 0, 1, 10_000, 20_000, 40_000), _inst(1, 0, 0, 10_000, 20_000, 40_000)]
    got = coral.schedule(inst, [Gpu(8 << 30, 1000, 1)])
    assert got[1] is not None and got[3] is not None and got[0] is None and got[2] is None


def _random_problem(rng):
    gpus = [Gpu(int(rng.integers(300, 2000)) * MB, int(rng.integers(500, 1001)), int(rng.integers(1, 4)))
            for _ in range(int(rng.integers(1, 4)))]
    inst = []
    for p in range(int(rng.integers(1, 5))):
        duty = int(rng.choice([50_000, 100_000, 150_000]))
        n_models = int(rng.integers(1, 5))
        cuts = np.sort(rng.choice(np.arange(1, duty // 1000), size=n_models, replace=False)) * 1000
        starts = np.concatenate([[0], cuts[:-1]])
        for m in range(n_models):
            for k in range(int(rng.integers(1, 4))):
                inst.append(Instance(p, m, k, int(starts[m]), int(cuts[m]), duty, int(rng.integers(20, 300)) * MB,
                                     int(rng.integers(10, 200)) * MB, int(rng.integers(50, 700))))
    order = rng.permutation(len(inst))
    return [inst[i] for i in order], gpus


def test_oracle_placements_are_valid_on_random_problems():
    rng = np.random.default_rng(0)
    placed_any = 0
    for _ in range(200):
        inst, gpus = _random_problem(rng)
        got = coral.schedule(inst, gpus)
        _check_valid(inst, gpus, got)
        placed_any += sum(g is not None for g in got)
    assert placed_any > 500


def test_library_matches_the_oracle_on_random_problems():
    rng = np.random.default_rng(1)
    some_unplaced = 0
    for _ in range(300):
        inst, gpus = _random_problem(rng)
        want = coral.schedule(inst, gpus)
        got = _lib(inst, gpus)
        assert got == want
        some_unplaced += sum(w is None for w in want)
    assert some_unplaced > 50


def test_library_on_the_hand_worked_cases_and_bad_arguments():
    inst = [_inst(0, 0, 0, 0, 10_000, 50_000), _inst(0, 1, 0, 40_000, 50_000, 50_000),
            _inst(1, 0, 0, 0, 18_000, 50_000), _inst(1, 1, 0, 30_000, 50_000, 50_000),
            _inst(2, 0, 0, 19_000, 29_000, 50_000)]
    gpus = [Gpu(8 << 30, 1000, 2)]
    assert _lib(inst, gpus) == coral.schedule(inst, gpus)
    assert _lib([], gpus) == []
    with pytest.raises(octo.OctoError):
        _lib([_inst(0, 0, 0, 10, 5, 100)], gpus)          # empty window
    with pytest.raises(octo.OctoError):
        _lib([_inst(0, 0, 0, 0, 200, 100)], gpus)         # window outside the duty cycle
    with pytest.raises(octo.OctoError):
        _lib(inst, [Gpu(1 << 30, 1000, 0)])               # a GPU without streams
