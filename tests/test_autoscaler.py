"""Local autoscaler (Algorithm 1): the library's C++ implementation against hand-worked updates,
against the plain restatement in oracle/autoscaler.py, and closed-loop properties the paper states
(growth slows as backpressure approaches one; the loop settles where the ITL SLO binds)."""
import math
import os

import numpy as np
import pytest

from oracle import autoscaler as ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "algorithm1_cases.txt")


@pytest.fixture(scope="module")
def b():
    from paper_2501_08090_b200 import build
    build.build()
    from paper_2501_08090_b200 import binding
    return binding


def cases():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#") or line.startswith("seq"):
            continue
        name, slo, bs, itl, tp, tc, bp, after = [x.strip() for x in line.split("|")]
        out.append((name, float(slo), float(bs), float(itl), None if tp == "-" else float(tp), float(tc),
                    float(bp), float(after)))
    return out


@pytest.mark.parametrize("case", cases(), ids=[c[0] for c in cases()])
def test_worked_updates_of_algorithm_1(b, case):
    _, slo, bs, itl, thr_prev, thr, want_bp, want_bs = case
    # the oracle restatement
    _, _, bp = ref.backpressure(itl, slo, thr_prev, thr)
    assert bp == pytest.approx(want_bp, rel=1e-12)
    assert ref.update(bs, bp) == pytest.approx(want_bs, rel=1e-12)
    # the library
    a = b.LocalAutoscaler(itl_slo_us=slo, initial_max_bs=bs)
    if thr_prev is not None:                       # plant the previous throughput: an increase that lands on bs
        a2 = b.LocalAutoscaler(itl_slo_us=slo, initial_max_bs=bs / 1.5)
        got, _ = a2.update(slo * 0.5, thr_prev)    # BP = 0.5 -> x1.5, and the baseline is kept
        assert got == pytest.approx(bs)
        a = a2
    got_bs, got_bp = a.update(itl, thr)
    assert got_bp == pytest.approx(want_bp, rel=1e-12)
    assert got_bs == pytest.approx(want_bs, rel=1e-12)
    assert a.max_bs == got_bs


def test_random_update_sequences_match_the_restatement(b):
    rng = np.random.default_rng(5)
    for trial in range(20):
        slo = float(rng.uniform(50, 500)); alpha = float(rng.uniform(0.1, 1.0))
        lo, hi = 1.0, float(rng.choice([64, 4096]))
        a = b.LocalAutoscaler(slo, 16.0, alpha=alpha, min_bs=lo, max_bs=hi)
        max_bs, prev = 16.0, None
        for _ in range(200):
            itl = float(rng.uniform(0.2, 2.5) * slo); thr = float(rng.uniform(0.0, 5000.0))
            if rng.random() < 0.05:
                thr = 0.0
            _, _, bp = ref.backpressure(itl, slo, prev, thr)
            new_bs = ref.update(max_bs, bp, alpha, lo, hi)
            prev = thr if new_bs > max_bs else None
            max_bs = new_bs
            got, got_bp = a.update(itl, thr)
            assert got == pytest.approx(max_bs, rel=1e-12)
            assert (math.isinf(bp) and math.isinf(got_bp)) or got_bp == pytest.approx(bp, rel=1e-12)


def test_a_decrease_does_not_trigger_the_next_one(b):
    """After a halving the throughput is lower, but that is not 'no gain from an increase'."""
    a = b.LocalAutoscaler(itl_slo_us=200.0, initial_max_bs=64.0)
    bs, _ = a.update(400.0, 1000.0)                # over the SLO: halve
    assert bs == 32.0
    bs, bp = a.update(100.0, 600.0)                # lower throughput at the smaller batch, ITL fine
    assert bp == pytest.approx(0.5) and bs == 48.0
    bs, bp = a.update(150.0, 500.0)                # now an increase is being judged: throughput fell 600 -> 500
    assert bp == pytest.approx(1.2) and bs == 24.0


def two_update_cases():
    out = []
    for line in open(GOLDEN):
        if line.startswith("seq"):
            f = [x.strip() for x in line.split("|")]
            out.append((f[1], *[float(x) for x in f[2:]]))
    return out


@pytest.mark.parametrize("case", two_update_cases(), ids=[c[0] for c in two_update_cases()])
def test_the_two_readings_of_previous_throughput(b, case):
    reading, slo, bs0, itl1, thr1, bs1, itl2, thr2, bp2, bs2 = case
    literal = reading == "literal"
    # the restatement
    _, _, bp = ref.backpressure(itl1, slo, None, thr1)
    after1 = ref.update(bs0, bp)
    assert after1 == bs1
    base = ref.next_baseline(thr1, bs0, after1, literal)
    _, _, bp = ref.backpressure(itl2, slo, base, thr2)
    assert bp == pytest.approx(bp2, rel=1e-12) and ref.update(after1, bp) == bs2
    # the library
    a = b.LocalAutoscaler(itl_slo_us=slo, initial_max_bs=bs0, literal_tbp=literal)
    assert a.update(itl1, thr1)[0] == bs1
    got_bs, got_bp = a.update(itl2, thr2)
    assert got_bp == pytest.approx(bp2, rel=1e-12) and got_bs == bs2


def test_literal_previous_throughput_collapses_in_closed_loop(b):
    """On a curve whose throughput still rises with the batch, the literal TBP rule turns the first
    halving into a cascade down to a batch of one and never recovers more than a step; the default
    reading keeps probing the SLO point."""
    sizes, us = linear_curve()
    slo, extra = 1000.0, 200.0                                # ITL(bs) = 230 + 4 bs  ->  bs* = 192
    lit = b.autoscaler_simulate(slo, 4.0, sizes, us, extra, demand=10000, iterations=400, literal_tbp=True)
    want = ref.simulate(list(sizes), list(us), extra, slo, 10000, 4.0, 400, literal_tbp=True)
    assert np.allclose(lit[0], [r[0] for r in want], rtol=1e-12)
    dflt = b.autoscaler_simulate(slo, 4.0, sizes, us, extra, demand=10000, iterations=400)
    assert lit[1][100:].min() == 1                            # the cascade reaches a batch of one ...
    assert np.mean(lit[1][100:]) < 0.5 * np.mean(dflt[1][100:])   # ... and the loop serves far fewer requests per step
    assert dflt[1][100:].min() >= 40                          # the default keeps probing between half the peak and the peak


def test_instance_slo_is_the_smallest(b):
    assert b.instance_slo([2e6, 2e5, 2e6]) == 2e5            # one interactive request among batch requests
    assert ref.instance_slo([2e6, 2e5, 2e6]) == 2e5
    with pytest.raises(b.CkvError):
        b.instance_slo([])


def linear_curve():
    sizes = np.array([1, 2, 4, 8, 16, 32, 64, 128, 256, 512], dtype=np.float64)
    return sizes, 30.0 + 4.0 * sizes                          # us per step, attention-like growth


def test_closed_loop_matches_restatement_and_settles_under_the_slo(b):
    sizes, us = linear_curve()
    slo, extra = 1000.0, 200.0                                # ITL(bs) = 230 + 4 bs  ->  bs* = 192
    got = b.autoscaler_simulate(slo, 4.0, sizes, us, extra, demand=10000, iterations=300)
    want = ref.simulate(list(sizes), list(us), extra, slo, 10000, 4.0, 300)
    for k, row in enumerate(want):
        assert got[0][k] == pytest.approx(row[0], rel=1e-12) and got[1][k] == row[1]
        assert got[2][k] == pytest.approx(row[2], rel=1e-12)
    bs_run, itl_run = got[1][100:], got[2][100:]
    best = 192                                                # largest batch whose ITL meets the SLO
    # a saw-tooth: probe upward, halve, probe again -- between half the peak and the peak, under the SLO
    assert bs_run.max() <= best * 1.05 and bs_run.min() >= bs_run.max() // 2 - 1
    assert (itl_run <= slo * 1.05).all()
    # growth slows as the backpressure approaches one (Section 4.2)
    ups = [(got[3][k], got[0][k] / got[0][k - 1]) for k in range(1, 300) if got[3][k] < 1.0 and got[0][k - 1] > 0]
    ups.sort()
    assert ups[0][1] > ups[-1][1] >= 1.0


def test_closed_loop_stays_between_half_the_slo_point_and_the_slo_point(b):
    sizes = np.array([1, 512], dtype=np.float64)
    us = 10.0 + 4.0 * sizes                                   # cheap fixed cost: throughput is flat early
    slo = 400.0                                               # ITL(bs) = 10 + 4 bs  ->  bs* = 97
    o = b.autoscaler_simulate(slo, 4.0, sizes, us, 0.0, demand=100000, iterations=3000)
    want = ref.simulate(list(sizes), list(us), 0.0, slo, 100000, 4.0, 3000)
    assert np.allclose(o[0], [r[0] for r in want], rtol=1e-12)
    tail_bs, tail_itl = o[1][2000:], o[2][2000:]
    assert 0.5 * 97 <= tail_bs.max() <= 97 * 1.05             # peaks: above half the SLO point ...
    assert (tail_itl <= slo * 1.05).all()                     # ... and never past it
    assert tail_bs.min() >= tail_bs.max() // 2 - 1


def test_closed_loop_respects_demand_and_clamps(b):
    sizes, us = linear_curve()
    o = b.autoscaler_simulate(1e6, 1.0, sizes, us, 0.0, demand=8, iterations=50, max_bs=4096.0)
    assert (o[1] <= 8).all() and o[1][-1] == 8                # never runs more than there is
    assert o[0].max() <= 4096.0
    tight = b.autoscaler_simulate(10.0, 64.0, sizes, us, 0.0, demand=1000, iterations=50)
    assert tight[0][-1] == 1.0 and tight[1][-1] == 1          # SLO below the curve: pinned at the minimum


def test_bad_arguments_are_rejected(b):
    with pytest.raises(b.CkvError):
        b.LocalAutoscaler(itl_slo_us=0.0, initial_max_bs=8)
    with pytest.raises(b.CkvError):
        b.LocalAutoscaler(itl_slo_us=100.0, initial_max_bs=8, alpha=0.0)
    a = b.LocalAutoscaler(100.0, 8)
    with pytest.raises(b.CkvError):
        a.update(0.0, 10.0)
    with pytest.raises(b.CkvError):
        b.autoscaler_simulate(100.0, 8, [4, 2], [10, 20], 0.0, 10, 5)      # sizes not increasing
