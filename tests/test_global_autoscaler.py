"""Global autoscaler primitives (Section 5): the library's C++ against hand-worked cases
(tests/golden/global_autoscaler_cases.txt), against the Python restatement in
oracle/global_autoscaler.py on random inputs, and against properties of the method."""
import os

import numpy as np
import pytest

from oracle import global_autoscaler as ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "global_autoscaler_cases.txt")


@pytest.fixture(scope="module")
def b():
    from paper_2501_08090_b200 import build
    build.build()
    from paper_2501_08090_b200 import binding
    return binding


def rows():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([x.strip() for x in line.split("|")])
    return out


def ints(s): return [int(x) for x in s.split()]
def flts(s): return [float(x) for x in s.split()]


@pytest.mark.parametrize("row", rows(), ids=[" ".join(r[:3]) for r in rows()])
def test_hand_worked_cases(b, row):
    kind = row[0]
    if kind == "wait":
        ahead, mu, sg, thr, z, want = int(row[1]), *map(float, row[2:7])
        assert ref.waiting_time(ahead, mu, sg, thr, z) == pytest.approx(want, rel=1e-12)
        assert b.waiting_time(ahead, mu, sg, thr, z) == pytest.approx(want, rel=1e-12)
    elif kind == "bbp":
        c, d = ints(row[1]), flts(row[2]); mu, sg, thr = map(float, row[3:6]); n, want = int(row[6]), int(row[7])
        assert ref.batch_backpressure(c, d, mu, sg, thr, n) == want
        assert b.batch_backpressure(c, d, mu, sg, thr, n) == want
    elif kind == "scale":
        c, d = ints(row[1]), flts(row[2]); mu, sg, thr = map(float, row[3:6])
        cur, active, cap, want = (int(x) for x in row[6:10])
        assert ref.batch_autoscale(c, d, mu, sg, thr, cur, active, cap) == want
        assert b.batch_autoscale(c, d, mu, sg, thr, cur, active, cap) == want
    elif kind == "ibp":
        busy, total = int(row[1]), int(row[2]); th, dl = float(row[3]), float(row[4]); fl, want = int(row[5]), int(row[6])
        assert ref.interactive_autoscale(busy, total, th, dl, fl) == want
        assert b.interactive_autoscale(busy, total, th, dl, fl) == want
    else:
        raise AssertionError(kind)


def test_request_groups_separate_interactive_from_batch_slos(b):
    # 10 s interactive TTFT SLOs and 1 h batch SLOs (Section 6 "Workloads"), some jitter
    rng = np.random.default_rng(0)
    slos = np.concatenate([10 + rng.uniform(-1, 1, 40), 3600 + rng.uniform(-200, 200, 25)])
    rng.shuffle(slos)
    grp, cent = b.request_groups(slos, 2)
    assert cent[0] == pytest.approx(10, abs=1) and cent[1] == pytest.approx(3600, abs=100)
    assert ((grp == 0) == (slos < 100)).all()
    rgrp, rcent = ref.request_groups(list(slos), 2)
    assert list(grp) == rgrp and np.allclose(cent, rcent, rtol=1e-12)


def test_random_parity_with_the_restatement(b):
    rng = np.random.default_rng(1)
    for trial in range(40):
        n = int(rng.integers(1, 60)); k = int(rng.integers(1, 6))
        slos = list(np.round(rng.choice([10, 60, 600, 3600], n) * rng.uniform(0.8, 1.2, n), 3))
        grp, cent = b.request_groups(slos, k)
        rgrp, rcent = ref.request_groups(slos, k)
        assert list(grp) == rgrp and np.allclose(cent, rcent, rtol=1e-12)
        g = int(rng.integers(1, 6))
        counts = [int(x) for x in rng.integers(0, 400, g)]
        deadlines = [float(x) for x in np.sort(rng.uniform(1, 4000, g))]
        mu, sg, thr = float(rng.uniform(50, 500)), float(rng.uniform(0, 200)), float(rng.uniform(200, 5000))
        z = float(rng.choice([0.0, 1.0, 2.33]))
        inst = int(rng.integers(1, 20))
        assert b.batch_backpressure(counts, deadlines, mu, sg, thr, inst, z) == ref.batch_backpressure(counts, deadlines, mu, sg, thr, inst, z)
        cur, act, cap = int(rng.integers(0, 5)), int(rng.integers(0, 3)), int(rng.integers(1, 40))
        assert b.batch_autoscale(counts, deadlines, mu, sg, thr, cur, act, cap, z) == ref.batch_autoscale(counts, deadlines, mu, sg, thr, cur, act, cap, z)
        busy, total = int(rng.integers(0, 30)), int(rng.integers(0, 60))
        th, dl, fl = float(rng.uniform(0.1, 0.9)), float(rng.uniform(0, 0.1)), int(rng.integers(0, 4))
        assert b.interactive_autoscale(busy, total, th, dl, fl) == ref.interactive_autoscale(busy, total, th, dl, fl)


def test_algorithm_2_adds_the_minimum_that_clears_the_backpressure(b):
    rng = np.random.default_rng(2)
    for _ in range(30):
        g = int(rng.integers(1, 5))
        counts = [int(x) for x in rng.integers(1, 500, g)]
        deadlines = [float(x) for x in np.sort(rng.uniform(5, 2000, g))]
        n = b.batch_autoscale(counts, deadlines, 200.0, 0.0, 1000.0, 0, 0, 10_000)
        assert b.batch_backpressure(counts, deadlines, 200.0, 0.0, 1000.0, n) == 0
        if n > 1:
            assert b.batch_backpressure(counts, deadlines, 200.0, 0.0, 1000.0, n - 1) > 0     # n - 1 was not enough


def test_waiting_time_grows_linearly_in_the_queue_and_shrinks_with_throughput(b):
    w1, w2 = b.waiting_time(100, 200, 0, 1000), b.waiting_time(200, 200, 0, 1000)
    assert w2 == pytest.approx(2 * w1) and b.waiting_time(100, 200, 0, 2000) == pytest.approx(w1 / 2)
    assert b.waiting_time(100, 200, 80, 1000, z=2.0) > w1                                     # conservative quantile


def test_interactive_band_prevents_hysteresis(b):
    theta, delta = 1 / 3, 0.05
    total = 30
    for busy in (9, 10, 11):                                     # IBP 0.30 .. 0.367: inside the band
        assert b.interactive_autoscale(busy, total, theta, delta) == total
    grown = b.interactive_autoscale(14, total, theta, delta)     # IBP 0.467: add instances
    assert grown == 42 and abs(14 / grown - theta) < 1e-9
    assert b.interactive_autoscale(5, total, theta, delta) == 15 # IBP 0.167: retire instances


def test_bad_arguments(b):
    with pytest.raises(b.CkvError):
        b.waiting_time(5, 100, 10, 0.0)
    with pytest.raises(b.CkvError):
        b.batch_backpressure([1], [1.0], 100, 0, 1000, 0)
    with pytest.raises(b.CkvError):
        b.interactive_autoscale(1, 1, 0.0, 0.1)
    with pytest.raises(b.CkvError):
        b.request_groups([], 2)
