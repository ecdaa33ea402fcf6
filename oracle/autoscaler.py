"""Plain restatement of the paper's batch-size autoscaling (Algorithm 1, Section 4.2 "Batch Size
Autoscaling", with the backpressure definitions of Section 4.1 "Local Backpressure").

TEST INFRASTRUCTURE ONLY, like the rest of oracle/: the library's C++ autoscaler shares no code
with this file and never imports it.

Per update (one per change of the running queue):
    LBP = ITL / ITL_SLO
    TBP = Throughput_prev / Throughput_curr          (no previous observation: 0)
    BP  = max(LBP, TBP)
    BP < 1 :  MaxBS <- alpha * (1/BP) * MaxBS + (1 - alpha) * MaxBS      (alpha = 0.5)
    else   :  MaxBS <- MaxBS / 2
The instance's ITL SLO is the smallest ITL SLO among the requests it runs.

Readings where the text leaves room: BP exactly 1 halves (the algorithm's `< 1` test decides, not
the prose's "greater than one"); MaxBS is kept as a real number clamped to [min_bs, max_bs]; the
batch the instance actually runs is floor(MaxBS) capped by the demand; a zero current throughput
counts as infinite backpressure.

Which throughput is "previous".  Printed rule (`literal_tbp=True` below): the throughput observed
at the update before, whatever that update did.  Default reading: Section 4.1 introduces TBP as
the check on whether a larger batch still buys throughput, so the previous throughput is kept
only across an update that INCREASED MaxBS; after a decrease (or at the start) there is none and
TBP = 0.  The literal rule is unstable in closed loop: on the rising part of the curve a halving
lowers the throughput, TBP reads above one at the next update, and each halving triggers the
next, down to a batch of one.  Both are implemented here and in the library and tested side by
side.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple


def backpressure(itl: float, itl_slo: float, thr_prev: Optional[float], thr_curr: float) -> Tuple[float, float, float]:
    lbp = itl / itl_slo
    if thr_prev is None:
        tbp = 0.0
    elif thr_curr <= 0.0:
        tbp = math.inf
    else:
        tbp = thr_prev / thr_curr
    return lbp, tbp, max(lbp, tbp)


def update(max_bs: float, bp: float, alpha: float = 0.5, min_bs: float = 1.0, max_cap: float = 1e9) -> float:
    if bp < 1.0:
        new = alpha * (1.0 / bp) * max_bs + (1.0 - alpha) * max_bs if bp > 0.0 else max_cap
    else:
        new = max_bs / 2.0
    return min(max(new, min_bs), max_cap)


def instance_slo(slos: Sequence[float]) -> float:
    return min(slos)


def interp_latency(batch_sizes: Sequence[float], us: Sequence[float], bs: float) -> float:
    """Piecewise-linear latency curve; beyond the last point the last slope continues."""
    n = len(batch_sizes)
    if n == 1 or bs <= batch_sizes[0]:
        return us[0]
    for i in range(1, n):
        if bs <= batch_sizes[i] or i == n - 1:
            x0, x1, y0, y1 = batch_sizes[i - 1], batch_sizes[i], us[i - 1], us[i]
            return y0 + (y1 - y0) * (bs - x0) / (x1 - x0)
    raise AssertionError


def next_baseline(thr: float, old_bs: float, new_bs: float, literal_tbp: bool) -> Optional[float]:
    """The 'previous throughput' the NEXT update will compare against (None: no TBP term)."""
    if literal_tbp or new_bs > old_bs:
        return thr
    return None


def simulate(batch_sizes: Sequence[float], us: Sequence[float], extra_us: float, itl_slo_us: float,
             demand: int, initial_max_bs: float, iterations: int, alpha: float = 0.5,
             min_bs: float = 1.0, max_cap: float = 1e9, literal_tbp: bool = False) -> List[Tuple[float, int, float, float]]:
    """Closed loop against a measured latency curve: rows of (MaxBS after the update, batch run,
    ITL in us, backpressure)."""
    max_bs, thr_prev, rows = float(initial_max_bs), None, []
    for _ in range(iterations):
        bs = max(1, min(int(math.floor(max_bs)), int(demand)))
        itl = interp_latency(batch_sizes, us, bs) + extra_us
        thr = bs / itl
        _, _, bp = backpressure(itl, itl_slo_us, thr_prev, thr)
        new_bs = update(max_bs, bp, alpha, min_bs, max_cap)
        thr_prev = next_baseline(thr, max_bs, new_bs, literal_tbp)
        max_bs = new_bs
        rows.append((max_bs, bs, itl, bp))
    return rows
