"""The paper's global autoscaler (Section 5 "Global Autoscaler") written out from its definitions:
request groups, the waiting-time estimate (Eq. 1), batch backpressure, Algorithm 2 and the
interactive over-provisioning band.  TEST INFRASTRUCTURE ONLY; the library's C++ shares no code
with it and never imports it.

What the paper fixes, and what each function below does with it:

 * Section 5.3 "Request Group Creation": requests in the queue are clustered by similar TTFT SLO
   (the paper cites MacQueen's k-means) and served first come first served inside a group.
   `request_groups` is Lloyd's iteration on the line.  Not fixed by the paper, chosen here: the
   k starting centroids are the sorted values at the mid-points of k equal slices; a value at the
   same distance from two centroids joins the lower one; an empty cluster keeps its centroid;
   groups are numbered by increasing centroid.
 * Eq. 1: W_q = sum_{i < q} O_i / Theta -- tokens ahead in the queue over the token throughput.
   The O_i are unknown and modelled by a fitted mean mu_o and deviation sigma_o; a sum of `a`
   such lengths is (CLT) Normal(a mu_o, a sigma_o^2), of which `waiting_time` takes the mean plus
   z deviations (z = 0: Eq. 1 with O_i -> mu_o; z > 0: the conservative estimate the evaluation
   section mentions for short queues).
 * BBP = number of request groups whose estimated waiting time exceeds their TTFT SLO.  A
   group's waiting time is taken for its LAST request (everything in earlier groups, and the rest
   of its own group, is ahead of it); what it is compared with is the time the group still has:
   the SLO less the age of its oldest member, passed in as `deadlines`.
 * Algorithm 2: keep adding one instance and re-evaluating BBP until it is 0; add that many;
   retire every batch instance when nothing is queued and nothing is being served.
 * Section 5.2: IBP = instances running interactive requests / (mixed + interactive instances)
   is held at Theta, in practice inside [Theta - delta, Theta + delta]; outside the band the
   instance count is reset to the smallest integer with IBP <= Theta.
"""
from __future__ import annotations

import math
from bisect import bisect_right
from fractions import Fraction
from typing import List, Sequence, Tuple


def request_groups(ttft_slos: Sequence[float], k: int, iters: int = 100) -> Tuple[List[int], List[float]]:
    """(group of every request, centroids in increasing order)."""
    xs = [float(x) for x in ttft_slos]
    n = len(xs)
    k = max(1, min(int(k), n))
    ranked = sorted(xs)
    # slice j of k equal slices covers ranks [j n / k, (j + 1) n / k); start at its middle rank
    cents = [ranked[min(n - 1, ((2 * j + 1) * n) // (2 * k))] for j in range(k)]
    owner = None
    for _ in range(iters):
        new_owner = []
        for x in xs:
            best, best_d = 0, abs(x - cents[0])
            for j in range(1, k):
                d = abs(x - cents[j])
                if d < best_d:
                    best, best_d = j, d
            new_owner.append(best)
        sums, sizes = [0.0] * k, [0] * k
        for x, j in zip(xs, new_owner):                    # in input order: the sums are sequential
            sums[j] += x
            sizes[j] += 1
        new_cents = [sums[j] / sizes[j] if sizes[j] else cents[j] for j in range(k)]
        settled = new_owner == owner and new_cents == cents
        owner, cents = new_owner, new_cents
        if settled:
            break
    order = sorted(range(k), key=lambda j: (cents[j], j))
    number = {old: new for new, old in enumerate(order)}
    return [number[j] for j in owner], [cents[j] for j in order]


def waiting_time(requests_ahead: int, mu_o: float, sigma_o: float, throughput: float, z: float = 0.0) -> float:
    """Seconds until a request with `requests_ahead` requests before it reaches the head."""
    a = float(requests_ahead)
    if a <= 0:
        return 0.0
    tokens_ahead = a * mu_o + z * sigma_o * math.sqrt(a)   # mean of the sum plus z of its deviations
    return tokens_ahead / throughput


def group_waits(counts: Sequence[int], mu_o: float, sigma_o: float, throughput: float, z: float = 0.0) -> List[float]:
    """W_g for every group in service order: the wait of the group's last request."""
    waits, before = [], 0
    for c in counts:
        waits.append(waiting_time(before + c - 1, mu_o, sigma_o, throughput, z) if c > 0 else 0.0)
        before += max(c, 0)
    return waits


def batch_backpressure(counts: Sequence[int], deadlines: Sequence[float], mu_o: float, sigma_o: float,
                       throughput_per_instance: float, instances: int, z: float = 0.0,
                       spare_throughput: float = 0.0) -> int:
    """BBP: how many non-empty groups would wait past the time they have left.

    `spare_throughput` is token throughput available besides the batch instances (the free
    capacity of mixed instances); with no throughput at all every non-empty group counts."""
    thr = throughput_per_instance * instances + spare_throughput
    if thr <= 0.0:
        return sum(1 for c in counts if c > 0)
    waits = group_waits(counts, mu_o, sigma_o, thr, z)
    return sum(1 for c, w, left in zip(counts, waits, deadlines) if c > 0 and w > left)


def batch_autoscale(counts, deadlines, mu_o, sigma_o, throughput_per_instance, current_instances: int,
                    active_requests: int, max_instances: int, z: float = 0.0) -> int:
    """Algorithm 2: the number of batch instances to run with."""
    if not any(c > 0 for c in counts):
        return current_instances if active_requests > 0 else 0     # nothing queued, nothing served: retire all
    n = max(current_instances, 1)
    while n < max_instances and batch_backpressure(counts, deadlines, mu_o, sigma_o, throughput_per_instance, n, z) > 0:
        n += 1
    return n


def interactive_autoscale(busy: int, total: int, theta: float, delta: float, floor: int = 1) -> int:
    """Interactive + mixed instance count that holds IBP = busy / total at theta (within +- delta)."""
    total = max(total, floor, 1)
    if theta - delta <= busy / total <= theta + delta:
        return total
    # smallest integer count with busy / count <= theta; theta is a ratio like 1/3, taken exactly
    ratio = Fraction(theta).limit_denominator(1_000_000)
    need = math.ceil(Fraction(busy) / ratio)
    return max(need, busy, floor)


def nearest_group(slo: float, centroids: Sequence[float]) -> int:
    """Group whose centroid is nearest to `slo` (the lower one at equal distance; 0 with no centroid)."""
    if not centroids:
        return 0
    hi = bisect_right(list(centroids), slo)
    if hi == 0:
        return 0
    if hi == len(centroids):
        hi -= 1
        # several equal centroids at the top: the lowest of them
        while hi > 0 and centroids[hi - 1] == centroids[hi]:
            hi -= 1
        return hi
    lo = hi - 1
    pick = lo if abs(slo - centroids[lo]) <= abs(centroids[hi] - slo) else hi
    while pick > 0 and abs(slo - centroids[pick - 1]) == abs(slo - centroids[pick]):
        pick -= 1
    return pick
