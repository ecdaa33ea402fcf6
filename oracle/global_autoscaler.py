"""Plain restatement of the paper's global autoscaler (Section 5 "Global Autoscaler"): request
groups, the waiting-time estimate (Eq. 1), batch backpressure, Algorithm 2 and the interactive
over-provisioning band.  TEST INFRASTRUCTURE ONLY; the library's C++ shares no code with it.

Readings where the text leaves room:
 * request groups: 1-D k-means (the paper cites MacQueen) on the TTFT SLO values, centroids
   initialised at evenly spaced quantiles of the sorted values, Lloyd iterations to a fixed point;
   groups are numbered by increasing centroid;
 * groups are served in order of increasing TTFT SLO (earliest deadline first), FCFS inside;
 * W_g (Algorithm 2's EstimateWaitingTime) is the time until the LAST request of group g reaches
   the head of the queue: Eq. 1 with q - 1 = (requests in earlier groups) + (requests in g) - 1,
   O_i replaced by its fitted mean mu_o, plus z standard deviations of the sum (CLT):
   W = ((q-1) mu_o + z sigma_o sqrt(q-1)) / (Theta * instances);  z = 0 is the plain mean;
 * a group's deadline is its smallest TTFT SLO minus the age of its oldest request;
 * Algorithm 2 starts from the instances already dispatched (at least one) and adds one at a time
   until BBP = 0 or a cap is reached;
 * interactive autoscaling: IBP = busy / total; outside [Theta - delta, Theta + delta] the total is
   set to ceil(busy / Theta) (never below busy, never below a floor).
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple


def request_groups(ttft_slos: Sequence[float], k: int, iters: int = 100) -> Tuple[List[int], List[float]]:
    """(group of every request, centroids in increasing order)."""
    n = len(ttft_slos)
    k = max(1, min(k, n))
    order = sorted(ttft_slos)
    cent = [order[min(n - 1, (2 * j + 1) * n // (2 * k))] for j in range(k)]
    assign = [0] * n
    for _ in range(iters):
        new_assign = [min(range(k), key=lambda j: (abs(x - cent[j]), j)) for x in ttft_slos]
        new_cent = []
        for j in range(k):
            members = [x for x, a in zip(ttft_slos, new_assign) if a == j]
            new_cent.append(sum(members) / len(members) if members else cent[j])
        if new_assign == assign and new_cent == cent:
            break
        assign, cent = new_assign, new_cent
    rank = sorted(range(k), key=lambda j: (cent[j], j))
    relabel = {old: new for new, old in enumerate(rank)}
    return [relabel[a] for a in assign], [cent[j] for j in rank]


def waiting_time(requests_ahead: int, mu_o: float, sigma_o: float, throughput: float, z: float = 0.0) -> float:
    """Eq. 1 with the CLT: tokens ahead ~ Normal(q mu, q sigma^2)."""
    if requests_ahead <= 0:
        return 0.0
    return (requests_ahead * mu_o + z * sigma_o * math.sqrt(requests_ahead)) / throughput


def batch_backpressure(counts: Sequence[int], deadlines: Sequence[float], mu_o: float, sigma_o: float,
                       throughput_per_instance: float, instances: int, z: float = 0.0) -> int:
    """Number of groups (given in service order) whose last request would wait past its deadline."""
    bbp, ahead = 0, 0
    for c, dl in zip(counts, deadlines):
        if c <= 0:
            continue
        w = waiting_time(ahead + c - 1, mu_o, sigma_o, throughput_per_instance * instances, z)
        if w > dl:
            bbp += 1
        ahead += c
    return bbp


def batch_autoscale(counts, deadlines, mu_o, sigma_o, throughput_per_instance, current_instances: int,
                    active_requests: int, max_instances: int, z: float = 0.0) -> int:
    """Algorithm 2: the batch-instance count to run with."""
    if sum(counts) == 0:
        return 0 if active_requests == 0 else current_instances          # retire all when nothing is served
    n = max(1, current_instances)
    while n < max_instances and batch_backpressure(counts, deadlines, mu_o, sigma_o, throughput_per_instance, n, z) > 0:
        n += 1
    return n


def interactive_autoscale(busy: int, total: int, theta: float, delta: float, floor: int = 1) -> int:
    """The interactive + mixed instance count that keeps IBP = busy / total within theta +- delta."""
    total = max(total, floor, 1)
    ibp = busy / total
    if theta - delta <= ibp <= theta + delta:
        return total
    return max(floor, busy, int(math.ceil(busy / theta - 1e-12)))
