"""The global autoscaler in time, as a plain event loop: the request life cycle of the paper's
Section 3 (global queue, interactive / mixed / batch instances, routing to the own class first and
to mixed instances otherwise, eviction of batch requests from mixed instances with their progress
kept) under the autoscaling of Section 5 (IBP band, request groups, Eq. 1, Algorithm 2).
TEST INFRASTRUCTURE ONLY: the library's C++ simulation shares no code with this file.

One heap holds every future event as (time, rank, id, stamp): rank orders simultaneous events
(0 completion, 1 instance ready, 2 arrival, 3 autoscaler tick), stamp invalidates entries whose
request was evicted or whose instance was removed in the meantime.  Instances and requests are
small objects; the queue is a heap keyed (group, arrival, id), rebuilt when groups are re-formed.

The arithmetic that fixes event times is written exactly as the interface states it:
finish = start + remaining / rate; on eviction remaining = max(remaining - (now - start) * rate, 0).
"""
from __future__ import annotations

import heapq
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

from . import global_autoscaler as ga

INTERACTIVE, MIXED, BATCH = 0, 1, 2
ARRIVE, START, EVICT, FINISH, ADD, READY, REMOVE, TICK = range(8)
CHIRON, IMMEDIATE = 0, 1


@dataclass
class SimConfig:
    slots_interactive: int
    slots_batch: int
    rate_interactive: float
    rate_batch: float
    startup_s: float
    tick_s: float
    theta: float = 1.0 / 3.0
    delta: float = 0.05
    floor_instances: int = 1
    initial_instances: int = 3
    max_batch_instances: int = 64
    groups_k: int = 4
    z: float = 0.0
    mu_o_prior: float = 256.0
    sigma_o_prior: float = 128.0
    policy: int = CHIRON
    horizon_s: float = 0.0


@dataclass
class _Req:
    rid: int
    arrival: float
    tokens: float
    slo: float
    kind: int
    remaining: float
    start: float = -1.0
    where: Optional["_Inst"] = None
    stamp: int = 0
    group: int = 0
    first_start: float = -1.0
    finished_at: float = -1.0
    evictions: int = 0
    queued: bool = False


@dataclass
class _Inst:
    iid: int
    cls: int
    added_at: float
    ready_at: float
    ready: bool = False
    gone: bool = False
    interactive: Dict[int, _Req] = field(default_factory=dict)
    batch: Dict[int, _Req] = field(default_factory=dict)

    def load(self) -> int:
        return len(self.interactive) + len(self.batch)


class Simulation:
    def __init__(self, cfg: SimConfig, arrival_s: Sequence[float], kind: Sequence[int],
                 output_tokens: Sequence[float], ttft_slo_s: Sequence[float]):
        self.cfg = cfg
        self.reqs = [_Req(i, float(a), float(o), float(s), int(k), float(o))
                     for i, (a, k, o, s) in enumerate(zip(arrival_s, kind, output_tokens, ttft_slo_s))]
        self.insts: List[_Inst] = []
        self.heap: List[Tuple[float, int, int, int]] = []
        self.queue: List[Tuple[int, float, int]] = []
        self.waiting: List[int] = []
        self.centroids: List[float] = []
        self.log: List[Tuple[float, int, int, int]] = []
        self.now = 0.0
        self.finished = 0
        self.added = [0, 0, 0]
        self.removed = [0, 0, 0]
        self.peak = [0, 0, 0]
        self.seconds = [0.0, 0.0, 0.0]
        self.tokens_served = 0.0
        self.fit = (0, 0.0, 0.0)                       # count, mean, sum of squared deviations
        want_int = max(1, math.floor(cfg.theta * cfg.initial_instances + 0.5))
        for _ in range(cfg.initial_instances):
            inst = self._new_instance(INTERACTIVE if self._count(INTERACTIVE) < want_int else MIXED, 0.0, initial=True)
            inst.ready = True
        for r in self.reqs:
            heapq.heappush(self.heap, (r.arrival, 2, r.rid, 0))
        self.tick_k = 1
        heapq.heappush(self.heap, (self.tick_k * cfg.tick_s, 3, 0, 0))

    # ---- bookkeeping
    def _live(self, cls: int) -> List[_Inst]:
        return [i for i in self.insts if i.cls == cls and not i.gone]          # ascending id by construction

    def _count(self, cls: int) -> int:
        return len(self._live(cls))

    def _rate(self, cls: int) -> float:
        return self.cfg.rate_batch if cls == BATCH else self.cfg.rate_interactive

    def _slots(self, cls: int) -> int:
        return self.cfg.slots_batch if cls == BATCH else self.cfg.slots_interactive

    def _emit(self, kind: int, a: int, b: int) -> None:
        self.log.append((self.now, kind, a, b))

    def _new_instance(self, cls: int, ready_at: float, initial: bool = False) -> _Inst:
        inst = _Inst(len(self.insts), cls, self.now, ready_at)
        self.insts.append(inst)
        self.peak[cls] = max(self.peak[cls], self._count(cls))
        if not initial:
            self.added[cls] += 1
            heapq.heappush(self.heap, (ready_at, 1, inst.iid, 0))
            self._emit(ADD, inst.iid, cls)
        return inst

    def _remove_instance(self, inst: _Inst) -> None:
        for rid in sorted(inst.batch):
            self._evict(self.reqs[rid])
        inst.gone = True
        self.removed[inst.cls] += 1
        self.seconds[inst.cls] += self.now - inst.added_at
        self._emit(REMOVE, inst.iid, inst.cls)

    # ---- requests
    def _enqueue(self, r: _Req) -> None:
        r.group = ga.nearest_group(r.slo, self.centroids)
        r.queued = True
        heapq.heappush(self.queue, (r.group, r.arrival, r.rid))

    def _start(self, r: _Req, inst: _Inst) -> None:
        r.where, r.start = inst, self.now
        if r.first_start < 0.0:
            r.first_start = self.now
        r.stamp += 1
        heapq.heappush(self.heap, (self.now + r.remaining / self._rate(inst.cls), 0, r.rid, r.stamp))
        (inst.interactive if r.kind == 0 else inst.batch)[r.rid] = r
        self._emit(START, r.rid, inst.iid)

    def _evict(self, r: _Req) -> None:
        inst = r.where
        r.remaining = max(r.remaining - (self.now - r.start) * self._rate(inst.cls), 0.0)
        r.stamp += 1                                       # its completion entry in the heap is void now
        del inst.batch[r.rid]
        self._emit(EVICT, r.rid, inst.iid)
        r.where = None
        r.evictions += 1
        self._enqueue(r)

    def _room(self, cls: int) -> Optional[_Inst]:
        for inst in self._live(cls):
            if inst.ready and inst.load() < self._slots(cls):
                return inst
        return None

    def _place_interactive(self, r: _Req) -> bool:
        inst = self._room(INTERACTIVE) or self._room(MIXED)
        if inst is None:
            for m in self._live(MIXED):
                if m.ready and m.batch:
                    victim = max(m.batch.values(), key=lambda b: (b.start, b.rid))
                    self._evict(victim)
                    inst = m
                    break
        if inst is None:
            return False
        self._start(r, inst)
        return True

    def _dispatch(self) -> None:
        while self.waiting and self._place_interactive(self.reqs[self.waiting[0]]):
            self.waiting.pop(0)
        while self.queue:
            inst = self._room(BATCH)
            if inst is None and not self.waiting:
                inst = self._room(MIXED)
            if inst is None:
                break
            _, _, rid = heapq.heappop(self.queue)
            self.reqs[rid].queued = False
            self._start(self.reqs[rid], inst)

    # ---- events
    def _arrive(self, r: _Req) -> None:
        self._emit(ARRIVE, r.rid, -1)
        if r.kind == 0:
            if self.waiting or not self._place_interactive(r):
                self.waiting.append(r.rid)
            self._dispatch()
            return
        self._enqueue(r)
        self._dispatch()
        if self.cfg.policy == IMMEDIATE and r.where is None:
            promised = self.cfg.slots_batch * sum(1 for i in self._live(BATCH) if not i.ready)
            if len(self.queue) > promised and self._count(BATCH) < self.cfg.max_batch_instances:
                self._new_instance(BATCH, self.now + self.cfg.startup_s)

    def _finish(self, r: _Req) -> None:
        inst = r.where
        del (inst.interactive if r.kind == 0 else inst.batch)[r.rid]
        r.finished_at, r.remaining, r.where = self.now, 0.0, None
        r.stamp += 1
        self.finished += 1
        self.tokens_served += r.tokens
        n, mean, m2 = self.fit
        n += 1
        d = r.tokens - mean
        mean += d / n
        m2 += d * (r.tokens - mean)
        self.fit = (n, mean, m2)
        self._emit(FINISH, r.rid, inst.iid)
        self._dispatch()
        if self.cfg.policy == IMMEDIATE and inst.cls == BATCH and inst.load() == 0:
            self._remove_instance(inst)

    def _regroup(self) -> None:
        members = sorted(self.queue)                       # queue order
        self.queue, self.centroids = [], []
        if not members:
            return
        slos = [self.reqs[rid].slo for _, _, rid in members]
        groups, self.centroids = ga.request_groups(slos, self.cfg.groups_k)
        for (_, arrival, rid), g in zip(members, groups):
            self.reqs[rid].group = g
            self.queue.append((g, arrival, rid))
        heapq.heapify(self.queue)

    def _scale_interactive(self) -> None:
        pool = self._live(INTERACTIVE) + self._live(MIXED)
        busy = sum(1 for i in pool if i.ready and i.interactive)
        total = len(pool)
        target = ga.interactive_autoscale(busy, total, self.cfg.theta, self.cfg.delta, self.cfg.floor_instances)
        if target > total:
            want_int = max(1, math.floor(self.cfg.theta * target + 0.5))
            for _ in range(target - total):
                cls = INTERACTIVE if self._count(INTERACTIVE) < want_int else MIXED
                self._new_instance(cls, self.now + self.cfg.startup_s)
        elif target < total:
            idle = [i for i in pool if not i.interactive]
            # still starting before ready, mixed before interactive, newest first
            idle.sort(key=lambda i: (i.ready, i.cls == INTERACTIVE, -i.iid))
            for inst in idle[:total - target]:
                self._remove_instance(inst)

    def _scale_batch(self) -> None:
        batch = self._live(BATCH)
        if not self.queue:
            if batch and all(i.load() == 0 for i in batch):
                for inst in batch:
                    self._remove_instance(inst)
            return
        by_group: Dict[int, List[_Req]] = {}
        for g, _, rid in self.queue:
            by_group.setdefault(g, []).append(self.reqs[rid])
        order = sorted(by_group)
        counts = [len(by_group[g]) for g in order]
        left = [min(r.arrival + r.slo - self.now for r in by_group[g]) for g in order]
        spare = 0.0
        for m in self._live(MIXED):
            if m.ready:
                spare += self.cfg.rate_interactive * float(self.cfg.slots_interactive - m.load())
        n_fit, mean, m2 = self.fit
        mu = mean if n_fit >= 2 else self.cfg.mu_o_prior
        sigma = math.sqrt(m2 / (n_fit - 1)) if n_fit >= 2 else self.cfg.sigma_o_prior
        per_instance = float(self.cfg.slots_batch) * self.cfg.rate_batch
        n = len(batch)
        while n < self.cfg.max_batch_instances and \
                ga.batch_backpressure(counts, left, mu, sigma, per_instance, n, self.cfg.z, spare) > 0:
            n += 1
        for _ in range(n - len(batch)):
            self._new_instance(BATCH, self.now + self.cfg.startup_s)

    def _tick(self) -> bool:
        """Returns True if the tick added an instance."""
        before = sum(self.added)
        self._regroup()
        self._scale_interactive()
        if self.cfg.policy == CHIRON:
            self._scale_batch()
        self._emit(TICK, self._count(INTERACTIVE) + self._count(MIXED), self._count(BATCH))
        self._dispatch()
        return sum(self.added) > before

    def run(self) -> "Simulation":
        n = len(self.reqs)
        while self.finished < n and self.heap:
            t, rank, ident, stamp = heapq.heappop(self.heap)
            if rank == 0 and self.reqs[ident].stamp != stamp:
                continue                                   # evicted since: void
            if rank == 1 and self.insts[ident].gone:
                continue
            if self.cfg.horizon_s > 0.0 and t > self.cfg.horizon_s:
                break
            self.now = t
            if rank == 0:
                self._finish(self.reqs[ident])
            elif rank == 1:
                self.insts[ident].ready = True
                self._emit(READY, ident, self.insts[ident].cls)
                self._dispatch()
            elif rank == 2:
                self._arrive(self.reqs[ident])
            else:
                grew = self._tick()
                self.tick_k += 1
                heapq.heappush(self.heap, (self.tick_k * self.cfg.tick_s, 3, 0, 0))
                if not grew and not self._anything_pending():
                    break                                  # nothing runs, starts or arrives any more: stuck
        for inst in self.insts:
            if not inst.gone:
                self.seconds[inst.cls] += self.now - inst.added_at
        return self

    def _anything_pending(self) -> bool:
        for t, rank, ident, stamp in self.heap:
            if rank == 0 and self.reqs[ident].stamp == stamp:
                return True
            if rank == 1 and not self.insts[ident].gone:
                return True
            if rank == 2:
                return True
        return False

    # ---- results
    def summary(self) -> dict:
        def met(r: _Req) -> bool:
            return r.first_start >= 0.0 and r.first_start - r.arrival <= r.slo
        inter = [r for r in self.reqs if r.kind == 0]
        batch = [r for r in self.reqs if r.kind == 1]
        return {
            "end_s": self.now, "finished": self.finished,
            "interactive_total": len(inter), "interactive_ttft_met": sum(met(r) for r in inter),
            "batch_total": len(batch), "batch_ttft_met": sum(met(r) for r in batch),
            "evictions": sum(r.evictions for r in self.reqs),
            "instances_added": list(self.added), "instances_removed": list(self.removed),
            "instance_seconds": list(self.seconds), "peak_instances": list(self.peak),
            "tokens_served": self.tokens_served,
        }


def simulate(cfg: SimConfig, arrival_s, kind, output_tokens, ttft_slo_s) -> Simulation:
    return Simulation(cfg, arrival_s, kind, output_tokens, ttft_slo_s).run()
