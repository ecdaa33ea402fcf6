#!/usr/bin/env python
"""Benchmark of the decode-iteration hot path: KV append + paged GQA decode attention.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-sweep]

One step = one pass of the whole hot path (append, split-KV plan, partial attention, combine; one
fused kernel per layer) for every layer of the workload over one seeded synthetic batch.  The headline workload is the
Llama-3-8B-shaped layer at batch 64 with contexts uniform in [512, 4096] ("llama8b_b64",
~600 MB of KV per step, several times the L2 size, so every step streams from HBM).

Prints ONE JSON line (rank 0).  `value` is the algorithmic bytes all ranks moved per second of
the slowest rank's device time, in TB/s; with N > 1 every rank is an independent serving
instance with its own batch (weak scaling, no collective on the data path).

`--impl reference` times the fp64 CPU oracle on the host cores instead, on a bounded sample of
the same workload (a deliberately slow baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2501_08090_b200 import workloads as wl  # noqa: E402

HEADLINE = "llama8b_b64"
METRIC = "decode_attention_hbm_bandwidth"
UNIT = "TB/s"
NORMALISED_TO_TBS = 8.0          # the metric is quoted as a fraction of 8 TB/s
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel on the headline
# workload, from the ncu capture summarised in profiles/paged_decode_attn_llama8b_b64.md.  Set to
# None whenever the kernel changes after the capture.
NCU_TRAFFIC_BYTES = 573.6e6    # dram read + write per launch of the attention kernel, mean of 2 captured launches (profiles/paged_decode_attn_llama8b_b64.md)


# ------------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Polls SM clock and clock-event reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reason_bits = [], 0
        self.max_mhz = None
        self.error = None
        self._stop_evt = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover - depends on the box
            self.error = repr(e)

    def _poll(self):
        nv = self.nv
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
        try:
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))

    def run(self):
        if self._h is None:
            return
        while not self._stop_evt.is_set():
            try:
                self._poll()
            except Exception as e:  # pragma: no cover
                self.error = repr(e)
                return
            time.sleep(self.period)

    def wait_first_sample(self, limit_s: float = 0.5):
        """The first NVML query of a process is slow; it is taken before the timed region opens."""
        t_end = time.perf_counter() + limit_s
        while self._h is not None and not self.samples and self.error is None and time.perf_counter() < t_end:
            time.sleep(0.0005)

    def stop(self) -> dict:
        self._stop_evt.set()
        self.join(timeout=2.0)
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        out = {"sm_mhz": int(statistics.median(self.samples)) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples)}
        if self.error:
            out["error"] = self.error
        return out


# ------------------------------------------------------------------------------- device workload

class DeviceWorkload:
    """A workload drawn on the GPU: pool, tables, per-layer q / k_new / v_new / out."""

    def __init__(self, name: str, device, seed_offset: int = 0, batch=None, num_layers=None):
        import torch
        from paper_2501_08090_b200 import binding
        w = rank_workload(name, seed_offset, num_layers)
        self.w, self.device = w, device
        self.lens = wl.seq_lens(w, batch)
        self.B = int(self.lens.size)
        self.num_pages = wl.num_pool_pages(w, self.lens)
        self.bt_host = wl.block_tables(self.lens, self.num_pages, w.seed, w.page_size)
        cfg = binding.make_config(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                  self.num_pages, self.bt_host.shape[1], self.B)
        pool = wl.device_normal_bf16((wl.pool_elems(w, self.num_pages),), w.seed, 1, device)
        self.kp = binding.KvPool(cfg, device=device, pool=pool)
        self.bt = torch.from_numpy(self.bt_host).to(device)
        self.sl = torch.from_numpy(self.lens).to(device)
        self.q = wl.device_normal_bf16((w.num_layers, self.B, w.num_q_heads, w.head_dim), w.seed, 2, device)
        self.k_new = wl.device_normal_bf16((w.num_layers, self.B, w.num_kv_heads, w.head_dim), w.seed, 3, device)
        self.v_new = wl.device_normal_bf16((w.num_layers, self.B, w.num_kv_heads, w.head_dim), w.seed, 4, device)
        self.out = torch.zeros_like(self.q)
        self.bytes = wl.algorithmic_bytes(w, self.lens)

    def step_calls(self):
        """Pre-marshalled (function, args) pairs of one step, so the timed loop is one C call per layer."""
        import torch
        from paper_2501_08090_b200 import binding
        lib, h = binding.lib, self.kp._h
        s = torch.cuda.current_stream().cuda_stream
        calls = []
        for layer in range(self.w.num_layers):
            calls.append((lib.decode_step, (h, layer, self.B, self.bt.data_ptr(), self.sl.data_ptr(),
                                            self.q[layer].data_ptr(), self.k_new[layer].data_ptr(),
                                            self.v_new[layer].data_ptr(), self.out[layer].data_ptr(), s)))
        return calls

    def run_steps(self, n: int) -> None:
        from paper_2501_08090_b200 import binding
        calls = self.step_calls()
        for _ in range(n):
            for fn, args in calls:
                rc = fn(*args)
                if rc != 0:
                    raise binding.CkvError(rc, binding.last_error())


def rank_workload(name: str, rank: int = 0, num_layers=None) -> "wl.Workload":
    """The workload of one serving instance: same shape on every rank, its own seeded batch."""
    over = {} if num_layers is None else {"num_layers": num_layers}
    if rank:
        over["seed"] = wl.workload(name).seed + 1000 * rank
    return wl.workload(name, **over)


def dist_setup(n_gpus: int):
    """(rank, world, local_rank); initialises NCCL only when launched under torchrun."""
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def reduce_max_sum(t_ms: float, units: float, world: int, device="cuda"):
    """Max over ranks of the time, sum over ranks of the units (bytes, launches ...)."""
    if world == 1:
        return t_ms, units
    import torch
    import torch.distributed as dist
    a = torch.tensor([t_ms], dtype=torch.float64, device=device)
    b = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(a, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(a.item()), float(b.item())


def barrier(world: int):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


# A launch takes the host a few microseconds, the first ones of a region more.  So that a short region
# holds the device time of its steps and not that latency, the launches are queued behind a spin kernel
# (torch's own, about 0.3 ms) that is enqueued after the synchronise and before the first event.
DELAY_CYCLES = 600_000


def timed_region(fn, world: int, device_index: int):
    """barrier+sync, CUDA events on the launch stream around fn(), barrier+sync; returns (ms, clocks)."""
    import torch
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(device_index)
    sampler.start()
    sampler.wait_first_sample()
    barrier(world)
    torch.cuda._sleep(DELAY_CYCLES)
    ev0.record()
    fn()
    ev1.record()
    barrier(world)
    clocks = sampler.stop()
    return ev0.elapsed_time(ev1), clocks


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------- CPU baseline (oracle)

def oracle_sample_inputs(name: str, rows):
    """Host inputs for the chosen requests of a workload, as a compact pool (oracle's arm only)."""
    w = wl.workload(name)
    lens_all = wl.seq_lens(w)
    lens = lens_all[list(rows)]
    npg = int(wl.pages_of(lens).sum())
    bt = wl.block_tables(lens, npg, w.seed)
    b = lens.size
    return dict(w=w, lens=lens, num_pages=npg, bt=bt,
                pool=wl.normal_bf16((wl.pool_elems(w, npg, 1),), w.seed, 11),
                q=wl.normal_bf16((b, w.num_q_heads, w.head_dim), w.seed, 12),
                k=wl.normal_bf16((b, w.num_kv_heads, w.head_dim), w.seed, 13),
                v=wl.normal_bf16((b, w.num_kv_heads, w.head_dim), w.seed, 14))


def oracle_step(inp) -> float:
    """One oracle pass (append + attention) over the sample; seconds."""
    from oracle import oracle
    from oracle.oracle import PoolShape
    w = inp["w"]
    sh = PoolShape(1, inp["num_pages"], w.num_q_heads, w.num_kv_heads, w.page_size, w.head_dim)
    t0 = time.perf_counter()
    rc = oracle.kv_append(inp["pool"], sh, 0, inp["bt"], inp["lens"], inp["k"], inp["v"])
    assert rc == 0
    oracle.decode_attention(inp["pool"], sh, 0, inp["bt"], inp["lens"], inp["q"])
    return time.perf_counter() - t0


def cpu_baseline(name: str, target_s: float = 12.0) -> dict:
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload."""
    from oracle import oracle
    w = wl.workload(name)
    total = w.batch
    probe = oracle_sample_inputs(name, range(min(2, total)))
    t_probe = oracle_step(probe)
    n = int(max(1, min(total, round(len(probe["lens"]) * target_s / max(t_probe, 1e-6)))))
    inp = oracle_sample_inputs(name, range(n))
    oracle_step(inp)                                   # untimed first pass (page faults, thread start)
    times = []
    while len(times) < 3 or (sum(times) < target_s and len(times) < 50):
        times.append(oracle_step(inp))
    t = sum(times) / len(times)
    nbytes = wl.algorithmic_bytes(w, inp["lens"], 1)["total"]
    return {"value": nbytes / t / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "first %d of %d requests of %s, one layer; mean of %d passes (%.1f s of CPU work)"
                      % (n, total, name, len(times), sum(times)),
            "us_per_step_sample": t * 1e6}


def oracle_beside(name: str, batch=None, max_tokens: int = 250_000, passes: int = 2) -> dict:
    """The oracle timed on a bounded sample of another workload: the first requests of the batch whose
    contexts add up to at most max_tokens (one layer), extrapolated to the whole step by algorithmic bytes."""
    from oracle import oracle
    from oracle.oracle import PoolShape
    w = wl.workload(name)
    lens_all = wl.seq_lens(w, batch)
    take = max(1, int(np.searchsorted(np.cumsum(lens_all.astype(np.int64)), max_tokens, side="right")))
    lens = lens_all[:take]
    if int(lens.sum()) > 4 * max_tokens:              # a single very long request: time a prefix of it
        lens = np.minimum(lens, max_tokens).astype(np.int32)
    npg = int(wl.pages_of(lens).sum())
    bt = wl.block_tables(lens, npg, w.seed)
    sh = PoolShape(1, npg, w.num_q_heads, w.num_kv_heads, w.page_size, w.head_dim)
    pool = wl.normal_bf16((wl.pool_elems(w, npg, 1),), w.seed, 11)
    q = wl.normal_bf16((lens.size, w.num_q_heads, w.head_dim), w.seed, 12)
    k = wl.normal_bf16((lens.size, w.num_kv_heads, w.head_dim), w.seed, 13)
    times = []
    for _ in range(passes + 1):
        t0 = time.perf_counter()
        assert oracle.kv_append(pool, sh, 0, bt, lens, k, k) == 0
        oracle.decode_attention(pool, sh, 0, bt, lens, q)
        times.append(time.perf_counter() - t0)
    t = min(times[1:])                                 # the first pass pays for page faults
    sample_bytes = wl.algorithmic_bytes(w, lens, 1)["total"]
    full_bytes = wl.algorithmic_bytes(w, lens_all)["total"]
    return {"value": sample_bytes / t / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d of %d requests (%d of %d tokens), 1 of %d layers; best of %d passes"
                      % (lens.size, lens_all.size, int(lens.sum()), int(lens_all.sum()), w.num_layers, passes),
            "us_per_step_extrapolated": t * 1e6 * full_bytes / sample_bytes}


def run_reference(args) -> None:
    """--impl reference: K timed oracle steps on a sample sized so the run ends within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    w = wl.workload(HEADLINE)
    budget_s = 150.0
    one = oracle_sample_inputs(HEADLINE, range(1))
    t_one = min(oracle_step(one), oracle_step(one))
    per_step = budget_s / max(1, args.steps + args.warmup)
    n = int(max(1, min(w.batch, per_step / max(t_one, 1e-6))))
    inp = oracle_sample_inputs(HEADLINE, range(n))
    for _ in range(args.warmup):
        oracle_step(inp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(inp)
    dt = time.perf_counter() - t0
    nbytes = wl.algorithmic_bytes(w, inp["lens"], 1)["total"]
    value = nbytes * args.steps / dt / 1e12
    sample = "first %d of %d requests of %s per step" % (n, w.batch, HEADLINE)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": HEADLINE, "sample": sample, "device": "host cpu"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------- our arm

def run_ours(args) -> None:
    import torch
    from paper_2501_08090_b200 import binding   # raises if the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    name = args.workload or HEADLINE
    dw = DeviceWorkload(name, dev, seed_offset=rank, batch=args.batch, num_layers=args.layers)
    w = dw.w
    K, W = args.steps, max(args.warmup, 3)

    # ---- the kernel standing alone: CUDA events around every single launch, which defeat programmatic
    # dependent launch, so no two launches overlap (`isolated`).  Taken first; it also leaves host and
    # device warm for the headline region.
    P = min(K, 2000)
    dw.run_steps(W)
    dw.kp.check_status()
    dw.kp.profile_enable(True)
    dw.run_steps(P)
    attn_ms, attn_n = dw.kp.profile_read()
    dw.kp.profile_enable(False)

    # ---- headline: K steps back to back, inputs resident in HBM
    dw.run_steps(W)
    dw.kp.check_status()
    n0 = dw.kp.launch_count()
    ms, clocks = timed_region(lambda: dw.run_steps(K), world, dev.index or 0)
    launches = dw.kp.launch_count() - n0
    dw.kp.check_status()
    ms_max, bytes_all = reduce_max_sum(ms, float(dw.bytes["total"]) * K, world)
    _, launches_all = reduce_max_sum(0.0, float(launches), world)
    _, tokens_all = reduce_max_sum(0.0, float(dw.B) * K, world)
    _, kv_all = reduce_max_sum(0.0, float(dw.bytes["kv"]) * K, world)
    value = bytes_all / (ms_max * 1e-3) / 1e12

    # ---- dominant kernel.  The timed region above holds `launches` launches of the attention kernel and
    # nothing else, so its average launch duration there is region time / launches.
    attn_bytes = dw.bytes["total"] // w.num_layers            # the fused kernel moves all of a step's bytes
    peak, peak_kind = measured_peak_gbs()
    us_launch = ms / max(1, launches) * 1e3
    achieved = attn_bytes / (us_launch * 1e-6) / 1e9
    isolated = attn_bytes / (attn_ms / attn_n * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "paged_decode_attn_kernel (fused append + plan + attention + combine)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_kind": "of " + peak_kind,
                "traffic": NCU_TRAFFIC_BYTES, "bytes_per_launch": attn_bytes, "us_per_launch": us_launch,
                "timing": "timed region / launches in it (one kernel per step, back to back)",
                "frac_of_8TBs": achieved / (NORMALISED_TO_TBS * 1e3),
                "isolated": {"us_per_launch": attn_ms / attn_n * 1e3, "achieved": isolated, "frac": isolated / peak,
                             "timing": "events around every launch, no overlap between launches"}}

    # ---- the same K steps in plain stream order (no programmatic dependent launch): every launch starts
    # after the one before has ended, with nothing but the stream's own gap between them
    dw.kp.set_overlap(False)
    dw.run_steps(W)
    ser_ms, _ = timed_region(lambda: dw.run_steps(K), world, dev.index or 0)
    dw.kp.set_overlap(True)
    dw.kp.check_status()
    ser_us = ser_ms * 1e3 / (K * w.num_layers)
    roofline["serialized"] = {"us_per_launch": ser_us, "achieved": attn_bytes / (ser_us * 1e-6) / 1e9,
                              "frac": attn_bytes / (ser_us * 1e-6) / 1e9 / peak,
                              "timing": "K steps back to back in plain stream order, launches not overlapped"}

    # ---- the read probe: the same tiles through the same rings, no arithmetic: the practical ceiling
    def probe_steps(n):
        for _ in range(n):
            for layer in range(w.num_layers):
                dw.kp.read_probe(layer, dw.bt, dw.sl)
    probe_steps(W)
    probe_ms, _ = timed_region(lambda: probe_steps(min(K, 500)), world, dev.index or 0)
    dw.kp.check_status()
    probe_us = probe_ms * 1e3 / (min(K, 500) * w.num_layers)
    probe_gbs = (dw.bytes["kv"] // w.num_layers) / (probe_us * 1e-6) / 1e9
    roofline["read_probe"] = {"us_per_launch": probe_us, "kv_gbs": probe_gbs,
                              "attention_kv_gbs": (dw.bytes["kv"] // w.num_layers) / (us_launch * 1e-6) / 1e9,
                              "frac_of_probe": probe_us / us_launch,
                              "what": "kv_read_probe: the attention kernel's loads without its arithmetic, back to back"}

    # ---- end to end through the host-buffer entry point (pinned memory, copies inside the timing)
    # Its step count does not follow K: the host side (launch path, host link) takes a few hundred calls to
    # settle, and a serving loop runs settled, so it is always 500 launches after as many warm-up ones.
    E = max(5, 500 // w.num_layers)
    pin = lambda t: t.cpu().pin_memory()
    hb = dict(bt=pin(dw.bt), sl=pin(dw.sl), q=pin(dw.q[0]), k=pin(dw.k_new[0]), v=pin(dw.v_new[0]))
    hout = torch.zeros_like(hb["q"]).pin_memory()
    h2d = sum(hb[k].numel() * hb[k].element_size() for k in hb)
    d2h = hout.numel() * hout.element_size()

    host_calls = [dw.kp.host_step_call(layer, hb["bt"], hb["sl"], hb["q"], hb["k"], hb["v"], hout)
                  for layer in range(w.num_layers)]

    def e2e_steps(n):
        for _ in range(n):
            for call in host_calls:
                call()
    e2e_steps(E)                                        # warm-up: the host side takes a few hundred calls to settle
    barrier(world)
    chunks = []
    for _ in range(5):                                  # E steps in five chunks; the median chunk is reported
        t0 = time.perf_counter()
        e2e_steps(E // 5)
        torch.cuda.synchronize()
        chunks.append(time.perf_counter() - t0)
    E = 5 * (E // 5)
    e2e_s = statistics.median(chunks) * 5
    e2e_ms_max, e2e_bytes = reduce_max_sum(e2e_s * 1e3, float(dw.bytes["total"]) * E, world)
    e2e = {"value": e2e_bytes / (e2e_ms_max * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d * w.num_layers,
           "d2h_bytes_per_step": d2h * w.num_layers, "steps": E, "us_per_step": e2e_ms_max / E * 1e3,
           "chunk_us_per_step": [round(c / (E // 5) * 1e6, 1) for c in chunks],
           "route": "decode_step_host, pinned host buffers: gather kernel in, output rows written to host memory by the "
                    "attention kernel, one synchronise per step"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": name, "batch": dw.B, "layers": w.num_layers, "q_heads": w.num_q_heads,
                   "kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "page_size": w.page_size,
                   "context": "uniform[512,4096]" if name == HEADLINE else "see the workload's recipe", "tokens_in_context": int(dw.lens.sum()),
                   "l2": "inputs larger than L2 (%.0f MB of KV per step)" % (dw.bytes["kv"] / 1e6),
                   "timing": "CUDA events around the K steps; their launches are queued behind a 0.3 ms spin kernel "
                             "enqueued after the synchronise, so the region holds device time, not launch latency",
                   "instances": "one independent batch per GPU"},
        "us_per_step": ms_max / K * 1e3, "tokens_per_s": tokens_all / (ms_max * 1e-3),
        "kv_gbs": kv_all / (ms_max * 1e-3) / 1e9, "frac_of_8TBs": value / NORMALISED_TO_TBS,
        # the same launch standing alone (events around every launch: what an engine that runs other
        # kernels between attention launches sees)
        "serialized_us_per_launch": ser_us,
        "isolated_us_per_launch": attn_ms / attn_n * 1e3, "isolated_frac_of_8TBs": isolated / (NORMALISED_TO_TBS * 1e3),
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches_all), "roofline": roofline,
    }

    if rank == 0 and world == 1:
        if not args.no_sweep:
            line["latency_sweep"] = run_sweep(dev)
            line["local_autoscaler"] = run_autoscaler(line["latency_sweep"])
            line["global_autoscaler"] = run_global_autoscaler(line["local_autoscaler"])
            line["global_autoscaler"]["simulation"] = run_global_simulation(line["local_autoscaler"])
            line["kv_swap"] = run_swap(dev)
            line["multi_token_step"] = run_multi_token(dw)
            dw.kp.close()
            del dw
            torch.cuda.empty_cache()
            line["other_workloads"] = run_other_workloads(dev)
            line["cuda_graph"] = run_cuda_graph(dev)
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(HEADLINE)
            add_oracle_timings(line)
    if name != HEADLINE:
        line["roofline"]["traffic"] = None            # the ncu figure belongs to the headline workload
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_sweep(dev) -> dict:
    """Latency against batch size on the mixed interactive/batch workload (nested prefixes)."""
    import torch
    del_later = DeviceWorkload("mixed_sweep", dev)
    dw = del_later
    flush = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)      # each half larger than the L2
    sizes = list(wl.SWEEP_BATCH_SIZES)
    med, mn = dw.kp.step_latency_sweep(sizes, dw.bt, dw.sl, dw.q, dw.k_new, dw.v_new, dw.out,
                                       warmup=3, iters=20, flush=flush)
    rows = []
    for b, m, lo in zip(sizes, med.tolist(), mn.tolist()):
        nb = wl.algorithmic_bytes(dw.w, dw.lens[:b])["total"]
        rows.append({"batch": b, "us_per_step": round(m, 2), "us_min": round(lo, 2),
                     "tokens_per_s": round(b / (m * 1e-6)), "tbs": round(nb / (m * 1e-6) / 1e12, 3)})
    dw.kp.close()
    return {"workload": "mixed_sweep", "l2": "before every timed step 256 MB are overwritten, then another 256 MB read (cold and clean L2)", "points": rows}


def add_oracle_timings(line: dict) -> None:
    """The oracle timed beside the other workloads of the line (rank 0, after the GPU work is done)."""
    for row in line.get("latency_sweep", {}).get("points", []):
        if row["batch"] in (1, 64, 512):
            row["cpu_baseline"] = oracle_beside("mixed_sweep", batch=row["batch"])
    for row in line.get("other_workloads", []):
        if "skipped" not in row:
            row["cpu_baseline"] = oracle_beside(row["workload"])


def run_swap(dev) -> dict:
    """Swap-out / swap-in of a 4096-page request image (8B shape, one layer: 256 MB) through the
    library's zero-copy kernels, beside torch's pinned-memory copies of the same bytes."""
    import torch
    from paper_2501_08090_b200 import binding
    n_pages, total_pages = 4096, 8192
    cfg = binding.make_config(1, 32, 8, 128, total_pages, n_pages, 1)
    kp = binding.KvPool(cfg, device=dev)
    kp.pool.normal_()
    ids = torch.randperm(total_pages, device=dev)[:n_pages].to(torch.int32)
    nbytes = kp.swap_image_bytes(n_pages)
    image = torch.empty(nbytes // 2, dtype=torch.int16).pin_memory()
    dev_buf = torch.empty(nbytes // 2, dtype=torch.int16, device=dev)

    def timed(fn, reps=5):
        fn(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record(); torch.cuda.synchronize()
        return nbytes * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9
    out = {"bytes": nbytes, "pages": n_pages,
           "swap_out_gbs": round(timed(lambda: kp.swap_out(ids, image)), 2),
           "swap_in_gbs": round(timed(lambda: kp.swap_in(ids, image)), 2),
           "memcpy_d2h_gbs": round(timed(lambda: image.copy_(dev_buf, non_blocking=True)), 2),
           "memcpy_h2d_gbs": round(timed(lambda: dev_buf.copy_(image, non_blocking=True)), 2)}
    kp.check_status()
    kp.close()
    return out


def run_multi_token(dw) -> dict:
    """kv_append_multi + decode_attention_multi on the headline batch: q_len new tokens per request
    share one pass over the KV stream while q_len x group <= 8 columns; q_len 4 takes two passes."""
    import torch
    w, rows = dw.w, []
    for q_len in (1, 2, 4):
        q = wl.device_normal_bf16((dw.B, q_len, w.num_q_heads, w.head_dim), w.seed, 20 + q_len, dw.device)
        k = wl.device_normal_bf16((dw.B, q_len, w.num_kv_heads, w.head_dim), w.seed, 30 + q_len, dw.device)
        out = torch.zeros_like(q)

        def step():
            dw.kp.kv_append_multi(0, q_len, dw.bt, dw.sl, k, k)
            dw.kp.decode_attention_multi(0, q_len, dw.bt, dw.sl, q, out)
        for _ in range(5):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 200
        e0.record()
        for _ in range(n):
            step()
        e1.record(); torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        passes = -(-q_len * w.group // 8)
        rows.append({"q_len": q_len, "passes": passes, "us_per_step": round(us, 2),
                     "kv_tbs": round(passes * dw.bytes["kv"] / us / 1e6, 3),
                     "new_tokens_per_s": round(dw.B * q_len / us * 1e6)})
    dw.kp.check_status()
    return {"workload": dw.w.name, "launches_per_step": "1 append + passes", "points": rows}


def run_other_workloads(dev) -> list:
    """The other full-size workloads, back to back like the headline: the skewed long-context batch
    and the 70B-shaped iteration with all 80 layers resident (about 80 GB of KV)."""
    import torch
    rows = []
    for name, steps in (("skewed_long", 300), ("llama70b_full", 5)):
        try:
            dw = DeviceWorkload(name, dev)
        except torch.cuda.OutOfMemoryError:
            rows.append({"workload": name, "skipped": "not enough free device memory"})
            continue
        dw.run_steps(2)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dw.run_steps(steps)
        e1.record()
        torch.cuda.synchronize()
        dw.kp.check_status()
        us = e0.elapsed_time(e1) * 1e3 / steps
        tbs = dw.bytes["total"] / us / 1e6
        rows.append({"workload": name, "batch": dw.B, "layers": dw.w.num_layers, "steps": steps,
                     "us_per_step": round(us, 1), "us_per_layer": round(us / dw.w.num_layers, 2),
                     "tokens_per_s": round(dw.B / us * 1e6), "tbs": round(tbs, 3),
                     "frac_of_8TBs": round(tbs / NORMALISED_TO_TBS, 4),
                     "kv_bytes_per_step": int(dw.bytes["kv"])})
        dw.kp.close()
        del dw
        torch.cuda.empty_cache()
    return rows


def run_cuda_graph(dev) -> dict:
    """Launch overhead: 32 back-to-back steps issued call by call against the same 32 steps captured
    once in a CUDA graph and replayed, on small and large batches of the mixed workload."""
    import torch
    rows = []
    stream = torch.cuda.Stream(device=dev)
    for b in (1, 8, 64):
        dw = DeviceWorkload("mixed_sweep", dev, batch=b)
        n, reps = 32, 20
        try:
            with torch.cuda.stream(stream):
                dw.run_steps(n)
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    dw.run_steps(n)
                e1.record(stream)
                stream.synchronize()
                eager_us = e0.elapsed_time(e1) * 1e3 / (n * reps)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    dw.run_steps(n)
                graph.replay()
                stream.synchronize()
                e0.record(stream)
                for _ in range(reps):
                    graph.replay()
                e1.record(stream)
                stream.synchronize()
                graph_us = e0.elapsed_time(e1) * 1e3 / (n * reps)
            dw.kp.check_status()
            rows.append({"batch": b, "eager_us_per_step": round(eager_us, 2), "graph_us_per_step": round(graph_us, 2)})
        except Exception as exc:                      # capture not possible here: report, do not fail the bench
            rows.append({"batch": b, "unavailable": str(exc)[:200]})
        dw.kp.close()
        del dw
    return {"workload": "mixed_sweep", "steps_per_graph": 32, "points": rows}


def run_autoscaler(sweep: dict) -> dict:
    """Algorithm 1 closed over the measured curve: ITL(batch) = layers x attention(batch) + a constant
    standing for weight streaming, against the paper's interactive (200 ms) and batch (2 s) ITL SLOs."""
    from paper_2501_08090_b200 import binding
    sizes = [p["batch"] for p in sweep["points"]]
    layers, weights_us = 32, 2300.0          # Llama-3-8B: 32 layers; ~16 GB of bf16 weights at ~7 TB/s
    us = [layers * p["us_per_step"] for p in sweep["points"]]
    out = {"model": "ITL = 32 layers x measured attention step + 2.3 ms weight streaming", "alpha": 0.5, "runs": []}
    for slo_ms in (200.0, 2000.0):
        max_bs, batch, itl, bp = binding.autoscaler_simulate(slo_ms * 1e3, 8.0, sizes, us, weights_us,
                                                             demand=1 << 20, iterations=400, max_bs=65536.0)
        tail = batch[200:]
        out["runs"].append({"itl_slo_ms": slo_ms, "peak_batch": int(tail.max()), "trough_batch": int(tail.min()),
                            "max_itl_ms": round(float(itl[200:].max()) / 1e3, 2),
                            "updates_to_first_halving": int(np.argmax(bp >= 1.0)) if (bp >= 1.0).any() else None})
    return out


def run_global_autoscaler(local: dict) -> dict:
    """Section 5 on top of the measured instance: one batch instance serves (peak batch of the 2 s ITL run)
    tokens every ITL; a queue of batch requests with a one-hour TTFT SLO (Section 6 "Workloads") is sized
    by Algorithm 2 for a range of queue lengths, and an interactive pool is held at Theta = 1/3."""
    from paper_2501_08090_b200 import binding
    run = local["runs"][-1]
    theta_tok_s = 0.75 * run["peak_batch"] / (run["max_itl_ms"] * 1e-3)       # saw-tooth mean: 3/4 of the peak
    mu_o, sigma_o = 256.0, 192.0                                             # output tokens per request (synthetic)
    out = {"tokens_per_s_per_instance": round(theta_tok_s), "mu_o": mu_o, "sigma_o": sigma_o, "z": 2.33,
           "ttft_slo_s": 3600.0, "batch_queue": [], "interactive": []}
    for queued in (10_000, 100_000, 1_000_000, 10_000_000):
        n = binding.batch_autoscale([queued], [3600.0], mu_o, sigma_o, theta_tok_s, 0, 0, 1 << 16, z=2.33)
        out["batch_queue"].append({"queued": queued, "instances": n,
                                   "wait_s": round(binding.waiting_time(queued - 1, mu_o, sigma_o, theta_tok_s * n, 2.33), 1)})
    total = 9
    for busy in (3, 5, 8, 4, 1):
        total = binding.interactive_autoscale(busy, total, 1.0 / 3.0, 0.05)
        out["interactive"].append({"busy": busy, "instances": total})
    return out


def run_global_simulation(local: dict) -> dict:
    """Sections 3 and 5 in time: a seeded Poisson trace of interactive and batch requests (Section 6
    "Workloads": TTFT SLOs of 10 s and one hour, here 10 s and 10 minutes to keep the run short) served by
    instances whose batch sizes and per-request token rates are what Algorithm 1 settled at on the measured
    latency curve; the deadline-driven policy beside immediate scaling (Section 2.3)."""
    from paper_2501_08090_b200 import binding
    inter, batch = local["runs"][0], local["runs"][-1]
    kw = dict(slots_interactive=max(1, inter["trough_batch"]), slots_batch=max(1, batch["trough_batch"]),
              rate_interactive=1e3 / inter["max_itl_ms"], rate_batch=1e3 / batch["max_itl_ms"],
              startup_s=30.0, tick_s=5.0, theta=1.0 / 3.0, delta=0.05, floor_instances=1, initial_instances=3,
              max_batch_instances=64, groups_k=4, z=2.33, mu_o_prior=200.0, sigma_o_prior=150.0, policy=0, horizon_s=0.0)
    # arrival rate that keeps about three interactive instances busy
    mean_tokens = float(wl.output_lengths(4000, 7).mean())
    rate = 0.9 * 3 * kw["slots_interactive"] * kw["rate_interactive"] / mean_tokens / 0.5
    trace = wl.request_trace(4000, rate, 1.0, 0.5, seed=7, batch_ttft_s=600.0)
    out = {"instance_model": {k: (round(v, 3) if isinstance(v, float) else v) for k, v in kw.items() if k.startswith(("slots", "rate"))},
           "requests": 4000, "arrival_rate_per_s": round(rate, 2), "policies": []}
    for policy, name in ((0, "deadline-driven (Algorithm 2 on request groups)"), (1, "immediate")):
        t0 = time.perf_counter()
        r = binding.global_simulate(binding.SimConfig(**dict(kw, policy=policy)), *trace)
        s = r["summary"]
        out["policies"].append({"policy": name, "events": r["events"], "wall_ms": round((time.perf_counter() - t0) * 1e3, 1),
                                "interactive_ttft_met": s["interactive_ttft_met"] / max(1, s["interactive_total"]),
                                "batch_ttft_met": s["batch_ttft_met"] / max(1, s["batch_total"]),
                                "instance_hours": [round(x / 3600.0, 3) for x in s["instance_seconds"]],
                                "scale_ups": s["instances_added"], "scale_downs": s["instances_removed"],
                                "hysteresis": round((sum(s["instances_added"]) + sum(s["instances_removed"])) / max(1, sum(s["instances_added"])), 2),
                                "evictions": s["evictions"], "end_s": round(s["end_s"], 1)})
    return out


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--no-sweep", action="store_true", help="skip the batch-size latency sweep")
    ap.add_argument("--workload", default=None, help="time another workload than the headline one (profiling runs)")
    ap.add_argument("--layers", type=int, default=None, help="number of layers of that workload to make resident")
    ap.add_argument("--batch", type=int, default=None, help="take only the first BATCH requests of that workload (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
