"""Seeded synthetic inputs for the decode-iteration hot path.

This module only DRAWS inputs: context lengths, block tables, and N(0,1) values rounded to
bf16.  It contains none of the attention or append arithmetic and imports neither the GPU
binding nor the CPU oracle; both are fed from here so that they see identical bytes.

The five workloads stand in for the paper's serving traces (ShareGPT-derived requests on
Llama-3.1 8B / 70B, Section 6 "Evaluation"), which are not available offline: only tensor
shapes and context-length distributions matter to this path.  Interactive requests have short
contexts, batch requests long ones (Section 2.1 "Workload Categories").

bf16 values travel as uint16 bit patterns on the host and as torch.bfloat16 on a device.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional

import numpy as np

PAGE_SIZE = 16


@dataclass(frozen=True)
class Workload:
    """One synthetic continuous batch: model shape, context lengths and pool sizing."""
    name: str
    seed: int
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    batch: int
    pool_factor: float          # physical pages = ceil(pool_factor * live pages)
    page_size: int = PAGE_SIZE
    fixed_num_pages: Optional[int] = None

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:
        """K and V bytes of one token in one layer (bf16)."""
        return 2 * self.num_kv_heads * self.head_dim * 2


WORKLOADS = {
    # Tiny GQA step: contexts {17, 64, 129, 256} hit the first slot of a fresh page (17, 129)
    # and the last slot of a page (64, 256); 31 of 64 pool pages are live.
    "tiny": Workload("tiny", 0, 1, 4, 1, 64, 4, 1.0, fixed_num_pages=64),
    # Llama-3-8B attention shape, batch 64, contexts uniform in [512, 4096], pool 2x live.
    "llama8b_b64": Workload("llama8b_b64", 1, 1, 32, 8, 128, 64, 2.0),
    # Mixed interactive/batch continuous batch on the 8B shape; batch sizes are nested prefixes
    # of one fixed list of 512 requests.
    "mixed_sweep": Workload("mixed_sweep", 2, 1, 32, 8, 128, 512, 1.25),
    # Llama-3-70B shape, all 80 layers resident, batch 96, contexts uniform in [1024, 4096].
    "llama70b_full": Workload("llama70b_full", 3, 80, 64, 8, 128, 96, 1.01),
    # Skewed batch: one 131072-token request and seven 1024-token ones.
    "skewed_long": Workload("skewed_long", 4, 1, 32, 8, 128, 8, 1.25),
}

SWEEP_BATCH_SIZES = (1, 2, 4, 8, 16, 32, 64, 128, 256, 512)


def workload(name: str, **overrides) -> Workload:
    """Look a workload up by name; keyword overrides give reduced variants (fewer layers...)."""
    w = WORKLOADS[name]
    return replace(w, **overrides) if overrides else w


# ----------------------------------------------------------------------------- lengths

def is_batch_request(i: int) -> bool:
    """Request i of the mixed list is a long-context batch request.

    Chosen so that every prefix of length B holds round(0.3 * B) batch requests (half up).
    """
    return math.floor(0.3 * (i + 1) + 0.5) > math.floor(0.3 * i + 0.5)


def seq_lens(w: Workload, batch: Optional[int] = None) -> np.ndarray:
    """Context lengths AFTER this step's append (tokens visible to attention), int32 [batch]."""
    rng = np.random.default_rng([w.seed, 0x5E9])
    if w.name == "tiny":
        lens = np.array([17, 64, 129, 256], dtype=np.int64)
    elif w.name == "llama8b_b64":
        lens = rng.integers(512, 4096, size=w.batch, endpoint=True)
    elif w.name == "mixed_sweep":
        n = WORKLOADS["mixed_sweep"].batch
        z = rng.standard_normal(n)
        interactive = np.minimum(8192, np.maximum(1, np.rint(np.exp(math.log(1024.0) + 0.8 * z))))
        long_ctx = rng.integers(8192, 32768, size=n, endpoint=True)
        is_batch = np.array([is_batch_request(i) for i in range(n)])
        lens = np.where(is_batch, long_ctx, interactive.astype(np.int64))
    elif w.name == "llama70b_full":
        lens = rng.integers(1024, 4096, size=w.batch, endpoint=True)
    elif w.name == "skewed_long":
        lens = np.array([131072] + [1024] * 7, dtype=np.int64)
    else:
        raise KeyError(w.name)
    b = w.batch if batch is None else batch
    if b > lens.size:
        raise ValueError("batch %d exceeds the workload's %d requests" % (b, lens.size))
    return lens[:b].astype(np.int32)


def pages_of(lens: np.ndarray, page_size: int = PAGE_SIZE) -> np.ndarray:
    return (lens.astype(np.int64) + page_size - 1) // page_size


def num_pool_pages(w: Workload, lens: np.ndarray) -> int:
    if w.fixed_num_pages is not None:
        return w.fixed_num_pages
    live = int(pages_of(lens, w.page_size).sum())
    return int(math.ceil(w.pool_factor * live))


def block_tables(lens: np.ndarray, num_pages: int, seed: int,
                 page_size: int = PAGE_SIZE, max_pages_per_req: Optional[int] = None) -> np.ndarray:
    """int32 [batch][max_pages_per_req], padded with -1.

    A seeded random permutation of the physical page ids is dealt out in consecutive runs, one
    run per request, so every request's pages are scattered over the whole pool.
    """
    n = pages_of(lens, page_size)
    if int(n.sum()) > num_pages:
        raise ValueError("pool of %d pages cannot hold %d live pages" % (num_pages, int(n.sum())))
    width = int(n.max()) if max_pages_per_req is None else int(max_pages_per_req)
    if width < int(n.max()):
        raise ValueError("max_pages_per_req too small")
    perm = np.random.default_rng([seed, 0xB10C]).permutation(num_pages).astype(np.int32)
    bt = np.full((lens.size, width), -1, dtype=np.int32)
    at = 0
    for r, cnt in enumerate(n.tolist()):
        bt[r, :cnt] = perm[at:at + cnt]
        at += cnt
    return bt


# ----------------------------------------------------------------------------- values

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, seed, stream: int) -> np.ndarray:
    """i.i.d. N(0,1) rounded once to bf16; uint16 bits of the given shape."""
    rng = np.random.default_rng([int(seed), int(stream), 0xA77])
    return f32_to_bf16_bits(rng.standard_normal(size=shape, dtype=np.float32))


def pool_elems(w: Workload, num_pages: int, num_layers: Optional[int] = None) -> int:
    layers = w.num_layers if num_layers is None else num_layers
    return layers * num_pages * w.num_kv_heads * 2 * w.page_size * w.head_dim


@dataclass
class HostInputs:
    """Everything one decode step consumes, as host numpy arrays (bf16 as uint16 bits)."""
    w: Workload
    num_pages: int
    seq_lens: np.ndarray        # int32 [B]
    block_tables: np.ndarray    # int32 [B][max_pages_per_req]
    pool: np.ndarray            # uint16 [layers][pages][Hkv][2][P][d], state BEFORE the append
    q: np.ndarray               # uint16 [layers][B][Hq][d]
    k_new: np.ndarray           # uint16 [layers][B][Hkv][d]
    v_new: np.ndarray           # uint16 [layers][B][Hkv][d]


def host_inputs(w: Workload, batch: Optional[int] = None,
                max_pages_per_req: Optional[int] = None) -> HostInputs:
    """Draw a full set of host inputs.  Meant for workloads whose pool fits host memory."""
    lens = seq_lens(w, batch)
    npg = num_pool_pages(w, lens)
    bt = block_tables(lens, npg, w.seed, w.page_size, max_pages_per_req)
    b = lens.size
    pool = normal_bf16((w.num_layers, npg, w.num_kv_heads, 2, w.page_size, w.head_dim), w.seed, 1)
    q = normal_bf16((w.num_layers, b, w.num_q_heads, w.head_dim), w.seed, 2)
    k_new = normal_bf16((w.num_layers, b, w.num_kv_heads, w.head_dim), w.seed, 3)
    v_new = normal_bf16((w.num_layers, b, w.num_kv_heads, w.head_dim), w.seed, 4)
    return HostInputs(w, npg, lens, bt, pool, q, k_new, v_new)


# ----------------------------------------------------------------------------- device fills

def device_normal_bf16(shape, seed: int, stream: int, device, chunk_elems: int = 1 << 28):
    """i.i.d. N(0,1) bf16 tensor drawn on `device` with a seeded torch generator, in chunks.

    Used where the pool is too large to draw on the host (tens of GB); the host reads back the
    pages it needs for checking.
    """
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed((int(seed) << 8) ^ int(stream) ^ 0xC41A0)
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for at in range(0, n, chunk_elems):
        m = min(chunk_elems, n - at)
        out[at:at + m].normal_(generator=gen)
    return out.view(*shape)


# ----------------------------------------------------------------------------- accounting

def algorithmic_bytes(w: Workload, lens: np.ndarray, num_layers: Optional[int] = None) -> dict:
    """Bytes one step must move (no partials, no padding of last pages), per component."""
    layers = w.num_layers if num_layers is None else num_layers
    b = int(lens.size)
    d2 = w.head_dim * 2
    kv = int(lens.astype(np.int64).sum()) * w.kv_bytes_per_token
    qo = b * w.num_q_heads * d2 * 2
    append = b * 2 * w.num_kv_heads * d2 * 2
    tables = int(pages_of(lens, w.page_size).sum()) * 4 + b * 4
    return {"kv": layers * kv, "q_out": layers * qo, "append": layers * append,
            "tables": layers * tables, "total": layers * (kv + qo + append + tables)}


# ----------------------------------------------------------------------------- request traces

def arrival_times(n: int, rate: float, cv: float, seed: int, start: float = 0.0) -> np.ndarray:
    """n arrival times with mean rate `rate` per second and inter-arrival coefficient of variation
    `cv`: Gamma inter-arrivals of shape 1 / cv^2 (cv = 1 is a Poisson process, Section 6
    "Workloads"; larger cv is burstier, Section 6 "Impact of Arrival Burstiness")."""
    rng = np.random.default_rng([int(seed), 0xA221])
    shape = 1.0 / (cv * cv)
    gaps = rng.gamma(shape, 1.0 / (shape * rate), size=n)
    return start + np.cumsum(gaps)


def output_lengths(n: int, seed: int, median: float = 180.0, sigma: float = 0.9, cap: int = 2048) -> np.ndarray:
    """Synthetic output-token counts: lognormal, clipped to [1, cap].  Stands in for the ShareGPT
    output-length distribution the paper's traces use (not available offline)."""
    rng = np.random.default_rng([int(seed), 0x0077])
    return np.clip(np.rint(np.exp(math.log(median) + sigma * rng.standard_normal(n))), 1, cap)


def request_trace(n: int, rate: float, cv: float, batch_fraction: float, seed: int,
                  interactive_ttft_s: float = 10.0, batch_ttft_s: float = 3600.0):
    """A trace of n requests in arrival order: (arrival_s, kind [0 interactive, 1 batch],
    output_tokens, ttft_slo_s) with the paper's two request classes (Section 6 "Workloads":
    interactive TTFT SLO 10 s, batch TTFT SLO one hour)."""
    arrival = arrival_times(n, rate, cv, seed)
    rng = np.random.default_rng([int(seed), 0x7A3C])
    kind = (rng.random(n) < batch_fraction).astype(np.int32)
    tokens = output_lengths(n, seed)
    slo = np.where(kind == 0, interactive_ttft_s, batch_ttft_s).astype(np.float64)
    return arrival, kind, tokens, slo
