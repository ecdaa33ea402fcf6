"""Shared helpers for the GPU parity tests: host <-> device marshalling and the tolerance."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

# Attention tolerance against the unrounded fp64 oracle: |err| <= ATOL + RTOL * |ref|.
# bf16 output rounding alone is 2^-9 relative (0.2 %); bf16 probabilities in the PV product and
# fp32 accumulation order add a few 1e-4 absolute on N(0,1) values.
ATOL, RTOL = 4e-3, 1.6e-2


def bits_to_dev(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    """uint16 bf16 bit patterns (host) -> torch.bfloat16 tensor on the device, same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor (any device) -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def widen(bits: np.ndarray) -> np.ndarray:
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def assert_close(gpu_bits: np.ndarray, ref: np.ndarray, what: str = "") -> float:
    got = widen(gpu_bits).reshape(ref.shape)
    err = np.abs(got - ref)
    bound = ATOL + RTOL * np.abs(ref)
    worst = float((err / bound).max())
    if not np.all(err <= bound) or not np.all(np.isfinite(got)):
        idx = np.unravel_index(np.argmax(err / bound), err.shape)
        raise AssertionError("%s: |err| %.3e exceeds %.3e at %s (got %.6f, ref %.6f); %d of %d outside"
                             % (what, err[idx], bound[idx], idx, got[idx], ref[idx],
                                int((err > bound).sum()), err.size))
    return worst


def pool_shape(w: wl.Workload, num_pages: int, num_layers: Optional[int] = None) -> PoolShape:
    return PoolShape(w.num_layers if num_layers is None else num_layers, num_pages,
                     w.num_q_heads, w.num_kv_heads, w.page_size, w.head_dim)


@dataclass
class DeviceStep:
    pool: object               # binding.KvPool
    bt: torch.Tensor
    sl: torch.Tensor
    q: torch.Tensor            # [layers][B][Hq][d]
    k_new: torch.Tensor
    v_new: torch.Tensor
    out: torch.Tensor


def make_device_step(h: wl.HostInputs, max_batch: Optional[int] = None) -> DeviceStep:
    """Upload a HostInputs to the GPU and create the library handle around it."""
    from paper_2501_08090_b200 import binding
    w = h.w
    cfg = binding.make_config(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, h.num_pages,
                              h.block_tables.shape[1], max_batch or max(1, h.seq_lens.size))
    pool_t = bits_to_dev(h.pool.reshape(-1))
    kp = binding.KvPool(cfg, pool=pool_t)
    bt = torch.from_numpy(h.block_tables).cuda()
    sl = torch.from_numpy(h.seq_lens).cuda()
    q = bits_to_dev(h.q); k = bits_to_dev(h.k_new); v = bits_to_dev(h.v_new)
    out = torch.full_like(q, float("nan"))
    return DeviceStep(kp, bt, sl, q, k, v, out)


def oracle_step(h: wl.HostInputs, layer: int = 0):
    """Oracle append + attention for one layer: (pool after append, fp64 out)."""
    sh = pool_shape(h.w, h.num_pages)
    pool = h.pool.copy().reshape(-1)
    rc = oracle.kv_append(pool, sh, layer, h.block_tables, h.seq_lens, h.k_new[layer], h.v_new[layer])
    assert rc == 0
    out = oracle.decode_attention(pool, sh, layer, h.block_tables, h.seq_lens, h.q[layer])
    return pool, out


def compact_requests(pool_dev: torch.Tensor, bt: np.ndarray, lens: np.ndarray, rows, layer: int):
    """Copy the pages of the chosen requests (one layer) to the host as a small dense pool.

    pool_dev: [layers][pages][Hkv][2][P][d] bf16 on the device.  Returns (uint16 pool
    [1][n][Hkv][2][P][d] flattened, remapped block tables, lens) for the oracle.
    """
    P = pool_dev.shape[4]
    rows = list(rows)
    counts = [int((int(lens[r]) + P - 1) // P) for r in rows]
    width = max(counts)
    new_bt = np.full((len(rows), width), -1, dtype=np.int32)
    ids = []
    at = 0
    for i, (r, cnt) in enumerate(zip(rows, counts)):
        ids.append(bt[r, :cnt])
        new_bt[i, :cnt] = np.arange(at, at + cnt, dtype=np.int32)
        at += cnt
    ids = torch.from_numpy(np.concatenate(ids).astype(np.int64)).to(pool_dev.device)
    sub = pool_dev[layer].index_select(0, ids)
    return dev_to_bits(sub).reshape(-1), new_bt, lens[rows].astype(np.int32), at


# ----------------------------------------------------------------------------- the plan's spec

def expected_plan(lens_np, Hkv, C, cost=3):
    """The partition spec restated: `cost` overhead units then one unit per 32-token tile for every
    (request, kv head); span s owns the tiles whose units lie in [s*q, (s+1)*q)."""
    tiles = (lens_np.astype(np.int64) + 31) // 32
    units = tiles + cost
    prefix = np.concatenate([[0], np.cumsum(units)]) * Hkv
    total = int(prefix[-1])
    q = max(1, -(-total // C))
    starts = np.full((C, 4), -1, dtype=np.int64)
    for c in range(C):
        b0, e0 = c * q, min((c + 1) * q, total)
        if b0 >= total:
            continue
        r = int(np.searchsorted(prefix, b0, side="right") - 1)
        rem = b0 - int(prefix[r])
        h, off = rem // int(units[r]), rem % int(units[r])
        tile = max(0, off - cost)
        v = int(prefix[r]) + h * int(units[r]) + cost + tile
        if v < e0:
            starts[c] = [r, h, tile, v]
    return total, q, starts.astype(np.int32)


def covered_tiles(lens_np, Hkv, C, cost=3, counts=None):
    """All (request, kv head, tile) triples the spans of the spec visit, in order.
    If `counts` is a list, the number of tiles of every span is appended to it."""
    tiles = (lens_np.astype(np.int64) + 31) // 32
    total, q, starts = expected_plan(lens_np, Hkv, C, cost)
    seen = []
    for c in range(C):
        r, h, tile, v = (int(x) for x in starts[c])
        before = len(seen)
        if counts is not None:
            counts.append(0)
        if r < 0:
            continue
        end = min((c + 1) * q, total)
        while v < end:
            seen.append((r, h, tile))
            v += 1; tile += 1
            if tile == tiles[r]:
                tile = 0; v += cost; h += 1
                if h == Hkv:
                    h = 0; r += 1
                    if r == lens_np.size:
                        break
        if counts is not None:
            counts[-1] = len(seen) - before
    return seen
