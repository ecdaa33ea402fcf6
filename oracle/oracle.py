"""ctypes front end of the fp64 C oracle (oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  The GPU library never imports this module and shares no code with it.

All arrays are numpy, on the host.  bf16 values travel as uint16 bit patterns.  The KV pool has
the byte format  bf16 [num_layers][num_pages][num_kv_heads][2 (K,V)][page_size][head_dim].
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        i32, i64, f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        vp = ctypes.c_void_p
        lib.oracle_num_threads.restype = i32
        lib.oracle_num_threads.argtypes = []
        lib.oracle_attention_dense_f64.restype = i32
        lib.oracle_attention_dense_f64.argtypes = [vp, vp, vp, i64, i32, f64, vp, vp]
        lib.oracle_attention_split_f64.restype = i32
        lib.oracle_attention_split_f64.argtypes = [vp, vp, vp, i64, i32, f64, vp, i32, vp]
        lib.oracle_kv_append.restype = i32
        lib.oracle_kv_append.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.oracle_decode_attention.restype = i32
        lib.oracle_decode_attention.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32,
                                                vp, vp, vp, vp]
        lib.oracle_kv_append_multi.restype = i32
        lib.oracle_kv_append_multi.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.oracle_decode_attention_multi.restype = i32
        lib.oracle_decode_attention_multi.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, i32,
                                                      vp, vp, vp, vp]
        _lib = lib
    return _lib


@dataclass(frozen=True)
class PoolShape:
    """Dimensions of a paged KV pool (bf16)."""
    num_layers: int
    num_pages: int
    num_q_heads: int
    num_kv_heads: int
    page_size: int
    head_dim: int

    @property
    def elems(self) -> int:
        return (self.num_layers * self.num_pages * self.num_kv_heads * 2
                * self.page_size * self.head_dim)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def attention_dense(q, K, V, scale: float, return_weights: bool = False):
    """softmax(scale * K q) weighted mean of V's rows, all fp64.  q [d], K [L][d], V [L][d]."""
    q = _c(q, np.float64); K = _c(K, np.float64); V = _c(V, np.float64)
    L, d = K.shape
    assert q.shape == (d,) and V.shape == (L, d)
    out = np.empty(d, dtype=np.float64)
    w = np.empty(L, dtype=np.float64) if return_weights else None
    rc = _load().oracle_attention_dense_f64(_p(q), _p(K), _p(V), L, d, float(scale), _p(out),
                                            _p(w) if w is not None else None)
    if rc != 0:
        raise ValueError("oracle_attention_dense_f64 failed: %d" % rc)
    return (out, w) if return_weights else out


def attention_split(q, K, V, scale: float, cuts):
    """Same result through split-KV partials at the given cut positions and an LSE combine."""
    q = _c(q, np.float64); K = _c(K, np.float64); V = _c(V, np.float64)
    L, d = K.shape
    cuts = _c(np.asarray(cuts, dtype=np.int64).reshape(-1), np.int64)
    out = np.empty(d, dtype=np.float64)
    rc = _load().oracle_attention_split_f64(_p(q), _p(K), _p(V), L, d, float(scale),
                                            _p(cuts), int(cuts.size), _p(out))
    if rc != 0:
        raise ValueError("oracle_attention_split_f64 failed: %d" % rc)
    return out


def kv_append(pool: np.ndarray, shape: PoolShape, layer: int, block_tables, seq_lens,
              k_new, v_new) -> int:
    """In-place append of each request's new token; returns the oracle's status code."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.size == shape.elems
    bt = _c(block_tables, np.int32); sl = _c(seq_lens, np.int32)
    k = _c(k_new, np.uint16); v = _c(v_new, np.uint16)
    batch, max_pages = bt.shape
    assert sl.shape == (batch,)
    assert k.size == batch * shape.num_kv_heads * shape.head_dim == v.size
    return int(_load().oracle_kv_append(_p(pool), shape.num_layers, shape.num_pages,
                                        shape.num_kv_heads, shape.page_size, shape.head_dim,
                                        layer, batch, max_pages, _p(bt), _p(sl), _p(k), _p(v)))


def decode_attention(pool: np.ndarray, shape: PoolShape, layer: int, block_tables, seq_lens,
                     q) -> np.ndarray:
    """fp64 attention output [batch][num_q_heads][head_dim] for one layer of the pool."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.size == shape.elems
    bt = _c(block_tables, np.int32); sl = _c(seq_lens, np.int32); qq = _c(q, np.uint16)
    batch, max_pages = bt.shape
    assert qq.size == batch * shape.num_q_heads * shape.head_dim
    out = np.zeros((batch, shape.num_q_heads, shape.head_dim), dtype=np.float64)
    rc = _load().oracle_decode_attention(_p(pool), shape.num_layers, shape.num_pages,
                                         shape.num_q_heads, shape.num_kv_heads, shape.page_size,
                                         shape.head_dim, layer, batch, max_pages,
                                         _p(bt), _p(sl), _p(qq), _p(out))
    if rc != 0:
        raise ValueError("oracle_decode_attention failed: %d" % rc)
    return out


def kv_append_multi(pool: np.ndarray, shape: PoolShape, layer: int, q_len: int, block_tables, seq_lens,
                    k_new, v_new) -> int:
    """In-place append of q_len new tokens per request (k_new, v_new [batch][q_len][Hkv][d])."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.size == shape.elems
    bt = _c(block_tables, np.int32); sl = _c(seq_lens, np.int32)
    k = _c(k_new, np.uint16); v = _c(v_new, np.uint16)
    batch, max_pages = bt.shape
    assert k.size == batch * q_len * shape.num_kv_heads * shape.head_dim == v.size
    return int(_load().oracle_kv_append_multi(_p(pool), shape.num_layers, shape.num_pages, shape.num_kv_heads,
                                              shape.page_size, shape.head_dim, layer, batch, q_len, max_pages,
                                              _p(bt), _p(sl), _p(k), _p(v)))


def decode_attention_multi(pool: np.ndarray, shape: PoolShape, layer: int, q_len: int, block_tables, seq_lens,
                           q) -> np.ndarray:
    """Causal attention of the q_len new tokens: fp64 [batch][q_len][Hq][d]."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.size == shape.elems
    bt = _c(block_tables, np.int32); sl = _c(seq_lens, np.int32); qq = _c(q, np.uint16)
    batch, max_pages = bt.shape
    assert qq.size == batch * q_len * shape.num_q_heads * shape.head_dim
    out = np.zeros((batch, q_len, shape.num_q_heads, shape.head_dim), dtype=np.float64)
    rc = _load().oracle_decode_attention_multi(_p(pool), shape.num_layers, shape.num_pages, shape.num_q_heads,
                                               shape.num_kv_heads, shape.page_size, shape.head_dim, layer, batch,
                                               q_len, max_pages, _p(bt), _p(sl), _p(qq), _p(out))
    if rc != 0:
        raise ValueError("oracle_decode_attention_multi failed: %d" % rc)
    return out
