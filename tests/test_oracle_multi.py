"""Pins for the oracle's multi-token step (q_len new tokens per request, causal among them).

Pinned by what does not re-use its code: q_len = 1 must be the single-token path; token i of a
multi-token step must equal a single-token step on the context truncated after token i (the
definition of causality); an independent numpy brute force with an explicit causal mask; and the
append must equal q_len single appends in order.
"""
import math

import numpy as np
import pytest

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl


def widen(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def setup(q_len, lens, Hq=8, Hkv=2, d=64, seed=3):
    lens = np.asarray(lens, dtype=np.int32)
    npg = int(wl.pages_of(lens).sum()) + 4
    bt = wl.block_tables(lens, npg, seed)
    sh = PoolShape(1, npg, Hq, Hkv, 16, d)
    pool = wl.normal_bf16((sh.elems,), seed, 1)
    B = lens.size
    q = wl.normal_bf16((B, q_len, Hq, d), seed, 2)
    k = wl.normal_bf16((B, q_len, Hkv, d), seed, 3)
    v = wl.normal_bf16((B, q_len, Hkv, d), seed, 4)
    return lens, bt, sh, pool, q, k, v


def test_one_new_token_is_the_single_token_path():
    lens, bt, sh, pool, q, k, v = setup(1, [17, 64, 129, 5])
    a, b = pool.copy(), pool.copy()
    assert oracle.kv_append_multi(a, sh, 0, 1, bt, lens, k, v) == 0
    assert oracle.kv_append(b, sh, 0, bt, lens, k[:, 0], v[:, 0]) == 0
    assert np.array_equal(a, b)
    multi = oracle.decode_attention_multi(a, sh, 0, 1, bt, lens, q)
    single = oracle.decode_attention(b, sh, 0, bt, lens, q[:, 0])
    assert np.array_equal(multi[:, 0], single)


@pytest.mark.parametrize("q_len", [2, 3, 4, 8])
def test_multi_append_equals_single_appends_in_order(q_len):
    lens, bt, sh, pool, q, k, v = setup(q_len, [q_len, 16, 17, 33, 100, 130])
    a, b = pool.copy(), pool.copy()
    assert oracle.kv_append_multi(a, sh, 0, q_len, bt, lens, k, v) == 0
    for i in range(q_len):
        step_lens = (lens - q_len + 1 + i).astype(np.int32)
        assert oracle.kv_append(b, sh, 0, bt, step_lens, k[:, i], v[:, i]) == 0
    assert np.array_equal(a, b)


@pytest.mark.parametrize("q_len", [2, 4, 5])
def test_token_i_equals_a_single_token_step_on_the_truncated_context(q_len):
    lens, bt, sh, pool, q, k, v = setup(q_len, [q_len, 20, 47, 48, 49, 200])
    assert oracle.kv_append_multi(pool, sh, 0, q_len, bt, lens, k, v) == 0
    multi = oracle.decode_attention_multi(pool, sh, 0, q_len, bt, lens, q)
    for i in range(q_len):
        trunc = (lens - q_len + 1 + i).astype(np.int32)
        single = oracle.decode_attention(pool, sh, 0, bt, trunc, q[:, i])
        assert np.array_equal(multi[:, i], single)


def test_against_numpy_brute_force_with_an_explicit_causal_mask():
    q_len, Hq, Hkv, d = 3, 4, 2, 64
    lens, bt, sh, pool, q, k, v = setup(q_len, [3, 40, 97], Hq, Hkv, d, seed=9)
    assert oracle.kv_append_multi(pool, sh, 0, q_len, bt, lens, k, v) == 0
    out = oracle.decode_attention_multi(pool, sh, 0, q_len, bt, lens, q)
    p6 = pool.reshape(1, sh.num_pages, Hkv, 2, 16, d)
    for r, L in enumerate(lens.tolist()):
        j = np.arange(L)
        pages = bt[r][j // 16]
        for h in range(Hq):
            K = widen(p6[0, pages, h // 2, 0, j % 16]); V = widen(p6[0, pages, h // 2, 1, j % 16])
            Q = widen(q[r, :, h])                                         # [q_len][d]
            logits = Q @ K.T / math.sqrt(d)                               # [q_len][L]
            pos = L - q_len + np.arange(q_len)[:, None]
            logits = np.where(j[None, :] <= pos, logits, -np.inf)        # causal: token sees itself and earlier
            w = np.exp(logits - logits.max(axis=1, keepdims=True))
            ref = (w / w.sum(axis=1, keepdims=True)) @ V
            assert np.allclose(out[r, :, h], ref, rtol=1e-12, atol=1e-13)
    # the last new token's own key/value are what was appended
    r, L = 2, int(lens[2])
    assert np.array_equal(p6[0, bt[r][(L - 1) // 16], :, 0, (L - 1) % 16], k[r, q_len - 1])


def test_bad_lengths_are_rejected():
    lens, bt, sh, pool, q, k, v = setup(4, [3])                           # fewer tokens than new tokens
    assert oracle.kv_append_multi(pool.copy(), sh, 0, 4, bt, lens, k, v) == -1
    with pytest.raises(ValueError):
        oracle.decode_attention_multi(pool, sh, 0, 4, bt, lens, q)
