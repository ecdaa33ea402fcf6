"""Pins for the fp64 oracle: things the mathematics fixes, none of which re-use its formula.

The paper prints no numbers for this path, so the pins are hand-computed cases
(tests/golden/hand_cases.txt), closed forms, invariants, an independently written numpy brute
force on dense (non-paged) tensors and torch's float64 softmax as a third opinion.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.txt")


# --------------------------------------------------------------------------- helpers

def _num(tok):
    return {"ln3": math.log(3.0), "ln2": math.log(2.0)}.get(tok) if tok in ("ln3", "ln2") else float(tok)


def _rows(field):
    return np.array([[_num(t) for t in row.split()] for row in field.split(";")], dtype=np.float64)


def load_hand_cases():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, scale, q, K, V, out, tol = [x.strip() for x in line.split("|")]
            cases.append((name, float(scale), _rows(q)[0], _rows(K), _rows(V), _rows(out)[0], float(tol)))
    return cases


HAND = load_hand_cases()


def brute_force_dense(q, K, V, scale):
    """Textbook softmax attention in numpy float64, written independently of the oracle."""
    logits = (K @ q) * scale
    p = np.exp(logits - logits.max())
    p = p / p.sum()
    return p @ V


def widen(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def gather_dense(pool, shape, layer, bt_row, L, kh):
    """Dense K, V [L][d] of one request / KV head, gathered with numpy fancy indexing."""
    P = shape.page_size
    p6 = pool.reshape(shape.num_layers, shape.num_pages, shape.num_kv_heads, 2, P, shape.head_dim)
    j = np.arange(L)
    pages = bt_row[j // P]
    K = widen(p6[layer, pages, kh, 0, j % P, :])
    V = widen(p6[layer, pages, kh, 1, j % P, :])
    return K, V


def tiny_inputs():
    return wl.host_inputs(wl.workload("tiny"))


def shape_of(h):
    w = h.w
    return PoolShape(w.num_layers, h.num_pages, w.num_q_heads, w.num_kv_heads, w.page_size, w.head_dim)


# --------------------------------------------------------------------------- the formula

@pytest.mark.parametrize("case", HAND, ids=[c[0] for c in HAND])
def test_hand_cases(case):
    _, scale, q, K, V, expected, tol = case
    out = oracle.attention_dense(q, K, V, scale)
    assert np.allclose(out, expected, rtol=0, atol=tol), (out, expected)


def test_hand_cases_reject_planted_mistakes():
    """The hand cases are sharp enough: each plausible slip fails at least one of them."""
    def no_scale(q, K, V, s): return brute_force_dense(q, K, V, 1.0)
    def kv_swapped(q, K, V, s): return brute_force_dense(q, V, K, s) if K.shape == V.shape else None
    def wrong_sign(q, K, V, s): return brute_force_dense(-q, K, V, s)
    def unnormalised(q, K, V, s):
        lg = (K @ q) * s
        return np.exp(lg - lg.max()) @ V
    def mean_only(q, K, V, s): return V.mean(axis=0)
    for wrong in (no_scale, kv_swapped, wrong_sign, unnormalised, mean_only):
        failed = False
        for _, scale, q, K, V, expected, tol in HAND:
            got = wrong(q, K, V, scale)
            if got is None or not np.allclose(got, expected, rtol=0, atol=1e-9):
                failed = True
        assert failed, wrong.__name__
    # and the correct brute force passes all of them
    for _, scale, q, K, V, expected, tol in HAND:
        assert np.allclose(brute_force_dense(q, K, V, scale), expected, rtol=0, atol=1e-12)


def test_length_one_returns_v():
    rng = np.random.default_rng(1)
    for d in (1, 64, 128):
        q = rng.standard_normal(d); K = rng.standard_normal((1, d)) * 50; V = rng.standard_normal((1, d))
        out = oracle.attention_dense(q, K, V, 1 / math.sqrt(d))
        assert np.array_equal(out, V[0])


def test_zero_query_and_equal_keys_give_mean():
    rng = np.random.default_rng(2)
    L, d = 37, 64
    V = rng.standard_normal((L, d)); K = rng.standard_normal((L, d))
    out = oracle.attention_dense(np.zeros(d), K, V, 0.125)
    assert np.allclose(out, V.mean(axis=0), rtol=0, atol=1e-14)
    Ksame = np.tile(rng.standard_normal(d), (L, 1))
    out = oracle.attention_dense(rng.standard_normal(d), Ksame, V, 0.125)
    assert np.allclose(out, V.mean(axis=0), rtol=0, atol=1e-14)


def test_dominant_key_and_large_scores_do_not_overflow():
    rng = np.random.default_rng(3)
    L, d, jstar = 50, 64, 31
    q = rng.standard_normal(d)
    K = np.zeros((L, d)); V = rng.standard_normal((L, d))
    scale = 1 / math.sqrt(d)
    t = 1000.0 / (scale * (q @ q))           # winning score = 1000, every other score = 0
    K[jstar] = t * q
    out, w = oracle.attention_dense(q, K, V, scale, return_weights=True)
    assert np.all(np.isfinite(out))
    assert abs(w[jstar] - 1.0) < 1e-15 and w.sum() == pytest.approx(1.0, abs=1e-15)
    assert np.allclose(out, V[jstar], rtol=0, atol=1e-15 * np.abs(V).max() * L)
    # all scores hugely negative: still finite, still a proper average
    out2 = oracle.attention_dense(q, -np.abs(t) * np.tile(q, (L, 1)), V, scale)
    assert np.allclose(out2, V.mean(axis=0), rtol=0, atol=1e-13)


def test_weights_sum_to_one_and_output_in_convex_hull():
    rng = np.random.default_rng(4)
    for L, d in ((1, 64), (17, 64), (300, 128)):
        q = rng.standard_normal(d); K = rng.standard_normal((L, d)); V = rng.standard_normal((L, d))
        out, w = oracle.attention_dense(q, K, V, 1 / math.sqrt(d), return_weights=True)
        assert abs(w.sum() - 1.0) < 1e-14 and np.all(w >= 0)
        assert np.all(out <= V.max(axis=0) + 1e-14) and np.all(out >= V.min(axis=0) - 1e-14)
        assert np.allclose(out, w @ V, rtol=0, atol=1e-14)


def test_softmax_shift_invariance():
    rng = np.random.default_rng(5)
    L, d = 129, 128
    q = rng.standard_normal(d); K = rng.standard_normal((L, d)); V = rng.standard_normal((L, d))
    u = rng.standard_normal(d) * 3
    a = oracle.attention_dense(q, K, V, 1 / math.sqrt(d))
    b = oracle.attention_dense(q, K + u, V, 1 / math.sqrt(d))
    assert np.allclose(a, b, rtol=1e-12, atol=1e-12)


def test_value_linearity():
    """out is linear in V: attention(q,K,aV1+bV2) = a*attention(q,K,V1) + b*attention(q,K,V2)."""
    rng = np.random.default_rng(6)
    L, d = 40, 64
    q = rng.standard_normal(d); K = rng.standard_normal((L, d))
    V1 = rng.standard_normal((L, d)); V2 = rng.standard_normal((L, d))
    s = 0.125
    lhs = oracle.attention_dense(q, K, 2.0 * V1 - 3.0 * V2, s)
    rhs = 2.0 * oracle.attention_dense(q, K, V1, s) - 3.0 * oracle.attention_dense(q, K, V2, s)
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("L,d", [(2, 64), (17, 64), (129, 64), (300, 128), (1000, 128)])
def test_dense_matches_numpy_brute_force_and_torch(L, d):
    rng = np.random.default_rng(100 + L)
    q = rng.standard_normal(d); K = rng.standard_normal((L, d)); V = rng.standard_normal((L, d))
    scale = 1 / math.sqrt(d)
    out = oracle.attention_dense(q, K, V, scale)
    assert np.allclose(out, brute_force_dense(q, K, V, scale), rtol=1e-12, atol=1e-13)
    tq, tK, tV = (torch.from_numpy(x) for x in (q, K, V))
    ref = (torch.softmax((tK @ tq) * scale, dim=-1) @ tV).numpy()
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------- split + combine

@pytest.mark.parametrize("cuts", [[], [1], [64], [128], [1, 2, 3], [16, 32, 100, 128], [5, 77, 128, 129]])
def test_split_combine_equals_direct(cuts):
    rng = np.random.default_rng(7)
    L, d = 130, 64
    q = rng.standard_normal(d) * 4; K = rng.standard_normal((L, d)) * 4; V = rng.standard_normal((L, d))
    scale = 1 / math.sqrt(d)
    direct = oracle.attention_dense(q, K, V, scale)
    split = oracle.attention_split(q, K, V, scale, cuts)
    assert np.allclose(split, direct, rtol=1e-12, atol=1e-13)
    assert np.allclose(split, brute_force_dense(q, K, V, scale), rtol=1e-12, atol=1e-13)


def test_split_combine_random_partitions_with_extreme_chunks():
    rng = np.random.default_rng(8)
    L, d = 257, 128
    q = rng.standard_normal(d); K = rng.standard_normal((L, d)); V = rng.standard_normal((L, d))
    K[200] = 40 * q                      # one chunk's maximum towers over the others
    scale = 1 / math.sqrt(d)
    direct = brute_force_dense(q, K, V, scale)
    for _ in range(20):
        k = int(rng.integers(1, 12))
        cuts = np.sort(rng.choice(np.arange(1, L), size=k, replace=False))
        assert np.allclose(oracle.attention_split(q, K, V, scale, cuts), direct, rtol=1e-12, atol=1e-13)


def test_split_rejects_bad_cuts():
    q = np.ones(4); K = np.ones((8, 4)); V = np.ones((8, 4))
    for bad in ([0], [8], [3, 3], [5, 2]):
        with pytest.raises(ValueError):
            oracle.attention_split(q, K, V, 1.0, bad)


# --------------------------------------------------------------------------- paging

def test_paged_matches_dense_brute_force_on_tiny_workload():
    h = tiny_inputs()
    sh = shape_of(h)
    pool = h.pool.copy().reshape(-1)
    assert oracle.kv_append(pool, sh, 0, h.block_tables, h.seq_lens, h.k_new[0], h.v_new[0]) == 0
    out = oracle.decode_attention(pool, sh, 0, h.block_tables, h.seq_lens, h.q[0])
    G = h.w.group
    scale = 1 / math.sqrt(h.w.head_dim)
    for r, L in enumerate(h.seq_lens.tolist()):
        for hq in range(h.w.num_q_heads):
            K, V = gather_dense(pool, sh, 0, h.block_tables[r], L, hq // G)
            # the appended token must be the last gathered row
            assert np.array_equal(K[-1], widen(h.k_new[0, r, hq // G]))
            assert np.array_equal(V[-1], widen(h.v_new[0, r, hq // G]))
            ref = brute_force_dense(widen(h.q[0, r, hq]), K, V, scale)
            assert np.allclose(out[r, hq], ref, rtol=1e-12, atol=1e-13)


def test_paged_random_shapes_against_brute_force_and_torch():
    rng = np.random.default_rng(9)
    for trial in range(6):
        d = (64, 128)[trial % 2]
        Hkv = int(rng.integers(1, 4)); G = (1, 2, 4, 8)[trial % 4]; Hq = Hkv * G
        B = int(rng.integers(1, 5)); layers = 2; layer = trial % 2
        lens = rng.integers(1, 301, size=B).astype(np.int32)
        npg = int(wl.pages_of(lens).sum()) + 5
        bt = wl.block_tables(lens, npg, seed=trial)
        sh = PoolShape(layers, npg, Hq, Hkv, 16, d)
        pool = wl.normal_bf16((sh.elems,), trial, 1)
        q = wl.normal_bf16((B, Hq, d), trial, 2)
        out = oracle.decode_attention(pool, sh, layer, bt, lens, q)
        scale = 1 / math.sqrt(d)
        for r in range(B):
            for hq in range(Hq):
                K, V = gather_dense(pool, sh, layer, bt[r], int(lens[r]), hq // G)
                qd = widen(q[r, hq])
                assert np.allclose(out[r, hq], brute_force_dense(qd, K, V, scale), rtol=1e-12, atol=1e-13)
                tref = torch.softmax(torch.from_numpy(K @ qd * scale), -1) @ torch.from_numpy(V)
                assert np.allclose(out[r, hq], tref.numpy(), rtol=1e-12, atol=1e-13)


def test_page_permutation_is_bit_exact_invariant():
    h = tiny_inputs()
    sh = shape_of(h)
    base = oracle.decode_attention(h.pool.reshape(-1), sh, 0, h.block_tables, h.seq_lens, h.q[0])
    perm = np.random.default_rng(11).permutation(h.num_pages)       # new id of old page p
    p6 = h.pool.reshape(1, h.num_pages, -1)
    moved = np.empty_like(p6)
    moved[:, perm, :] = p6
    bt2 = np.where(h.block_tables >= 0, perm[np.maximum(h.block_tables, 0)], -1).astype(np.int32)
    out = oracle.decode_attention(moved.reshape(-1), sh, 0, bt2, h.seq_lens, h.q[0])
    assert np.array_equal(out, base)


def test_paged_length_one_returns_appended_v_exactly():
    w = wl.workload("tiny")
    sh = PoolShape(1, 8, w.num_q_heads, w.num_kv_heads, 16, w.head_dim)
    pool = wl.normal_bf16((sh.elems,), 5, 1)
    lens = np.array([1, 1], dtype=np.int32)
    bt = np.array([[6], [2]], dtype=np.int32)
    k = wl.normal_bf16((2, 1, 64), 5, 3); v = wl.normal_bf16((2, 1, 64), 5, 4)
    q = wl.normal_bf16((2, 4, 64), 5, 2)
    assert oracle.kv_append(pool, sh, 0, bt, lens, k, v) == 0
    out = oracle.decode_attention(pool, sh, 0, bt, lens, q)
    for r in range(2):
        for hq in range(4):
            assert np.array_equal(out[r, hq], widen(v[r, 0]))


def test_gqa_head_mapping():
    rng = np.random.default_rng(12)
    Hkv, G, d, B = 2, 4, 64, 2
    lens = np.array([40, 17], dtype=np.int32)
    npg = 8
    bt = wl.block_tables(lens, npg, seed=3)
    sh = PoolShape(1, npg, Hkv * G, Hkv, 16, d)
    pool = wl.normal_bf16((sh.elems,), 12, 1)
    q = wl.normal_bf16((B, Hkv * G, d), 12, 2)
    q[:, 1:4] = q[:, 0:1]                                   # heads 0..3 share one query
    out = oracle.decode_attention(pool, sh, 0, bt, lens, q)
    for g in range(1, 4):
        assert np.array_equal(out[:, g], out[:, 0])
    assert not np.array_equal(out[:, 4], out[:, 0])
    # swapping the two KV heads' data while swapping the query groups swaps the outputs
    p6 = pool.reshape(1, npg, Hkv, 2, 16, d)
    swapped = p6[:, :, ::-1].copy().reshape(-1)
    q2 = np.concatenate([q[:, 4:8], q[:, 0:4]], axis=1)
    out2 = oracle.decode_attention(swapped, sh, 0, bt, lens, q2)
    assert np.array_equal(out2[:, 0:4], out[:, 4:8]) and np.array_equal(out2[:, 4:8], out[:, 0:4])


def test_layers_are_independent():
    w = wl.workload("tiny", num_layers=3)
    h = wl.host_inputs(w)
    sh = shape_of(h)
    pool = h.pool.reshape(-1)
    for layer in range(3):
        out = oracle.decode_attention(pool, sh, layer, h.block_tables, h.seq_lens, h.q[layer])
        single = PoolShape(1, sh.num_pages, sh.num_q_heads, sh.num_kv_heads, 16, sh.head_dim)
        sl = h.pool[layer].reshape(-1)
        ref = oracle.decode_attention(np.ascontiguousarray(sl), single, 0, h.block_tables, h.seq_lens, h.q[layer])
        assert np.array_equal(out, ref)


# --------------------------------------------------------------------------- append

def test_append_replaces_exactly_the_target_rows_and_is_idempotent():
    h = tiny_inputs()
    sh = shape_of(h)
    before = h.pool.copy()
    pool = h.pool.copy().reshape(-1)
    assert oracle.kv_append(pool, sh, 0, h.block_tables, h.seq_lens, h.k_new[0], h.v_new[0]) == 0
    after = pool.reshape(before.shape)
    expect = before.copy()
    P = 16
    for r, L in enumerate(h.seq_lens.tolist()):
        page = h.block_tables[r, (L - 1) // P]; slot = (L - 1) % P
        expect[0, page, :, 0, slot, :] = h.k_new[0, r]
        expect[0, page, :, 1, slot, :] = h.v_new[0, r]
    assert np.array_equal(after, expect)
    changed_rows = int((after != before).any(axis=-1).sum())
    assert changed_rows <= 4 * 1 * 2                       # B * Hkv * (K and V)
    assert changed_rows >= 4 * 1 * 2 - 1                   # identical random rows are not expected
    again = pool.copy()
    assert oracle.kv_append(again, sh, 0, h.block_tables, h.seq_lens, h.k_new[0], h.v_new[0]) == 0
    assert np.array_equal(again, pool)


def test_append_page_boundaries():
    """L % 16 == 1 opens a fresh page at slot 0; L % 16 == 0 fills the last slot of a page."""
    sh = PoolShape(2, 6, 2, 2, 16, 64)
    zero = np.zeros(sh.elems, dtype=np.uint16)
    lens = np.array([17, 32, 1, 16], dtype=np.int32)
    bt = np.array([[0, 5], [3, 1], [2, -1], [4, -1]], dtype=np.int32)
    k = np.arange(4 * 2 * 64, dtype=np.uint16).reshape(4, 2, 64) + 1
    v = k + 1000
    pool = zero.copy()
    assert oracle.kv_append(pool, sh, 1, bt, lens, k, v) == 0
    p6 = pool.reshape(2, 6, 2, 2, 16, 64)
    assert not p6[0].any()                                   # layer 0 untouched
    for r, (page, slot) in enumerate([(5, 0), (1, 15), (2, 0), (4, 15)]):
        assert np.array_equal(p6[1, page, :, 0, slot], k[r])
        assert np.array_equal(p6[1, page, :, 1, slot], v[r])
    assert int((p6 != 0).any(axis=-1).sum()) == 4 * 2 * 2


def test_invalid_inputs_are_reported_not_followed():
    sh = PoolShape(1, 4, 2, 1, 16, 64)
    pool = np.zeros(sh.elems, dtype=np.uint16)
    k = np.ones((1, 1, 64), dtype=np.uint16)
    assert oracle.kv_append(pool, sh, 0, np.array([[9]], np.int32), np.array([1], np.int32), k, k) == -4
    assert oracle.kv_append(pool, sh, 0, np.array([[0]], np.int32), np.array([0], np.int32), k, k) == -1
    assert oracle.kv_append(pool, sh, 0, np.array([[0]], np.int32), np.array([17], np.int32), k, k) == -1
    assert not pool.any()
    with pytest.raises(ValueError):
        oracle.decode_attention(pool, sh, 0, np.array([[7]], np.int32), np.array([3], np.int32),
                                np.ones((1, 2, 64), np.uint16))
