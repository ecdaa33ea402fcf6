"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded inputs.

Append and block-table indexing are bit-exact (whole-pool comparison); attention is within
|err| <= 4e-3 + 1.6e-2*|ref| elementwise.
"""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

from helpers import (assert_close, bits_to_dev, dev_to_bits, expected_plan, make_device_step, oracle_step,
                     pool_shape, widen)

pytestmark = pytest.mark.gpu


def binding():
    from paper_2501_08090_b200 import binding as b
    return b


def run_step(h, layer=0, partition=None, fused=False):
    ds = make_device_step(h)
    if partition is not None:
        ds.pool.set_partition(partition)
    if fused:
        ds.pool.decode_step(layer, ds.bt, ds.sl, ds.q[layer], ds.k_new[layer], ds.v_new[layer], ds.out[layer])
    else:
        ds.pool.kv_append(layer, ds.bt, ds.sl, ds.k_new[layer], ds.v_new[layer])
        ds.pool.decode_attention(layer, ds.bt, ds.sl, ds.q[layer], ds.out[layer])
    bits = ds.pool.check_status()
    assert bits == 0
    return ds


def custom_inputs(lens, Hq, Hkv, d, seed, layers=1, extra_pages=3, max_pages=None):
    w = wl.Workload("custom", seed, layers, Hq, Hkv, d, len(lens), 1.0)
    lens = np.asarray(lens, dtype=np.int32)
    npg = int(wl.pages_of(lens).sum()) + extra_pages
    bt = wl.block_tables(lens, npg, seed, 16, max_pages)
    B = lens.size
    return wl.HostInputs(
        w, npg, lens, bt,
        wl.normal_bf16((layers, npg, Hkv, 2, 16, d), seed, 1),
        wl.normal_bf16((layers, B, Hq, d), seed, 2),
        wl.normal_bf16((layers, B, Hkv, d), seed, 3),
        wl.normal_bf16((layers, B, Hkv, d), seed, 4))


# --------------------------------------------------------------------------- config 1

def test_tiny_workload_append_bit_exact_and_attention_within_tolerance():
    h = wl.host_inputs(wl.workload("tiny"))
    ref_pool, ref_out = oracle_step(h)
    ds = run_step(h)
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)           # every byte of the pool
    assert_close(dev_to_bits(ds.out[0]), ref_out, "tiny")


@pytest.mark.parametrize("partition", [1, 2, 3, 5, 31, 37, 148, 592, 1021, 2048])
def test_partition_invariance_on_tiny_workload(partition):
    h = wl.host_inputs(wl.workload("tiny"))
    _, ref_out = oracle_step(h)
    ds = run_step(h, partition=partition)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "tiny/partition=%d" % partition)


# --------------------------------------------------------------------------- fused append + attention

@pytest.mark.parametrize("Hq,Hkv,d", [(4, 1, 64), (8, 2, 128), (32, 8, 128), (64, 8, 128), (5, 1, 128)])
def test_decode_step_equals_append_then_attention(Hq, Hkv, d):
    lens = [1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 49, 64, 65, 96, 97, 129, 300, 1000, 2049]
    h = custom_inputs(lens, Hq, Hkv, d, seed=Hq * 7 + d)
    ref_pool, ref_out = oracle_step(h)
    for partition in (None, 1, 9, 2048):
        ds = run_step(h, partition=partition, fused=True)
        assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)           # every byte of the pool
        assert_close(dev_to_bits(ds.out[0]), ref_out, "fused Hq=%d Hkv=%d d=%d part=%s" % (Hq, Hkv, d, partition))


def test_decode_step_on_tiny_workload_and_with_poisoned_unused_slots():
    h = wl.host_inputs(wl.workload("tiny"))
    ref_pool, ref_out = oracle_step(h)
    ds = run_step(h, fused=True)
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "tiny fused")
    # the slot being appended to may hold anything before the step, NaN included
    h = custom_inputs([5, 17, 70, 130, 1, 64, 33], 8, 2, 128, seed=19, extra_pages=2)
    P = 16
    live = np.zeros((h.num_pages, P), dtype=bool)
    for r, L in enumerate(h.seq_lens.tolist()):
        for j in range(L - 1):                                              # everything but the new token
            live[h.block_tables[r, j // P], j % P] = True
    pool = h.pool.reshape(1, h.num_pages, 2, 2, P, 128)
    dead_pages, dead_slots = np.nonzero(~live)
    pool[0, dead_pages, :, :, dead_slots, :] = 0x7FC0
    ref_pool, ref_out = oracle_step(h)
    assert np.all(np.isfinite(ref_out))
    ds = run_step(h, fused=True)
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "fused, NaN in the target slots")


def test_decode_step_reports_bad_append_pages_without_writing():
    b = binding()
    h = custom_inputs([50, 60], 8, 2, 128, seed=54)
    h.block_tables[0, 3] = -7                                    # the append target of request 0
    ds = make_device_step(h)
    before = dev_to_bits(ds.pool.pool).copy()
    ds.pool.decode_step(0, ds.bt, ds.sl, ds.q[0], ds.k_new[0], ds.v_new[0], ds.out[0])
    assert ds.pool.check_status(raise_on_error=False) & b.STATUS_BAD_PAGE
    after = dev_to_bits(ds.pool.pool).reshape(1, h.num_pages, 2, 2, 16, 128)
    changed = (after != before.reshape(after.shape)).any(axis=-1)
    assert int(changed.sum()) == 1 * 2 * 2                       # request 1 only


# --------------------------------------------------------------------------- shapes and edges

@pytest.mark.parametrize("Hq,Hkv,d", [(1, 1, 64), (2, 1, 64), (8, 1, 64), (8, 2, 128), (32, 8, 128),
                                       (64, 8, 128), (6, 2, 128), (5, 1, 128), (7, 1, 64)])
def test_group_sizes_and_head_dims(Hq, Hkv, d):
    h = custom_inputs([1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 300, 1000], Hq, Hkv, d, seed=Hq * 131 + d)
    ref_pool, ref_out = oracle_step(h)
    for partition in (None, 7):
        ds = run_step(h, partition=partition)
        assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
        assert_close(dev_to_bits(ds.out[0]), ref_out, "Hq=%d Hkv=%d d=%d" % (Hq, Hkv, d))


def test_length_one_returns_v_bit_exact():
    h = custom_inputs([1, 1, 1], 8, 2, 128, seed=77)
    ds = run_step(h)
    out = dev_to_bits(ds.out[0])
    for r in range(3):
        for hq in range(8):
            assert np.array_equal(out[r, hq], h.v_new[0, r, hq // 4])


def test_single_request_batch_and_every_length_around_tile_edges():
    for L in (1, 2, 16, 17, 31, 32, 33, 47, 48, 49, 63, 64, 65, 79, 80, 81, 128, 191, 192, 193, 257):
        h = custom_inputs([L], 4, 1, 64, seed=L)
        ref_pool, ref_out = oracle_step(h)
        ds = run_step(h)
        assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
        assert_close(dev_to_bits(ds.out[0]), ref_out, "L=%d" % L)


def test_multi_layer_pools_are_addressed_per_layer():
    h = custom_inputs([40, 130, 700], 8, 2, 128, seed=5, layers=3)
    sh = pool_shape(h.w, h.num_pages)
    ds = make_device_step(h)
    ref_pool = h.pool.copy().reshape(-1)
    for layer in (2, 0, 1):
        ds.pool.kv_append(layer, ds.bt, ds.sl, ds.k_new[layer], ds.v_new[layer])
        ds.pool.decode_attention(layer, ds.bt, ds.sl, ds.q[layer], ds.out[layer])
        assert oracle.kv_append(ref_pool, sh, layer, h.block_tables, h.seq_lens, h.k_new[layer], h.v_new[layer]) == 0
    assert ds.pool.check_status() == 0
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    for layer in range(3):
        ref = oracle.decode_attention(ref_pool, sh, layer, h.block_tables, h.seq_lens, h.q[layer])
        assert_close(dev_to_bits(ds.out[layer]), ref, "layer %d" % layer)


def test_unused_slots_and_pages_full_of_nan_do_not_leak():
    """Slots past a context's end and pages no request owns may hold anything, NaN included."""
    h = custom_inputs([5, 17, 70, 130, 1, 64], 8, 2, 128, seed=9, extra_pages=4)
    P = 16
    live = np.zeros((h.num_pages, P), dtype=bool)
    for r, L in enumerate(h.seq_lens.tolist()):
        for j in range(L):
            live[h.block_tables[r, j // P], j % P] = True
    pool = h.pool.reshape(1, h.num_pages, 2, 2, P, 128)
    dead_pages, dead_slots = np.nonzero(~live)
    pool[0, dead_pages, :, :, dead_slots, :] = 0x7FC0                         # bf16 quiet NaN
    assert np.isnan(widen(pool)).sum() > 1000
    _, ref_out = oracle_step(h)
    assert np.all(np.isfinite(ref_out))
    ds = run_step(h)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "nan-poisoned")


def test_large_norm_keys_do_not_overflow():
    h = custom_inputs([200, 333, 64], 4, 1, 128, seed=21)
    pool = h.pool.reshape(1, h.num_pages, 1, 2, 16, 128)
    k = widen(pool[0, :, :, 0])
    pool[0, :, :, 0] = wl.f32_to_bf16_bits((k * 24.0).astype(np.float32))   # scores ~ N(0, 24^2): up to +-100
    _, ref_out = oracle_step(h)
    ds = run_step(h)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "large-norm keys")
    ds2 = run_step(h, partition=5)
    assert_close(dev_to_bits(ds2.out[0]), ref_out, "large-norm keys, split")


def test_requests_may_share_pages_for_reading():
    h = custom_inputs([100, 100], 8, 2, 128, seed=31)
    h.block_tables[1, :6] = h.block_tables[0, :6]                # common 96-token prefix
    ref_pool, ref_out = oracle_step(h)
    ds = run_step(h)
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "shared prefix")


def test_block_table_wider_than_needed_and_padding_never_read():
    h = custom_inputs([33, 500], 8, 2, 128, seed=41, max_pages=77)
    assert h.block_tables.shape[1] == 77 and (h.block_tables[0, 3:] == -1).all()
    _, ref_out = oracle_step(h)
    ds = run_step(h)
    assert_close(dev_to_bits(ds.out[0]), ref_out, "wide table")


# --------------------------------------------------------------------------- invalid data

def test_invalid_length_sets_status_zero_fills_row_and_writes_nothing():
    b = binding()
    h = custom_inputs([50, 60, 70], 8, 2, 128, seed=51)
    h.seq_lens[1] = 0
    ds = make_device_step(h)
    before = dev_to_bits(ds.pool.pool).copy()
    ds.pool.kv_append(0, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0])
    ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
    with pytest.raises(b.CkvError) as e:
        ds.pool.check_status()
    assert e.value.code == b.CKV_EBOUNDS
    out = dev_to_bits(ds.out[0])
    assert not out[1].any()                                      # zero-filled row
    after = dev_to_bits(ds.pool.pool).reshape(1, h.num_pages, 2, 2, 16, 128)
    changed = (after != before.reshape(after.shape)).any(axis=-1)
    assert int(changed.sum()) == 2 * 2 * 2                       # only requests 0 and 2 appended
    # the valid requests are still right
    good = custom_inputs([50, 60, 70], 8, 2, 128, seed=51)
    good_rows = [0, 2]
    sub = wl.HostInputs(good.w, good.num_pages, good.seq_lens[good_rows], good.block_tables[good_rows],
                        good.pool, good.q[:, good_rows], good.k_new[:, good_rows], good.v_new[:, good_rows])
    _, ref = oracle_step(sub)
    assert_close(out[good_rows], ref, "valid rows beside an invalid one")
    assert ds.pool.check_status() == 0                           # the word was cleared


def test_too_long_length_and_bad_page_id_are_reported_without_faulting():
    b = binding()
    h = custom_inputs([50, 60], 8, 2, 128, seed=52)
    h.seq_lens[0] = h.block_tables.shape[1] * 16 + 1
    ds = make_device_step(h)
    ds.pool.kv_append(0, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0])
    ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
    assert ds.pool.check_status(raise_on_error=False) & b.STATUS_BAD_LENGTH

    h = custom_inputs([50, 60], 8, 2, 128, seed=53)
    h.block_tables[1, 1] = h.num_pages + 100
    h.block_tables[0, 3] = -7                                    # the append target of request 0
    ds = make_device_step(h)
    before = dev_to_bits(ds.pool.pool).copy()
    ds.pool.kv_append(0, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0])
    ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
    assert ds.pool.check_status(raise_on_error=False) & b.STATUS_BAD_PAGE
    after = dev_to_bits(ds.pool.pool).reshape(1, h.num_pages, 2, 2, 16, 128)
    changed = (after != before.reshape(after.shape)).any(axis=-1)
    assert int(changed.sum()) == 1 * 2 * 2                       # request 1 only


# --------------------------------------------------------------------------- the plan

def check_plan(kp, lens_np, Hkv):
    sl = torch.from_numpy(lens_np).cuda()
    hdr, starts = kp.decode_plan(sl)
    C = kp.get_partition()
    total, q, want = expected_plan(lens_np, Hkv, C)
    assert hdr["total_units"] == total and hdr["num_spans"] == C
    assert hdr["units_per_span"] == q
    assert hdr["spans_with_units"] == -(-total // q)
    assert np.array_equal(starts, want)
    return hdr


def test_plan_partitions_tiles_evenly_and_deterministically():
    b = binding()
    for name in ("tiny", "llama8b_b64", "skewed_long"):
        w = wl.workload(name)
        lens = wl.seq_lens(w)
        cfg = b.make_config(1, w.num_q_heads, w.num_kv_heads, w.head_dim, 64, int(wl.pages_of(lens).max()), lens.size)
        kp = b.KvPool(cfg)
        for C in (kp.get_partition(), 1, 7, 296, 2048):
            kp.set_partition(C)
            hdr = check_plan(kp, lens, w.num_kv_heads)
            hdr2, _ = kp.decode_plan(torch.from_numpy(lens).cuda())
            assert hdr == hdr2
        kp.close()


def test_attention_kernel_derives_the_same_partition_as_the_plan():
    h = custom_inputs([700, 90, 2000, 64, 1500, 333, 800, 16, 5000], 8, 2, 128, seed=71)
    ds = make_device_step(h)
    for C in (ds.pool.get_partition(), 5, 77):
        ds.pool.set_partition(C)
        ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
        trace, starts = ds.pool.read_span_trace()
        _, _, want = expected_plan(h.seq_lens, 2, C)
        assert np.array_equal(starts, want)
        busy = want[:, 0] >= 0
        assert np.all(trace[busy, 3] >= trace[busy, 0]) and np.all(trace[busy, 1] > 0)
    assert ds.pool.check_status() == 0


def test_read_probe_streams_the_batch_and_reports_bad_pages():
    b = binding()
    h = custom_inputs([700, 90, 2000, 64, 1500, 333, 800, 16, 5000], 8, 2, 128, seed=73)
    ds = make_device_step(h)
    before = dev_to_bits(ds.pool.pool).copy()
    for C in (ds.pool.get_partition(), 5, 2048):
        ds.pool.set_partition(C)
        n0 = ds.pool.launch_count()
        ds.pool.read_probe(0, ds.bt, ds.sl)
        assert ds.pool.launch_count() - n0 == 1
        assert ds.pool.check_status() == 0
    assert np.array_equal(dev_to_bits(ds.pool.pool), before)              # a probe writes nothing
    bad = ds.bt.clone()
    bad[2, 3] = h.num_pages + 5
    ds.pool.read_probe(0, bad, ds.sl)
    assert ds.pool.check_status(raise_on_error=False) & b.STATUS_BAD_PAGE


# --------------------------------------------------------------------------- merge stages

@pytest.mark.parametrize("Hq,Hkv", [(4, 1), (8, 1), (8, 2)])
def test_every_merge_stage_matches_oracle(Hq, Hkv):
    """One long context cut into C spans exercises each way partials are merged: inside one CTA
    through shared memory (C <= 4 spans), two CTAs with the later one fetching the other's partial
    (5..8), a flat merge of up to 24 CTA partials (in several rounds where they do not fit the ring
    at once: 8 columns, C = 96), and the two-level merge beyond that -- with a short request
    behind it so that the last span also holds a whole (request, kv head)."""
    h = custom_inputs([9000, 70], Hq, Hkv, 128, seed=500 + Hq + Hkv)
    ref_pool, ref_out = oracle_step(h)
    for fused in (False, True):
        for C in (1, 2, 3, 4, 5, 6, 8, 9, 12, 40, 96, 97, 130, 400):
            ds = run_step(h, partition=C, fused=fused)
            assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
            assert_close(dev_to_bits(ds.out[0]), ref_out, "merge stages C=%d fused=%s" % (C, fused))
            ds.pool.close()


def test_results_are_bit_identical_from_run_to_run():
    """Which warp or CTA arrives last at a merge differs from launch to launch; the bits of the
    output must not (partials are folded in the order of their index, whoever does the folding)."""
    rng = np.random.default_rng(5)
    lens = rng.integers(300, 3000, size=48).tolist() + [20000]
    h = custom_inputs(lens, 8, 2, 128, seed=77)
    ds = make_device_step(h)
    ds.pool.kv_append(0, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0])
    first = None
    for C in (None, 40):
        if C is not None:
            ds.pool.set_partition(C)
            first = None
        for _ in range(25):
            ds.out.fill_(float("nan"))
            ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
            got = dev_to_bits(ds.out[0]).copy()
            if first is None:
                first = got
            assert np.array_equal(got, first)
    assert ds.pool.check_status() == 0


# --------------------------------------------------------------------------- configs 2, 5

def device_workload(name, batch=None, num_layers=None):
    """Draw a workload directly on the GPU; returns everything needed for GPU run and checks."""
    b = binding()
    w = wl.workload(name) if num_layers is None else wl.workload(name, num_layers=num_layers)
    lens = wl.seq_lens(w, batch)
    npg = wl.num_pool_pages(w, lens)
    bt = wl.block_tables(lens, npg, w.seed, 16)
    B = lens.size
    cfg = b.make_config(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, npg, bt.shape[1], B)
    pool_t = wl.device_normal_bf16((w.num_layers, npg, w.num_kv_heads, 2, 16, w.head_dim), w.seed, 1, "cuda:0")
    kp = b.KvPool(cfg, pool=pool_t.view(-1))
    q = wl.device_normal_bf16((w.num_layers, B, w.num_q_heads, w.head_dim), w.seed, 2, "cuda:0")
    k = wl.device_normal_bf16((w.num_layers, B, w.num_kv_heads, w.head_dim), w.seed, 3, "cuda:0")
    v = wl.device_normal_bf16((w.num_layers, B, w.num_kv_heads, w.head_dim), w.seed, 4, "cuda:0")
    out = torch.full_like(q, float("nan"))
    return w, lens, npg, bt, kp, pool_t, q, k, v, out


def full_parity(name, partitions=(None,)):
    w, lens, npg, bt, kp, pool_t, q, k, v, out = device_workload(name)
    sh = pool_shape(w, npg)
    host_pool = dev_to_bits(pool_t).reshape(-1)                  # state before the append
    hq, hk, hv = dev_to_bits(q), dev_to_bits(k), dev_to_bits(v)
    assert oracle.kv_append(host_pool, sh, 0, bt, lens, hk[0], hv[0]) == 0
    ref = oracle.decode_attention(host_pool, sh, 0, bt, lens, hq[0])
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    kp.kv_append(0, btd, sld, k[0], v[0])
    assert np.array_equal(dev_to_bits(pool_t).reshape(-1), host_pool)
    worst = []
    for part in partitions:
        if part is not None:
            kp.set_partition(part)
        out.fill_(float("nan"))
        kp.decode_attention(0, btd, sld, q[0], out[0])
        assert kp.check_status() == 0
        worst.append(assert_close(dev_to_bits(out[0]), ref, "%s partition=%s" % (name, part)))
    kp.close()
    return worst


def full_parity_fused(name, partitions=(None,)):
    w, lens, npg, bt, kp, pool_t, q, k, v, out = device_workload(name)
    sh = pool_shape(w, npg)
    host_pool = dev_to_bits(pool_t).reshape(-1)                  # state before the step
    pristine = pool_t.clone()
    hq, hk, hv = dev_to_bits(q), dev_to_bits(k), dev_to_bits(v)
    assert oracle.kv_append(host_pool, sh, 0, bt, lens, hk[0], hv[0]) == 0
    ref = oracle.decode_attention(host_pool, sh, 0, bt, lens, hq[0])
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    for part in partitions:
        if part is not None:
            kp.set_partition(part)
        pool_t.copy_(pristine)                                   # every run appends into a pre-step pool
        out.fill_(float("nan"))
        kp.decode_step(0, btd, sld, q[0], k[0], v[0], out[0])
        assert kp.check_status() == 0
        assert np.array_equal(dev_to_bits(pool_t).reshape(-1), host_pool)
        assert_close(dev_to_bits(out[0]), ref, "%s fused partition=%s" % (name, part))
    kp.close()


def test_llama8b_batch64_fused_step_full_parity():
    full_parity_fused("llama8b_b64", partitions=(None, 100))


def test_skewed_long_context_fused_step_full_parity():
    full_parity_fused("skewed_long", partitions=(None, 2048))


def test_llama8b_batch64_full_parity():
    full_parity("llama8b_b64", partitions=(None, 296, 100, 2048))


def test_skewed_long_context_full_parity():
    full_parity("skewed_long", partitions=(None, 37, 2048))


# --------------------------------------------------------------------------- host-buffer entry and sweep

@pytest.mark.parametrize("pinned,route,launches", [(True, "auto", 2), (True, "staged", 2), (True, "direct", 1),
                                                   (True, "copy", 1), (False, "auto", 1), (False, "direct", 1)])
def test_decode_step_host_matches_oracle(pinned, route, launches):
    """Pinned buffers take a zero-copy route (staged through a gather kernel, or read directly by
    the attention kernel; output rows written straight to the host buffer), pageable ones the copy
    route whatever was asked for; every route must give the oracle's step."""
    from paper_2501_08090_b200 import binding as b
    h = custom_inputs([700, 90, 2000, 64, 1500, 333, 800, 16, 4000], 8, 2, 128, seed=67)
    ref_pool, ref_out = oracle_step(h)
    ds = make_device_step(h)
    ds.pool.set_host_route({"auto": b.HOST_ROUTE_AUTO, "staged": b.HOST_ROUTE_STAGED, "direct": b.HOST_ROUTE_DIRECT,
                            "copy": b.HOST_ROUTE_COPY}[route])
    host = lambda a: torch.from_numpy(np.ascontiguousarray(a).copy())
    pin = (lambda a: host(a).pin_memory()) if pinned else host
    q = pin(h.q[0].view(np.int16)).view(torch.bfloat16)
    k = pin(h.k_new[0].view(np.int16)).view(torch.bfloat16)
    v = pin(h.v_new[0].view(np.int16)).view(torch.bfloat16)
    out = torch.zeros_like(q)
    out = out.pin_memory() if pinned else out
    bt, sl = pin(h.block_tables), pin(h.seq_lens)
    n0 = ds.pool.launch_count()
    ds.pool.decode_step_host(0, bt, sl, q, k, v, out)
    assert ds.pool.launch_count() - n0 == launches
    assert ds.pool.check_status() == 0
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    assert_close(dev_to_bits(out), ref_out, "decode_step_host pinned=%s route=%s" % (pinned, route))
    # the pre-marshalled form issues the same step (same lengths: the append rewrites the same rows)
    out.zero_()
    ds.pool.host_step_call(0, bt, sl, q, k, v, out)()
    assert ds.pool.check_status() == 0
    assert_close(dev_to_bits(out), ref_out, "host_step_call pinned=%s route=%s" % (pinned, route))
    ds.pool.close()


def test_step_latency_sweep_runs_nested_prefixes_and_counts_launches():
    h = custom_inputs([700, 90, 2000, 64, 1500, 333, 800, 16], 8, 2, 128, seed=61, layers=2)
    ds = make_device_step(h)
    n0 = ds.pool.launch_count()
    med, mn = ds.pool.step_latency_sweep([1, 2, 4, 8], ds.bt, ds.sl, ds.q, ds.k_new, ds.v_new, ds.out,
                                         warmup=2, iters=5)
    assert med.shape == (4,) and np.all(med > 0) and np.all(mn > 0) and np.all(mn <= med)
    assert ds.pool.launch_count() - n0 == 4 * (2 + 5) * 2 * 1    # sizes * steps * layers * one fused kernel
    # the last sweep point ran the full batch on both layers: outputs must be the oracle's
    sh = pool_shape(h.w, h.num_pages)
    ref_pool = h.pool.copy().reshape(-1)
    for layer in range(2):
        assert oracle.kv_append(ref_pool, sh, layer, h.block_tables, h.seq_lens, h.k_new[layer], h.v_new[layer]) == 0
    assert np.array_equal(dev_to_bits(ds.pool.pool), ref_pool)
    for layer in range(2):
        ref = oracle.decode_attention(ref_pool, sh, layer, h.block_tables, h.seq_lens, h.q[layer])
        assert_close(dev_to_bits(ds.out[layer]), ref, "sweep layer %d" % layer)


def test_profile_events_bracket_the_attention_kernel():
    h = wl.host_inputs(wl.workload("tiny"))
    ds = make_device_step(h)
    ds.pool.profile_enable(True)
    for _ in range(5):
        ds.pool.decode_attention(0, ds.bt, ds.sl, ds.q[0], ds.out[0])
    ms, n = ds.pool.profile_read()
    assert n == 5 and 0 < ms < 50
    ds.pool.profile_enable(False)


def test_arguments_are_validated_on_the_host():
    b = binding()
    h = wl.host_inputs(wl.workload("tiny"))
    ds = make_device_step(h)
    with pytest.raises(b.CkvError) as e:
        ds.pool.kv_append(1, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0])         # layer out of range
    assert e.value.code == b.CKV_EINVAL
    with pytest.raises(b.CkvError):
        ds.pool.set_partition(0)
    with pytest.raises(b.CkvError):
        ds.pool.set_partition(3000)
    big = torch.ones(9, dtype=torch.int32, device="cuda")
    big_bt = torch.zeros((9, ds.bt.shape[1]), dtype=torch.int32, device="cuda")
    big_q = torch.zeros((9,) + tuple(ds.q[0].shape[1:]), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.CkvError) as e:
        ds.pool.decode_attention(0, big_bt, big, big_q, torch.zeros_like(big_q))   # batch > max_batch
    assert e.value.code == b.CKV_EINVAL
    # tensors too small for the batch, or a table with another row width, never reach the device
    with pytest.raises(ValueError):
        ds.pool.decode_attention(0, ds.bt, big, ds.q[0], ds.out[0])
    with pytest.raises(ValueError):
        ds.pool.decode_attention(0, ds.bt[:, :-1].contiguous(), ds.sl, ds.q[0], ds.out[0])
    with pytest.raises(ValueError):
        ds.pool.decode_step(0, ds.bt, ds.sl, ds.q[0], ds.k_new[0][:-1], ds.v_new[0], ds.out[0])
    with pytest.raises(ValueError):
        ds.pool.decode_step(0, ds.bt, ds.sl, ds.q[0][:-1], ds.k_new[0], ds.v_new[0], ds.out[0])
    with pytest.raises(ValueError):
        ds.pool.kv_append(0, ds.bt, ds.sl, ds.k_new[0], ds.v_new[0][:-1])
    # and nothing above disturbed the pool: a regular step still matches
    ds.pool.decode_step(0, ds.bt, ds.sl, ds.q[0], ds.k_new[0], ds.v_new[0], ds.out[0])
    assert ds.pool.check_status() == 0
