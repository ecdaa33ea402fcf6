"""The seeded input recipes: shapes, ranges, mix ratios, determinism, bf16 rounding."""
import numpy as np
import torch

from paper_2501_08090_b200 import workloads as wl


def test_tiny_lengths_and_pool():
    w = wl.workload("tiny")
    lens = wl.seq_lens(w)
    assert lens.tolist() == [17, 64, 129, 256]
    assert int(wl.pages_of(lens).sum()) == 31 and wl.num_pool_pages(w, lens) == 64
    assert w.kv_bytes_per_token == 256 and int(lens.sum()) * 256 == 119296


def test_uniform_workloads_ranges_and_determinism():
    for name, lo, hi in (("llama8b_b64", 512, 4096), ("llama70b_full", 1024, 4096)):
        w = wl.workload(name)
        a, b = wl.seq_lens(w), wl.seq_lens(w)
        assert np.array_equal(a, b) and a.dtype == np.int32 and a.size == w.batch
        assert a.min() >= lo and a.max() <= hi
        assert w.kv_bytes_per_token == 4096


def test_mixed_sweep_prefixes_hold_thirty_percent_batch_requests():
    w = wl.workload("mixed_sweep")
    full = wl.seq_lens(w)
    flags = np.array([wl.is_batch_request(i) for i in range(512)])
    expect = {1: 0, 2: 1, 4: 1, 8: 2, 16: 5, 32: 10, 64: 19, 128: 38, 256: 77, 512: 154}
    for b in wl.SWEEP_BATCH_SIZES:
        assert int(flags[:b].sum()) == expect[b]
        assert np.array_equal(wl.seq_lens(w, b), full[:b])          # nested prefixes
    assert np.all(full[flags] >= 8192) and np.all(full[flags] <= 32768)
    assert np.all(full[~flags] >= 1) and np.all(full[~flags] <= 8192)
    med = np.median(full[~flags])
    assert 800 < med < 1300                                        # lognormal median 1024


def test_skewed_lengths():
    assert wl.seq_lens(wl.workload("skewed_long")).tolist() == [131072] + [1024] * 7


def test_block_tables_are_a_scattered_partition_of_distinct_pages():
    w = wl.workload("llama8b_b64")
    lens = wl.seq_lens(w)
    npg = wl.num_pool_pages(w, lens)
    assert npg == 2 * int(wl.pages_of(lens).sum())
    bt = wl.block_tables(lens, npg, w.seed)
    n = wl.pages_of(lens)
    live = np.concatenate([bt[r, :n[r]] for r in range(lens.size)])
    assert live.min() >= 0 and live.max() < npg and np.unique(live).size == live.size
    for r in range(lens.size):
        assert np.all(bt[r, n[r]:] == -1)
    assert np.array_equal(bt, wl.block_tables(lens, npg, w.seed))
    assert not np.array_equal(bt, wl.block_tables(lens, npg, w.seed + 1))
    assert np.abs(np.diff(live[:200].astype(np.int64))).mean() > 100     # not contiguous runs


def test_bf16_rounding_is_nearest_even_and_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40], np.float32)])
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    # exact ties: 1 + 2^-8 rounds down to even (1.0), 1 + 3*2^-8 rounds up to 1 + 2^-6
    assert wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(np.array([1.00390625], np.float32)))[0] == 1.0
    assert wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(np.array([1.01171875], np.float32)))[0] == 1.015625
    assert np.array_equal(wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(bits)), bits)


def test_normal_values_have_unit_variance_and_independent_streams():
    a = wl.bf16_bits_to_f32(wl.normal_bf16((200000,), 1, 1))
    b = wl.bf16_bits_to_f32(wl.normal_bf16((200000,), 1, 2))
    assert abs(a.mean()) < 0.01 and abs(a.std() - 1) < 0.01
    assert abs(np.corrcoef(a, b)[0, 1]) < 0.01
    assert np.array_equal(wl.normal_bf16((1000,), 1, 1), wl.normal_bf16((1000,), 1, 1))


def test_algorithmic_bytes_formula():
    w = wl.workload("tiny")
    lens = wl.seq_lens(w)
    acc = wl.algorithmic_bytes(w, lens)
    assert acc["kv"] == 119296
    assert acc["q_out"] == 4 * 4 * 64 * 2 * 2
    assert acc["append"] == 4 * 2 * 1 * 64 * 2 * 2
    assert acc["tables"] == 31 * 4 + 4 * 4
    assert acc["total"] == sum(acc[k] for k in ("kv", "q_out", "append", "tables"))
