"""decode_attention_noalloc: the entry point for callers that cannot allocate a workspace.

Some users of this library have nowhere to put split-KV partials: an engine that gave all free
device memory to the KV pool at start-up, a plugin under a framework that owns the allocator, a
latency-critical loop that cannot take cudaMalloc's device-wide synchronisation.  For them the
partials live in a fixed array inside the library.  This test drives that entry point through the
C ABI and checks it against the fp64 oracle and against decode_attention (which uses a
caller-provided workspace) on two calls in a row -- the second call finds the array as the first
one left it.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

from helpers import ATOL, RTOL, assert_close, bits_to_dev, dev_to_bits, widen

pytestmark = pytest.mark.gpu


def _inputs(lens, seed, Hq=32, Hkv=8, d=128):
    lens = np.asarray(lens, dtype=np.int32)
    npg = int(wl.pages_of(lens).sum()) + 5
    bt = wl.block_tables(lens, npg, seed)
    B = lens.size
    return dict(lens=lens, npg=npg, bt=bt, Hq=Hq, Hkv=Hkv, d=d,
                pool=wl.normal_bf16((npg, Hkv, 2, 16, d), seed, 1),
                q=wl.normal_bf16((B, Hq, d), seed, 2))


def _oracle(inp):
    sh = PoolShape(1, inp["npg"], inp["Hq"], inp["Hkv"], 16, inp["d"])
    return oracle.decode_attention(inp["pool"].reshape(-1), sh, 0, inp["bt"], inp["lens"], inp["q"])


def _run_both(b, inp, num_spans=0, sync=True):
    """(output of decode_attention, output of decode_attention_noalloc) as float64 arrays."""
    B = inp["lens"].size
    cfg = b.make_config(1, inp["Hq"], inp["Hkv"], inp["d"], inp["npg"], inp["bt"].shape[1], B)
    pool = bits_to_dev(inp["pool"].reshape(-1))
    bt = torch.from_numpy(inp["bt"]).cuda()
    sl = torch.from_numpy(inp["lens"]).cuda()
    q = bits_to_dev(inp["q"])
    ref = torch.full_like(q, float("nan"))
    got = torch.full_like(q, float("nan"))

    kp = b.KvPool(cfg, pool=pool)                      # existing entry point: workspace from the caller
    if num_spans:
        kp.set_partition(num_spans)
    kp.decode_attention(0, bt, sl, q, ref)
    assert kp.check_status() == 0
    kp.close()

    bits = b.decode_attention_noalloc(cfg, pool, 0, bt, sl, q, got, num_spans=num_spans, sync=sync)
    assert bits == 0
    if not sync:
        torch.cuda.synchronize()                   # the call only enqueued work
    assert_close(dev_to_bits(got), _oracle(inp), "decode_attention_noalloc against the oracle")
    return widen(dev_to_bits(ref)), widen(dev_to_bits(got))


def test_noalloc_matches_decode_attention_on_two_calls_in_a_row():
    from paper_2501_08090_b200 import binding as b
    torch.cuda.set_device(0)
    # call 1: long contexts, so most (request, kv head) pairs are split and merged from partials
    first = _inputs([5000, 700, 3000, 64, 1], seed=901)
    # call 2: another batch, other lengths; the array still holds call 1's partials and counters
    second = _inputs([17, 2048, 129, 9000, 333, 4096, 15], seed=902)
    for inp in (first, second):
        ref, got = _run_both(b, inp)
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref))
    # and once more with a narrow partition and the small head size
    third = _inputs([300, 77, 1000], seed=903, Hq=4, Hkv=1, d=64)
    ref, got = _run_both(b, third, num_spans=7)
    assert np.all(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref))
    # enqueue-only form (no status pointer): the caller synchronises
    ref, got = _run_both(b, second, sync=False)
    assert np.all(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref))


def test_noalloc_rejects_partitions_beyond_its_built_in_scratch():
    from paper_2501_08090_b200 import binding as b
    torch.cuda.set_device(0)
    inp = _inputs([100, 200], seed=904)
    cfg = b.make_config(1, inp["Hq"], inp["Hkv"], inp["d"], inp["npg"], inp["bt"].shape[1], 2)
    pool = bits_to_dev(inp["pool"].reshape(-1))
    bt = torch.from_numpy(inp["bt"]).cuda()
    sl = torch.from_numpy(inp["lens"]).cuda()
    q = bits_to_dev(inp["q"])
    out = torch.zeros_like(q)
    with pytest.raises(b.CkvError) as e:
        b.decode_attention_noalloc(cfg, pool, 0, bt, sl, q, out, num_spans=641)
    assert e.value.code == b.CKV_EINVAL and "640" in str(e.value)
    torch.cuda.synchronize()
    assert not dev_to_bits(out).any()                  # nothing was launched
    assert b.decode_attention_noalloc(cfg, pool, 0, bt, sl, q, out, num_spans=640) == 0
    assert dev_to_bits(out).any()
