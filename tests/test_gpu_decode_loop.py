"""A real decode loop on the GPU: contexts grow by one token per step, steps are enqueued back to
back with no synchronisation between them (so consecutive kernels overlap their prologues), and
every step's output plus the final pool are compared with the oracle run step by step.

Also a randomized sweep over shapes, lengths and partitions.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

from helpers import assert_close, bits_to_dev, dev_to_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("Hq,Hkv,d,fused", [(8, 2, 128, True), (8, 2, 128, False), (4, 1, 64, True)])
def test_decode_loop_with_growing_contexts(Hq, Hkv, d, fused):
    from paper_2501_08090_b200 import binding as b
    steps, B = 40, 6
    start = np.array([1, 15, 30, 63, 100, 250], dtype=np.int32)          # lengths before the first step
    final = start + steps
    npg = int(wl.pages_of(final).sum()) + 3
    bt = wl.block_tables(final, npg, seed=11)                              # tables sized for the final lengths
    sh = PoolShape(1, npg, Hq, Hkv, 16, d)
    pool_h = wl.normal_bf16((sh.elems,), 77, 1)
    q_h = wl.normal_bf16((steps, B, Hq, d), 77, 2)
    k_h = wl.normal_bf16((steps, B, Hkv, d), 77, 3)
    v_h = wl.normal_bf16((steps, B, Hkv, d), 77, 4)

    cfg = b.make_config(1, Hq, Hkv, d, npg, bt.shape[1], B)
    kp = b.KvPool(cfg, pool=bits_to_dev(pool_h))
    btd = torch.from_numpy(bt).cuda()
    lens_d = torch.from_numpy(np.stack([start + s + 1 for s in range(steps)]).astype(np.int32)).cuda()
    q, k, v = bits_to_dev(q_h), bits_to_dev(k_h), bits_to_dev(v_h)
    out = torch.full_like(q, float("nan"))
    for s in range(steps):                                                 # enqueue everything, no sync
        if fused:
            kp.decode_step(0, btd, lens_d[s], q[s], k[s], v[s], out[s])
        else:
            kp.kv_append(0, btd, lens_d[s], k[s], v[s])
            kp.decode_attention(0, btd, lens_d[s], q[s], out[s])
    assert kp.check_status() == 0
    got = dev_to_bits(out)

    ref_pool = pool_h.copy()
    for s in range(steps):
        lens = (start + s + 1).astype(np.int32)
        assert oracle.kv_append(ref_pool, sh, 0, bt, lens, k_h[s], v_h[s]) == 0
        ref = oracle.decode_attention(ref_pool, sh, 0, bt, lens, q_h[s])
        assert_close(got[s], ref, "step %d" % s)
    assert np.array_equal(dev_to_bits(kp.pool), ref_pool)
    kp.close()


def test_randomized_shapes_lengths_and_partitions():
    from paper_2501_08090_b200 import binding as b
    rng = np.random.default_rng(2024)
    for trial in range(24):
        d = (64, 128)[trial % 2]
        Hkv = int(rng.integers(1, 9))
        G = int(rng.integers(1, 9))
        Hq = Hkv * G
        B = int(rng.integers(1, 12))
        kind = trial % 3
        hi = (40, 700, 5000)[kind]
        lens = rng.integers(1, hi + 1, size=B).astype(np.int32)
        npg = int(wl.pages_of(lens).sum()) + int(rng.integers(0, 6))
        bt = wl.block_tables(lens, npg, seed=trial, max_pages_per_req=int(wl.pages_of(lens).max()) + int(rng.integers(0, 40)))
        sh = PoolShape(1, npg, Hq, Hkv, 16, d)
        pool_h = wl.normal_bf16((sh.elems,), trial, 1)
        q_h = wl.normal_bf16((B, Hq, d), trial, 2)
        k_h = wl.normal_bf16((B, Hkv, d), trial, 3)
        v_h = wl.normal_bf16((B, Hkv, d), trial, 4)
        ref_pool = pool_h.copy()
        assert oracle.kv_append(ref_pool, sh, 0, bt, lens, k_h, v_h) == 0
        ref = oracle.decode_attention(ref_pool, sh, 0, bt, lens, q_h)

        cfg = b.make_config(1, Hq, Hkv, d, npg, bt.shape[1], B)
        btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
        q, k, v = bits_to_dev(q_h), bits_to_dev(k_h), bits_to_dev(v_h)
        for part in (None, int(rng.integers(1, 2049))):
            kp = b.KvPool(cfg, pool=bits_to_dev(pool_h))
            if part is not None:
                kp.set_partition(part)
            out = torch.full_like(q, float("nan"))
            kp.decode_step(0, btd, sld, q, k, v, out)
            assert kp.check_status() == 0
            what = "trial %d Hq=%d Hkv=%d d=%d B=%d part=%s" % (trial, Hq, Hkv, d, B, part)
            assert np.array_equal(dev_to_bits(kp.pool), ref_pool), what
            assert_close(dev_to_bits(out), ref, what)
            kp.close()


def test_fused_loop_at_full_size_with_poisoned_future_slots():
    """The decode loop at the 8B shape, batch 64: 72 fused steps enqueued behind one another with
    no synchronisation, every context growing by one token per step.  Every slot that no step has
    written yet -- and every unused page -- holds bf16 NaN, so a tile copy that read a row before
    the preceding step's store of it landed shows up as a NaN output row instead of hiding inside
    the tolerance.  All outputs must be finite; every step is compared with the oracle, and so is
    the final pool, byte for byte."""
    from paper_2501_08090_b200 import binding as b
    w = wl.workload("llama8b_b64")
    steps, B, Hq, Hkv, d = 72, w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    start = wl.seq_lens(w) - 1                                             # lengths before the first step
    # a few contexts that cross a tile boundary (multiple of 32) early in the loop
    start[:4] = [1023, 2047 - 3, 511 + 17, 4000]
    final = start + steps
    npg = int(wl.pages_of(final).sum()) + 64
    bt = wl.block_tables(final, npg, seed=5)
    sh = PoolShape(1, npg, Hq, Hkv, 16, d)
    pool_h = np.full(sh.elems, 0x7FC0, dtype=np.uint16)                    # NaN everywhere ...
    view = pool_h.reshape(npg, Hkv, 2, 16, d)
    for r in range(B):                                                     # ... except the tokens that exist
        pos = np.arange(int(start[r]))
        view[bt[r, pos // 16], :, :, pos % 16, :] = wl.normal_bf16((pos.size, Hkv, 2, d), 91, 100 + r)
    q_h = wl.normal_bf16((steps, B, Hq, d), 91, 2)
    k_h = wl.normal_bf16((steps, B, Hkv, d), 91, 3)
    v_h = wl.normal_bf16((steps, B, Hkv, d), 91, 4)

    cfg = b.make_config(1, Hq, Hkv, d, npg, bt.shape[1], B)
    kp = b.KvPool(cfg, pool=bits_to_dev(pool_h))
    btd = torch.from_numpy(bt).cuda()
    lens_d = torch.from_numpy(np.stack([start + s + 1 for s in range(steps)]).astype(np.int32)).cuda()
    q, k, v = bits_to_dev(q_h), bits_to_dev(k_h), bits_to_dev(v_h)
    out = torch.full_like(q, float("nan"))
    hold = torch.empty(1 << 28, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for _ in range(4):
        hold.fill_(1)                                                      # the launches below queue up behind this
    for s in range(steps):
        kp.decode_step(0, btd, lens_d[s], q[s], k[s], v[s], out[s])
    assert kp.check_status() == 0
    got = dev_to_bits(out)
    assert np.all(np.isfinite(wl.bf16_bits_to_f32(got))), "a step read a slot before its store landed"

    ref_pool = pool_h.copy()
    for s in range(steps):
        lens = (start + s + 1).astype(np.int32)
        assert oracle.kv_append(ref_pool, sh, 0, bt, lens, k_h[s], v_h[s]) == 0
        ref = oracle.decode_attention(ref_pool, sh, 0, bt, lens, q_h[s])
        assert_close(got[s], ref, "step %d" % s)
    assert np.array_equal(dev_to_bits(kp.pool), ref_pool)

    # the same loop in plain stream order (no launch overlaps its predecessor): same bits
    kp.pool.copy_(bits_to_dev(pool_h))
    kp.set_overlap(False)
    out2 = torch.full_like(q, float("nan"))
    for s in range(steps):
        kp.decode_step(0, btd, lens_d[s], q[s], k[s], v[s], out2[s])
    assert kp.check_status() == 0
    assert np.array_equal(dev_to_bits(out2), got)
    assert np.array_equal(dev_to_bits(kp.pool), ref_pool)
    kp.close()
