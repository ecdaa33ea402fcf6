"""GPU parity of the multi-token step (q_len new tokens per request, causal among them) against the
oracle: pool bit-exact after the append, attention within the tolerance, across group sizes,
lengths that put the new tokens across tile and page boundaries, and partitions."""
import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

from helpers import assert_close, bits_to_dev, dev_to_bits

pytestmark = pytest.mark.gpu


def run_case(q_len, Hq, Hkv, d, lens, seed, partitions=(None,)):
    from paper_2501_08090_b200 import binding as b
    lens = np.asarray(lens, dtype=np.int32)
    B = lens.size
    npg = int(wl.pages_of(lens).sum()) + 3
    bt = wl.block_tables(lens, npg, seed)
    sh = PoolShape(1, npg, Hq, Hkv, 16, d)
    pool_h = wl.normal_bf16((sh.elems,), seed, 1)
    q_h = wl.normal_bf16((B, q_len, Hq, d), seed, 2)
    k_h = wl.normal_bf16((B, q_len, Hkv, d), seed, 3)
    v_h = wl.normal_bf16((B, q_len, Hkv, d), seed, 4)
    ref_pool = pool_h.copy()
    assert oracle.kv_append_multi(ref_pool, sh, 0, q_len, bt, lens, k_h, v_h) == 0
    ref = oracle.decode_attention_multi(ref_pool, sh, 0, q_len, bt, lens, q_h)

    cfg = b.make_config(1, Hq, Hkv, d, npg, bt.shape[1], B)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    q, k, v = bits_to_dev(q_h), bits_to_dev(k_h), bits_to_dev(v_h)
    for part in partitions:
        kp = b.KvPool(cfg, pool=bits_to_dev(pool_h))
        if part is not None:
            kp.set_partition(part)
        out = torch.full_like(q, float("nan"))
        kp.kv_append_multi(0, q_len, btd, sld, k, v)
        kp.decode_attention_multi(0, q_len, btd, sld, q, out)
        assert kp.check_status() == 0
        what = "q_len=%d Hq=%d Hkv=%d d=%d part=%s" % (q_len, Hq, Hkv, d, part)
        assert np.array_equal(dev_to_bits(kp.pool), ref_pool), what
        assert_close(dev_to_bits(out), ref, what)
        kp.close()


EDGE_LENS = [8, 9, 15, 16, 17, 31, 32, 33, 34, 35, 36, 47, 48, 49, 63, 64, 65, 66, 67, 96, 97, 129, 300, 1000, 2050]


@pytest.mark.parametrize("q_len,Hq,Hkv,d", [(2, 8, 2, 128), (2, 32, 8, 128), (4, 4, 2, 128), (4, 2, 1, 64),
                                            (8, 2, 2, 128), (8, 1, 1, 64), (3, 4, 2, 64), (1, 8, 1, 128),
                                            # more (new token, head) pairs than one launch holds: 2, 3, 4 and 8 passes
                                            (3, 32, 8, 128), (5, 8, 2, 128), (4, 8, 1, 128), (8, 16, 2, 64)])
def test_multi_token_step_matches_oracle(q_len, Hq, Hkv, d):
    lens = [L for L in EDGE_LENS if L >= q_len]
    run_case(q_len, Hq, Hkv, d, lens, seed=q_len * 100 + Hq, partitions=(None, 1, 11, 2048))


@pytest.mark.parametrize("n_tiles", [12, 13, 16, 17, 24, 25, 64, 65, 80, 257, 300])
@pytest.mark.parametrize("q_len", [1, 4])
def test_two_level_merge_of_many_partials(n_tiles, q_len):
    """One request cut into one partial per tile (2048 spans for a handful of units): group sizes 8, 16 and
    32, full and ragged last groups, a last group of one, and (q_len 4) groups in which the early new
    tokens see nothing at all."""
    for tail in (1, 32):
        run_case(q_len, 2, 1, 128, [(n_tiles - 1) * 32 + tail], seed=n_tiles + tail, partitions=(2048,))
    run_case(q_len, 4, 2, 64, [(n_tiles - 1) * 32 + 7, 40, n_tiles * 32], seed=n_tiles, partitions=(2048, 700))


def test_new_tokens_straddling_every_tile_boundary():
    for L in range(30, 40):                                    # the 4 new tokens walk across the 32-token boundary
        run_case(4, 4, 2, 128, [L, 4, L + 32], seed=L)


def test_multi_token_limits_are_checked_on_the_host():
    from paper_2501_08090_b200 import binding as b
    cfg = b.make_config(1, 32, 8, 128, 16, 4, 2)
    kp = b.KvPool(cfg)
    z = torch.zeros(2, 9, 32, 128, dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros(2, 4, dtype=torch.int32, device="cuda")
    sl = torch.full((2,), 10, dtype=torch.int32, device="cuda")
    for bad in (0, 9):
        with pytest.raises(b.CkvError) as e:
            kp.decode_attention_multi(0, bad, bt, sl, z, z.clone())
        assert e.value.code == b.CKV_EINVAL and "q_len" in str(e.value)
    n0 = kp.launch_count()
    kp.decode_attention_multi(0, 3, bt, sl, z[:, :3].contiguous(), z[:, :3].clone())   # 3 new tokens x group 4: two passes
    assert kp.launch_count() - n0 == 2
    kp.close()


def test_too_short_requests_are_flagged_and_zero_filled():
    from paper_2501_08090_b200 import binding as b
    cfg = b.make_config(1, 4, 2, 128, 16, 4, 3)
    kp = b.KvPool(cfg)
    kp.pool.normal_()
    q = torch.randn(3, 2, 4, 128, device="cuda").to(torch.bfloat16)
    out = torch.full_like(q, float("nan"))
    bt = torch.arange(12, dtype=torch.int32, device="cuda").view(3, 4)
    sl = torch.tensor([5, 1, 40], dtype=torch.int32, device="cuda")     # request 1 has fewer tokens than q_len
    kp.decode_attention_multi(0, 2, bt, sl, q, out)
    assert kp.check_status(raise_on_error=False) & b.STATUS_BAD_LENGTH
    o = out.float().cpu().numpy()
    assert not o[1].any() and np.isfinite(o[[0, 2]]).all()
    kp.close()
