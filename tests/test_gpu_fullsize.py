"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The pools here are tens of GB, drawn on the device; the oracle cannot hold them, so it is run on
sampled requests: their pages are copied to the host BEFORE the append as a small compact pool with
remapped block tables, the oracle appends and attends on that copy, and the GPU's output rows and
(after the append) the same pages are compared with it -- attention within tolerance, pages
bit-exact.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from oracle.oracle import PoolShape
from paper_2501_08090_b200 import workloads as wl

from helpers import assert_close, compact_requests, dev_to_bits, widen

pytestmark = pytest.mark.gpu


def _device_workload(name, num_layers=None):
    from paper_2501_08090_b200 import binding as b
    w = wl.workload(name) if num_layers is None else wl.workload(name, num_layers=num_layers)
    lens = wl.seq_lens(w)
    npg = wl.num_pool_pages(w, lens)
    bt = wl.block_tables(lens, npg, w.seed, 16)
    B = lens.size
    cfg = b.make_config(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, npg, bt.shape[1], B)
    pool = wl.device_normal_bf16((w.num_layers, npg, w.num_kv_heads, 2, 16, w.head_dim), w.seed, 1, "cuda:0")
    kp = b.KvPool(cfg, pool=pool.view(-1))
    q = wl.device_normal_bf16((w.num_layers, B, w.num_q_heads, w.head_dim), w.seed, 2, "cuda:0")
    k = wl.device_normal_bf16((w.num_layers, B, w.num_kv_heads, w.head_dim), w.seed, 3, "cuda:0")
    v = wl.device_normal_bf16((w.num_layers, B, w.num_kv_heads, w.head_dim), w.seed, 4, "cuda:0")
    out = torch.full_like(q, float("nan"))
    return w, lens, npg, bt, kp, pool, q, k, v, out


def _oracle_on_sample(w, pool_dev, bt, lens, rows, layer, q, k, v):
    """Oracle append + attention for the sampled requests of one layer, from a pre-append copy."""
    sub_pool, sub_bt, sub_lens, n = compact_requests(pool_dev, bt, lens, rows, layer)
    sh = PoolShape(1, n, w.num_q_heads, w.num_kv_heads, 16, w.head_dim)
    hq = dev_to_bits(q[layer][rows]); hk = dev_to_bits(k[layer][rows]); hv = dev_to_bits(v[layer][rows])
    assert oracle.kv_append(sub_pool, sh, 0, sub_bt, sub_lens, hk, hv) == 0
    ref = oracle.decode_attention(sub_pool, sh, 0, sub_bt, sub_lens, hq)
    return sub_pool, ref


def _pick(lens, n, seed, always=()):
    rng = np.random.default_rng(seed)
    rows = set(int(x) for x in always)
    rows.update([int(np.argmax(lens)), int(np.argmin(lens))])
    while len(rows) < min(n, lens.size):
        rows.add(int(rng.integers(0, lens.size)))
    return sorted(rows)


def test_mixed_sweep_full_batch_and_nested_prefixes():
    w, lens, npg, bt, kp, pool, q, k, v, out = _device_workload("mixed_sweep")
    rows = _pick(lens, 14, seed=3, always=(0, 1, 2, 3))
    sub_pool_ref, ref = _oracle_on_sample(w, pool, bt, lens, rows, 0, q, k, v)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()

    kp.kv_append(0, btd, sld, k[0], v[0])
    sub_after, _, _, _ = compact_requests(pool, bt, lens, rows, 0)
    assert np.array_equal(sub_after, sub_pool_ref)                         # sampled pages, bit-exact
    kp.decode_attention(0, btd, sld, q[0], out[0])
    assert kp.check_status() == 0
    got = dev_to_bits(out[0])
    assert_close(got[rows], ref, "mixed_sweep B=512")

    # nested prefixes: a request's output does not depend on who else is in the batch
    for B in (1, 2, 4, 8, 64, 256):
        out.fill_(float("nan"))
        kp.kv_append(0, btd[:B], sld[:B], k[0][:B], v[0][:B])
        kp.decode_attention(0, btd[:B], sld[:B], q[0][:B], out[0][:B])
        assert kp.check_status() == 0
        got = dev_to_bits(out[0])
        inside = [i for i, r in enumerate(rows) if r < B]
        assert inside
        assert_close(got[[rows[i] for i in inside]], ref[inside], "mixed_sweep B=%d" % B)
        assert np.isnan(widen(got[B:])).all()                              # rows outside the batch stay untouched
    kp.close()


def test_mixed_sweep_through_decode_step_the_call_the_sweep_times():
    """step_latency_sweep and bench.py time decode_step (append + attention in one kernel): the full
    batch of 512 and the nested prefixes through that call, sampled rows against the oracle, sampled
    pages bit-exact."""
    w, lens, npg, bt, kp, pool, q, k, v, out = _device_workload("mixed_sweep")
    rows = _pick(lens, 14, seed=4, always=(0, 1, 2, 3, 7, 15, 31))
    sub_pool_ref, ref = _oracle_on_sample(w, pool, bt, lens, rows, 0, q, k, v)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    for B in (512, 1, 2, 4, 8, 16, 32, 64, 128, 256):
        out.fill_(float("nan"))
        kp.decode_step(0, btd[:B], sld[:B], q[0][:B], k[0][:B], v[0][:B], out[0][:B])
        assert kp.check_status() == 0
        got = dev_to_bits(out[0])
        inside = [i for i, r in enumerate(rows) if r < B]
        assert inside
        assert_close(got[[rows[i] for i in inside]], ref[inside], "mixed_sweep decode_step B=%d" % B)
        assert torch.isfinite(out[0][:B].float()).all()
        assert np.isnan(widen(got[B:])).all()
        if B == 512:
            sub_after, _, _, _ = compact_requests(pool, bt, lens, rows, 0)
            assert np.array_equal(sub_after, sub_pool_ref)
    kp.close()


def test_llama70b_two_layers_append_touches_exactly_the_target_rows():
    """Reduced-layer variant where a second copy of the pool fits: global untouched-bytes check."""
    w, lens, npg, bt, kp, pool, q, k, v, out = _device_workload("llama70b_full", num_layers=2)
    before = pool.clone()
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    for layer in range(2):
        kp.kv_append(layer, btd, sld, k[layer], v[layer])
    assert kp.check_status() == 0
    changed = (pool.view(torch.int16) != before.view(torch.int16)).view(-1, w.head_dim).any(dim=1)
    assert int(changed.sum()) == 2 * lens.size * w.num_kv_heads * 2
    # the changed rows are exactly (layer, page of L-1, head, K|V, slot of L-1)
    idx = torch.nonzero(changed).flatten().cpu().numpy()
    want = []
    for layer in range(2):
        for r, L in enumerate(lens.tolist()):
            page, slot = int(bt[r, (L - 1) // 16]), (L - 1) % 16
            for h in range(w.num_kv_heads):
                for kv in range(2):
                    want.append((((layer * npg + page) * w.num_kv_heads + h) * 2 + kv) * 16 + slot)
    assert np.array_equal(np.sort(idx), np.sort(np.array(want)))
    kp.close()


def test_llama70b_all_80_layers_sampled_parity():
    w, lens, npg, bt, kp, pool, q, k, v, out = _device_workload("llama70b_full")
    assert w.num_layers == 80 and pool.numel() * 2 > 79e9
    layers = (0, 1, 13, 27, 39, 52, 66, 79)                                # every request of the batch on these ...
    rows = list(range(lens.size))
    refs = {layer: _oracle_on_sample(w, pool, bt, lens, rows, layer, q, k, v) for layer in layers}
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    for layer in range(w.num_layers):                                      # one whole decode iteration
        kp.decode_step(layer, btd, sld, q[layer], k[layer], v[layer], out[layer])
    assert kp.check_status() == 0
    assert torch.isfinite(out.float()).all()                               # ... and nothing non-finite on the other 72
    for layer in layers:
        sub_ref, ref = refs[layer]
        sub_after, _, _, _ = compact_requests(pool, bt, lens, rows, layer)
        assert np.array_equal(sub_after, sub_ref)
        assert_close(dev_to_bits(out[layer][rows]), ref, "llama70b layer %d" % layer)
    kp.close()


def test_skewed_long_is_bit_reproducible_over_many_launches():
    """A fold's result must not depend on which warp or CTA arrives last: the rounds it is taken in, and
    so its rounding, are a function of the partition alone.  The long request of this batch is cut into
    about 18 CTA partials per kv head; 20 000 back-to-back fused steps on the same inputs must write
    the same bits every time (a round size that followed the number of merges a warp happened to
    inherit showed up as one bf16 ulp in one element about once in 400 launches)."""
    w, lens, npg, bt, kp, pool, q, k, v, out = _device_workload("skewed_long")
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    kp.decode_step(0, btd, sld, q[0], k[0], v[0], out[0])
    assert kp.check_status() == 0
    first = out[0].clone()
    differing = 0
    for _ in range(1000):
        for _ in range(20):
            kp.decode_step(0, btd, sld, q[0], k[0], v[0], out[0])
        differing += 0 if torch.equal(out[0], first) else 1
    assert kp.check_status() == 0
    assert differing == 0
    kp.close()
