"""KV swap-out / swap-in (eviction of a request's KV cache to host memory and back).

CPU part: the oracle's gather/scatter is pinned by brute-force loops and a round trip.
GPU part: the library's image equals the oracle's bit for bit, a request swapped out, overwritten
and swapped back into DIFFERENT physical pages attends exactly as before, and bad page ids are
flagged without touching memory.
"""
import numpy as np
import pytest
import torch

from oracle import swap as oswap
from paper_2501_08090_b200 import workloads as wl


def test_oracle_swap_is_a_page_gather_and_its_inverse():
    layers, pages, Hkv, P, d = 3, 10, 2, 16, 8
    pool = np.arange(layers * pages * Hkv * 2 * P * d, dtype=np.uint16).reshape(layers, pages, Hkv, 2, P, d)
    ids = np.array([7, 2, 9], dtype=np.int32)
    img = oswap.swap_out(pool, ids)
    assert img.shape == (layers, 3, Hkv, 2, P, d)
    for l in range(layers):                                     # brute force, element by element
        for i, pg in enumerate(ids):
            for h in range(Hkv):
                for kv in range(2):
                    assert np.array_equal(img[l, i, h, kv], pool[l, pg, h, kv])
    scrambled = pool.copy()
    scrambled[:, ids] = 0
    new_ids = np.array([0, 5, 1], dtype=np.int32)               # restart in other physical pages
    oswap.swap_in(scrambled, new_ids, img)
    for i in range(3):
        assert np.array_equal(scrambled[:, new_ids[i]], pool[:, ids[i]])
    untouched = [p for p in range(pages) if p not in set(ids) | set(new_ids)]
    assert np.array_equal(scrambled[:, untouched], pool[:, untouched])


@pytest.mark.gpu
def test_gpu_swap_round_trip_into_other_pages_keeps_attention_identical():
    from paper_2501_08090_b200 import binding as b
    from helpers import bits_to_dev, dev_to_bits
    layers, Hq, Hkv, d = 3, 8, 2, 128
    lens = np.array([700, 33, 1500], dtype=np.int32)
    npg = int(wl.pages_of(lens).sum()) + 120
    bt = wl.block_tables(lens, npg, seed=8)
    pool_h = wl.normal_bf16((layers, npg, Hkv, 2, 16, d), 8, 1)
    q_h = wl.normal_bf16((layers, 3, Hq, d), 8, 2)
    cfg = b.make_config(layers, Hq, Hkv, d, npg, bt.shape[1], 3)
    kp = b.KvPool(cfg, pool=bits_to_dev(pool_h.reshape(-1)))
    btd, sld, q = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda(), bits_to_dev(q_h)
    before = torch.zeros_like(q)
    for l in range(layers):
        kp.decode_attention(l, btd, sld, q[l], before[l])

    victim = 2                                                   # evict the longest request
    n = int(wl.pages_of(lens)[victim])
    ids = bt[victim, :n].copy()
    image = torch.empty(kp.swap_image_bytes(n) // 2, dtype=torch.int16).pin_memory()
    kp.swap_out(torch.from_numpy(ids).cuda(), image)
    torch.cuda.synchronize()
    want = oswap.swap_out(pool_h, ids)
    assert np.array_equal(image.numpy().view(np.uint16).reshape(want.shape), want)          # bit-exact image

    # its pages are reused by someone else ...
    pv = kp.pool_view()
    pv[:, torch.from_numpy(ids.astype(np.int64)).cuda()] = float("nan")
    # ... and it restarts in other free pages
    used = set(int(x) for r in range(3) for x in bt[r, :int(wl.pages_of(lens)[r])])
    free = np.array([p for p in range(npg) if p not in used][:n], dtype=np.int32)
    assert free.size == n
    kp.swap_in(torch.from_numpy(free).cuda(), image)
    bt2 = bt.copy(); bt2[victim, :n] = free
    after = torch.zeros_like(q)
    bt2d = torch.from_numpy(bt2).cuda()
    for l in range(layers):
        kp.decode_attention(l, bt2d, sld, q[l], after[l])
    assert kp.check_status() == 0
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))                    # same bits
    ref_pool = pool_h.copy()
    ref_pool[:, ids] = 0x7FC0
    oswap.swap_in(ref_pool, free, want)
    got_pool = dev_to_bits(kp.pool).reshape(ref_pool.shape)
    live = np.ones(npg, bool); live[ids] = False
    assert np.array_equal(got_pool[:, live], ref_pool[:, live])
    kp.close()


@pytest.mark.gpu
def test_gpu_swap_rejects_unpinned_images_and_flags_bad_pages():
    from paper_2501_08090_b200 import binding as b
    cfg = b.make_config(2, 8, 2, 128, 16, 4, 2)
    kp = b.KvPool(cfg)
    kp.pool.zero_()
    ids = torch.tensor([3, 99, -1], dtype=torch.int32, device="cuda")
    image = torch.ones(kp.swap_image_bytes(3) // 2, dtype=torch.int16)
    with pytest.raises(ValueError):
        kp.swap_out(ids, image)                                  # pageable memory
    small = torch.ones(10, dtype=torch.int16).pin_memory()
    with pytest.raises(b.CkvError) as e:
        kp.swap_out(ids, small)
    assert e.value.code == b.CKV_ENOMEM
    pinned = image.pin_memory()
    kp.swap_in(ids, pinned)
    assert kp.check_status(raise_on_error=False) & b.STATUS_BAD_PAGE
    pv = kp.pool_view().view(torch.int16)
    assert bool((pv[:, 3] == 1).all()) and int((pv != 0).sum()) == pv[:, 3].numel()          # only page 3 written
    kp.close()
