"""The give-up path of the bounded device-side waits: a wait that runs out must turn into
CKV_ETIMEOUT on the host, leave the context usable, and leave the handle in a state from which the
next step is correct.  The wait is made to run out harmlessly: a one-warp kernel waits 200 us on a
barrier phase that nothing completes (no copy is issued, nothing can fault or hang)."""
import time

import numpy as np
import pytest
import torch

from paper_2501_08090_b200 import workloads as wl

from helpers import assert_close, dev_to_bits, make_device_step, oracle_step

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_handle_recovers():
    from paper_2501_08090_b200 import binding as b
    h = wl.host_inputs(wl.workload("llama8b_b64"), batch=6)
    ds = make_device_step(h)
    kp = ds.pool
    ws = kp.workspace.view(torch.int32)
    assert kp.check_status() == 0

    t0 = time.perf_counter()
    kp.wait_limit_selftest(200_000)                                        # 200 us
    with pytest.raises(b.CkvError) as e:
        kp.check_status()
    assert e.value.code == b.CKV_ETIMEOUT
    assert time.perf_counter() - t0 < 5.0                                  # it gave up, it did not hang
    # the bits are reported once and then cleared; the half-way arrival counter is cleared too
    assert kp.check_status() == 0
    kp.wait_limit_selftest(50_000)
    assert kp.check_status(raise_on_error=False) == b.STATUS_WAIT_LIMIT
    torch.cuda.synchronize()

    # the context is alive and the next step on the same handle is right: long contexts, so
    # pairs are merged across CTAs through the arrival counters the self-test disturbed
    ref_pool, ref = oracle_step(h)
    kp.decode_step(0, ds.bt, ds.sl, ds.q[0], ds.k_new[0], ds.v_new[0], ds.out[0])
    assert kp.check_status() == 0
    assert np.array_equal(dev_to_bits(kp.pool), ref_pool)
    assert_close(dev_to_bits(ds.out[0]), ref, "step after a timed-out wait")
    kp.close()


def test_selftest_limit_is_validated():
    from paper_2501_08090_b200 import binding as b
    h = wl.host_inputs(wl.workload("tiny"))
    ds = make_device_step(h)
    for bad in (0, 999, 10**9):
        with pytest.raises(b.CkvError) as e:
            ds.pool.wait_limit_selftest(bad)
        assert e.value.code == b.CKV_EINVAL
    assert ds.pool.check_status() == 0
    ds.pool.close()
