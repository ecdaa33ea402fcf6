"""Host-only checks of the C ABI: the library loads without a GPU, exports every function the
header declares, and validates configurations and arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADERS = [os.path.join(ROOT, "include", n) for n in sorted(os.listdir(os.path.join(ROOT, "include"))) if n.endswith(".h")]


@pytest.fixture(scope="module")
def b():
    from paper_2501_08090_b200 import build
    build.build()
    from paper_2501_08090_b200 import binding
    return binding


def declared_functions():
    names = []
    for header in HEADERS:
        text = open(header).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b([a-z_0-9]+)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


def test_every_declared_function_is_exported(b):
    names = declared_functions()
    assert {"kv_pool_create", "kv_append", "decode_attention", "step_latency_sweep"} <= set(names)
    lib = ctypes.CDLL(b.LIBRARY)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(b.EXPORTS)


def test_sizes_follow_the_pool_layout(b):
    cfg = b.make_config(1, 4, 1, 64, 64, 16, 4)
    assert b.kv_pool_bytes(cfg) == 64 * 1 * 2 * 16 * 64 * 2
    cfg = b.make_config(80, 64, 8, 128, 1000, 256, 96)
    assert b.kv_pool_bytes(cfg) == 80 * 1000 * 8 * 2 * 16 * 128 * 2
    ws = b.kv_workspace_bytes(cfg)
    assert ws > 0 and ws % 256 == 0
    bigger = b.make_config(80, 64, 8, 128, 1000, 256, 512)
    assert b.kv_workspace_bytes(bigger) > ws


@pytest.mark.parametrize("kw,needle", [
    (dict(head_dim=96), "head_dim"),
    (dict(page_size=32), "page_size"),
    (dict(num_q_heads=7, num_kv_heads=2), "multiple"),
    (dict(num_q_heads=16, num_kv_heads=1), "group"),
    (dict(num_pages=0), "num_pages"),
    (dict(max_batch=0), "max_batch"),
    (dict(max_batch=10000), "max_batch"),
    (dict(num_layers=0), "num_layers"),
    (dict(num_layers=4096, num_pages=1 << 20), "rows"),
])
def test_invalid_configurations_are_rejected_with_a_message(b, kw, needle):
    base = dict(num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=128, num_pages=16,
                max_pages_per_req=4, max_batch=4, page_size=16)
    base.update(kw)
    cfg = b.make_config(**base)
    assert b.kv_pool_bytes(cfg) == 0
    assert needle in b.last_error()
    assert b.kv_workspace_bytes(cfg) == 0


def test_create_rejects_null_and_misaligned_buffers_before_any_cuda_call(b):
    cfg = b.make_config(1, 8, 2, 128, 16, 4, 4)
    h = ctypes.c_void_p()
    need_p, need_w = b.kv_pool_bytes(cfg), b.kv_workspace_bytes(cfg)
    rc = b.lib.kv_pool_create(ctypes.byref(cfg), None, need_p, 4096, need_w, 0, ctypes.byref(h))
    assert rc == b.CKV_EINVAL and not h.value
    rc = b.lib.kv_pool_create(ctypes.byref(cfg), 4096 + 16, need_p, 8192, need_w, 0, ctypes.byref(h))
    assert rc == b.CKV_EINVAL and "aligned" in b.last_error()
    rc = b.lib.kv_pool_create(ctypes.byref(cfg), 4096, need_p - 1, 8192, need_w, 0, ctypes.byref(h))
    assert rc == b.CKV_ENOMEM
    rc = b.lib.kv_pool_create(ctypes.byref(cfg), 4096, need_p, 8192, need_w - 1, 0, ctypes.byref(h))
    assert rc == b.CKV_ENOMEM
    rc = b.lib.kv_pool_create(ctypes.byref(cfg), 4096, need_p, 8192, need_w, 0, None)
    assert rc == b.CKV_EINVAL


def test_null_handles_are_errors_not_crashes(b):
    assert b.lib.kv_append(None, 0, 1, None, None, None, None, None) == b.CKV_EINVAL
    assert b.lib.decode_attention(None, 0, 1, None, None, None, None, None) == b.CKV_EINVAL
    assert b.lib.kv_check_status(None, None, None) == b.CKV_EINVAL
    assert b.lib.kv_pool_destroy(None) == b.CKV_EINVAL
    assert b.lib.ckv_launch_count(None) == 0


def test_missing_library_is_a_loud_import_error(b, monkeypatch):
    import importlib
    monkeypatch.setattr(b, "LIBRARY", os.path.join(ROOT, "no_such_dir", "libchiron_kv.so"))
    with pytest.raises(ImportError):
        b._load()
