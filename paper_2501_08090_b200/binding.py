"""ctypes binding of libchiron_kv.so (see include/chiron_kv.h): argument marshalling only.

Every computation runs in the library's CUDA kernels.  There is no fallback: if the shared
library has not been built, importing this module raises.  torch is used for device memory and
streams, nothing else.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIBRARY = os.path.join(_HERE, "libchiron_kv.so")

CKV_OK, CKV_EINVAL, CKV_ENOMEM, CKV_ECUDA, CKV_EBOUNDS, CKV_ETIMEOUT = 0, -1, -2, -3, -4, -5
STATUS_BAD_LENGTH, STATUS_BAD_PAGE, STATUS_WAIT_LIMIT = 1, 2, 4
HOST_ROUTE_AUTO, HOST_ROUTE_STAGED, HOST_ROUTE_DIRECT, HOST_ROUTE_COPY = 0, 1, 2, 3
TILE_TOKENS, PIECE_COST_TILES = 32, 3      # the plan's tile size and per-piece overhead units

EXPORTS = (
    "kv_pool_bytes", "kv_workspace_bytes", "kv_pool_create", "kv_pool_destroy", "kv_append",
    "decode_attention", "decode_plan", "ckv_set_partition", "ckv_get_partition", "kv_check_status",
    "decode_step_host", "step_latency_sweep", "ckv_profile_enable", "ckv_profile_read",
    "ckv_launch_count", "ckv_last_error", "ckv_read_span_trace", "ckv_set_overlap",
    "decode_attention_noalloc", "decode_step", "kv_swap_out", "kv_swap_in",
    "kv_append_multi", "decode_attention_multi", "kv_read_probe", "ckv_wait_limit_selftest", "ckv_set_host_route",
    "local_autoscaler_instance_slo", "local_autoscaler_create", "local_autoscaler_destroy",
    "local_autoscaler_update", "local_autoscaler_get", "local_autoscaler_simulate",
    "global_request_groups", "global_waiting_time", "global_batch_backpressure", "global_batch_autoscale",
    "global_interactive_autoscale", "global_autoscaler_simulate",
)


class CkvError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("chiron_kv error %d: %s" % (code, message))
        self.code = code


class AutoscalerConfig(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_double), ("itl_slo_us", ctypes.c_double),
                ("min_bs", ctypes.c_double), ("max_bs", ctypes.c_double), ("tbp_mode", ctypes.c_int32)]


class SimConfig(ctypes.Structure):
    """ckv_sim_config of include/chiron_autoscaler.h."""
    _fields_ = [("slots_interactive", ctypes.c_int32), ("slots_batch", ctypes.c_int32),
                ("rate_interactive", ctypes.c_double), ("rate_batch", ctypes.c_double),
                ("startup_s", ctypes.c_double), ("tick_s", ctypes.c_double),
                ("theta", ctypes.c_double), ("delta", ctypes.c_double),
                ("floor_instances", ctypes.c_int32), ("initial_instances", ctypes.c_int32),
                ("max_batch_instances", ctypes.c_int32), ("groups_k", ctypes.c_int32),
                ("z", ctypes.c_double), ("mu_o_prior", ctypes.c_double), ("sigma_o_prior", ctypes.c_double),
                ("policy", ctypes.c_int32), ("horizon_s", ctypes.c_double)]


class SimSummary(ctypes.Structure):
    """ckv_sim_summary of include/chiron_autoscaler.h."""
    _fields_ = [("end_s", ctypes.c_double), ("finished", ctypes.c_int32),
                ("interactive_total", ctypes.c_int32), ("interactive_ttft_met", ctypes.c_int32),
                ("batch_total", ctypes.c_int32), ("batch_ttft_met", ctypes.c_int32),
                ("evictions", ctypes.c_int32),
                ("instances_added", ctypes.c_int32 * 3), ("instances_removed", ctypes.c_int32 * 3),
                ("instance_seconds", ctypes.c_double * 3), ("peak_instances", ctypes.c_int32 * 3),
                ("tokens_served", ctypes.c_double)]


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "num_layers", "num_q_heads", "num_kv_heads", "head_dim", "page_size", "num_pages",
        "max_pages_per_req", "max_batch")]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIBRARY):
        raise ImportError(
            "libchiron_kv.so is missing at %s: build it with `python -m paper_2501_08090_b200.build` "
            "(nvcc, sm_100a).  There is no CPU fallback." % LIBRARY)
    lib = ctypes.CDLL(LIBRARY)
    i32, i64, vp, sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t
    cfgp = ctypes.POINTER(Config)
    lib.kv_pool_bytes.restype = sz; lib.kv_pool_bytes.argtypes = [cfgp]
    lib.kv_workspace_bytes.restype = sz; lib.kv_workspace_bytes.argtypes = [cfgp]
    lib.kv_pool_create.restype = i32
    lib.kv_pool_create.argtypes = [cfgp, vp, sz, vp, sz, i32, ctypes.POINTER(vp)]
    lib.kv_pool_destroy.restype = i32; lib.kv_pool_destroy.argtypes = [vp]
    lib.kv_append.restype = i32; lib.kv_append.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.decode_attention.restype = i32; lib.decode_attention.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.decode_step.restype = i32; lib.decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.kv_swap_out.restype = i32; lib.kv_swap_out.argtypes = [vp, i32, vp, vp, sz, vp]
    lib.kv_swap_in.restype = i32; lib.kv_swap_in.argtypes = [vp, i32, vp, vp, sz, vp]
    lib.kv_append_multi.restype = i32; lib.kv_append_multi.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.decode_attention_multi.restype = i32; lib.decode_attention_multi.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.kv_read_probe.restype = i32; lib.kv_read_probe.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.ckv_wait_limit_selftest.restype = i32; lib.ckv_wait_limit_selftest.argtypes = [vp, ctypes.c_uint64, vp]
    lib.decode_plan.restype = i32; lib.decode_plan.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.ckv_set_partition.restype = i32; lib.ckv_set_partition.argtypes = [vp, i32]
    lib.ckv_set_overlap.restype = i32; lib.ckv_set_overlap.argtypes = [vp, i32]
    lib.ckv_get_partition.restype = i32; lib.ckv_get_partition.argtypes = [vp]
    lib.ckv_set_host_route.restype = i32; lib.ckv_set_host_route.argtypes = [vp, i32]
    lib.kv_check_status.restype = i32; lib.kv_check_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.decode_step_host.restype = i32; lib.decode_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.step_latency_sweep.restype = i32
    lib.step_latency_sweep.argtypes = [vp, i32, vp, i32, vp, vp, vp, vp, vp, vp, i32, i32, vp, sz, vp, vp, vp]
    lib.ckv_profile_enable.restype = i32; lib.ckv_profile_enable.argtypes = [vp, i32]
    lib.ckv_profile_read.restype = i32
    lib.ckv_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32)]
    lib.ckv_read_span_trace.restype = i32; lib.ckv_read_span_trace.argtypes = [vp, vp, vp, vp]
    lib.decode_attention_noalloc.restype = i32
    lib.decode_attention_noalloc.argtypes = [cfgp, vp, i32, i32, vp, vp, vp, vp, i32, vp, ctypes.POINTER(ctypes.c_uint32)]
    f64 = ctypes.c_double
    f64p, i32p, acfgp = ctypes.POINTER(f64), ctypes.POINTER(i32), ctypes.POINTER(AutoscalerConfig)
    lib.local_autoscaler_instance_slo.restype = i32; lib.local_autoscaler_instance_slo.argtypes = [vp, i32, f64p]
    lib.local_autoscaler_create.restype = i32; lib.local_autoscaler_create.argtypes = [acfgp, f64, ctypes.POINTER(vp)]
    lib.local_autoscaler_destroy.restype = i32; lib.local_autoscaler_destroy.argtypes = [vp]
    lib.local_autoscaler_update.restype = i32; lib.local_autoscaler_update.argtypes = [vp, f64, f64, f64p, f64p]
    lib.local_autoscaler_get.restype = i32; lib.local_autoscaler_get.argtypes = [vp, f64p]
    lib.local_autoscaler_simulate.restype = i32
    lib.local_autoscaler_simulate.argtypes = [acfgp, f64, i32, vp, vp, f64, i32, i32, vp, vp, vp, vp]
    lib.global_request_groups.restype = i32; lib.global_request_groups.argtypes = [vp, i32, i32, vp, vp]
    lib.global_waiting_time.restype = i32; lib.global_waiting_time.argtypes = [i32, f64, f64, f64, f64, f64p]
    lib.global_batch_backpressure.restype = i32
    lib.global_batch_backpressure.argtypes = [vp, vp, i32, f64, f64, f64, i32, f64, i32p]
    lib.global_batch_autoscale.restype = i32
    lib.global_batch_autoscale.argtypes = [vp, vp, i32, f64, f64, f64, i32, i32, i32, f64, i32p]
    lib.global_interactive_autoscale.restype = i32
    lib.global_interactive_autoscale.argtypes = [i32, i32, f64, f64, i32, i32p]
    lib.global_autoscaler_simulate.restype = i32
    lib.global_autoscaler_simulate.argtypes = [ctypes.POINTER(SimConfig), i32, vp, vp, vp, vp, vp, vp, vp,
                                               ctypes.POINTER(SimSummary), vp, vp, i32, ctypes.POINTER(i64)]
    lib.ckv_launch_count.restype = i64; lib.ckv_launch_count.argtypes = [vp]
    lib.ckv_last_error.restype = ctypes.c_char_p; lib.ckv_last_error.argtypes = []
    return lib


lib = _load()


def last_error() -> str:
    return lib.ckv_last_error().decode("utf-8", "replace")


def _check(rc: int) -> None:
    if rc != CKV_OK:
        raise CkvError(rc, last_error())


def make_config(num_layers, num_q_heads, num_kv_heads, head_dim, num_pages, max_pages_per_req,
                max_batch, page_size=16) -> Config:
    return Config(num_layers, num_q_heads, num_kv_heads, head_dim, page_size, num_pages,
                  max_pages_per_req, max_batch)


def kv_pool_bytes(cfg: Config) -> int:
    return int(lib.kv_pool_bytes(ctypes.byref(cfg)))


def kv_workspace_bytes(cfg: Config) -> int:
    return int(lib.kv_workspace_bytes(ctypes.byref(cfg)))


def _dev_ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


class KvPool:
    """A paged bf16 KV cache in caller-owned device memory plus the library's scratch.

    `pool` (bf16, kv_pool_bytes) and `workspace` (uint8, kv_workspace_bytes) may be passed in;
    otherwise they are allocated with torch on `device`.  The tensors are kept alive here.
    """

    def __init__(self, cfg: Config, device="cuda:0", pool: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None):
        self.cfg = cfg
        self.device = torch.device(device)
        need_pool, need_ws = kv_pool_bytes(cfg), kv_workspace_bytes(cfg)
        if need_pool == 0 or need_ws == 0:
            raise CkvError(CKV_EINVAL, last_error())
        if pool is None:
            pool = torch.empty(need_pool // 2, dtype=torch.bfloat16, device=self.device)
        if workspace is None:
            workspace = torch.empty(need_ws, dtype=torch.uint8, device=self.device)
        self.pool, self.workspace = pool, workspace
        self._h = ctypes.c_void_p()
        index = self.device.index if self.device.index is not None else torch.cuda.current_device()
        _check(lib.kv_pool_create(ctypes.byref(cfg), _dev_ptr(pool), pool.numel() * pool.element_size(),
                                  _dev_ptr(workspace), workspace.numel() * workspace.element_size(),
                                  index, ctypes.byref(self._h)))

    # -- lifetime
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            lib.kv_pool_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def pool_view(self) -> torch.Tensor:
        """[layers][pages][Hkv][2][P][d] view of the pool tensor."""
        c = self.cfg
        n = c.num_layers * c.num_pages * c.num_kv_heads * 2 * c.page_size * c.head_dim
        return self.pool.view(-1)[:n].view(c.num_layers, c.num_pages, c.num_kv_heads, 2, c.page_size, c.head_dim)

    def _check_sizes(self, batch: int, block_tables, q_len: int = 1, q=None, kv=(), out=None) -> None:
        """The C ABI takes bare pointers and cannot see a tensor that is too small or a table with
        another row width; the device would read past it.  Checked here, where the sizes are known."""
        c = self.cfg
        if block_tables.numel() < batch * c.max_pages_per_req or \
                (block_tables.dim() == 2 and block_tables.shape[1] != c.max_pages_per_req):
            raise ValueError("block_tables must be [batch=%d][max_pages_per_req=%d], got %s"
                             % (batch, c.max_pages_per_req, tuple(block_tables.shape)))
        need_q = batch * q_len * c.num_q_heads * c.head_dim
        need_kv = batch * q_len * c.num_kv_heads * c.head_dim
        for name, t, need in [("q", q, need_q), ("out", out, need_q)] + [("k_new / v_new", t, need_kv) for t in kv]:
            if t is not None and t.numel() < need:
                raise ValueError("%s holds %d elements, %d needed for batch %d" % (name, t.numel(), need, batch))

    # -- the hot path
    def kv_append(self, layer: int, block_tables, seq_lens, k_new, v_new, stream=None) -> None:
        batch = int(seq_lens.shape[0])
        self._check_sizes(batch, block_tables, kv=(k_new, v_new))
        _check(lib.kv_append(self._h, layer, batch, _dev_ptr(block_tables, torch.int32),
                             _dev_ptr(seq_lens, torch.int32), _dev_ptr(k_new, torch.bfloat16),
                             _dev_ptr(v_new, torch.bfloat16), _stream_ptr(stream)))

    def decode_attention(self, layer: int, block_tables, seq_lens, q, out, stream=None) -> None:
        batch = int(seq_lens.shape[0])
        self._check_sizes(batch, block_tables, q=q, out=out)
        _check(lib.decode_attention(self._h, layer, batch, _dev_ptr(block_tables, torch.int32),
                                    _dev_ptr(seq_lens, torch.int32), _dev_ptr(q, torch.bfloat16),
                                    _dev_ptr(out, torch.bfloat16), _stream_ptr(stream)))

    def decode_step(self, layer: int, block_tables, seq_lens, q, k_new, v_new, out, stream=None) -> None:
        """kv_append + decode_attention of one layer in a single kernel."""
        batch = int(seq_lens.shape[0])
        self._check_sizes(batch, block_tables, q=q, kv=(k_new, v_new), out=out)
        _check(lib.decode_step(self._h, layer, batch, _dev_ptr(block_tables, torch.int32),
                               _dev_ptr(seq_lens, torch.int32), _dev_ptr(q, torch.bfloat16),
                               _dev_ptr(k_new, torch.bfloat16), _dev_ptr(v_new, torch.bfloat16),
                               _dev_ptr(out, torch.bfloat16), _stream_ptr(stream)))

    def kv_append_multi(self, layer: int, q_len: int, block_tables, seq_lens, k_new, v_new, stream=None) -> None:
        """Append q_len new tokens per request (k_new, v_new [batch][q_len][Hkv][d])."""
        self._check_sizes(int(seq_lens.shape[0]), block_tables, q_len=int(q_len), kv=(k_new, v_new))
        _check(lib.kv_append_multi(self._h, layer, int(seq_lens.shape[0]), int(q_len),
                                   _dev_ptr(block_tables, torch.int32), _dev_ptr(seq_lens, torch.int32),
                                   _dev_ptr(k_new, torch.bfloat16), _dev_ptr(v_new, torch.bfloat16), _stream_ptr(stream)))

    def decode_attention_multi(self, layer: int, q_len: int, block_tables, seq_lens, q, out, stream=None) -> None:
        """Causal attention of the q_len new tokens (q, out [batch][q_len][Hq][d])."""
        self._check_sizes(int(seq_lens.shape[0]), block_tables, q_len=int(q_len), q=q, out=out)
        _check(lib.decode_attention_multi(self._h, layer, int(seq_lens.shape[0]), int(q_len),
                                          _dev_ptr(block_tables, torch.int32), _dev_ptr(seq_lens, torch.int32),
                                          _dev_ptr(q, torch.bfloat16), _dev_ptr(out, torch.bfloat16), _stream_ptr(stream)))

    def swap_image_bytes(self, n_pages: int) -> int:
        c = self.cfg
        return c.num_layers * int(n_pages) * c.num_kv_heads * 2 * c.page_size * c.head_dim * 2

    def swap_out(self, page_ids, image, stream=None) -> None:
        """Copy the listed pages (all layers) into `image`, a pinned host tensor."""
        self._swap(lib.kv_swap_out, page_ids, image, stream)

    def swap_in(self, page_ids, image, stream=None) -> None:
        """Copy `image` (pinned host tensor) into the listed pages (all layers)."""
        self._swap(lib.kv_swap_in, page_ids, image, stream)

    def _swap(self, fn, page_ids, image, stream):
        if image.is_cuda or not image.is_contiguous() or not image.is_pinned():
            raise ValueError("the swap image must be a contiguous pinned host tensor")
        _check(fn(self._h, int(page_ids.shape[0]), _dev_ptr(page_ids, torch.int32), image.data_ptr(),
                  image.numel() * image.element_size(), _stream_ptr(stream)))

    def read_probe(self, layer: int, block_tables, seq_lens, stream=None) -> None:
        """Stream the KV tiles decode_attention would read for this batch, without the arithmetic."""
        self._check_sizes(int(seq_lens.shape[0]), block_tables)
        _check(lib.kv_read_probe(self._h, layer, int(seq_lens.shape[0]), _dev_ptr(block_tables, torch.int32),
                                 _dev_ptr(seq_lens, torch.int32), _stream_ptr(stream)))

    def wait_limit_selftest(self, limit_ns: int, stream=None) -> None:
        """Make a bounded device-side wait run out on purpose (see ckv_wait_limit_selftest)."""
        _check(lib.ckv_wait_limit_selftest(self._h, int(limit_ns), _stream_ptr(stream)))

    def decode_plan(self, seq_lens, stream=None):
        """(header dict, int32 [num_spans][4] array of span starts)."""
        batch = int(seq_lens.shape[0])
        header = np.zeros(4, dtype=np.int32)
        starts = np.zeros((self.get_partition(), 4), dtype=np.int32)
        _check(lib.decode_plan(self._h, batch, _dev_ptr(seq_lens, torch.int32), _stream_ptr(stream),
                               header.ctypes.data, starts.ctypes.data))
        keys = ("total_units", "units_per_span", "num_spans", "spans_with_units")
        return dict(zip(keys, header.tolist())), starts

    def set_partition(self, num_spans: int) -> None:
        _check(lib.ckv_set_partition(self._h, int(num_spans)))

    def set_overlap(self, enable: bool) -> None:
        _check(lib.ckv_set_overlap(self._h, 1 if enable else 0))

    def get_partition(self) -> int:
        return int(lib.ckv_get_partition(self._h))

    def check_status(self, stream=None, raise_on_error: bool = True) -> int:
        bits = ctypes.c_uint32(0)
        rc = lib.kv_check_status(self._h, _stream_ptr(stream), ctypes.byref(bits))
        if rc != CKV_OK and raise_on_error:
            raise CkvError(rc, last_error())
        return int(bits.value)

    def decode_step_host(self, layer: int, block_tables, seq_lens, q, k_new, v_new, out, stream=None) -> None:
        """Host (CPU, ideally pinned) tensors in, host tensor out; synchronises."""
        for t in (block_tables, seq_lens, q, k_new, v_new, out):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("decode_step_host takes contiguous host tensors")
        batch = int(seq_lens.shape[0])
        self._check_sizes(batch, block_tables, q=q, kv=(k_new, v_new), out=out)
        _check(lib.decode_step_host(self._h, layer, batch, block_tables.data_ptr(), seq_lens.data_ptr(),
                                    q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                    _stream_ptr(stream)))

    def set_host_route(self, route: int) -> None:
        """How decode_step_host moves its buffers: HOST_ROUTE_AUTO / STAGED / DIRECT / COPY."""
        _check(lib.ckv_set_host_route(self._h, int(route)))

    def host_step_call(self, layer: int, block_tables, seq_lens, q, k_new, v_new, out, stream=None):
        """decode_step_host with its arguments marshalled once: returns a callable that issues one
        step per call (for loops that reuse the same host buffers; the buffers must stay alive)."""
        for t in (block_tables, seq_lens, q, k_new, v_new, out):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("decode_step_host takes contiguous host tensors")
        self._check_sizes(int(seq_lens.shape[0]), block_tables, q=q, kv=(k_new, v_new), out=out)
        keep = (block_tables, seq_lens, q, k_new, v_new, out)
        args = (self._h, int(layer), int(seq_lens.shape[0]), block_tables.data_ptr(), seq_lens.data_ptr(),
                q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(), _stream_ptr(stream))
        fn = lib.decode_step_host

        def call(_keep=keep):
            rc = fn(*args)
            if rc != CKV_OK:
                raise CkvError(rc, last_error())
        return call

    def step_latency_sweep(self, batch_sizes: Sequence[int], block_tables, seq_lens, q, k_new, v_new, out,
                           warmup: int = 3, iters: int = 20, flush: Optional[torch.Tensor] = None,
                           stream=None):
        """Median and minimum microseconds per step for each batch size (numpy float64 arrays)."""
        sizes = np.asarray(list(batch_sizes), dtype=np.int32)
        med = np.zeros(sizes.size, dtype=np.float64)
        mn = np.zeros(sizes.size, dtype=np.float64)
        stride = int(seq_lens.shape[0])
        self._check_sizes(stride, block_tables)
        c = self.cfg                                   # q, k_new, v_new, out: [layers][stride][heads][d]
        for name, t, heads in (("q", q, c.num_q_heads), ("out", out, c.num_q_heads),
                               ("k_new", k_new, c.num_kv_heads), ("v_new", v_new, c.num_kv_heads)):
            if t.numel() < c.num_layers * stride * heads * c.head_dim:
                raise ValueError("%s holds %d elements, %d needed for %d layers of batch %d"
                                 % (name, t.numel(), c.num_layers * stride * heads * c.head_dim, c.num_layers, stride))
        fl_ptr = _dev_ptr(flush) if flush is not None else None
        fl_bytes = flush.numel() * flush.element_size() if flush is not None else 0
        _check(lib.step_latency_sweep(self._h, int(sizes.size), sizes.ctypes.data, stride,
                                      _dev_ptr(block_tables, torch.int32), _dev_ptr(seq_lens, torch.int32),
                                      _dev_ptr(q, torch.bfloat16), _dev_ptr(k_new, torch.bfloat16),
                                      _dev_ptr(v_new, torch.bfloat16), _dev_ptr(out, torch.bfloat16),
                                      int(warmup), int(iters), fl_ptr, fl_bytes, _stream_ptr(stream),
                                      med.ctypes.data, mn.ctypes.data))
        return med, mn

    def profile_enable(self, enable: bool) -> None:
        _check(lib.ckv_profile_enable(self._h, 1 if enable else 0))

    def profile_read(self):
        ms = ctypes.c_double(0.0)
        n = ctypes.c_int32(0)
        _check(lib.ckv_profile_read(self._h, ctypes.byref(ms), ctypes.byref(n)))
        return float(ms.value), int(n.value)

    def read_span_trace(self, stream=None):
        """(uint64 [spans][8]: ns of warp start, first tile landed, last tile computed, span finished;
        ns spent waiting for data, ns spent between pieces; tiles; pieces.
        int32 [spans][4] span starts as the attention kernel derived them)."""
        trace = np.zeros((self.get_partition(), 8), dtype=np.uint64)
        starts = np.zeros((self.get_partition(), 4), dtype=np.int32)
        _check(lib.ckv_read_span_trace(self._h, _stream_ptr(stream), trace.ctypes.data, starts.ctypes.data))
        return trace, starts

    def launch_count(self) -> int:
        return int(lib.ckv_launch_count(self._h))


def decode_attention_noalloc(cfg: Config, pool: torch.Tensor, layer: int, block_tables, seq_lens, q, out,
                             num_spans: int = 0, stream=None, sync: bool = True) -> int:
    """decode_attention for callers that cannot allocate a workspace: partial results go into a fixed
    array inside the library (at most 640 spans).  Runs on the current CUDA device.  With `sync`
    the stream is synchronised and the device status bits are returned (and raised if non-zero)."""
    batch = int(seq_lens.shape[0])
    if block_tables.numel() < batch * cfg.max_pages_per_req or \
            (block_tables.dim() == 2 and block_tables.shape[1] != cfg.max_pages_per_req):
        raise ValueError("block_tables must be [batch=%d][max_pages_per_req=%d], got %s"
                         % (batch, cfg.max_pages_per_req, tuple(block_tables.shape)))
    if min(q.numel(), out.numel()) < batch * cfg.num_q_heads * cfg.head_dim:
        raise ValueError("q / out too small for batch %d" % batch)
    if pool.numel() * pool.element_size() < kv_pool_bytes(cfg):
        raise ValueError("pool tensor smaller than kv_pool_bytes(cfg)")
    bits = ctypes.c_uint32(0)
    rc = lib.decode_attention_noalloc(ctypes.byref(cfg), _dev_ptr(pool), int(layer), int(seq_lens.shape[0]),
                                      _dev_ptr(block_tables, torch.int32), _dev_ptr(seq_lens, torch.int32),
                                      _dev_ptr(q, torch.bfloat16), _dev_ptr(out, torch.bfloat16), int(num_spans),
                                      _stream_ptr(stream), ctypes.byref(bits) if sync else None)
    _check(rc)
    return int(bits.value)


class LocalAutoscaler:
    """Per-instance batch-size autoscaler (Algorithm 1); host-only, thin wrapper over the C ABI."""

    def __init__(self, itl_slo_us: float, initial_max_bs: float, alpha: float = 0.5,
                 min_bs: float = 1.0, max_bs: float = 1e9, literal_tbp: bool = False):
        self.cfg = AutoscalerConfig(alpha, itl_slo_us, min_bs, max_bs, 1 if literal_tbp else 0)
        self._h = ctypes.c_void_p()
        rc = lib.local_autoscaler_create(ctypes.byref(self.cfg), float(initial_max_bs), ctypes.byref(self._h))
        if rc != CKV_OK:
            raise CkvError(rc, "local_autoscaler_create: bad configuration")

    def update(self, itl_us: float, throughput: float):
        """(new maximum batch size, backpressure)."""
        bs, bp = ctypes.c_double(0.0), ctypes.c_double(0.0)
        rc = lib.local_autoscaler_update(self._h, float(itl_us), float(throughput), ctypes.byref(bs), ctypes.byref(bp))
        if rc != CKV_OK:
            raise CkvError(rc, "local_autoscaler_update: bad argument")
        return bs.value, bp.value

    @property
    def max_bs(self) -> float:
        v = ctypes.c_double(0.0)
        lib.local_autoscaler_get(self._h, ctypes.byref(v))
        return v.value

    def close(self):
        if self._h.value:
            lib.local_autoscaler_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def instance_slo(itl_slos_us) -> float:
    a = np.ascontiguousarray(itl_slos_us, dtype=np.float64)
    out = ctypes.c_double(0.0)
    rc = lib.local_autoscaler_instance_slo(a.ctypes.data, int(a.size), ctypes.byref(out))
    if rc != CKV_OK:
        raise CkvError(rc, "local_autoscaler_instance_slo: bad argument")
    return out.value


def autoscaler_simulate(itl_slo_us: float, initial_max_bs: float, batch_sizes, us_per_step, extra_us: float,
                        demand: int, iterations: int, alpha: float = 0.5, min_bs: float = 1.0, max_bs: float = 1e9,
                        literal_tbp: bool = False):
    """Closed loop of Algorithm 1 over a latency curve: arrays (MaxBS, batch run, ITL us, backpressure)."""
    cfg = AutoscalerConfig(alpha, itl_slo_us, min_bs, max_bs, 1 if literal_tbp else 0)
    x = np.ascontiguousarray(batch_sizes, dtype=np.float64)
    y = np.ascontiguousarray(us_per_step, dtype=np.float64)
    o_bs = np.zeros(iterations, np.float64); o_b = np.zeros(iterations, np.int32)
    o_itl = np.zeros(iterations, np.float64); o_bp = np.zeros(iterations, np.float64)
    rc = lib.local_autoscaler_simulate(ctypes.byref(cfg), float(initial_max_bs), int(x.size), x.ctypes.data,
                                       y.ctypes.data, float(extra_us), int(demand), int(iterations),
                                       o_bs.ctypes.data, o_b.ctypes.data, o_itl.ctypes.data, o_bp.ctypes.data)
    if rc != CKV_OK:
        raise CkvError(rc, "local_autoscaler_simulate: bad argument")
    return o_bs, o_b, o_itl, o_bp


# ----------------------------------------------------------------------------- global autoscaler

def _rc(rc: int, what: str) -> None:
    if rc != CKV_OK:
        raise CkvError(rc, what + ": bad argument")


def request_groups(ttft_slos, k: int):
    """(group index of every request, centroids in increasing order): 1-D k-means on TTFT SLOs."""
    x = np.ascontiguousarray(ttft_slos, dtype=np.float64)
    kk = max(1, min(int(k), int(x.size)))
    grp = np.zeros(x.size, dtype=np.int32)
    cent = np.zeros(kk, dtype=np.float64)
    _rc(lib.global_request_groups(x.ctypes.data, int(x.size), int(k), grp.ctypes.data, cent.ctypes.data), "global_request_groups")
    return grp, cent


def waiting_time(requests_ahead: int, mu_o: float, sigma_o: float, throughput: float, z: float = 0.0) -> float:
    out = ctypes.c_double(0.0)
    _rc(lib.global_waiting_time(int(requests_ahead), float(mu_o), float(sigma_o), float(throughput), float(z),
                                ctypes.byref(out)), "global_waiting_time")
    return out.value


def batch_backpressure(counts, deadlines, mu_o, sigma_o, throughput_per_instance, instances, z=0.0) -> int:
    c = np.ascontiguousarray(counts, dtype=np.int32); d = np.ascontiguousarray(deadlines, dtype=np.float64)
    out = ctypes.c_int32(0)
    _rc(lib.global_batch_backpressure(c.ctypes.data, d.ctypes.data, int(c.size), float(mu_o), float(sigma_o),
                                      float(throughput_per_instance), int(instances), float(z), ctypes.byref(out)),
        "global_batch_backpressure")
    return out.value


def batch_autoscale(counts, deadlines, mu_o, sigma_o, throughput_per_instance, current_instances,
                    active_requests, max_instances, z=0.0) -> int:
    c = np.ascontiguousarray(counts, dtype=np.int32); d = np.ascontiguousarray(deadlines, dtype=np.float64)
    out = ctypes.c_int32(0)
    _rc(lib.global_batch_autoscale(c.ctypes.data, d.ctypes.data, int(c.size), float(mu_o), float(sigma_o),
                                   float(throughput_per_instance), int(current_instances), int(active_requests),
                                   int(max_instances), float(z), ctypes.byref(out)), "global_batch_autoscale")
    return out.value


def interactive_autoscale(busy: int, total: int, theta: float, delta: float, floor: int = 1) -> int:
    out = ctypes.c_int32(0)
    _rc(lib.global_interactive_autoscale(int(busy), int(total), float(theta), float(delta), int(floor),
                                         ctypes.byref(out)), "global_interactive_autoscale")
    return out.value


SIM_POLICY_CHIRON, SIM_POLICY_IMMEDIATE = 0, 1
SIM_EVENTS = ("ARRIVE", "START", "EVICT", "FINISH", "ADD", "READY", "REMOVE", "TICK")


def global_simulate(cfg: SimConfig, arrival_s, kind, output_tokens, ttft_slo_s, log_cap: int = 0):
    """Run the global autoscaler's discrete-event simulation (host-only).

    Returns a dict: per-request arrays `first_start_s`, `finish_s`, `evictions`; `summary` (a plain
    dict of ckv_sim_summary); `events` = number of events that occurred; and, if log_cap > 0,
    `log` = list of (time, kind, a, b) rows (at most log_cap)."""
    a = np.ascontiguousarray(arrival_s, dtype=np.float64)
    k = np.ascontiguousarray(kind, dtype=np.int32)
    o = np.ascontiguousarray(output_tokens, dtype=np.float64)
    s = np.ascontiguousarray(ttft_slo_s, dtype=np.float64)
    n = int(a.size)
    if not (k.size == n and o.size == n and s.size == n):
        raise ValueError("the four request arrays must have one entry per request")
    first = np.zeros(n, np.float64); fin = np.zeros(n, np.float64); ev = np.zeros(n, np.int32)
    summ = SimSummary()
    lt = np.zeros(max(1, log_cap), np.float64); lr = np.zeros((max(1, log_cap), 3), np.int32)
    rows = ctypes.c_int64(0)
    rc = lib.global_autoscaler_simulate(ctypes.byref(cfg), n, a.ctypes.data, k.ctypes.data, o.ctypes.data,
                                        s.ctypes.data, first.ctypes.data, fin.ctypes.data, ev.ctypes.data,
                                        ctypes.byref(summ), lt.ctypes.data if log_cap else None,
                                        lr.ctypes.data if log_cap else None, int(log_cap), ctypes.byref(rows))
    _rc(rc, "global_autoscaler_simulate")
    summary = {name: (list(getattr(summ, name)) if hasattr(getattr(summ, name), "__len__") else getattr(summ, name))
               for name, _ in SimSummary._fields_}
    out = {"first_start_s": first, "finish_s": fin, "evictions": ev, "summary": summary, "events": int(rows.value)}
    if log_cap:
        m = min(int(rows.value), log_cap)
        out["log"] = [(float(lt[i]), int(lr[i, 0]), int(lr[i, 1]), int(lr[i, 2])) for i in range(m)]
    return out
