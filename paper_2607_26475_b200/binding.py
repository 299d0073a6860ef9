"""Thin ctypes binding of the C-ABI library (`include/dd.h`, instrumentation in `include/dd_bench.h`):
argument marshalling only.

Every step of the path runs in the library's CUDA kernels. torch is used for device and
pinned memory and for streams; tensors are passed as raw pointers. There is no CPU
fallback: importing this module raises if `libdd.so` has not been built
(`python -m paper_2607_26475_b200.build`).
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdd.so")

DD_OK = 0
DD_ERR_INVALID_ARG = -1
DD_ERR_NOT_PINNED = -2
DD_ERR_CUDA = -3
DD_ERR_TIMEOUT = -4
DD_ERR_INDEX_RANGE = -5
DD_ERR_STATE = -6
DD_ERR_WAIT_EXPIRED = -7
DD_GATHER_LOADS = 0
DD_GATHER_BULK = 1
DD_GATHER_STAGED = 2
DD_GATHER_STATS_FIELDS = 7
DD_TRACE_FIELDS = 8
DD_ATTN_AUTO = 0
DD_ATTN_SPLIT = 1
DD_ATTN_STREAM = 2
DD_ATTN_TC = 3
DD_SELECT_AUTO = 0
DD_SELECT_TWO_KERNELS = 1

EXPORTS = [
    "dd_create", "dd_destroy", "dd_slot_bytes", "dd_ring_bytes", "dd_scratch_bytes", "dd_slot_ptr",
    "dd_strerror", "dd_last_error_message", "dd_device_error", "dd_sync", "dd_build_landmarks",
    "dd_select_topk", "dd_gather_kv_from_host", "dd_sparse_decode_attn", "dd_bind", "dd_prime",
    "dd_decode_layer_step", "dd_get_indices", "dd_static_scratch_capacity", "dd_sparse_decode_attn_static",
    "dd_select_topk_chunked", "dd_sparse_decode_attn_causal", "dd_decode_layer_step_causal", "dd_diff_indices",
    "dd_fetch_missing_from_host", "dd_get_merged_indices", "dd_miss_stats", "dd_probe_attn_loads", "dd_probe_select_loads",
    "dd_trace_begin", "dd_trace_end", "dd_trace_read", "dd_decode_step_host", "dd_last_device_error",
    "dd_gather_stats", "dd_set_bulk_wait", "dd_test_pick_cluster", "dd_test_stage_plan", "dd_test_attn_split",
]


class DDConfig(C.Structure):
    """Mirror of `dd_config`."""
    _fields_ = [
        ("n_layers", C.c_int), ("batch", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
        ("head_dim", C.c_int), ("page_tokens", C.c_int), ("max_pages", C.c_int), ("k_pages", C.c_int),
        ("forced_recent_pages", C.c_int), ("n_q_tokens", C.c_int), ("ring_depth", C.c_int),
        ("gather_mode", C.c_int), ("gather_ctas", C.c_int), ("select_mode", C.c_int), ("attn_splits", C.c_int),
        ("compute_stream", C.c_void_p), ("copy_stream", C.c_void_p),
        ("ring_mem", C.c_void_p), ("ring_bytes", C.c_size_t),
        ("landmark_chunk_tokens", C.c_int), ("miss_correction", C.c_int), ("urgent_stream", C.c_void_p),
        ("select_stream", C.c_void_p), ("stage_min_run_pages", C.c_int), ("stage_block_pages", C.c_int), ("attn_mode", C.c_int),
    ]


class DDError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"dd error {code}: {message}")
        self.code = code


PICK_FITS = C.CFUNCTYPE(C.c_int, C.c_int, C.c_size_t, C.c_void_p)


def _load() -> C.CDLL:
    from . import build as _build
    try:
        _build.build()          # compiles with nvcc when the library is missing or older than its sources
    except Exception as e:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing and could not be built ({e}); build it with "
                              "`python -m paper_2607_26475_b200.build` (there is no CPU fallback)") from e
    lib = C.CDLL(LIB_PATH)
    vp, ip = C.c_void_p, C.c_int
    lib.dd_create.argtypes = [C.POINTER(DDConfig), C.POINTER(vp)]
    lib.dd_destroy.argtypes = [vp]
    for name in ("dd_slot_bytes", "dd_ring_bytes", "dd_scratch_bytes"):
        getattr(lib, name).argtypes = [C.POINTER(DDConfig)]
        getattr(lib, name).restype = C.c_size_t
    lib.dd_slot_ptr.argtypes = [vp, ip, C.POINTER(vp)]
    lib.dd_strerror.argtypes = [ip]
    lib.dd_strerror.restype = C.c_char_p
    lib.dd_last_error_message.argtypes = [vp]
    lib.dd_last_error_message.restype = C.c_char_p
    lib.dd_device_error.argtypes = [vp, C.c_double, C.POINTER(ip), C.POINTER(ip)]
    lib.dd_sync.argtypes = [vp, C.c_double]
    lib.dd_build_landmarks.argtypes = [vp, vp, vp, vp, vp]
    lib.dd_select_topk.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp]
    lib.dd_gather_kv_from_host.argtypes = [vp, vp, vp, vp, ip, vp]
    lib.dd_sparse_decode_attn.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp]
    lib.dd_bind.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, vp]
    lib.dd_prime.argtypes = [vp, vp]
    lib.dd_decode_layer_step.argtypes = [vp, ip, ip, vp, vp]
    lib.dd_get_indices.argtypes = [vp, ip, ip, C.POINTER(vp)]
    lib.dd_select_topk_chunked.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp, vp]
    lib.dd_sparse_decode_attn_causal.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp, vp, vp]
    lib.dd_decode_layer_step_causal.argtypes = [vp, ip, ip, vp, vp, vp, vp]
    lib.dd_diff_indices.argtypes = [vp, vp, vp, ip, vp, vp]
    lib.dd_fetch_missing_from_host.argtypes = [vp, vp, ip, vp]
    lib.dd_get_merged_indices.argtypes = [vp, ip, C.POINTER(vp)]
    lib.dd_miss_stats.argtypes = [vp, C.POINTER(C.c_ulonglong), C.POINTER(C.c_ulonglong), ip]
    lib.dd_decode_step_host.argtypes = [vp, ip, vp, vp]
    lib.dd_trace_begin.argtypes = [vp, ip]
    lib.dd_trace_end.argtypes = [vp, C.POINTER(ip)]
    lib.dd_trace_read.argtypes = [vp, ip, ip, vp]
    lib.dd_probe_attn_loads.argtypes = [vp, ip, vp]
    lib.dd_probe_select_loads.argtypes = [vp, vp, vp, vp]
    lib.dd_last_device_error.argtypes = [vp, C.POINTER(ip), C.POINTER(ip)]
    lib.dd_gather_stats.argtypes = [vp, C.POINTER(C.c_ulonglong), ip]
    lib.dd_set_bulk_wait.argtypes = [vp, C.c_double, ip]
    lib.dd_test_pick_cluster.argtypes = [ip, ip, ip, ip, ip, ip, PICK_FITS, vp, C.POINTER(ip), C.POINTER(C.c_size_t), C.POINTER(ip), C.POINTER(ip)]
    lib.dd_test_stage_plan.argtypes = [vp, vp, ip, ip, ip, ip, ip, ip, C.c_longlong, vp, C.c_longlong, vp, vp, vp, vp, vp, vp]
    lib.dd_test_attn_split.argtypes = [ip, ip, ip, ip, ip, C.POINTER(ip), C.POINTER(ip), C.POINTER(ip)]
    lib.dd_static_scratch_capacity.argtypes = []
    lib.dd_static_scratch_capacity.restype = C.c_size_t
    lib.dd_sparse_decode_attn_static.argtypes = [ip] * 8 + [vp] * 7
    return lib


lib = _load()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


class _DevMem:
    """Raw device memory as a CUDA-array-interface object, so that torch can view it."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False),
                                         "version": 2, "strides": None}


def _view(ptr: int, shape, kind: str) -> torch.Tensor:
    """Zero-copy torch view of library-owned device memory (kind: 'i4' or 'bf16')."""
    if kind == "bf16":
        return torch.as_tensor(_DevMem(ptr, shape, "<i2"), device="cuda").view(torch.bfloat16)
    return torch.as_tensor(_DevMem(ptr, shape, "<" + kind), device="cuda")


def _stream(s) -> int:
    if s is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def sparse_decode_attn_static(q, slot, idx, ctx_len, out, out_lse=None, *, n_splits=1, page_tokens=16, stream=None):
    """Attention over a gathered slot without a context and without any allocation: for callers that are
    not allowed to allocate device memory. The library's built-in scratch array (8 MiB per GPU) is shared
    by every call on the device, so calls must not overlap on the GPU; the first call on a device should
    come before any stream capture. q [B, Tq, Hq, d], slot [B, Hkv, 2, k*T, d], idx [B, Hkv, k]."""
    B, Tq, Hq, d = q.shape
    Hkv, k = idx.shape[1], idx.shape[2]
    rc = lib.dd_sparse_decode_attn_static(B, Hq, Hkv, d, page_tokens, k, Tq, n_splits, _ptr(q), _ptr(slot), _ptr(idx),
                                          _ptr(ctx_len), _ptr(out), _ptr(out_lse), _stream(stream))
    if rc != DD_OK:
        raise DDError(rc, lib.dd_last_error_message(None).decode())


class Context:
    """Owns one `dd_ctx`. Method names follow the C entry points (without the `dd_` prefix)."""

    def __init__(self, *, n_layers, batch, max_pages, k_pages, n_q_heads=32, n_kv_heads=8, head_dim=128,
                 page_tokens=16, forced_recent_pages=0, n_q_tokens=2, ring_depth=2, gather_mode=DD_GATHER_LOADS,
                 gather_ctas=0, select_mode=DD_SELECT_AUTO, attn_splits=0, compute_stream=None, copy_stream=None, ring=None,
                 miss_correction=False, urgent_stream=None, landmark_chunk_tokens=0, select_stream=None,
                 stage_min_run_pages=0, stage_block_pages=0, attn_mode=DD_ATTN_AUTO):
        if not torch.cuda.is_available():
            raise RuntimeError("the sparse decode path needs a CUDA device; there is no CPU fallback")
        self.compute_stream = compute_stream if compute_stream is not None else torch.cuda.current_stream()
        self.copy_stream = copy_stream if copy_stream is not None else torch.cuda.Stream()
        self._ring = ring
        self.urgent_stream = urgent_stream
        if miss_correction and urgent_stream is None:
            self.urgent_stream = torch.cuda.Stream(priority=-1)
        self.cfg = DDConfig(n_layers, batch, n_q_heads, n_kv_heads, head_dim, page_tokens, max_pages, k_pages,
                            forced_recent_pages, n_q_tokens, ring_depth, gather_mode, gather_ctas, select_mode, attn_splits,
                            self.compute_stream.cuda_stream, self.copy_stream.cuda_stream,
                            _ptr(ring), ring.numel() * ring.element_size() if ring is not None else 0,
                            landmark_chunk_tokens, 1 if miss_correction else 0,
                            self.urgent_stream.cuda_stream if self.urgent_stream is not None else None,
                            select_stream.cuda_stream if select_stream is not None else None,
                            stage_min_run_pages, stage_block_pages, attn_mode)
        self.select_stream = select_stream
        self._h = C.c_void_p()
        self._keep = []
        rc = lib.dd_create(C.byref(self.cfg), C.byref(self._h))
        if rc != DD_OK:
            raise DDError(rc, lib.dd_last_error_message(None).decode())

    # -- plumbing
    def _check(self, rc: int):
        if rc != DD_OK:
            raise DDError(rc, lib.dd_last_error_message(self._h).decode())

    def close(self):
        if self._h:
            rc = lib.dd_destroy(self._h)
            self._h = C.c_void_p()
            if rc != DD_OK:
                raise DDError(rc, "dd_destroy failed")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def slot_bytes(self) -> int:
        return lib.dd_slot_bytes(C.byref(self.cfg))

    def ring_bytes(self) -> int:
        return lib.dd_ring_bytes(C.byref(self.cfg))

    def scratch_bytes(self) -> int:
        return lib.dd_scratch_bytes(C.byref(self.cfg))

    def slot_ptr(self, slot: int) -> int:
        p = C.c_void_p()
        self._check(lib.dd_slot_ptr(self._h, slot, C.byref(p)))
        return p.value

    def slot_tensor(self, slot: int) -> torch.Tensor:
        """A copy of ring slot `slot` as [B, Hkv, 2, k*T, d] bf16 (synchronises; for tests)."""
        c = self.cfg
        shape = (c.batch, c.n_kv_heads, 2, c.k_pages * c.page_tokens, c.head_dim)
        torch.cuda.synchronize()
        return _view(self.slot_ptr(slot), shape, "bf16").clone()

    def sync(self, timeout_s: float = 60.0):
        self._check(lib.dd_sync(self._h, timeout_s))

    def device_error(self, timeout_s: float = 60.0):
        code, detail = C.c_int(), C.c_int()
        self._check(lib.dd_device_error(self._h, timeout_s, C.byref(code), C.byref(detail)))
        return code.value, detail.value

    def last_device_error(self):
        """(code, detail) of the first device-side error since the last device_error(), without synchronising."""
        code, detail = C.c_int(), C.c_int()
        self._check(lib.dd_last_device_error(self._h, C.byref(code), C.byref(detail)))
        return code.value, detail.value

    def gather_stats(self, reset=False) -> dict:
        """Host-side counters of the staged gather (see dd_gather_stats)."""
        a = (C.c_ulonglong * DD_GATHER_STATS_FIELDS)()
        self._check(lib.dd_gather_stats(self._h, a, 1 if reset else 0))
        names = ("gathers", "copies", "copied_bytes", "pages_staged", "pages_zero_copy", "host_wait_us", "host_issue_us")
        return dict(zip(names, [int(x) for x in a]))

    def set_bulk_wait(self, wait_seconds: float, inflate_first_stage: bool = False):
        self._check(lib.dd_set_bulk_wait(self._h, wait_seconds, 1 if inflate_first_stage else 0))

    # -- entry points
    def build_landmarks(self, kv_layer, ctx_len, landmarks, stream=None):
        self._check(lib.dd_build_landmarks(self._h, _ptr(kv_layer), _ptr(ctx_len), _ptr(landmarks), _stream(stream)))

    def select_topk(self, q, q_token, landmarks, n_pages, out_idx, out_scores=None, stream=None):
        self._check(lib.dd_select_topk(self._h, _ptr(q), q_token, _ptr(landmarks), _ptr(n_pages), _ptr(out_idx),
                                       _ptr(out_scores), _stream(stream)))

    def select_topk_chunked(self, q, q_token, landmarks, n_pages, ctx_len, out_idx, out_scores=None, stream=None):
        self._check(lib.dd_select_topk_chunked(self._h, _ptr(q), q_token, _ptr(landmarks), _ptr(n_pages), _ptr(ctx_len),
                                               _ptr(out_idx), _ptr(out_scores), _stream(stream)))

    def gather_kv_from_host(self, host_kv_layer, idx, n_pages, slot, stream=None):
        self._check(lib.dd_gather_kv_from_host(self._h, _ptr(host_kv_layer), _ptr(idx), _ptr(n_pages), slot,
                                               _stream(stream)))

    def sparse_decode_attn(self, q, slot, idx, ctx_len, out, out_lse=None, stream=None):
        self._check(lib.dd_sparse_decode_attn(self._h, _ptr(q), slot, _ptr(idx), _ptr(ctx_len), _ptr(out),
                                              _ptr(out_lse), _stream(stream)))

    def sparse_decode_attn_causal(self, q, slot, idx, ctx_len, k_new, v_new, out, out_lse=None, stream=None):
        self._check(lib.dd_sparse_decode_attn_causal(self._h, _ptr(q), slot, _ptr(idx), _ptr(ctx_len), _ptr(k_new),
                                                     _ptr(v_new), _ptr(out), _ptr(out_lse), _stream(stream)))

    def decode_layer_step_causal(self, step, layer, q, k_new, v_new, out):
        self._check(lib.dd_decode_layer_step_causal(self._h, step, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)))

    def bind(self, landmarks_per_layer, host_kv_per_layer, n_pages, ctx_len):
        L = self.cfg.n_layers
        assert len(landmarks_per_layer) == L and len(host_kv_per_layer) == L
        self._keep = [landmarks_per_layer, host_kv_per_layer, n_pages, ctx_len]    # keep the tensors alive
        lm = (C.c_void_p * L)(*[_ptr(t) for t in landmarks_per_layer])
        kv = (C.c_void_p * L)(*[_ptr(t) for t in host_kv_per_layer])
        self._check(lib.dd_bind(self._h, lm, kv, _ptr(n_pages), _ptr(ctx_len)))

    def prime(self, q_init):
        self._check(lib.dd_prime(self._h, _ptr(q_init)))

    def decode_layer_step(self, step, layer, q, out):
        self._check(lib.dd_decode_layer_step(self._h, step, layer, _ptr(q), _ptr(out)))

    def diff_indices(self, pred_idx, true_idx, slot, merged_idx, stream=None):
        self._check(lib.dd_diff_indices(self._h, _ptr(pred_idx), _ptr(true_idx), slot, _ptr(merged_idx), _stream(stream)))

    def fetch_missing_from_host(self, host_kv_layer, slot, stream=None):
        self._check(lib.dd_fetch_missing_from_host(self._h, _ptr(host_kv_layer), slot, _stream(stream)))

    def get_merged_indices(self, slot) -> torch.Tensor:
        """A copy of the repaired page list [B, Hkv, k] int32 of ring slot `slot` (synchronises)."""
        p = C.c_void_p()
        self._check(lib.dd_get_merged_indices(self._h, slot, C.byref(p)))
        c = self.cfg
        torch.cuda.synchronize()
        return _view(p.value, (c.batch, c.n_kv_heads, c.k_pages), "i4").clone()

    def miss_stats(self, reset=False):
        """(missing pages, selected pages) accumulated by the corrected layer steps (synchronises)."""
        a, b = C.c_ulonglong(), C.c_ulonglong()
        self._check(lib.dd_miss_stats(self._h, C.byref(a), C.byref(b), 1 if reset else 0))
        return a.value, b.value

    def trace_begin(self, max_layer_steps: int):
        self._check(lib.dd_trace_begin(self._h, max_layer_steps))

    def trace_end(self):
        """Stops the trace and returns it as a [n, DD_TRACE_FIELDS] float32 numpy array of microseconds (see
        dd_trace_begin in dd_bench.h)."""
        import numpy as np
        n = C.c_int()
        self._check(lib.dd_trace_end(self._h, C.byref(n)))
        out = np.zeros((n.value, DD_TRACE_FIELDS), dtype=np.float32)
        if n.value:
            self._check(lib.dd_trace_read(self._h, 0, n.value, out.ctypes.data_as(C.c_void_p)))
        return out

    def probe_attn_loads(self, slot, stream=None):
        self._check(lib.dd_probe_attn_loads(self._h, slot, _stream(stream)))

    def probe_select_loads(self, landmarks, n_pages, stream=None):
        self._check(lib.dd_probe_select_loads(self._h, _ptr(landmarks), _ptr(n_pages), _stream(stream)))

    def decode_step_host(self, step, q_host, out_host):
        """One whole step from pinned host tensors [L, B, Tq, Hq, d] (asynchronous on the compute stream)."""
        self._check(lib.dd_decode_step_host(self._h, step, _ptr(q_host), _ptr(out_host)))

    def get_indices(self, step_parity, layer) -> torch.Tensor:
        """A copy of the index set [B, Hkv, k] int32 used at (step parity, layer) (synchronises)."""
        p = C.c_void_p()
        self._check(lib.dd_get_indices(self._h, step_parity, layer, C.byref(p)))
        c = self.cfg
        torch.cuda.synchronize()
        return _view(p.value, (c.batch, c.n_kv_heads, c.k_pages), "i4").clone()
