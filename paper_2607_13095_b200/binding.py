"""Thin ctypes binding of libhswa.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors owned by the caller; this module passes their device pointers and the current
torch stream to the library.  Every step of the path runs inside the library's kernels; there is no Python or
CPU fallback, and a missing or unloadable library raises at import of the symbols.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

HSWA_OK = 0
HSWA_ERR_INVALID_ARG = 1
HSWA_ERR_UNSUPPORTED = 2
HSWA_ERR_WORKSPACE = 3
HSWA_ERR_CUDA = 4
HSWA_ERR_BOUNDS = 5
HSWA_ERR_TIMEOUT = 6

EXPORTS = [
    "hswa_create", "hswa_destroy", "hswa_workspace_bytes", "hswa_validate_batch", "hswa_kv_append",
    "hswa_decode_attn", "hswa_decode_attn_mtp", "hswa_decode_attn_shared_prefix", "hswa_decode_attn_static_ws", "hswa_prefill_attn", "hswa_step_advance", "hswa_get_async_error", "hswa_status_string",
    "hswa_window_safe_len", "hswa_swa_window_gather", "hswa_swa_window_scatter",
    "hswa_decode_workspace_need", "hswa_selftest_wait_timeout", "hswa_set_overlap",
    "hswa_swa_release", "hswa_swa_valid_mask", "hswa_prefix_hit_len", "hswa_set_prefill_order", "hswa_set_block_trace",
    "hswa_probe_read_stream",
]


class hswa_config(C.Structure):
    _fields_ = [
        ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("window", C.c_int32), ("ring_pages", C.c_int32),
        ("sm_scale", C.c_float), ("out_dtype", C.c_int32),
    ]


class hswa_layer(C.Structure):
    _fields_ = [("pool", C.c_void_p), ("num_pages", C.c_int64), ("is_swa", C.c_int32)]


class hswa_batch(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("ctx_len", C.c_void_p), ("q_indptr", C.c_void_p), ("block_table", C.c_void_p),
        ("max_blocks", C.c_int32), ("ring_table", C.c_void_p), ("ring_head", C.c_void_p),
        ("max_q_len", C.c_int32), ("total_q", C.c_int32), ("max_ctx_len", C.c_int32),
    ]


class HswaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


_lib = None


def lib_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> C.CDLL:
    """Load libhswa.so (building it in-tree first when it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build() if build_if_missing else _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2607_13095_b200.build`")
    lib = C.CDLL(path)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.hswa_create.restype = C.c_int
    lib.hswa_create.argtypes = [C.POINTER(hswa_config), C.POINTER(vp)]
    lib.hswa_destroy.restype = None
    lib.hswa_destroy.argtypes = [vp]
    lib.hswa_workspace_bytes.restype = sz
    lib.hswa_workspace_bytes.argtypes = [vp, i32, i32, i32]
    lib.hswa_decode_workspace_need.restype = sz
    lib.hswa_decode_workspace_need.argtypes = [vp, i32, i32, i32, i32, i32]
    lib.hswa_set_prefill_order.restype = C.c_int
    lib.hswa_set_prefill_order.argtypes = [vp, i32]
    lib.hswa_set_block_trace.restype = C.c_int
    lib.hswa_set_block_trace.argtypes = [vp, vp, i64]
    lib.hswa_probe_read_stream.restype = C.c_int
    lib.hswa_probe_read_stream.argtypes = [vp, vp, sz, vp]
    lib.hswa_set_overlap.restype = C.c_int
    lib.hswa_set_overlap.argtypes = [vp, i32]
    lib.hswa_selftest_wait_timeout.restype = C.c_int
    lib.hswa_selftest_wait_timeout.argtypes = [vp, i64, vp]
    lib.hswa_validate_batch.restype = C.c_int
    lib.hswa_validate_batch.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp]
    lib.hswa_kv_append.restype = C.c_int
    lib.hswa_kv_append.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp, vp]
    lib.hswa_decode_attn.restype = C.c_int
    lib.hswa_decode_attn.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp, vp, vp, vp, vp, sz, vp]
    lib.hswa_decode_attn_mtp.restype = C.c_int
    lib.hswa_decode_attn_mtp.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), i32, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.hswa_decode_attn_shared_prefix.restype = C.c_int
    lib.hswa_decode_attn_shared_prefix.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), i32, vp, vp, vp, vp, vp,
                                                   vp, sz, vp]
    lib.hswa_decode_attn_static_ws.restype = C.c_int
    lib.hswa_decode_attn_static_ws.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp, vp, vp, vp, vp]
    lib.hswa_prefill_attn.restype = C.c_int
    lib.hswa_prefill_attn.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp, vp, i32, vp, vp, vp,
                                      sz, vp]
    lib.hswa_window_safe_len.restype = C.c_int64
    lib.hswa_window_safe_len.argtypes = [C.c_int64, i32, vp]
    lib.hswa_swa_window_gather.restype = C.c_int
    lib.hswa_swa_window_gather.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp]
    lib.hswa_swa_window_scatter.restype = C.c_int
    lib.hswa_swa_window_scatter.argtypes = [vp, C.POINTER(hswa_layer), C.POINTER(hswa_batch), vp, vp]
    lib.hswa_swa_release.restype = C.c_int
    lib.hswa_swa_release.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.hswa_swa_valid_mask.restype = C.c_int
    lib.hswa_swa_valid_mask.argtypes = [vp, i32, vp, vp, i64, vp, vp]
    lib.hswa_prefix_hit_len.restype = C.c_int64
    lib.hswa_prefix_hit_len.argtypes = [i64, i32, vp, vp]
    lib.hswa_step_advance.restype = C.c_int
    lib.hswa_step_advance.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.hswa_get_async_error.restype = C.c_int
    lib.hswa_get_async_error.argtypes = [vp, vp, C.POINTER(i32 * 4)]
    lib.hswa_status_string.restype = C.c_char_p
    lib.hswa_status_string.argtypes = [C.c_int]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().hswa_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, what: str):
    if status != HSWA_OK:
        raise HswaError(status, what)


class Handle:
    """Owns an hswa_handle*."""

    def __init__(self, num_q_heads, num_kv_heads, head_dim, page_size, window=128, ring_pages=0, sm_scale=0.0,
                 out_dtype=torch.bfloat16):
        self._h = C.c_void_p()
        self.cfg = hswa_config(num_q_heads, num_kv_heads, head_dim, page_size, window, ring_pages, sm_scale,
                               1 if out_dtype == torch.float32 else 0)
        self.out_dtype = out_dtype
        _check(load().hswa_create(C.byref(self.cfg), C.byref(self._h)), "hswa_create")
        self.ring_pages = ring_pages or (-(-window // page_size) + 1)

    def close(self):
        if self._h:
            load().hswa_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def ptr(self):
        return self._h


class Layer:
    """One layer's pool: bf16 CUDA tensor [num_pages][2][Hkv][P][D]."""

    def __init__(self, pool: torch.Tensor, is_swa: bool):
        assert pool.dtype == torch.bfloat16 and pool.dim() == 5 and pool.is_contiguous()
        self.pool = pool
        self.is_swa = bool(is_swa)
        self.c = hswa_layer(pool.data_ptr(), pool.shape[0], int(self.is_swa))


class Batch:
    """One step's batch: int32 CUDA tensors plus the host-known bounds."""

    def __init__(self, ctx_len, block_table, ring_table, ring_head, q_indptr=None, *, max_q_len=1, total_q=None,
                 max_ctx_len=0):
        for t in (ctx_len, block_table, ring_table, ring_head):
            assert t.dtype == torch.int32 and t.is_cuda and t.is_contiguous()
        self.ctx_len, self.block_table, self.ring_table, self.ring_head, self.q_indptr = (
            ctx_len, block_table, ring_table, ring_head, q_indptr)
        B = int(ctx_len.shape[0])
        self.batch = B
        self.total_q = B if total_q is None else int(total_q)
        self.max_q_len = int(max_q_len)
        self.c = hswa_batch(
            B, ctx_len.data_ptr(), None if q_indptr is None else q_indptr.data_ptr(), block_table.data_ptr(),
            int(block_table.shape[1]) if block_table.dim() == 2 else 0, ring_table.data_ptr(), ring_head.data_ptr(),
            self.max_q_len, self.total_q, int(max_ctx_len))


def hswa_workspace_bytes(h: Handle, max_batch: int, max_total_q: int, max_ctx_len: int) -> int:
    return int(load().hswa_workspace_bytes(h.ptr, max_batch, max_total_q, max_ctx_len))


def hswa_decode_workspace_need(h: Handle, is_swa: bool, batch: int, max_ctx_len: int, shared_prefix_len: int = 0,
                               q_len: int = 1) -> int:
    return int(load().hswa_decode_workspace_need(h.ptr, int(bool(is_swa)), batch, max_ctx_len, shared_prefix_len, q_len))


def hswa_set_overlap(h: Handle, enabled: bool):
    _check(load().hswa_set_overlap(h.ptr, int(bool(enabled))), "hswa_set_overlap")


PREFILL_ORDER_BY_REQUEST, PREFILL_ORDER_LAST_TILE_FIRST, PREFILL_ORDER_LONGEST_REQUEST_FIRST, PREFILL_ORDER_LONGEST_TILE_FIRST = 0, 1, 2, 3


def hswa_set_prefill_order(h: Handle, mode: int):
    _check(load().hswa_set_prefill_order(h.ptr, int(mode)), "hswa_set_prefill_order")


def hswa_set_block_trace(h: Handle, buf: Optional[torch.Tensor]):
    """buf: int64 CUDA tensor [capacity][4] (zeroed by the caller) or None to switch the trace off."""
    if buf is None:
        _check(load().hswa_set_block_trace(h.ptr, None, 0), "hswa_set_block_trace")
        return
    assert buf.dtype == torch.int64 and buf.is_cuda and buf.is_contiguous() and buf.dim() == 2 and buf.shape[1] == 4
    _check(load().hswa_set_block_trace(h.ptr, C.c_void_p(buf.data_ptr()), int(buf.shape[0])), "hswa_set_block_trace")


def hswa_probe_read_stream(h: Handle, buf: torch.Tensor):
    """Stream a CUDA tensor's bytes (a multiple of 32 KB) through shared memory; time it with events."""
    _check(load().hswa_probe_read_stream(h.ptr, _ptr(buf), buf.numel() * buf.element_size(), _stream()), "hswa_probe_read_stream")


def hswa_selftest_wait_timeout(h: Handle, limit_clocks: int):
    _check(load().hswa_selftest_wait_timeout(h.ptr, int(limit_clocks), _stream()), "hswa_selftest_wait_timeout")


def hswa_validate_batch(h: Handle, layer: Layer, batch: Batch):
    _check(load().hswa_validate_batch(h.ptr, C.byref(layer.c), C.byref(batch.c), _stream()), "hswa_validate_batch")


def hswa_kv_append(h: Handle, layer: Layer, batch: Batch, k_new: torch.Tensor, v_new: torch.Tensor):
    _check(load().hswa_kv_append(h.ptr, C.byref(layer.c), C.byref(batch.c), _ptr(k_new), _ptr(v_new), _stream()),
           "hswa_kv_append")


def hswa_decode_attn(h: Handle, layer: Layer, batch: Batch, q, k_new, v_new, out, lse=None, workspace=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().hswa_decode_attn(h.ptr, C.byref(layer.c), C.byref(batch.c), _ptr(q), _ptr(k_new), _ptr(v_new),
                                   _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes, _stream()), "hswa_decode_attn")


def hswa_decode_attn_mtp(h: Handle, layer: Layer, batch: Batch, q_len: int, q, k_new, v_new, out, lse=None, workspace=None):
    """Multi-token decode: q [B][q_len][Hq][D], k_new / v_new [B][q_len][Hkv][D], causal within the q_len drafts."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().hswa_decode_attn_mtp(h.ptr, C.byref(layer.c), C.byref(batch.c), int(q_len), _ptr(q), _ptr(k_new),
                                       _ptr(v_new), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes, _stream()),
           "hswa_decode_attn_mtp")


def hswa_decode_attn_shared_prefix(h: Handle, layer: Layer, batch: Batch, shared_prefix_len: int, q, k_new, v_new, out,
                                   lse=None, workspace=None):
    """Cascade decode: every request of the batch shares its first shared_prefix_len cached tokens (same pages)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().hswa_decode_attn_shared_prefix(h.ptr, C.byref(layer.c), C.byref(batch.c), int(shared_prefix_len), _ptr(q),
                                                 _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                                 _stream()), "hswa_decode_attn_shared_prefix")


STATIC_WS_BYTES = 64 << 20


def hswa_decode_attn_static_ws(h: Handle, layer: Layer, batch: Batch, q, k_new, v_new, out, lse=None):
    """Decode attention for callers that cannot allocate: the split-K scratch is a fixed STATIC_WS_BYTES array
    inside the library (shared by all calls on the device, so keep them on one stream).  Make the first call
    on a device outside any stream capture."""
    _check(load().hswa_decode_attn_static_ws(h.ptr, C.byref(layer.c), C.byref(batch.c), _ptr(q), _ptr(k_new),
                                             _ptr(v_new), _ptr(out), _ptr(lse), _stream()),
           "hswa_decode_attn_static_ws")


def hswa_prefill_attn(h: Handle, layer: Layer, batch: Batch, q, k_new, v_new, fuse_append, out, lse=None,
                      workspace=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().hswa_prefill_attn(h.ptr, C.byref(layer.c), C.byref(batch.c), _ptr(q), _ptr(k_new), _ptr(v_new),
                                    int(bool(fuse_append)), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                    _stream()), "hswa_prefill_attn")


def hswa_window_safe_len(match_len: int, window: int, swa_valid) -> int:
    """Largest usable hit length given the donor's per-position SWA validity (any uint8 buffer / numpy array)."""
    import numpy as np
    v = np.ascontiguousarray(swa_valid, dtype=np.uint8)
    assert v.shape[0] >= match_len
    return int(load().hswa_window_safe_len(int(match_len), int(window), C.c_void_p(v.ctypes.data)))


def _any_ptr(t: torch.Tensor):
    assert t.is_contiguous() and (t.is_cuda or t.is_pinned()), "buffer must be a CUDA tensor or pinned host memory"
    return C.c_void_p(t.data_ptr())


def hswa_swa_window_gather(h: Handle, layer: Layer, batch: Batch, buf: torch.Tensor):
    _check(load().hswa_swa_window_gather(h.ptr, C.byref(layer.c), C.byref(batch.c), _any_ptr(buf), _stream()),
           "hswa_swa_window_gather")


def hswa_swa_window_scatter(h: Handle, layer: Layer, batch: Batch, buf: torch.Tensor):
    _check(load().hswa_swa_window_scatter(h.ptr, C.byref(layer.c), C.byref(batch.c), _any_ptr(buf), _stream()),
           "hswa_swa_window_scatter")


def hswa_swa_release(h: Handle, batch: int, ctx_len: torch.Tensor, release: Optional[torch.Tensor],
                     swa_valid_from: torch.Tensor):
    """release: uint8 CUDA tensor [B] (None: every request releases); swa_valid_from: int32 CUDA tensor [B], in place."""
    assert swa_valid_from.dtype == torch.int32 and (release is None or release.dtype == torch.uint8)
    _check(load().hswa_swa_release(h.ptr, batch, _ptr(ctx_len), _ptr(release), _ptr(swa_valid_from), _stream()),
           "hswa_swa_release")


def hswa_swa_valid_mask(h: Handle, batch: int, ctx_len: torch.Tensor, swa_valid_from: torch.Tensor, mask: torch.Tensor):
    """mask: uint8 [B][stride], CUDA or pinned host."""
    assert mask.dtype == torch.uint8 and mask.dim() == 2 and mask.shape[0] == batch
    _check(load().hswa_swa_valid_mask(h.ptr, batch, _ptr(ctx_len), _ptr(swa_valid_from), int(mask.shape[1]), _any_ptr(mask),
                                      _stream()), "hswa_swa_valid_mask")


def hswa_prefix_hit_len(match_len: int, window: int, full_valid, swa_valid) -> int:
    import numpy as np
    f = np.ascontiguousarray(full_valid, dtype=np.uint8)
    s = np.ascontiguousarray(swa_valid, dtype=np.uint8)
    assert f.shape[0] >= match_len and s.shape[0] >= match_len
    return int(load().hswa_prefix_hit_len(int(match_len), int(window), C.c_void_p(f.ctypes.data), C.c_void_p(s.ctypes.data)))


def hswa_step_advance(h: Handle, batch: int, ctx_len: torch.Tensor, ring_head: torch.Tensor, q_indptr=None):
    _check(load().hswa_step_advance(h.ptr, batch, _ptr(ctx_len), _ptr(ring_head), _ptr(q_indptr), _stream()),
           "hswa_step_advance")


def hswa_get_async_error(h: Handle):
    """Synchronise the current stream and return (status, request, index, value); clears the error word."""
    info = (C.c_int32 * 4)()
    st = load().hswa_get_async_error(h.ptr, _stream(), C.byref(info))
    return int(st), int(info[1]), int(info[2]), int(info[3])
