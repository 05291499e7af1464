"""ctypes front end of the fp64 CPU oracle (hswa_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of the bench.
The product package never imports this module, and this module never imports the product package.

All tensors cross this boundary as numpy arrays: bf16 data as uint16 bit patterns, tables as int32.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hswa_oracle.c")
_SO = os.path.join(_HERE, "_build", "libhswa_oracle.so")


def build(force: bool = False) -> str:
    """Compile hswa_oracle.c with gcc (-O2, no fast-math, OpenMP over independent rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_SO), exist_ok=True)
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


class _Config(C.Structure):
    _fields_ = [
        ("num_q_heads", C.c_int32),
        ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32),
        ("page_size", C.c_int32),
        ("window", C.c_int32),
        ("ring_pages", C.c_int32),
        ("sm_scale", C.c_double),
    ]


class _Layer(C.Structure):
    _fields_ = [
        ("pool", C.c_void_p),
        ("num_pages", C.c_int64),
        ("is_swa", C.c_int32),
        ("stride_page", C.c_int64),
        ("stride_kv", C.c_int64),
        ("stride_head", C.c_int64),
        ("stride_slot", C.c_int64),
        ("stride_d", C.c_int64),
    ]


class _Batch(C.Structure):
    _fields_ = [
        ("batch", C.c_int32),
        ("ctx_len", C.c_void_p),
        ("q_indptr", C.c_void_p),
        ("block_table", C.c_void_p),
        ("max_blocks", C.c_int32),
        ("ring_table", C.c_void_p),
        ("ring_head", C.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.orc_locate.restype = C.c_int
        lib.orc_kv_append.restype = C.c_int
        lib.orc_attention.restype = C.c_int
        lib.orc_step_advance.restype = C.c_int
        lib.orc_window_safe_len.restype = C.c_int64
        lib.orc_window_safe_len.argtypes = [C.c_int64, C.c_int32, C.c_void_p]
        lib.orc_window_gather.restype = C.c_int
        lib.orc_window_scatter.restype = C.c_int
        lib.orc_attended_keys.restype = C.c_int64
        lib.orc_swa_release.restype = C.c_int
        lib.orc_release_due.restype = C.c_int
        lib.orc_swa_valid_mask.restype = C.c_int
        lib.orc_prefix_hit_len.restype = C.c_int64
        lib.orc_attended_keys.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
        _lib = lib
    return _lib


@dataclass
class OracleConfig:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    window: int = 128
    ring_pages: int = 0  # 0 -> ceil(W / P) + 1
    sm_scale: float = 0.0  # 0 -> 1 / sqrt(D)

    def __post_init__(self):
        if self.ring_pages == 0:
            self.ring_pages = -(-self.window // self.page_size) + 1
        if self.sm_scale == 0.0:
            self.sm_scale = 1.0 / float(np.sqrt(self.head_dim))

    @property
    def ring_slots(self) -> int:
        return self.ring_pages * self.page_size

    def c(self) -> _Config:
        return _Config(self.num_q_heads, self.num_kv_heads, self.head_dim, self.page_size, self.window,
                       self.ring_pages, self.sm_scale)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


class OracleLayer:
    """One layer's pool as a uint16 numpy array of shape [num_pages][2][Hkv][P][D] (any strides)."""

    def __init__(self, pool: np.ndarray, is_swa: bool):
        assert pool.dtype == np.uint16 and pool.ndim == 5 and pool.shape[1] == 2
        self.pool = pool
        self.is_swa = bool(is_swa)

    def c(self) -> _Layer:
        st = [s // 2 for s in self.pool.strides]
        return _Layer(self.pool.ctypes.data, self.pool.shape[0], int(self.is_swa), st[0], st[1], st[2], st[3], st[4])


class OracleBatch:
    def __init__(self, ctx_len, block_table, ring_table, ring_head, q_indptr=None):
        self.ctx_len = _i32(ctx_len)
        self.block_table = _i32(block_table)
        self.ring_table = _i32(ring_table)
        self.ring_head = _i32(ring_head)
        self.q_indptr = None if q_indptr is None else _i32(q_indptr)
        self.batch = int(self.ctx_len.shape[0])
        assert self.block_table.ndim == 2 and self.block_table.shape[0] == self.batch
        assert self.ring_table.ndim == 2 and self.ring_table.shape[0] == self.batch

    @property
    def total_q(self) -> int:
        return self.batch if self.q_indptr is None else int(self.q_indptr[-1])

    def c(self) -> _Batch:
        return _Batch(
            self.batch,
            self.ctx_len.ctypes.data,
            None if self.q_indptr is None else self.q_indptr.ctypes.data,
            self.block_table.ctypes.data,
            int(self.block_table.shape[1]),
            self.ring_table.ctypes.data,
            self.ring_head.ctypes.data,
        )


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with status {rc}")


def locate(cfg: OracleConfig, is_swa: bool, batch: OracleBatch, r: int, p: int):
    """(page, slot) of logical position p of request r."""
    lib = _load()
    page, slot = C.c_int64(), C.c_int32()
    cc, cb = cfg.c(), batch.c()
    _check(lib.orc_locate(C.byref(cc), C.c_int32(int(is_swa)), C.byref(cb), C.c_int32(r), C.c_int64(p),
                          C.byref(page), C.byref(slot)), "locate")
    return page.value, slot.value


def kv_append(cfg: OracleConfig, layer: OracleLayer, batch: OracleBatch, k_new, v_new, want_offsets=False):
    """Append in place into layer.pool; optionally return int64 element offsets [T][2][Hkv]."""
    lib = _load()
    k_new, v_new = _u16(k_new), _u16(v_new)
    T = batch.total_q
    assert k_new.shape == (T, cfg.num_kv_heads, cfg.head_dim) == v_new.shape
    offs = np.zeros((T, 2, cfg.num_kv_heads), dtype=np.int64) if want_offsets else None
    cc, cl, cb = cfg.c(), layer.c(), batch.c()
    _check(lib.orc_kv_append(C.byref(cc), C.byref(cl), C.byref(cb), C.c_void_p(k_new.ctypes.data),
                             C.c_void_p(v_new.ctypes.data),
                             C.c_void_p(offs.ctypes.data) if want_offsets else None), "kv_append")
    return offs


def attention(cfg: OracleConfig, layer: OracleLayer, batch: OracleBatch, q, k_new=None, v_new=None, rows=None):
    """fp64 attention.  rows=None -> all (token, head) rows, shapes [T][Hq][D] and [T][Hq];
    rows=(tok[], head[]) -> shapes [n][D] and [n]."""
    lib = _load()
    q = _u16(q)
    T = batch.total_q
    assert q.shape == (T, cfg.num_q_heads, cfg.head_dim)
    if k_new is not None:
        k_new, v_new = _u16(k_new), _u16(v_new)
        assert k_new.shape == (T, cfg.num_kv_heads, cfg.head_dim) == v_new.shape
    if rows is None:
        n = T * cfg.num_q_heads
        tok = head = None
    else:
        tok, head = _i32(rows[0]), _i32(rows[1])
        n = int(tok.shape[0])
    out = np.zeros((n, cfg.head_dim), dtype=np.float64)
    lse = np.zeros((n,), dtype=np.float64)
    cc, cl, cb = cfg.c(), layer.c(), batch.c()
    _check(lib.orc_attention(
        C.byref(cc), C.byref(cl), C.byref(cb), C.c_void_p(q.ctypes.data),
        None if k_new is None else C.c_void_p(k_new.ctypes.data),
        None if v_new is None else C.c_void_p(v_new.ctypes.data),
        C.c_int64(n), None if tok is None else C.c_void_p(tok.ctypes.data),
        None if head is None else C.c_void_p(head.ctypes.data),
        C.c_void_p(out.ctypes.data), C.c_void_p(lse.ctypes.data)), "attention")
    if rows is None:
        return out.reshape(T, cfg.num_q_heads, cfg.head_dim), lse.reshape(T, cfg.num_q_heads)
    return out, lse


def step_advance(cfg: OracleConfig, ctx_len: np.ndarray, ring_head: np.ndarray, q_indptr=None):
    """In-place step advance of int32 arrays ctx_len and ring_head."""
    lib = _load()
    assert ctx_len.dtype == np.int32 and ring_head.dtype == np.int32
    qi = None if q_indptr is None else _i32(q_indptr)
    cc = cfg.c()
    _check(lib.orc_step_advance(C.byref(cc), C.c_int32(ctx_len.shape[0]), C.c_void_p(ctx_len.ctypes.data),
                                C.c_void_p(ring_head.ctypes.data),
                                None if qi is None else C.c_void_p(qi.ctypes.data)), "step_advance")


def attended_keys(cfg: OracleConfig, is_swa: bool, p: int) -> int:
    cc = cfg.c()
    return int(_load().orc_attended_keys(C.byref(cc), C.c_int32(int(is_swa)), C.c_int64(p)))


def window_safe_len(match_len: int, window: int, swa_valid) -> int:
    """Largest hit length <= match_len whose tail still has valid SWA slots (uint8 mask per donor position)."""
    v = np.ascontiguousarray(swa_valid, dtype=np.uint8)
    assert v.shape[0] >= match_len
    return int(_load().orc_window_safe_len(int(match_len), int(window), C.c_void_p(v.ctypes.data)))


def window_gather(cfg: OracleConfig, layer: OracleLayer, batch: OracleBatch) -> np.ndarray:
    """Compact copy [B][W-1][2][Hkv][D] of the cached positions the next token's window needs."""
    buf = np.zeros((batch.batch, cfg.window - 1, 2, cfg.num_kv_heads, cfg.head_dim), dtype=np.uint16)
    cc, cl, cb = cfg.c(), layer.c(), batch.c()
    _check(_load().orc_window_gather(C.byref(cc), C.byref(cl), C.byref(cb), C.c_void_p(buf.ctypes.data)), "window_gather")
    return buf


def window_scatter(cfg: OracleConfig, layer: OracleLayer, batch: OracleBatch, buf: np.ndarray):
    """Write a compact window buffer into the ring slots of the batch (in place)."""
    buf = _u16(buf)
    assert buf.shape == (batch.batch, cfg.window - 1, 2, cfg.num_kv_heads, cfg.head_dim)
    cc, cl, cb = cfg.c(), layer.c(), batch.c()
    _check(_load().orc_window_scatter(C.byref(cc), C.byref(cl), C.byref(cb), C.c_void_p(buf.ctypes.data)), "window_scatter")


def swa_release(cfg: OracleConfig, ctx_len, release, swa_valid_from: np.ndarray):
    """In-place update of int32 swa_valid_from after a step (ctx_len: lengths after the advance; release: uint8
    flags per request or None for all)."""
    assert swa_valid_from.dtype == np.int32
    ctx = _i32(ctx_len)
    rel = None if release is None else np.ascontiguousarray(release, dtype=np.uint8)
    cc = cfg.c()
    _check(_load().orc_swa_release(C.byref(cc), C.c_int32(ctx.shape[0]), C.c_void_p(ctx.ctypes.data),
                                   None if rel is None else C.c_void_p(rel.ctypes.data),
                                   C.c_void_p(swa_valid_from.ctypes.data)), "swa_release")


RELEASE_CHUNK_END, RELEASE_REQUEST_END, RELEASE_DECODE_TOKEN = 0, 1, 2


def release_due(kind: int, decoded: int = 0, every_n: int = 0) -> bool:
    return bool(_load().orc_release_due(C.c_int32(kind), C.c_int64(decoded), C.c_int64(every_n)))


def swa_valid_mask(length: int, swa_valid_from: int) -> np.ndarray:
    mask = np.zeros(max(length, 1), dtype=np.uint8)
    _check(_load().orc_swa_valid_mask(C.c_int64(length), C.c_int64(swa_valid_from), C.c_void_p(mask.ctypes.data)),
           "swa_valid_mask")
    return mask[:length]


def prefix_hit_len(match_len: int, window: int, full_valid, swa_valid) -> int:
    """Largest usable hit length <= match_len given per-token Full and SWA status of the cached prefix."""
    f = np.ascontiguousarray(full_valid, dtype=np.uint8)
    s = np.ascontiguousarray(swa_valid, dtype=np.uint8)
    assert f.shape[0] >= match_len and s.shape[0] >= match_len
    return int(_load().orc_prefix_hit_len(C.c_int64(match_len), C.c_int32(window), C.c_void_p(f.ctypes.data),
                                          C.c_void_p(s.ctypes.data)))


def num_threads() -> int:
    """Threads the OpenMP runtime will use for orc_attention."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        try:
            return max(1, int(env.split(",")[0]))
        except ValueError:
            pass
    return len(os.sched_getaffinity(0))
