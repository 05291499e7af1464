"""Work accounting for the bench: the bytes and (query, key) pairs the method must touch per step.

Roofline numerators only; no kernel detail and nothing the kernels or the CPU checker execute.
The key-count rule follows the paper's Sec. 2.1 (an SWA layer attends inside a window of W = 128 keys,
a Full layer over the whole sequence), which is what makes the hybrid stack cost about 1/7 of an all-Full
stack at long lengths.
"""
from __future__ import annotations

import numpy as np

from .workloads import Workload


def attended_keys(is_swa: bool, p, window: int):
    """Keys visible to the query at absolute position p (numpy-broadcastable)."""
    p = np.asarray(p, dtype=np.int64)
    return np.minimum(p + 1, window) if is_swa else p + 1


def decode_algorithmic_bytes(w: Workload) -> int:
    """Bytes one decode step must move: visible KV of every layer, plus q, out and the new KV row."""
    d, t = w.dims, w.tables
    total = 0
    per_req_io = (2 * d.num_q_heads * d.head_dim * 2) + d.kv_bytes_per_token
    for is_swa in w.layer_is_swa:
        keys = attended_keys(is_swa, t.ctx_len, d.window).sum()
        total += int(keys) * d.kv_bytes_per_token + t.batch * per_req_io
    return total


def decode_unique_bytes(w: Workload) -> int:
    """Like decode_algorithmic_bytes, but the KV of a prefix whose pages all requests share (paper Sec. 3.1.3:
    equal prefixes share physical pages) is counted once per Full layer instead of once per request: the bytes a
    sharing-aware kernel has to bring from HBM.  SWA layers hold private rings, so nothing is shared there."""
    d, t = w.dims, w.tables
    shared = t.shared_prefix_pages * d.page_size
    total = 0
    per_req_io = (2 * d.num_q_heads * d.head_dim * 2) + d.kv_bytes_per_token
    for is_swa in w.layer_is_swa:
        keys = int(attended_keys(is_swa, t.ctx_len, d.window).sum())
        if not is_swa and t.batch > 0:
            keys -= (t.batch - 1) * shared
        total += keys * d.kv_bytes_per_token + t.batch * per_req_io
    return total


def decode_layer_bytes(w: Workload, is_swa: bool, unique: bool = False) -> int:
    """Algorithmic bytes of one layer of the given kind in one decode step (logical, or with the shared prefix
    counted once)."""
    d, t = w.dims, w.tables
    keys = int(attended_keys(is_swa, t.ctx_len, d.window).sum())
    if unique and not is_swa and t.batch > 0:
        keys -= (t.batch - 1) * t.shared_prefix_pages * d.page_size
    return keys * d.kv_bytes_per_token + t.batch * ((2 * d.num_q_heads * d.head_dim * 2) + d.kv_bytes_per_token)


def prefill_compulsory_bytes(w: Workload, is_swa: bool) -> int:
    """Bytes one prefill layer must move: Q read, output written (bf16), the chunk's K/V read once, the cached keys
    the chunk can see read once (Full: the whole context; SWA: at most W - 1 ring positions), and the appended K/V
    written (SWA: the last min(n, C) tokens)."""
    d, t = w.dims, w.tables
    T = int(t.q_len.astype(np.int64).sum())
    qo = 2 * T * d.num_q_heads * d.head_dim * 2
    chunk_kv = T * d.kv_bytes_per_token
    ctx = t.ctx_len.astype(np.int64)
    n = t.q_len.astype(np.int64)
    if is_swa:
        cached = int(np.minimum(ctx, d.window - 1)[n > 0].sum())
        written = int(np.minimum(n, d.ring_slots).sum())
    else:
        cached = int(ctx[n > 0].sum())
        written = T
    return qo + chunk_kv + (cached + written) * d.kv_bytes_per_token


def prefill_pairs_per_head(w: Workload, is_swa: bool) -> int:
    """Unmasked (query, key) pairs per query head over the whole batch for one layer."""
    d, t = w.dims, w.tables
    total = 0
    for c, n in zip(t.ctx_len.astype(np.int64), t.q_len.astype(np.int64)):
        p = c + np.arange(n, dtype=np.int64)
        total += int(attended_keys(is_swa, p, d.window).sum())
    return total


def prefill_flops(w: Workload, is_swa: bool) -> int:
    """4 * D flops per unmasked pair per query head (QK^T and PV, multiply + add)."""
    return 4 * w.dims.head_dim * w.dims.num_q_heads * prefill_pairs_per_head(w, is_swa)
