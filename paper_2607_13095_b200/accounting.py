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
