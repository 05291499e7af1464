"""Test-side scenario builder: logical K/V sequences placed into paged / ring pools by the CPU oracle.

Everything here runs on the host.  The logical sequences are the ground truth a brute-force check uses;
the pools are what the oracle's storage model (and the CUDA library) read.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import workloads as wl

POISON_K = 0.0     # a leaked key gets an ordinary softmax weight ...
POISON_V = 1000.0  # ... and drags the output far outside any tolerance


def oracle_config(d: wl.Dims, sm_scale: float = 0.0) -> orc.OracleConfig:
    return orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages,
                            sm_scale)


def poison_pool(num_pages: int, d: wl.Dims) -> np.ndarray:
    pool = np.empty((num_pages, 2, d.num_kv_heads, d.page_size, d.head_dim), dtype=np.uint16)
    pool[:, 0] = wl.bf16_bits_const(POISON_K, (1,))[0]
    pool[:, 1] = wl.bf16_bits_const(POISON_V, (1,))[0]
    return pool


@dataclass
class Scenario:
    dims: wl.Dims
    cfg: orc.OracleConfig
    tables: wl.Tables
    k_seq: List[np.ndarray]      # per request [ctx + n][Hkv][D] bf16 bits (logical ground truth)
    v_seq: List[np.ndarray]
    q: np.ndarray                # [T][Hq][D]
    k_new: np.ndarray            # [T][Hkv][D]
    v_new: np.ndarray
    full_pool: np.ndarray        # state BEFORE this step's append
    swa_pool: np.ndarray

    def batch(self) -> orc.OracleBatch:
        t = self.tables
        return orc.OracleBatch(t.ctx_len, t.block_table, t.ring_table, t.ring_head, t.q_indptr)

    def layer(self, is_swa: bool, copy: bool = True) -> orc.OracleLayer:
        pool = self.swa_pool if is_swa else self.full_pool
        return orc.OracleLayer(pool.copy() if copy else pool, is_swa)


def build_scenario(d: wl.Dims, ctx_len, q_len, seed: int, *, scale: float = 1.0, sm_scale: float = 0.0,
                   shared_prefix_tokens: int = 0, ring_keep: Optional[int] = None, permute: bool = True,
                   ring_head=None, slack: float = 1.25, share_pages: bool = True) -> Scenario:
    """Random logical sequences; history [0, ctx) placed in the Full pool, the last `ring_keep`
    (default W - 1, the minimum the window needs) history tokens placed in the ring; everything else in
    both pools is poison."""
    cfg = oracle_config(d, sm_scale)
    t = wl.make_tables(d, ctx_len, q_len, seed, shared_prefix_tokens=shared_prefix_tokens if share_pages else 0,
                       permute=permute, ring_head=ring_head, slack=slack)
    B, Hkv, Hq, D = t.batch, d.num_kv_heads, d.num_q_heads, d.head_dim
    shared_k = wl.bf16_bits_normal(seed * 1000 + 1, (shared_prefix_tokens, Hkv, D), scale)
    shared_v = wl.bf16_bits_normal(seed * 1000 + 2, (shared_prefix_tokens, Hkv, D), scale)
    k_seq, v_seq = [], []
    for r in range(B):
        L = int(t.ctx_len[r] + t.q_len[r])
        k = wl.bf16_bits_normal(seed * 1000 + 10 + 2 * r, (L, Hkv, D), scale)
        v = wl.bf16_bits_normal(seed * 1000 + 11 + 2 * r, (L, Hkv, D), scale)
        k[:shared_prefix_tokens] = shared_k
        v[:shared_prefix_tokens] = shared_v
        k_seq.append(k)
        v_seq.append(v)
    T = t.total_q
    q = wl.bf16_bits_normal(seed * 1000 + 3, (T, Hq, D), scale)
    k_new = np.zeros((T, Hkv, D), dtype=np.uint16)
    v_new = np.zeros((T, Hkv, D), dtype=np.uint16)
    for r in range(B):
        c, a, b = int(t.ctx_len[r]), int(t.q_indptr[r]), int(t.q_indptr[r + 1])
        k_new[a:b] = k_seq[r][c:]
        v_new[a:b] = v_seq[r][c:]
    # history into the Full pool: an append of ctx tokens starting from an empty cache
    full_pool = poison_pool(t.num_full_pages, d)
    hist_ptr = np.zeros(B + 1, dtype=np.int32)
    hist_ptr[1:] = np.cumsum(t.ctx_len)
    if hist_ptr[-1] > 0:
        hk = np.concatenate([k_seq[r][: t.ctx_len[r]] for r in range(B)])
        hv = np.concatenate([v_seq[r][: t.ctx_len[r]] for r in range(B)])
        hb = orc.OracleBatch(np.zeros(B, np.int32), t.block_table, t.ring_table, t.ring_head, hist_ptr)
        orc.kv_append(cfg, orc.OracleLayer(full_pool, False), hb, hk, hv)
    # the last `keep` history tokens into the ring
    swa_pool = poison_pool(t.num_ring_pages, d)
    keep_max = d.window - 1 if ring_keep is None else ring_keep
    keep = np.minimum(t.ctx_len, keep_max).astype(np.int32)
    rp = np.zeros(B + 1, dtype=np.int32)
    rp[1:] = np.cumsum(keep)
    if rp[-1] > 0:
        rk = np.concatenate([k_seq[r][t.ctx_len[r] - keep[r]: t.ctx_len[r]] for r in range(B)])
        rv = np.concatenate([v_seq[r][t.ctx_len[r] - keep[r]: t.ctx_len[r]] for r in range(B)])
        rb = orc.OracleBatch(t.ctx_len - keep, t.block_table, t.ring_table,
                             np.mod(t.ring_head - keep, d.ring_slots), rp)
        orc.kv_append(cfg, orc.OracleLayer(swa_pool, True), rb, rk, rv)
    return Scenario(d, cfg, t, k_seq, v_seq, q, k_new, v_new, full_pool, swa_pool)


def brute_force_attention(sc: Scenario, is_swa: bool):
    """Dense score matrix + explicit boolean mask + softmax in numpy fp64, from the LOGICAL sequences."""
    d, t = sc.dims, sc.tables
    G = d.group
    out = np.zeros((t.total_q, d.num_q_heads, d.head_dim))
    lse = np.zeros((t.total_q, d.num_q_heads))
    for r in range(t.batch):
        c, n = int(t.ctx_len[r]), int(t.q_len[r])
        if n == 0:
            continue
        K = wl.bits_to_f64(sc.k_seq[r])
        V = wl.bits_to_f64(sc.v_seq[r])
        Q = wl.bits_to_f64(sc.q[t.q_indptr[r]: t.q_indptr[r + 1]])
        pos_q = c + np.arange(n)[:, None]
        pos_k = np.arange(c + n)[None, :]
        mask = pos_k <= pos_q
        if is_swa:
            mask &= pos_k > pos_q - d.window
        for h in range(d.num_q_heads):
            S = sc.cfg.sm_scale * (Q[:, h, :] @ K[:, h // G, :].T)
            S = np.where(mask, S, -np.inf)
            m = S.max(axis=1, keepdims=True)
            E = np.exp(S - m)
            E = np.where(mask, E, 0.0)
            den = E.sum(axis=1, keepdims=True)
            out[t.q_indptr[r]: t.q_indptr[r + 1], h] = (E @ V[:, h // G, :]) / den
            lse[t.q_indptr[r]: t.q_indptr[r + 1], h] = (m + np.log(den))[:, 0]
    return out, lse
