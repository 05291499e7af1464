"""Seeded synthetic inputs for the hybrid-SWA attention path.

This module only draws random numbers and lays out bookkeeping (lengths, page ids, ring heads).  It holds
none of the method's arithmetic: no attention, no position -> slot mapping, no append.  It imports neither
the CUDA binding nor the CPU checker, so both sides can be fed from it.

Workload shapes follow the paper's serving setting (Sec. 2.1: 60 SWA layers with window 128 and 10 Full
layers, i.e. 6:1; Sec. 5.2: 16K-token prefill chunks against long cached prefixes and length buckets up to
256K and beyond; Sec. 3.1.4: multi-user shared system prompts).  The paper measures on production traffic,
which is not public; these inputs stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Dims:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    window: int = 128

    @property
    def ring_pages(self) -> int:  # R = ceil(W / P) + 1
        return -(-self.window // self.page_size) + 1

    @property
    def ring_slots(self) -> int:  # C = R * P
        return self.ring_pages * self.page_size

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:  # K and V rows of all KV heads, bf16
        return 2 * self.num_kv_heads * self.head_dim * 2

    @property
    def page_bytes(self) -> int:
        return self.kv_bytes_per_token * self.page_size


TINY = Dims(num_q_heads=4, num_kv_heads=1, head_dim=64, page_size=16)
BIG = Dims(num_q_heads=64, num_kv_heads=8, head_dim=128, page_size=64)


def hybrid_layer_flags(num_layers: int) -> List[bool]:
    """is_swa per layer for a 6:1 interleave: layer 0 of every 7 is Full."""
    return [(l % 7) != 0 for l in range(num_layers)]


def bf16_bits_normal(seed: int, shape, scale: float = 1.0) -> np.ndarray:
    """N(0,1) * scale rounded to bf16, returned as uint16 bit patterns (host)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    x = torch.randn(tuple(shape), generator=g, dtype=torch.float32) * scale
    return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_const(value: float, shape) -> np.ndarray:
    x = torch.full(tuple(shape), float(value), dtype=torch.float32)
    return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64 (data plumbing for tests)."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@dataclass
class Tables:
    """Bookkeeping of one batch: lengths and page ids.  All int32 numpy arrays."""
    dims: Dims
    ctx_len: np.ndarray          # [B] tokens cached before the step
    q_len: np.ndarray            # [B] new tokens in the step
    q_indptr: np.ndarray         # [B+1]
    block_table: np.ndarray      # [B][max_blocks] page ids in a Full pool
    num_full_pages: int          # pages a Full pool must have
    ring_table: np.ndarray       # [B][R] page ids in an SWA pool
    num_ring_pages: int
    ring_head: np.ndarray        # [B] in [0, C)
    shared_prefix_pages: int = 0

    @property
    def batch(self) -> int:
        return int(self.ctx_len.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.q_indptr[-1])

    @property
    def max_q_len(self) -> int:
        return int(self.q_len.max()) if self.batch else 0

    @property
    def max_ctx_len(self) -> int:
        return int(self.ctx_len.max()) if self.batch else 0


def make_tables(dims: Dims, ctx_len, q_len, seed: int, shared_prefix_tokens: int = 0, slack: float = 1.25,
                permute: bool = True, ring_head: Optional[np.ndarray] = None,
                extra_blocks: int = 0) -> Tables:
    """Allocate page ids for a batch.

    Every request gets ceil((ctx + n) / P) Full pages and R ring pages.  With shared_prefix_tokens > 0
    (a multiple of P, <= every ctx) the leading block-table entries of all requests name the SAME
    physical pages.  Physical ids are a random permutation of a pool `slack` times larger than needed
    (identity order when permute is False); unused block-table entries are -1.
    """
    rng = np.random.default_rng(seed)
    P, R, Cs = dims.page_size, dims.ring_pages, dims.ring_slots
    ctx_len = np.asarray(ctx_len, dtype=np.int64)
    q_len = np.asarray(q_len, dtype=np.int64)
    B = int(ctx_len.shape[0])
    assert shared_prefix_tokens % P == 0 and (B == 0 or shared_prefix_tokens <= ctx_len.min())
    n_shared = shared_prefix_tokens // P
    need = [int(-(-(int(c) + int(n)) // P)) for c, n in zip(ctx_len, q_len)]
    max_blocks = max(need + [1]) + extra_blocks
    n_private = sum(x - n_shared for x in need)
    n_needed = n_shared + n_private
    num_full_pages = max(int(np.ceil(n_needed * slack)), n_needed, 1)
    ids = rng.permutation(num_full_pages) if permute else np.arange(num_full_pages)
    block_table = np.full((B, max_blocks), -1, dtype=np.int32)
    shared_ids = ids[:n_shared]
    cur = n_shared
    for r in range(B):
        block_table[r, :n_shared] = shared_ids
        k = need[r] - n_shared
        block_table[r, n_shared:need[r]] = ids[cur:cur + k]
        cur += k
    num_ring_pages = max(int(np.ceil(B * R * slack)), B * R, 1)
    rids = rng.permutation(num_ring_pages) if permute else np.arange(num_ring_pages)
    ring_table = rids[:B * R].reshape(B, R).astype(np.int32)
    if ring_head is None:
        ring_head = rng.integers(0, Cs, B)
    q_indptr = np.zeros(B + 1, dtype=np.int32)
    q_indptr[1:] = np.cumsum(q_len)
    return Tables(dims, ctx_len.astype(np.int32), q_len.astype(np.int32), q_indptr, block_table, num_full_pages,
                  ring_table, num_ring_pages, np.asarray(ring_head, dtype=np.int32), n_shared)


# ---------------------------------------------------------------------------------------------------
# The five named workloads.  Lengths come from numpy's default_rng(seed).integers(lo, hi + 1, B).
# ---------------------------------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    dims: Dims
    layer_is_swa: List[bool]
    tables: Tables
    seed: int
    value_scale: float = 1.0
    notes: dict = field(default_factory=dict)


def config1(kind: str = "decode", seed: int = 1) -> Workload:
    """Tiny hybrid pair: 1 Full + 1 SWA layer, GQA 4:1, D 64, P 16, contexts (100, 512);
    kind 'decode' = one decode step, 'prefill' = one 64-token chunk."""
    n = 1 if kind == "decode" else 64
    t = make_tables(TINY, [100, 512], [n, n], seed)
    return Workload(f"cfg1-{kind}", TINY, [False, True], t, seed, value_scale=1.0 / 8.0)


def config2(seed: int = 2, batch: int = 64) -> Workload:
    """Decode, one hybrid block (1 Full + 6 SWA), batch 64, contexts U[4k, 32k]."""
    ctx = np.random.default_rng(seed).integers(4096, 32768 + 1, batch)
    t = make_tables(BIG, ctx, np.ones(batch, dtype=np.int64), seed, slack=1.0)
    return Workload("cfg2-decode-b64-4k-32k", BIG, hybrid_layer_flags(7), t, seed)


def config3(seed: int = 3, batch: int = 8, chunk: int = 8192) -> Workload:
    """Chunked prefill: 8 requests, cached context U[0, 16k], new chunk of 8192 tokens each."""
    ctx = np.random.default_rng(seed).integers(0, 16384 + 1, batch)
    t = make_tables(BIG, ctx, np.full(batch, chunk, dtype=np.int64), seed, slack=1.0)
    return Workload("cfg3-prefill-b8-chunk8192", BIG, hybrid_layer_flags(7), t, seed)


def config4(seed: int = 4, batch: int = 128, prefix: int = 16384) -> Workload:
    """Prefix-cache-hit decode: 128 requests share a 16k-token prefix (same physical pages),
    unique suffixes U[256, 4k]."""
    suf = np.random.default_rng(seed).integers(256, 4096 + 1, batch)
    t = make_tables(BIG, prefix + suf, np.ones(batch, dtype=np.int64), seed, shared_prefix_tokens=prefix,
                    slack=1.0)
    return Workload("cfg4-prefixhit-decode-b128", BIG, hybrid_layer_flags(7), t, seed,
                    notes={"suffix_sum": int(suf.sum())})


def config5(seed: int = 5, batch: int = 16, num_layers: int = 70) -> Workload:
    """Full-stack long-context decode: 70 layers (60 SWA + 10 Full), batch 16, contexts U[64k, 256k]."""
    ctx = np.random.default_rng(seed).integers(65536, 262144 + 1, batch)
    t = make_tables(BIG, ctx, np.ones(batch, dtype=np.int64), seed, slack=1.0)
    return Workload("cfg5-fullstack-decode-b16-64k-256k", BIG, hybrid_layer_flags(num_layers), t, seed)
