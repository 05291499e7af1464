"""Host <-> device plumbing for the GPU parity tests."""
from __future__ import annotations

import numpy as np
import torch

from paper_2607_13095_b200 import binding as hb


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def make_handle(d, out_dtype=torch.float32, sm_scale=0.0) -> hb.Handle:
    return hb.Handle(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages, sm_scale,
                     out_dtype)


def dev_batch(t, decode: bool) -> hb.Batch:
    """binding.Batch from workloads.Tables (decode: q_indptr = NULL)."""
    return hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head),
                    None if decode else dev_i32(t.q_indptr), max_q_len=1 if decode else t.max_q_len,
                    total_q=t.total_q, max_ctx_len=t.max_ctx_len)


def workspace_for(h, t) -> torch.Tensor:
    n = hb.hswa_workspace_bytes(h, max(t.batch, 1), max(t.total_q, 1), t.max_ctx_len)
    return torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")
