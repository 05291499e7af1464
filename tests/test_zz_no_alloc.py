"""GPU test of hswa_decode_attn_static_ws, the decode entry point for callers that may not allocate device
memory (fixed memory budget, or a section where cudaMalloc's device-wide synchronisation is not allowed).
Its scratch is a fixed array inside the library, shared by every call, so the test makes two calls in a row
with different batches and checks each against hswa_decode_attn with a caller-allocated workspace (the two run
the same kernels with the same split plan, so they must agree bit for bit) and against the CPU oracle.
This file sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import binding as hb
from paper_2607_13095_b200 import workloads as wl
from helpers import build_scenario
from gpu_utils import dev_batch, dev_i32, make_handle, to_dev_bf16, workspace_for

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _both(sc, is_swa):
    d, t = sc.dims, sc.tables
    h = make_handle(d)
    q, k, v = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    res = []
    for static in (False, True):
        layer = hb.Layer(to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool), is_swa)
        out = torch.full((t.batch, d.num_q_heads, d.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((t.batch, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        if static:
            hb.hswa_decode_attn_static_ws(h, layer, dev_batch(t, True), q, k, v, out, lse)
        else:
            hb.hswa_decode_attn(h, layer, dev_batch(t, True), q, k, v, out, lse, workspace_for(h, t))
        assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
        res.append((out.cpu().numpy(), lse.cpu().numpy(), layer.pool.view(torch.int16).cpu().numpy()))
    (o0, l0, p0), (o1, l1, p1) = res
    assert np.isfinite(o1).all()
    # same kernels, same split plan, only the scratch address differs: identical bits
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)
    assert np.array_equal(p0, p1)  # the fused append wrote the same bytes
    # and both are right: the oracle on the same inputs
    ol = sc.layer(is_swa)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(o1 - ref).max() <= TOL and np.abs(l1 - ref_lse).max() <= TOL
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(p1.view(np.uint16), ol.pool)


def test_static_ws_matches_workspace_entry_twice_in_a_row():
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    first = build_scenario(d, [9000, 5000, 2049, 70, 12000], [1] * 5, seed=21)   # several splits per request
    second = build_scenario(d, [4100, 300], [1, 1], seed=22)                      # smaller: stale partials remain
    _both(first, False)
    _both(second, False)
    _both(second, True)   # SWA layers use no scratch but must work through the same entry point


def test_static_ws_rejects_oversized_batch():
    d = wl.Dims(num_q_heads=64, num_kv_heads=8, head_dim=128, page_size=64)
    sc = build_scenario(d, [100, 200], [1, 1], seed=23)
    t = sc.tables
    h = make_handle(d)
    layer = hb.Layer(to_dev_bf16(sc.full_pool), False)
    out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    b = dev_batch(t, True)
    # claim a context bound whose partials cannot fit 64 MiB: 2 * 64 rows * 16384 splits * 520 B ~ 1 GiB
    # (with a block table wide enough for that bound, as the call requires)
    claim = 32 * 1024 * 1024
    wide = dev_i32(np.zeros((2, claim // d.page_size + 1)))
    big = hb.Batch(b.ctx_len, wide, b.ring_table, b.ring_head, None, max_q_len=1, total_q=2, max_ctx_len=claim)
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn_static_ws(h, layer, big, to_dev_bf16(sc.q), None, None, out)
    assert e.value.status == hb.HSWA_ERR_WORKSPACE
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
