"""GPU-box tests of the C-ABI boundary's host logic and failure paths: workspace sizing, shapes the library
refuses before launching anything, the bounded-wait status path, and early-start chaining next to foreign
kernels.  (A handle can only be created where an sm_100 device is present, hence the gpu mark; most of these
tests launch little or nothing.)"""
import numpy as np
import pytest
import torch

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import binding as hb
from paper_2607_13095_b200 import workloads as wl
from helpers import build_scenario
from gpu_utils import dev_batch, dev_i32, make_handle, to_dev_bf16, to_host_bits, workspace_for

pytestmark = pytest.mark.gpu
TOL = 1e-2


def test_workspace_bound_covers_every_accepted_call():
    """hswa_workspace_bytes(max_batch, max_total_q, max_ctx) must be at least the exact need of every decode call
    with a batch and a context inside those bounds, for the plain, shared-prefix and multi-token entry points."""
    d = wl.BIG
    h = make_handle(d)
    batches = [1, 2, 3, 5, 8, 16, 31, 32, 33, 64, 100, 128, 255, 256]
    ctxs = [0, 1, 63, 255, 256, 257, 1023, 4095, 4096, 4097, 20000, 65535, 65536, 131071, 300000]
    prefixes = [0, 128, 192, 4096, 16384, 65536]
    checked = 0
    for max_b in (1, 7, 64, 256):
        for max_ctx in (0, 300, 4096, 40000, 300000):
            for q_len in (1, 2, 4):
                bound = hb.hswa_workspace_bytes(h, max_b, max_b * q_len, max_ctx)
                for b in [x for x in batches if x <= max_b]:
                    for c in [x for x in ctxs if x <= max_ctx]:
                        for pre in (prefixes if q_len == 1 else [0]):
                            if pre > c:
                                continue
                            need = hb.hswa_decode_workspace_need(h, False, b, c, pre, q_len)
                            assert need <= bound, (max_b, max_ctx, q_len, b, c, pre, need, bound)
                            checked += 1
                assert hb.hswa_decode_workspace_need(h, True, max_b, max_ctx, 0, q_len) == 0   # rings need no scratch
    assert checked > 3000


def test_exact_workspace_need_is_the_acceptance_threshold():
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    sc = build_scenario(d, [9000, 5000, 70], [1, 1, 1], seed=41)
    t = sc.tables
    h = make_handle(d)
    layer = hb.Layer(to_dev_bf16(sc.full_pool), False)
    q, k, v = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    need = hb.hswa_decode_workspace_need(h, False, t.batch, t.max_ctx_len, 0, 1)
    assert need > 0 and need % 256 == 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn(h, layer, dev_batch(t, True), q, k, v, out, None, ws[: need - 256])
    assert e.value.status == hb.HSWA_ERR_WORKSPACE
    hb.hswa_decode_attn(h, layer, dev_batch(t, True), q, k, v, out, None, ws)
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    ref, _ = orc.attention(sc.cfg, sc.layer(False), sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(out.cpu().numpy() - ref).max() <= TOL


def test_mtp_rejects_windows_too_long_for_either_ring_kernel_without_launching():
    """Multi-token decode on a ring needs the whole window staged at once.  Windows of a few hundred tokens fit the
    compact kernel's shared memory; beyond that the streaming kernel only serves rings of at most three 64-slot
    tiles, so such a shape is refused on the host (single-token decode still serves it)."""
    d = wl.Dims(num_q_heads=8, num_kv_heads=1, head_dim=128, page_size=64, window=600)   # R = 11, C = 704
    sc = build_scenario(d, [900, 40], [2, 2], seed=42)
    t = sc.tables
    h = make_handle(d)
    swa = hb.Layer(to_dev_bf16(sc.swa_pool), True)
    before = to_host_bits(swa.pool)
    q, k, v = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    out = torch.full((t.batch, 2, d.num_q_heads, d.head_dim), 7.0, dtype=torch.float32, device="cuda")
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None,
                 max_q_len=1, total_q=t.batch, max_ctx_len=t.max_ctx_len)
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn_mtp(h, swa, b, 2, q, k, v, out, None, workspace_for(h, t))
    assert e.value.status == hb.HSWA_ERR_UNSUPPORTED
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    assert (out == 7.0).all() and np.array_equal(to_host_bits(swa.pool), before)   # nothing ran


@pytest.mark.parametrize("W,P,D,G", [(200, 64, 128, 8), (190, 32, 64, 4), (33, 16, 128, 3), (64, 64, 64, 8), (1, 16, 64, 2),
                                     (600, 64, 128, 8)])
@pytest.mark.parametrize("nq", [1, 2, 3, 4])
def test_ring_decode_other_windows_and_token_counts(W, P, D, G, nq):
    """SWA decode for windows other than the paper's 128, every page size, one to four tokens per request, contexts
    around every boundary (empty, shorter than the window, ring wrap)."""
    d = wl.Dims(num_q_heads=G * 2, num_kv_heads=2, head_dim=D, page_size=P, window=W)
    C = d.ring_slots
    if nq > C - W + 1:
        pytest.skip("append-then-attend limit of the ring")
    if W == 600 and nq > 1:
        pytest.skip("refused on the host: see the test above")
    ctx = sorted({0, 1, 2, W - 2, W - 1, W, W + 1, P - 1, P, C - 1, C, C + 1, 3 * C + 5, 2000} - {-1})
    B = len(ctx)
    sc = build_scenario(d, ctx, [nq] * B, seed=48 + nq, ring_keep=C)
    t = sc.tables
    h = make_handle(d)
    pool = to_dev_bf16(sc.swa_pool)
    layer = hb.Layer(pool, True)
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None, max_q_len=1,
                 total_q=B, max_ctx_len=t.max_ctx_len)
    out = torch.full((B * nq, d.num_q_heads, d.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B * nq, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    q, k, v = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    if nq == 1:
        hb.hswa_decode_attn(h, layer, b, q, k, v, out, lse, None)
    else:
        hb.hswa_decode_attn_mtp(h, layer, b, nq, q, k, v, out, lse, None)
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    ol = sc.layer(True)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL and np.abs(lse.cpu().numpy() - ref_lse).max() <= TOL
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(to_host_bits(pool), ol.pool)


def test_single_token_decode_serves_long_rings():
    d = wl.Dims(num_q_heads=8, num_kv_heads=1, head_dim=128, page_size=64, window=200)   # C = 320: five tiles
    sc = build_scenario(d, [500, 40, 199, 200, 201], [1] * 5, seed=43)
    t = sc.tables
    h = make_handle(d)
    swa = hb.Layer(to_dev_bf16(sc.swa_pool), True)
    out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_decode_attn(h, swa, dev_batch(t, True), to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new), out,
                        None, workspace_for(h, t))
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    ol = sc.layer(True)
    ref, _ = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(out.cpu().numpy() - ref).max() <= TOL
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(to_host_bits(swa.pool), ol.pool)


def test_decode_rejects_block_table_that_cannot_cover_the_host_bound():
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    sc = build_scenario(d, [100, 200], [1, 1], seed=44)
    t = sc.tables
    h = make_handle(d)
    layer = hb.Layer(to_dev_bf16(sc.full_pool), False)
    out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    b = dev_batch(t, True)
    claim = hb.Batch(b.ctx_len, b.block_table, b.ring_table, b.ring_head, None, max_q_len=1, total_q=2,
                     max_ctx_len=int(t.block_table.shape[1]) * d.page_size)   # position max_ctx_len has no table entry
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn(h, layer, claim, to_dev_bf16(sc.q), None, None, out, None, workspace_for(h, t))
    assert e.value.status == hb.HSWA_ERR_INVALID_ARG


def test_bounded_wait_runs_out_and_reports_timeout():
    """Failure detection without a fault: a kernel whose consumer waits on a barrier nobody arms gives up after the
    limit, records HSWA_ERR_TIMEOUT and returns; the context stays usable and the word is cleared by the read."""
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    h = make_handle(d)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    hb.hswa_selftest_wait_timeout(h, 2_000_000)   # about a millisecond of SM clocks
    t1.record()
    st = hb.hswa_get_async_error(h)
    assert st == (hb.HSWA_ERR_TIMEOUT, -1, 0, 7), st
    assert t0.elapsed_time(t1) < 1000.0            # it did give up at the limit
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    with pytest.raises(hb.HswaError):
        hb.hswa_selftest_wait_timeout(h, 0)
    # the library still works on this context
    sc = build_scenario(d, [300, 70], [1, 1], seed=45)
    t = sc.tables
    layer = hb.Layer(to_dev_bf16(sc.full_pool), False)
    out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_decode_attn(h, layer, dev_batch(t, True), to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new), out,
                        None, workspace_for(h, t))
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    ref, _ = orc.attention(sc.cfg, sc.layer(False), sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(out.cpu().numpy() - ref).max() <= TOL


@pytest.mark.parametrize("is_swa", [False, True])
def test_early_start_chain_next_to_foreign_kernels(is_swa):
    """Consecutive fused decodes through one handle may overlap (the later kernel streams its cache before the
    earlier one has finished).  Between two such calls this test (a) runs a foreign kernel that rewrites the NEXT
    layer's q / k_new / v_new (legal: the library waits before touching those) and (b) calls the same layer twice in
    a row (the second call must not start early on the pool the first one appends to).  Every result is compared
    with the oracle replaying the same sequence."""
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    sc = build_scenario(d, [700, 130, 5000, 64], [1] * 4, seed=46)
    t = sc.tables
    h = make_handle(d)
    pools = [to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool) for _ in range(3)]
    layers = [hb.Layer(p, is_swa) for p in pools]
    b = dev_batch(t, True)
    ws = workspace_for(h, t)
    q_src, k_src, v_src = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    q, k, v = torch.zeros_like(q_src), torch.zeros_like(k_src), torch.zeros_like(v_src)
    outs = [torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda") for _ in range(4)]
    scales = [1.0, 0.5, 2.0]
    for i in range(3):
        # foreign kernels between two library calls: the next layer's inputs are produced late, on the same stream
        q.copy_(q_src * scales[i])
        k.copy_(k_src * scales[i])
        v.copy_(v_src * scales[i])
        hb.hswa_decode_attn(h, layers[i], b, q, k, v, outs[i], None, ws)
    # same layer again, right behind its own fused decode, reading the row that call appended
    hb.hswa_decode_attn(h, layers[2], b, q, None, None, outs[3], None, ws)
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    for i in range(3):
        scaled = [to_host_bits((x * scales[i]).contiguous()) for x in (q_src, k_src, v_src)]
        ol = sc.layer(is_swa)
        ref, _ = orc.attention(sc.cfg, ol, sc.batch(), *scaled)
        assert np.abs(outs[i].cpu().numpy() - ref).max() <= TOL, i
        orc.kv_append(sc.cfg, ol, sc.batch(), scaled[1], scaled[2])
        assert np.array_equal(to_host_bits(pools[i]), ol.pool), i
    assert np.abs(outs[3].cpu().numpy() - ref).max() <= TOL   # append-then-attend equals the fused call


def test_overlap_switched_off_allows_foreign_pool_writes():
    """With hswa_set_overlap(h, 0) every kernel waits for all earlier work on the stream, so a caller may fill the
    next layer's pool with its own kernel between two fused decode calls."""
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    sc = build_scenario(d, [700, 130, 5000, 64], [1] * 4, seed=47)
    t = sc.tables
    h = make_handle(d)
    hb.hswa_set_overlap(h, False)
    b = dev_batch(t, True)
    ws = workspace_for(h, t)
    q, k, v = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    for is_swa in (False, True):
        src = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
        first = hb.Layer(src.clone(), is_swa)
        second = hb.Layer(torch.zeros_like(src), is_swa)   # wrong contents until the foreign kernel below runs
        outs = [torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda") for _ in range(2)]
        hb.hswa_decode_attn(h, first, b, q, k, v, outs[0], None, ws)
        second.pool.copy_(src)                              # foreign kernel writes the next layer's pool
        hb.hswa_decode_attn(h, second, b, q, k, v, outs[1], None, ws)
        assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
        ol = sc.layer(is_swa)
        ref, _ = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
        orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
        for o, layer in zip(outs, (first, second)):
            assert np.abs(o.cpu().numpy() - ref).max() <= TOL
            assert np.array_equal(to_host_bits(layer.pool), ol.pool)
