"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on the same seeded
inputs.  Indexing and pool bytes must match bit for bit; attention outputs (fp32 output mode) within
1e-2 max abs error (bf16 inputs, fp32 accumulation)."""
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


def dims(G, D, P, Hkv=2, W=128):
    return wl.Dims(num_q_heads=G * Hkv, num_kv_heads=Hkv, head_dim=D, page_size=P, window=W)


def check_no_async_error(h):
    st = hb.hswa_get_async_error(h)
    assert st[0] == hb.HSWA_OK, st


# ---------------------------------------------------------------------------------------------------------
def run_append(sc, is_swa, decode):
    h = make_handle(sc.dims)
    pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
    layer = hb.Layer(pool, is_swa)
    hb.hswa_validate_batch(h, layer, dev_batch(sc.tables, decode))
    hb.hswa_kv_append(h, layer, dev_batch(sc.tables, decode), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new))
    check_no_async_error(h)
    ol = sc.layer(is_swa)
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    got = to_host_bits(pool)
    assert np.array_equal(got, ol.pool), "pool bytes differ after append"


@pytest.mark.parametrize("is_swa", [False, True])
def test_append_config1(is_swa):
    for kind in ("decode", "prefill"):
        w = wl.config1(kind)
        sc = build_scenario(w.dims, w.tables.ctx_len, w.tables.q_len, seed=1, scale=w.value_scale, ring_keep=w.dims.ring_slots)
        run_append(sc, is_swa, decode=False)
        if kind == "decode":
            run_append(sc, is_swa, decode=True)


@pytest.mark.parametrize("d", [dims(4, 64, 16, 1), dims(8, 128, 64), dims(2, 128, 32, 3)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_append_sweep(d, is_swa):
    C, P = d.ring_slots, d.page_size
    ctx = [0, 1, P - 1, P, C - 1, C + 1, 3 * C + 5, 700]
    q_len = [2 * C + 3, 1, C, 17, 0, C + 1, 65, 300]
    sc = build_scenario(d, ctx, q_len, seed=5, ring_keep=C)
    run_append(sc, is_swa, decode=False)


# ---------------------------------------------------------------------------------------------------------
def run_decode(sc, is_swa, fused, out_dtype=torch.float32, check_pool=True):
    d, t = sc.dims, sc.tables
    h = make_handle(d, out_dtype, sc.cfg.sm_scale)
    pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
    layer = hb.Layer(pool, is_swa)
    b = dev_batch(t, decode=True)
    q, k_new, v_new = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    out = torch.full((t.batch, d.num_q_heads, d.head_dim), float("nan"), dtype=out_dtype, device="cuda")
    lse = torch.full((t.batch, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    ws = workspace_for(h, t)
    if fused:
        hb.hswa_decode_attn(h, layer, b, q, k_new, v_new, out, lse, ws)
    else:
        hb.hswa_kv_append(h, layer, b, k_new, v_new)
        hb.hswa_decode_attn(h, layer, b, q, None, None, out, lse, ws)
    check_no_async_error(h)
    ol = sc.layer(is_swa)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    got = out.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max() if t.batch else 0.0
    lerr = np.abs(lse.cpu().numpy() - ref_lse).max() if t.batch else 0.0
    assert np.isfinite(got).all()
    if check_pool:
        orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
        assert np.array_equal(to_host_bits(pool), ol.pool), "pool bytes differ after fused append"
    return err, lerr


@pytest.mark.parametrize("is_swa", [False, True])
@pytest.mark.parametrize("fused", [True, False])
def test_decode_config1(is_swa, fused):
    w = wl.config1("decode")
    sc = build_scenario(w.dims, w.tables.ctx_len, w.tables.q_len, seed=1, scale=w.value_scale)
    err, lerr = run_decode(sc, is_swa, fused)
    assert err <= TOL and lerr <= TOL, (err, lerr)


@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(4, 64, 16, 1)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_decode_ignores_nonfinite_stale_slots(d, is_swa):
    """Slots that hold no valid token (stale ring slots, page tails, unused pages) are filled with +inf (K) and
    NaN (V) instead of the finite poison: decode must neither read them into a score that counts nor let
    0 * NaN reach the output (Sec. 3.1.3: reading an invalid slot degrades correctness)."""
    W, C = d.window, d.ring_slots
    ctx = [0, 1, 5, 63, 64, 100, W - 1, W, W + 1, C, C + 7, 1000, 2049]
    sc = build_scenario(d, ctx, [1] * len(ctx), seed=91)
    poison_dead_slots_nonfinite(sc)
    for fused in (True, False):
        err, lerr = run_decode(sc, is_swa, fused)
        assert err <= TOL and lerr <= TOL, (fused, err, lerr)


@pytest.mark.parametrize("d", [dims(4, 64, 16, 1), dims(8, 128, 64), dims(1, 128, 64, 3), dims(3, 64, 32),
                               dims(8, 128, 16), dims(5, 64, 64)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_decode_sweep(d, is_swa):
    W, P, C = d.window, d.page_size, d.ring_slots
    ctx = sorted({0, 1, 2, 62, 63, 64, 65, W - 2, W - 1, W, W + 1, P - 1, P, P + 1, C - 1, C, C + 1, 3 * C + 5,
                  255, 256, 257, 2047, 2048, 2049, 5000})
    sc = build_scenario(d, ctx, [1] * len(ctx), seed=7)
    for fused in (True, False):
        err, lerr = run_decode(sc, is_swa, fused)
        assert err <= TOL and lerr <= TOL, (fused, err, lerr)


@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(4, 64, 16, 1), dims(3, 64, 32, 2, W=33), dims(5, 128, 32, 3, W=100),
                               dims(8, 128, 16, 2, W=128)], ids=str)
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("n_per_sm", [3, 4], ids=["over3", "over4"])
def test_decode_swa_many_rings(d, out_dtype, n_per_sm):
    """SWA decode on batches with more rings than three (four) per SM: the compact single-token kernel serves them --
    between three and four per SM at head_dim 128 in its form with four blocks per SM, whose late V granules take the K
    area -- and some of its blocks walk a second ring.  Contexts cross every window / page / ring boundary, ring heads
    are random, every dead slot holds +inf / NaN; with and without the fused append; fp32 and bf16 output (the bf16
    result is the fp32 one rounded once: half a bf16 ulp on top of the bar)."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    B = (n_per_sm * sms + 40 + d.num_kv_heads - 1) // d.num_kv_heads
    W, P, C = d.window, d.page_size, d.ring_slots
    base = [0, 1, 2, 15, 16, 17, W - 2, W - 1, W, W + 1, P - 1, P, P + 1, C - 1, C, C + 1, 2 * C + 5, 300, 517]
    ctx = [base[i % len(base)] + (i // len(base)) % 3 for i in range(B)]
    sc = build_scenario(d, ctx, [1] * B, seed=23)
    poison_dead_slots_nonfinite(sc)
    tol = TOL if out_dtype == torch.float32 else 2 * TOL
    for fused in (True, False):
        err, lerr = run_decode(sc, True, fused, out_dtype=out_dtype)
        assert err <= tol and lerr <= TOL, (fused, err, lerr)


def test_decode_long_split_and_bf16_out():
    d = dims(8, 128, 64, 2)
    sc = build_scenario(d, [40000, 9000, 33, 20481], [1, 1, 1, 1], seed=9)
    err, lerr = run_decode(sc, False, True)
    assert err <= TOL and lerr <= TOL, (err, lerr)
    err, _ = run_decode(sc, False, True, out_dtype=torch.bfloat16)
    assert err <= TOL, err
    err, _ = run_decode(sc, True, True, out_dtype=torch.bfloat16)
    assert err <= TOL, err


def test_decode_large_values_and_shared_prefix():
    d = dims(8, 128, 64, 2)
    sc = build_scenario(d, [64 * 5 + 3, 64 * 5 + 100, 64 * 9], [1, 1, 1], seed=10, shared_prefix_tokens=64 * 5)
    assert (sc.tables.block_table[:, :5] == sc.tables.block_table[0, :5]).all()
    for is_swa in (False, True):
        err, lerr = run_decode(sc, is_swa, True)
        assert err <= TOL and lerr <= TOL, (err, lerr)


def test_decode_page_permutation_bit_identical():
    d = dims(8, 128, 64, 2)
    outs = []
    for permute in (True, False):
        sc = build_scenario(d, [5000, 300, 2049], [1, 1, 1], seed=11, permute=permute,
                            ring_head=np.array([5, 100, 191]))
        h = make_handle(d)
        t = sc.tables
        res = []
        for is_swa in (False, True):
            layer = hb.Layer(to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool), is_swa)
            out = torch.zeros((t.batch, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
            hb.hswa_decode_attn(h, layer, dev_batch(t, True), to_dev_bf16(sc.q), to_dev_bf16(sc.k_new),
                                to_dev_bf16(sc.v_new), out, None, workspace_for(h, t))
            res.append(out.cpu())
        outs.append(res)
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


# ---------------------------------------------------------------------------------------------------------
def poison_dead_slots_nonfinite(sc):
    """Every slot of both pools that holds no token (its whole row still carries the finite poison the scenario was
    built with) gets +inf in K and NaN in V.  Whole rows only: a valid row may contain an element whose bits happen
    to equal the poison's."""
    from helpers import POISON_K, POISON_V
    pk, pv = wl.bf16_bits_const(POISON_K, (1,))[0], wl.bf16_bits_const(POISON_V, (1,))[0]
    for pool in (sc.full_pool, sc.swa_pool):
        dead_k = (pool[:, 0] == pk).all(axis=-1)
        dead_v = (pool[:, 1] == pv).all(axis=-1)
        assert dead_k.any() and dead_v.any()
        pool[:, 0][dead_k] = 0x7F80  # +inf
        pool[:, 1][dead_v] = 0x7FC0  # NaN


def run_prefill(sc, is_swa, fuse_append=True, out_dtype=torch.float32, arrays=False):
    d, t = sc.dims, sc.tables
    h = make_handle(d, out_dtype, sc.cfg.sm_scale)
    pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
    layer = hb.Layer(pool, is_swa)
    b = dev_batch(t, decode=False)
    q, k_new, v_new = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    out = torch.full((t.total_q, d.num_q_heads, d.head_dim), float("nan"), dtype=out_dtype, device="cuda")
    lse = torch.full((t.total_q, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    hb.hswa_prefill_attn(h, layer, b, q, k_new, v_new, fuse_append, out, lse, workspace_for(h, t))
    check_no_async_error(h)
    ol = sc.layer(is_swa)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    if fuse_append:
        orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(to_host_bits(pool), ol.pool), "pool bytes differ after prefill"
    if arrays:
        return got, ref, np.abs(lse.cpu().numpy() - ref_lse).max()
    return np.abs(got - ref).max(), np.abs(lse.cpu().numpy() - ref_lse).max()


@pytest.mark.parametrize("is_swa", [False, True])
@pytest.mark.parametrize("fuse_append", [True, False])
def test_prefill_config1(is_swa, fuse_append):
    w = wl.config1("prefill")
    sc = build_scenario(w.dims, w.tables.ctx_len, w.tables.q_len, seed=1, scale=w.value_scale)
    err, lerr = run_prefill(sc, is_swa, fuse_append)
    assert err <= TOL and lerr <= TOL, (err, lerr)


@pytest.mark.parametrize("d", [dims(4, 64, 16, 1), dims(8, 128, 64), dims(2, 128, 32, 3), dims(1, 64, 64)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_prefill_sweep(d, is_swa):
    C, P, W = d.ring_slots, d.page_size, d.window
    ctx = [0, 1, W - 1, W, P + 1, C - 1, 3 * C + 5, 700, 0, 130]
    q_len = [2 * C + 3, 1, 64, 65, 17, C + 1, 66, 300, 129, 0]
    sc = build_scenario(d, ctx, q_len, seed=13)
    err, lerr = run_prefill(sc, is_swa)
    assert err <= TOL and lerr <= TOL, (err, lerr)


def test_prefill_wrong_order_on_ring_is_detected():
    """Contract guard: appending a long chunk to a ring BEFORE attending loses keys the chunk's first queries
    need, so the library's attend-then-append order is the only valid one on SWA layers."""
    d = dims(4, 64, 16, 1)
    sc = build_scenario(d, [512], [64], seed=14, ring_keep=d.ring_slots)
    t = sc.tables
    h = make_handle(d)
    pool = to_dev_bf16(sc.swa_pool)
    layer = hb.Layer(pool, True)
    b = dev_batch(t, decode=False)
    q, k_new, v_new = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    hb.hswa_kv_append(h, layer, b, k_new, v_new)          # wrong: append first
    out = torch.zeros((t.total_q, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_prefill_attn(h, layer, b, q, k_new, v_new, False, out, None, None)
    ref, _ = orc.attention(sc.cfg, sc.layer(True), sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(out.cpu().numpy() - ref).max() > TOL


# ---------------------------------------------------------------------------------------------------------
def test_step_advance_matches_oracle():
    d = dims(8, 128, 64)
    t = wl.make_tables(d, [0, 5, 1000, 191], [1, 200, 64, 7], seed=3)
    h = make_handle(d)
    for q_indptr in (t.q_indptr, None):
        ctx, head = dev_i32(t.ctx_len), dev_i32(t.ring_head)
        hb.hswa_step_advance(h, t.batch, ctx, head, None if q_indptr is None else dev_i32(q_indptr))
        ectx, ehead = t.ctx_len.copy(), t.ring_head.copy()
        orc.step_advance(orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size), ectx, ehead, q_indptr)
        assert np.array_equal(ctx.cpu().numpy(), ectx) and np.array_equal(head.cpu().numpy(), ehead)


def test_multi_step_decode_history():
    """Prefill a prompt, then decode several tokens with fused append and step advance; every step must match
    the oracle run on the same evolving state (ring wraps included)."""
    d = dims(4, 64, 16, 1)
    sc = build_scenario(d, [0, 37], [150, 120], seed=15)
    t = sc.tables
    h = make_handle(d)
    steps = 40
    big_t = wl.make_tables(d, [0, 37], [150 + steps, 120 + steps], seed=15, ring_head=t.ring_head)
    # device state (block table sized for the whole history)
    pools = {False: to_dev_bf16(np.resize(sc.full_pool, (big_t.num_full_pages,) + sc.full_pool.shape[1:])),
             True: to_dev_bf16(sc.swa_pool)}
    o_pools = {False: np.resize(sc.full_pool, (big_t.num_full_pages,) + sc.full_pool.shape[1:]).copy(),
               True: sc.swa_pool.copy()}
    # history already present in sc pools was placed with sc.tables' block table: rebuild with big_t instead
    sc2 = build_scenario(d, [0, 37], [150, 120], seed=15, ring_head=t.ring_head)
    bt = big_t.block_table
    ctx = dev_i32(t.ctx_len)
    head = dev_i32(t.ring_head)
    octx, ohead = t.ctx_len.copy(), t.ring_head.copy()
    # place the 37-token history of request 1 through the library itself (append on both layers)
    hist_b = hb.Batch(dev_i32([0, 0]), dev_i32(bt), dev_i32(big_t.ring_table), dev_i32(np.mod(t.ring_head - t.ctx_len, d.ring_slots)),
                      dev_i32([0, 0, 37]), max_q_len=37, total_q=37, max_ctx_len=0)
    hk, hv = sc2.k_seq[1][:37], sc2.v_seq[1][:37]
    ohist = orc.OracleBatch(np.zeros(2, np.int32), bt, big_t.ring_table, np.mod(t.ring_head - t.ctx_len, d.ring_slots),
                            np.array([0, 0, 37], np.int32))
    for is_swa in (False, True):
        pools[is_swa].view(torch.int16).fill_(0)
        o_pools[is_swa][:] = 0
        hb.hswa_kv_append(h, hb.Layer(pools[is_swa], is_swa), hist_b, to_dev_bf16(hk), to_dev_bf16(hv))
        orc.kv_append(sc2.cfg, orc.OracleLayer(o_pools[is_swa], is_swa), ohist, hk, hv)
    # step 0: prefill
    qi = t.q_indptr
    for step in range(steps + 1):
        if step == 0:
            q_bits, k_bits, v_bits, q_indptr = sc2.q, sc2.k_new, sc2.v_new, qi
        else:
            q_bits = wl.bf16_bits_normal(1000 + step, (2, d.num_q_heads, d.head_dim))
            k_bits = wl.bf16_bits_normal(2000 + step, (2, d.num_kv_heads, d.head_dim))
            v_bits = wl.bf16_bits_normal(3000 + step, (2, d.num_kv_heads, d.head_dim))
            q_indptr = None
        T = q_bits.shape[0]
        ob = orc.OracleBatch(octx.copy(), bt, big_t.ring_table, ohead.copy(), q_indptr)
        gb = hb.Batch(ctx, dev_i32(bt), dev_i32(big_t.ring_table), head, None if q_indptr is None else dev_i32(q_indptr),
                      max_q_len=150 if step == 0 else 1, total_q=T, max_ctx_len=int(octx.max()))
        for is_swa in (False, True):
            layer = hb.Layer(pools[is_swa], is_swa)
            out = torch.zeros((T, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
            ws = torch.empty(hb.hswa_workspace_bytes(h, 2, T, 400) + 256, dtype=torch.uint8, device="cuda")
            if step == 0:
                hb.hswa_prefill_attn(h, layer, gb, to_dev_bf16(q_bits), to_dev_bf16(k_bits), to_dev_bf16(v_bits), True, out, None, ws)
            else:
                hb.hswa_decode_attn(h, layer, gb, to_dev_bf16(q_bits), to_dev_bf16(k_bits), to_dev_bf16(v_bits), out, None, ws)
            ol = orc.OracleLayer(o_pools[is_swa], is_swa)
            ref, _ = orc.attention(sc2.cfg, ol, ob, q_bits, k_bits, v_bits)
            orc.kv_append(sc2.cfg, ol, ob, k_bits, v_bits)
            assert np.abs(out.cpu().numpy() - ref).max() <= TOL, (step, is_swa)
            assert np.array_equal(to_host_bits(pools[is_swa]), o_pools[is_swa]), (step, is_swa)
        hb.hswa_step_advance(h, 2, ctx, head, None if q_indptr is None else dev_i32(q_indptr))
        orc.step_advance(sc2.cfg, octx, ohead, q_indptr)
        assert np.array_equal(ctx.cpu().numpy(), octx) and np.array_equal(head.cpu().numpy(), ohead)
    check_no_async_error(h)


# ---------------------------------------------------------------------------------------------------------
def test_validate_batch_reports_bad_ids():
    d = dims(8, 128, 64)
    sc = build_scenario(d, [300, 70], [1, 1], seed=16)
    t = sc.tables
    h = make_handle(d)
    full = hb.Layer(to_dev_bf16(sc.full_pool), False)
    swa = hb.Layer(to_dev_bf16(sc.swa_pool), True)
    hb.hswa_validate_batch(h, full, dev_batch(t, True))
    hb.hswa_validate_batch(h, swa, dev_batch(t, True))
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    # corrupt the HOST copy of the block table, then validate: the error word names request and entry
    bad = t.block_table.copy()
    bad[1, 0] = t.num_full_pages + 7
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(bad), dev_i32(t.ring_table), dev_i32(t.ring_head), max_ctx_len=300)
    hb.hswa_validate_batch(h, full, b)
    st = hb.hswa_get_async_error(h)
    assert st == (hb.HSWA_ERR_BOUNDS, 1, 0, t.num_full_pages + 7), st
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK  # cleared
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32([0, d.ring_slots]), max_ctx_len=300)
    hb.hswa_validate_batch(h, swa, b)
    st = hb.hswa_get_async_error(h)
    assert st[0] == hb.HSWA_ERR_BOUNDS and st[1] == 1, st
    # a decode over the corrupted table skips the bad page, records the error and returns
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(bad), dev_i32(t.ring_table), dev_i32(t.ring_head), max_ctx_len=300)
    out = torch.zeros((2, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_decode_attn(h, full, b, to_dev_bf16(sc.q), None, None, out, None, workspace_for(h, t))
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_ERR_BOUNDS
    # an append over a corrupted table records the error, skips that row and writes every other row
    bad = t.block_table.copy()
    bad[1, 70 // d.page_size] = -5   # request 1's new token (position 70) lands in this entry
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(bad), dev_i32(t.ring_table), dev_i32(t.ring_head), max_ctx_len=300)
    k_new, v_new = to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    before = to_host_bits(full.pool)
    hb.hswa_kv_append(h, full, b, k_new, v_new)
    st = hb.hswa_get_async_error(h)
    assert st == (hb.HSWA_ERR_BOUNDS, 1, 70 // d.page_size, -5), st
    ol = orc.OracleLayer(before.copy(), False)
    only0 = orc.OracleBatch(t.ctx_len[:1], t.block_table[:1], t.ring_table[:1], t.ring_head[:1])
    orc.kv_append(sc.cfg, ol, only0, sc.k_new[:1], sc.v_new[:1])
    assert np.array_equal(to_host_bits(full.pool), ol.pool)   # request 0 appended, request 1 skipped, nothing else touched
    bad_ring = t.ring_table.copy()
    bad_ring[0, :] = t.num_ring_pages + 3
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(bad_ring), dev_i32(t.ring_head), max_ctx_len=300)
    before = to_host_bits(swa.pool)
    hb.hswa_kv_append(h, swa, b, k_new, v_new)
    st = hb.hswa_get_async_error(h)
    assert st[0] == hb.HSWA_ERR_BOUNDS and st[1] == 0 and st[3] == t.num_ring_pages + 3, st
    ol = orc.OracleLayer(before.copy(), True)
    only1 = orc.OracleBatch(t.ctx_len[1:], t.block_table[1:], t.ring_table[1:], t.ring_head[1:])
    orc.kv_append(sc.cfg, ol, only1, sc.k_new[1:], sc.v_new[1:])
    assert np.array_equal(to_host_bits(swa.pool), ol.pool)
    # a length above the host bound the launch was planned for is reported, by the validator and by the decode kernel
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), max_ctx_len=200)
    hb.hswa_validate_batch(h, full, b)
    assert hb.hswa_get_async_error(h) == (hb.HSWA_ERR_BOUNDS, 0, -1, 300)
    hb.hswa_decode_attn(h, full, b, to_dev_bf16(sc.q), None, None, out, None, workspace_for(h, t))
    assert hb.hswa_get_async_error(h) == (hb.HSWA_ERR_BOUNDS, 0, -1, 300)


def test_host_side_argument_errors():
    d = dims(8, 128, 64)
    sc = build_scenario(d, [5000, 70], [1, 1], seed=17)
    t = sc.tables
    h = make_handle(d)
    full = hb.Layer(to_dev_bf16(sc.full_pool), False)
    b = dev_batch(t, True)
    q = to_dev_bf16(sc.q)
    out = torch.zeros((2, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn(h, full, b, q, None, None, out, None, None)   # split-K needs a workspace
    assert e.value.status == hb.HSWA_ERR_WORKSPACE
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn(h, full, b, q, to_dev_bf16(sc.k_new), None, out, None, workspace_for(h, t))
    assert e.value.status == hb.HSWA_ERR_INVALID_ARG
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn(h, full, dev_batch(t, False), q, None, None, out, None, workspace_for(h, t))
    assert e.value.status == hb.HSWA_ERR_INVALID_ARG                     # decode takes no q_indptr
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_prefill_attn(h, full, dev_batch(t, False), q, None, None, True, out)
    assert e.value.status == hb.HSWA_ERR_INVALID_ARG                     # prefill needs k_new / v_new
    # empty batch is a no-op
    empty = hb.Batch(dev_i32(np.zeros(0)), dev_i32(np.zeros((0, 1))), dev_i32(np.zeros((0, 3))), dev_i32(np.zeros(0)),
                     max_q_len=1, total_q=0)
    hb.hswa_decode_attn(h, full, empty, q, None, None, out, None, None)
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)


# ---------------------------------------------------------------------------------------------------------
# tcgen05 prefill kernel (head_dim 128, page 64, even GQA group)
@pytest.mark.parametrize("case", ["one_tile", "two_tiles", "ctx_small", "ragged"])
@pytest.mark.parametrize("is_swa", [False, True])
def test_prefill_tc_small(case, is_swa):
    d = dims(2, 128, 64, 1)
    ctx, q_len = {"one_tile": ([0], [128]), "two_tiles": ([0], [256]), "ctx_small": ([70], [128]),
                  "ragged": ([0, 130, 64], [100, 129, 1])}[case]
    sc = build_scenario(d, ctx, q_len, seed=31)
    err, lerr = run_prefill(sc, is_swa)
    assert err <= TOL and lerr <= TOL, (err, lerr)


@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(2, 128, 64, 3), dims(4, 128, 64, 1)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_prefill_tc_sweep(d, is_swa):
    ctx = [0, 1, 63, 64, 65, 127, 128, 129, 191, 192, 193, 500, 5000]
    q_len = [300, 128, 129, 1, 127, 256, 64, 700, 0, 5, 130, 257, 400]
    sc = build_scenario(d, ctx, q_len, seed=32)
    got32, ref, lerr = run_prefill(sc, is_swa, arrays=True)
    assert np.abs(got32 - ref).max() <= TOL and lerr <= TOL, (np.abs(got32 - ref).max(), lerr)
    # bf16 output is the fp32 output rounded once (round to nearest even): same bits as rounding the fp32-mode result.
    # Against the oracle that is the fp32-mode error (<= 1e-2, just checked) plus at most half a bf16 ulp,
    # abs(out) * 2^-8 -- 0.0078 for a value of 2, which rows with 1-3 keys do reach -- and stays within 1e-2 outright
    # wherever the values are small.
    got16, _, _ = run_prefill(sc, is_swa, fuse_append=False, out_dtype=torch.bfloat16, arrays=True)
    want16 = torch.from_numpy(got32.astype(np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)
    assert np.array_equal(got16, want16)
    err = np.abs(got16 - ref)
    assert (err <= TOL + np.abs(ref) * 2.0 ** -8).all()
    assert (err[np.abs(ref) < 0.5] <= TOL).all()


@pytest.mark.parametrize("W", [64, 96, 33])
@pytest.mark.parametrize("G", [8, 4, 2])
def test_prefill_tc_other_windows(W, G):
    """Windows other than the paper's 128: the streaming SWA kernel is bypassed and the packed / tile kernels
    must apply the general window mask."""
    d = dims(G, 128, 64, 1, W=W)
    ctx = [0, 1, W - 1, W, 200, 64]
    q_len = [300, 130, 257, 129, 1, 700]
    sc = build_scenario(d, ctx, q_len, seed=41 + W)
    err, lerr = run_prefill(sc, True)
    assert err <= TOL and lerr <= TOL, (err, lerr)
    err, lerr = run_decode(build_scenario(d, [0, 1, W - 1, W, 5 * W + 3], [1] * 5, seed=42 + W), True, True)
    assert err <= TOL and lerr <= TOL, (err, lerr)


def test_prefill_tc_long_context_and_many_requests():
    d = dims(8, 128, 64, 1)
    ctx = [20000, 0, 4097] + [int(x) for x in np.random.default_rng(7).integers(0, 700, 13)]
    q_len = [300, 2049, 128] + [int(x) for x in np.random.default_rng(8).integers(0, 400, 13)]
    sc = build_scenario(d, ctx, q_len, seed=43)
    for is_swa in (False, True):
        err, lerr = run_prefill(sc, is_swa)
        assert err <= TOL and lerr <= TOL, (is_swa, err, lerr)


@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(2, 128, 64, 3), dims(4, 64, 16, 1)], ids=str)
@pytest.mark.parametrize("is_swa", [False, True])
def test_prefill_ignores_nonfinite_dead_slots(d, is_swa):
    """As test_decode_ignores_nonfinite_stale_slots, for chunked prefill: slots that hold no token (page tails behind
    the cached context, ring slots never written or past the ring's last page, unused pages) hold +inf (K) and NaN
    (V).  Their probabilities are exactly 0, and 0 * NaN must not reach the output through the PV product either
    (Sec. 3.1.3).  Contexts that end inside a 128-key tile, inside a page, and rings that are not full yet."""
    W, C = d.window, d.ring_slots
    ctx = [0, 1, 5, 63, 64, 65, 100, W - 1, W, W + 1, C - 1, C, C + 7, 1000, 2049]
    q_len = [130, 64, 300, 129, 1, 128, 257, 70, 200, 16, 140, 131, 5, 260, 129]
    sc = build_scenario(d, ctx, q_len, seed=92)
    poison_dead_slots_nonfinite(sc)
    for fuse_append in (True, False):
        err, lerr = run_prefill(sc, is_swa, fuse_append)
        assert err <= TOL and lerr <= TOL, (fuse_append, err, lerr)


@pytest.mark.parametrize("case", ["many_short_streams", "one_long_stream", "two_long_streams", "fewer_units_than_sms"])
def test_prefill_swa_stream_walk(case):
    """The streaming SWA kernel (group of 8, W = 128) hands each persistent block a run of 16-token sub-tiles that may
    begin in the middle of one (request, KV head) stream, skip streams that have no token past the 128th, and end in
    another stream: mixes of chunk lengths that put several stream switches, many empty streams, or a single
    sub-tile into one block's run, with ragged last sub-tiles, against the oracle in both output types."""
    rng = np.random.default_rng(61)
    if case == "many_short_streams":      # one long request sets the stride of the unit space; the rest own 0-3 sub-tiles
        d = dims(8, 128, 64, 2)
        q_len = [3001] + [int(x) for x in rng.integers(100, 180, 63)]
    elif case == "one_long_stream":       # every block starts and ends inside the same stream
        d = dims(8, 128, 64, 1)
        q_len = [128 + 16 * 148 * 3 + 5]
    elif case == "two_long_streams":      # blocks in the middle of the grid cross from one KV head / request to the next
        d = dims(8, 128, 64, 2)
        q_len = [128 + 16 * 203 + 9, 128 + 16 * 77 + 16]
    else:                                 # fewer sub-tiles than SMs: one unit per block
        d = dims(8, 128, 64, 1)
        q_len = [129, 160, 145, 128, 7]
    ctx = [int(x) for x in rng.integers(0, 300, len(q_len))]
    sc = build_scenario(d, ctx, q_len, seed=62)
    got32, ref, lerr = run_prefill(sc, True, arrays=True)
    assert np.abs(got32 - ref).max() <= TOL and lerr <= TOL, (np.abs(got32 - ref).max(), lerr)
    got16, _, _ = run_prefill(sc, True, fuse_append=False, out_dtype=torch.bfloat16, arrays=True)
    want16 = torch.from_numpy(got32.astype(np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)
    assert np.array_equal(got16, want16)


# ---------------------------------------------------------------------------------------------------------
# cascade decode over a shared prefix
@pytest.mark.parametrize("G,Hkv,B,prefix_pages", [(8, 2, 40, 37), (8, 1, 5, 2), (8, 2, 33, 64), (4, 2, 6, 8)])
def test_decode_shared_prefix(G, Hkv, B, prefix_pages):
    d = dims(G, 128, 64, Hkv)
    prefix = 64 * prefix_pages
    rng = np.random.default_rng(50 + B)
    ctx = [prefix + int(x) for x in rng.integers(0, 700, B)]
    ctx[0] = prefix          # a request whose whole context is the shared prefix
    sc = build_scenario(d, ctx, [1] * B, seed=51, shared_prefix_tokens=prefix)
    t = sc.tables
    assert (t.block_table[:, :prefix_pages] == t.block_table[0, :prefix_pages]).all()
    h = make_handle(d)
    q, k_new, v_new = to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new)
    ws = workspace_for(h, t)
    for is_swa in (False, True):
        pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
        layer = hb.Layer(pool, is_swa)
        out = torch.full((B, d.num_q_heads, d.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((B, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        hb.hswa_decode_attn_shared_prefix(h, layer, dev_batch(t, True), prefix, q, k_new, v_new, out, lse, ws)
        check_no_async_error(h)
        ol = sc.layer(is_swa)
        ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= TOL and np.abs(lse.cpu().numpy() - ref_lse).max() <= TOL
        orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
        assert np.array_equal(to_host_bits(pool), ol.pool)
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn_shared_prefix(h, layer, dev_batch(t, True), 65, q, k_new, v_new, out, lse, ws)
    assert e.value.status == hb.HSWA_ERR_INVALID_ARG


# ---------------------------------------------------------------------------------------------------------
# multi-token (MTP) decode
@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(4, 64, 16, 1), dims(3, 128, 32)], ids=str)
@pytest.mark.parametrize("nq", [2, 4])
@pytest.mark.parametrize("is_swa", [False, True])
def test_decode_mtp(d, nq, is_swa):
    W, P, C = d.window, d.page_size, d.ring_slots
    ctx = sorted({0, 1, 63, 64, W - 2, W - 1, W, W + 1, P - 1, P, C - 1, C, C + 1, 3 * C + 5, 2047, 2048, 2049, 5000})
    B = len(ctx)
    sc = build_scenario(d, ctx, [nq] * B, seed=60 + nq, ring_keep=C)
    t = sc.tables
    h = make_handle(d)
    pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
    layer = hb.Layer(pool, is_swa)
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None, max_q_len=1,
                 total_q=B, max_ctx_len=t.max_ctx_len)
    out = torch.full((B * nq, d.num_q_heads, d.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B * nq, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(hb.hswa_workspace_bytes(h, B, B * nq, t.max_ctx_len + nq) + 256, dtype=torch.uint8, device="cuda")
    hb.hswa_decode_attn_mtp(h, layer, b, nq, to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new), out, lse, ws)
    check_no_async_error(h)
    ol = sc.layer(is_swa)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)   # oracle: q_indptr with nq per request
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL and np.abs(lse.cpu().numpy() - ref_lse).max() <= TOL
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(to_host_bits(pool), ol.pool)


@pytest.mark.parametrize("nq", [2, 3, 4])
def test_decode_mtp_tensor_core_walk(nq):
    """Full layers at the serving shape (group of 8, head_dim 128, page 64) take the tensor-core multi-token kernel:
    148 persistent blocks share the flat sequence of 128-key tiles evenly, so a block's slice starts and ends in the
    middle of (request, KV head) streams and holds several of them.  Contexts from 0 to 40 000 tokens, lengths that
    end on, just before and just behind tile and page boundaries (the new tokens then straddle two tiles), more
    requests than one 32-wide scan step, and every dead slot of the pool filled with +inf (K) / NaN (V): outputs
    and lse against the oracle, pool bytes after the append bit-exact."""
    d = dims(8, 128, 64, 2)
    rng = np.random.default_rng(70 + nq)
    ctx = [40000, 0, 1, 125, 126, 127, 128, 129, 254, 255, 256, 63, 64, 65, 8191, 8192, 8193, 16383, 20000, 3000] + \
          [int(x) for x in rng.integers(0, 6000, 20)]
    B = len(ctx)
    sc = build_scenario(d, ctx, [nq] * B, seed=71 + nq)
    poison_dead_slots_nonfinite(sc)
    t = sc.tables
    h = make_handle(d)
    pool = to_dev_bf16(sc.full_pool)
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None, max_q_len=1,
                 total_q=B, max_ctx_len=t.max_ctx_len)
    out = torch.full((B * nq, d.num_q_heads, d.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B * nq, d.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    need = hb.hswa_decode_workspace_need(h, False, B, t.max_ctx_len, 0, nq)
    assert 0 < need <= hb.hswa_workspace_bytes(h, B, B * nq, t.max_ctx_len + nq)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    hb.hswa_decode_attn_mtp(h, hb.Layer(pool, False), b, nq, to_dev_bf16(sc.q), to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new),
                            out, lse, ws)
    check_no_async_error(h)
    ol = sc.layer(False)
    ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL and np.abs(lse.cpu().numpy() - ref_lse).max() <= TOL
    orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
    assert np.array_equal(to_host_bits(pool), ol.pool)
    # one byte less of workspace than the stated need is refused on the host
    short = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(hb.HswaError) as e:
        hb.hswa_decode_attn_mtp(h, hb.Layer(pool, False), b, nq, to_dev_bf16(sc.q), to_dev_bf16(sc.k_new),
                                to_dev_bf16(sc.v_new), out, lse, short)
    assert e.value.status == hb.HSWA_ERR_WORKSPACE


# ---------------------------------------------------------------------------------------------------------
# window-only data movement for SWA prefix reuse
@pytest.mark.parametrize("d", [dims(8, 128, 64), dims(4, 64, 16, 1), dims(2, 128, 32, 3, W=33)], ids=str)
@pytest.mark.parametrize("host_buf", [False, True])
def test_window_gather_scatter(d, host_buf):
    W, C = d.window, d.ring_slots
    ctx = [0, 1, W - 2, W - 1, W, C - 1, C + 1, 3 * C + 5]
    B = len(ctx)
    donor = build_scenario(d, ctx, [1] * B, seed=70)
    h = make_handle(d)
    layer = hb.Layer(to_dev_bf16(donor.swa_pool), True)
    shape = (B, W - 1, 2, d.num_kv_heads, d.head_dim)
    buf = torch.full(shape, 7.0, dtype=torch.bfloat16)
    buf = buf.pin_memory() if host_buf else buf.cuda()
    hb.hswa_swa_window_gather(h, layer, dev_batch(donor.tables, True), buf)
    check_no_async_error(h)
    ref = orc.window_gather(donor.cfg, donor.layer(True), donor.batch())
    assert np.array_equal(to_host_bits(buf.cuda()), ref)
    # seed fresh rings (other pages, other heads) from the buffer: pool bytes must equal the oracle's scatter
    fresh = wl.make_tables(d, ctx, [1] * B, seed=71)
    from helpers import poison_pool
    dst_pool = to_dev_bf16(poison_pool(fresh.num_ring_pages, d))
    dst = hb.Layer(dst_pool, True)
    hb.hswa_swa_window_scatter(h, dst, dev_batch(fresh, True), buf)
    check_no_async_error(h)
    odst = orc.OracleLayer(poison_pool(fresh.num_ring_pages, d), True)
    ob = orc.OracleBatch(fresh.ctx_len, fresh.block_table, fresh.ring_table, fresh.ring_head)
    orc.window_scatter(donor.cfg, odst, ob, ref)
    assert np.array_equal(to_host_bits(dst_pool), odst.pool)
    # a decode step on the seeded rings reproduces the donor's output
    out = torch.zeros((B, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_decode_attn(h, dst, dev_batch(fresh, True), to_dev_bf16(donor.q), to_dev_bf16(donor.k_new), to_dev_bf16(donor.v_new),
                        out, None, None)
    want, _ = orc.attention(donor.cfg, donor.layer(True), donor.batch(), donor.q, donor.k_new, donor.v_new)
    assert np.abs(out.cpu().numpy() - want).max() <= TOL
    with pytest.raises(hb.HswaError):
        hb.hswa_swa_window_gather(h, hb.Layer(to_dev_bf16(donor.full_pool), False), dev_batch(donor.tables, True), buf)


# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_stress(seed):
    """Seeded random shapes, lengths and layer kinds through prefill, decode, multi-token decode and cascade."""
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    P = int(rng.choice([16, 32, 64]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    W = int(rng.choice([128, 128, 128, 64, 17]))
    d = dims(G, D, P, Hkv, W=W)
    B = int(rng.integers(1, 9))
    big = rng.random() < 0.3
    ctx = [int(x) for x in rng.integers(0, 6000 if big else 700, B)]
    is_swa = bool(rng.integers(0, 2))
    kind = rng.choice(["prefill", "decode", "mtp", "cascade"])
    if kind == "prefill":
        q_len = [int(x) for x in rng.integers(0, 500, B)]
        if sum(q_len) == 0:
            q_len[0] = 1
        sc = build_scenario(d, ctx, q_len, seed=seed)
        err, lerr = run_prefill(sc, is_swa)
    elif kind == "decode":
        sc = build_scenario(d, ctx, [1] * B, seed=seed)
        err, lerr = run_decode(sc, is_swa, bool(rng.integers(0, 2)))
    elif kind == "mtp":
        nq = int(rng.integers(2, 5))
        if is_swa and nq > d.ring_slots - W + 1:
            nq = 2
        sc = build_scenario(d, ctx, [nq] * B, seed=seed, ring_keep=d.ring_slots)
        t = sc.tables
        h = make_handle(d)
        pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
        b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None,
                     max_q_len=1, total_q=B, max_ctx_len=t.max_ctx_len)
        out = torch.zeros((B * nq, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
        lse = torch.zeros((B * nq, d.num_q_heads), dtype=torch.float32, device="cuda")
        ws = torch.empty(hb.hswa_workspace_bytes(h, B, B * nq, t.max_ctx_len + nq) + 256, dtype=torch.uint8, device="cuda")
        hb.hswa_decode_attn_mtp(h, hb.Layer(pool, is_swa), b, nq, to_dev_bf16(sc.q), to_dev_bf16(sc.k_new),
                                to_dev_bf16(sc.v_new), out, lse, ws)
        check_no_async_error(h)
        ol = sc.layer(is_swa)
        ref, ref_lse = orc.attention(sc.cfg, ol, sc.batch(), sc.q, sc.k_new, sc.v_new)
        orc.kv_append(sc.cfg, ol, sc.batch(), sc.k_new, sc.v_new)
        assert np.array_equal(to_host_bits(pool), ol.pool)
        err, lerr = np.abs(out.cpu().numpy() - ref).max(), np.abs(lse.cpu().numpy() - ref_lse).max()
    else:
        prefix = P * int(rng.integers(1, 12))
        ctx = [prefix + c for c in ctx]
        sc = build_scenario(d, ctx, [1] * B, seed=seed, shared_prefix_tokens=prefix)
        t = sc.tables
        h = make_handle(d)
        pool = to_dev_bf16(sc.swa_pool if is_swa else sc.full_pool)
        out = torch.zeros((B, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
        lse = torch.zeros((B, d.num_q_heads), dtype=torch.float32, device="cuda")
        hb.hswa_decode_attn_shared_prefix(h, hb.Layer(pool, is_swa), dev_batch(t, True), prefix, to_dev_bf16(sc.q),
                                          to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new), out, lse, workspace_for(h, t))
        check_no_async_error(h)
        ref, ref_lse = orc.attention(sc.cfg, sc.layer(is_swa), sc.batch(), sc.q, sc.k_new, sc.v_new)
        err, lerr = np.abs(out.cpu().numpy() - ref).max(), np.abs(lse.cpu().numpy() - ref_lse).max()
    assert err <= TOL and lerr <= TOL, (kind, d, is_swa, err, lerr)


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_many_rings_swa_decode(seed):
    """Seeded random shapes with more rings than two, three or four per SM (the regimes of the compact single-token
    ring kernel and its form with four blocks per SM): random window up to 128, page size, group size, head count,
    ring heads and a mix of short and long contexts, every dead slot filled with +inf / NaN."""
    rng = np.random.default_rng(7000 + seed)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    D = int(rng.choice([64, 128]))
    P = int(rng.choice([16, 32, 64]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 4]))
    W = int(rng.choice([128, 128, 100, 64, 17]))
    d = dims(G, D, P, Hkv, W=W)
    per_sm = float(rng.choice([2.2, 3.3, 4.4]))
    B = int(per_sm * sms / Hkv) + 1
    ctx = [int(x) for x in np.where(rng.random(B) < 0.5, rng.integers(0, W + 3, B), rng.integers(W, 900, B))]
    sc = build_scenario(d, ctx, [1] * B, seed=seed)
    poison_dead_slots_nonfinite(sc)
    err, lerr = run_decode(sc, True, bool(rng.integers(0, 2)))
    assert err <= TOL and lerr <= TOL, (d, B, err, lerr)


@pytest.mark.parametrize("sm_scale", [1.0, 3.0])
def test_peaked_softmax_exercises_lazy_rescale(sm_scale):
    """Large score scale: row maxima keep growing from tile to tile by more than the 2^8 slack of the lazy
    rescale, so the O-rescale path of the tcgen05 kernels (and the split combine with far-apart maxima) runs."""
    d = dims(8, 128, 64, 1)
    sc = build_scenario(d, [3000, 0, 777], [300, 520, 129], seed=81, sm_scale=sm_scale)
    # Nearly one-hot rows: the weight of the dominant key is rounded to bf16 before the PV product (2^-9 relative)
    # while the row sum keeps fp32, and the output is rounded to bf16 once more; neither averages out over keys
    # here, so the bound is 2^-8 max|v| instead of the 1e-2 that holds at the model's 1/sqrt(D) scale.
    vmax = float(np.abs(wl.bits_to_f64(sc.full_pool[:, 1])).max())
    tol = max(TOL, 2.0 ** -8 * max(vmax, float(np.abs(wl.bits_to_f64(sc.v_new)).max())))
    for is_swa in (False, True):
        err, lerr = run_prefill(sc, is_swa)
        assert err <= tol and lerr <= 2 * TOL * max(1.0, sm_scale), (is_swa, err, lerr, tol)
    prefix = 64 * 40
    sc = build_scenario(d, [prefix + 5, prefix + 2100, prefix], [1, 1, 1], seed=82, sm_scale=sm_scale, shared_prefix_tokens=prefix)
    t = sc.tables
    h = make_handle(d, sm_scale=sm_scale)
    out = torch.zeros((3, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
    hb.hswa_decode_attn_shared_prefix(h, hb.Layer(to_dev_bf16(sc.full_pool), False), dev_batch(t, True), prefix, to_dev_bf16(sc.q),
                                      to_dev_bf16(sc.k_new), to_dev_bf16(sc.v_new), out, None, workspace_for(h, t))
    check_no_async_error(h)
    ref, _ = orc.attention(sc.cfg, sc.layer(False), sc.batch(), sc.q, sc.k_new, sc.v_new)
    assert np.abs(out.cpu().numpy() - ref).max() <= TOL
    err, lerr = run_decode(build_scenario(d, [9000, 130], [1, 1], seed=83, sm_scale=sm_scale), False, True)
    assert err <= TOL, err
