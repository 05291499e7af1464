"""GPU parity of the SWA-aware prefix reuse path (paper Sec. 3.1.3 items 1-3, Sec. 3.1.1 data movement, Sec. 3.1.2
layerwise loadback): two donor requests live through prefill chunks and decode steps with out-of-window releases;
their per-position SWA status then clips a new request's hit to the window-safe length; the window is gathered
from the donor's ring, scattered into a fresh ring, and the new request's first decode step on shared Full pages
and the seeded ring is compared with the oracle replaying the same chain.  Every integer (boundaries, masks, hit
lengths, pool bytes) must match exactly, outputs within 1e-2."""
import numpy as np
import pytest
import torch

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import binding as hb
from paper_2607_13095_b200 import workloads as wl
from helpers import oracle_config, poison_pool
from gpu_utils import dev_i32, make_handle, to_dev_bf16, to_host_bits

pytestmark = pytest.mark.gpu
TOL = 1e-2


def rand_bits(seed, shape):
    return wl.bf16_bits_normal(seed, shape)


@pytest.mark.parametrize("d,every_n", [(wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64), 16),
                                       (wl.Dims(num_q_heads=4, num_kv_heads=1, head_dim=64, page_size=16), 5)], ids=["big", "tiny"])
def test_release_then_window_safe_hit_then_seeded_decode(d, every_n):
    W, P, C = d.window, d.page_size, d.ring_slots
    cfg = oracle_config(d)
    h = make_handle(d)
    B = 2
    chunks = [[300, 250], [131]]            # prefill chunks per donor
    n_decode = [37, 2 * C + 3]              # decode tokens per donor (the second wraps its ring twice)
    total = [sum(c) + n for c, n in zip(chunks, n_decode)]
    t = wl.make_tables(d, [0, 0], total, seed=81)
    k_seq = [rand_bits(810 + r, (total[r], d.num_kv_heads, d.head_dim)) for r in range(B)]
    v_seq = [rand_bits(820 + r, (total[r], d.num_kv_heads, d.head_dim)) for r in range(B)]
    pools = {s: to_dev_bf16(poison_pool(t.num_ring_pages if s else t.num_full_pages, d)) for s in (False, True)}
    o_pools = {s: poison_pool(t.num_ring_pages if s else t.num_full_pages, d) for s in (False, True)}
    layers = {s: hb.Layer(pools[s], s) for s in (False, True)}
    bt, rt = dev_i32(t.block_table), dev_i32(t.ring_table)
    ctx, head = dev_i32([0, 0]), dev_i32(t.ring_head)
    valid_from = dev_i32([0, 0])
    octx, ohead, ofrom = np.zeros(B, np.int32), t.ring_head.copy(), np.zeros(B, np.int32)
    ws = torch.empty(hb.hswa_workspace_bytes(h, B, B, max(total)) + 256, dtype=torch.uint8, device="cuda")

    # the life of the donors: one request per step keeps the bookkeeping simple (the other has 0 new tokens)
    events = []
    for r in range(B):
        events += [("chunk", r, n) for n in chunks[r]]
    for i in range(max(n_decode)):
        events.append(("decode", None, i))
    decoded = np.zeros(B, np.int64)
    for kind, who, arg in events:
        if kind == "chunk":
            n = np.zeros(B, np.int64)
            n[who] = arg
        else:
            n = np.array([1 if arg < n_decode[r] else 0 for r in range(B)], np.int64)
            decoded += n
        q_indptr = np.zeros(B + 1, np.int32)
        q_indptr[1:] = np.cumsum(n)
        T = int(q_indptr[-1])
        k_new = np.concatenate([k_seq[r][octx[r]: octx[r] + n[r]] for r in range(B)])
        v_new = np.concatenate([v_seq[r][octx[r]: octx[r] + n[r]] for r in range(B)])
        q = rand_bits(830 + len(events) + int(octx.sum()), (T, d.num_q_heads, d.head_dim))
        gb = hb.Batch(ctx, bt, rt, head, dev_i32(q_indptr), max_q_len=int(n.max()), total_q=T, max_ctx_len=int(octx.max()))
        ob = orc.OracleBatch(octx.copy(), t.block_table, t.ring_table, ohead.copy(), q_indptr)
        for s in (False, True):
            out = torch.zeros((T, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
            hb.hswa_prefill_attn(h, layers[s], gb, to_dev_bf16(q), to_dev_bf16(k_new), to_dev_bf16(v_new), True, out, None, ws)
            ol = orc.OracleLayer(o_pools[s], s)
            ref, _ = orc.attention(cfg, ol, ob, q, k_new, v_new)
            orc.kv_append(cfg, ol, ob, k_new, v_new)
            assert np.abs(out.cpu().numpy() - ref).max() <= TOL, (kind, who, arg, s)
        hb.hswa_step_advance(h, B, ctx, head, dev_i32(q_indptr))
        orc.step_advance(cfg, octx, ohead, q_indptr)
        # release policy (the scheduler's): a chunk end releases; in decode every every_n generated tokens
        if kind == "chunk":
            flags = (n > 0).astype(np.uint8)
        else:
            flags = np.array([n[r] > 0 and orc.release_due(orc.RELEASE_DECODE_TOKEN, int(decoded[r]), every_n) for r in range(B)],
                             np.uint8)
        hb.hswa_swa_release(h, B, ctx, torch.from_numpy(flags).cuda(), valid_from)
        orc.swa_release(cfg, octx, flags, ofrom)
        assert np.array_equal(valid_from.cpu().numpy(), ofrom), (kind, who, arg)
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    assert octx.tolist() == total
    for s in (False, True):
        assert np.array_equal(to_host_bits(pools[s]), o_pools[s])

    # per-position SWA status, on the device and into pinned host memory, against the oracle
    stride = max(total) + 37
    for mask in (torch.full((B, stride), 9, dtype=torch.uint8, device="cuda"), torch.full((B, stride), 9, dtype=torch.uint8).pin_memory()):
        hb.hswa_swa_valid_mask(h, B, ctx, valid_from, mask)
        torch.cuda.synchronize()
        got = mask.cpu().numpy()
        for r in range(B):
            want = np.zeros(stride, np.uint8)
            want[: total[r]] = orc.swa_valid_mask(total[r], int(ofrom[r]))
            assert np.array_equal(got[r], want), r
    masks = got

    # two new requests match the donors' prefixes: window-safe hit lengths (library, host arithmetic) vs the oracle
    full_ok = [np.ones(total[r], np.uint8) for r in range(B)]
    # the first diverges from its donor two tokens before the end: its window [L - (W - 1), L) is still there (the last
    # release was a few decode tokens ago); the second matches a prefix whose tail was released long ago
    match = [total[0] - 2, int(ofrom[1]) + 50]
    assert match[0] - (W - 1) >= int(ofrom[0]) > 0
    hits = [hb.hswa_prefix_hit_len(match[r], W, full_ok[r], masks[r]) for r in range(B)]
    assert hits == [orc.prefix_hit_len(match[r], W, full_ok[r], masks[r]) for r in range(B)]
    assert hits[0] == match[0] and hits[1] == 0             # the second would read released slots: a miss
    # strict O(W) storage: a prefix much shorter than what the ring still holds is no longer window-safe
    assert hb.hswa_prefix_hit_len(int(ofrom[0]) + W - 2, W, full_ok[0], masks[0]) == 0
    # an evicted Full segment ends the prefix at its first token whatever the SWA status
    holed = full_ok[0].copy()
    holed[200:264] = 0
    assert hb.hswa_prefix_hit_len(match[0], W, holed, np.ones(total[0], np.uint8)) == 200 == \
        orc.prefix_hit_len(match[0], W, holed, np.ones(total[0], np.uint8))

    # reuse of donor 0 at L = hits[0]: gather its window as of length L (same ring, head moved back by ctx - L) ...
    L = hits[0]
    back = total[0] - L
    view = hb.Batch(dev_i32([L]), bt[:1].contiguous(), rt[:1].contiguous(), dev_i32([(int(ohead[0]) - back) % C]),
                    None, max_q_len=1, total_q=1, max_ctx_len=L)
    oview = orc.OracleBatch(np.array([L], np.int32), t.block_table[:1], t.ring_table[:1],
                            np.array([(int(ohead[0]) - back) % C], np.int32))
    buf = torch.zeros((1, W - 1, 2, d.num_kv_heads, d.head_dim), dtype=torch.bfloat16, device="cuda")
    hb.hswa_swa_window_gather(h, layers[True], view, buf)
    ref_buf = orc.window_gather(cfg, orc.OracleLayer(o_pools[True], True), oview)
    assert np.array_equal(to_host_bits(buf), ref_buf)
    for j in range(W - 1):                                  # and it is the donor's logical tail
        assert np.array_equal(ref_buf[0, j, 0], k_seq[0][L - (W - 1) + j])
    # ... scatter it into the new request's fresh ring (its own pages and head), share the donor's Full pages
    nt = wl.make_tables(d, [L], [1], seed=82)
    new_ring = to_dev_bf16(poison_pool(nt.num_ring_pages, d))
    o_new_ring = poison_pool(nt.num_ring_pages, d)
    # Full pages: the donor's, up to and including the page position L falls into (the donor is finished and its
    # tokens from L on are dropped, so the new request takes that page over and writes there)
    new_bt = np.ascontiguousarray(t.block_table[0, : L // P + 1], dtype=np.int32)[None, :]
    nb = hb.Batch(dev_i32([L]), dev_i32(new_bt), dev_i32(nt.ring_table), dev_i32(nt.ring_head), None, max_q_len=1, total_q=1,
                  max_ctx_len=L)
    onb = orc.OracleBatch(np.array([L], np.int32), new_bt, nt.ring_table, nt.ring_head)
    hb.hswa_swa_window_scatter(h, hb.Layer(new_ring, True), nb, buf)
    orc.window_scatter(cfg, orc.OracleLayer(o_new_ring, True), onb, ref_buf)
    assert np.array_equal(to_host_bits(new_ring), o_new_ring)
    new_from = dev_i32([max(0, L - (W - 1))])               # a seeded ring starts with exactly the window
    # first decode step of the new request: a different token than the donor generated at position L
    q = rand_bits(840, (1, d.num_q_heads, d.head_dim))
    k_new, v_new = rand_bits(841, (1, d.num_kv_heads, d.head_dim)), rand_bits(842, (1, d.num_kv_heads, d.head_dim))
    for s, pool, opool in ((False, pools[False], o_pools[False]), (True, new_ring, o_new_ring)):
        out = torch.zeros((1, d.num_q_heads, d.head_dim), dtype=torch.float32, device="cuda")
        hb.hswa_decode_attn(h, hb.Layer(pool, s), nb, to_dev_bf16(q), to_dev_bf16(k_new), to_dev_bf16(v_new), out, None, ws)
        ol = orc.OracleLayer(opool, s)
        ref, _ = orc.attention(cfg, ol, onb, q, k_new, v_new)
        orc.kv_append(cfg, ol, onb, k_new, v_new)
        assert np.abs(out.cpu().numpy() - ref).max() <= TOL, s
        assert np.array_equal(to_host_bits(pool), opool), s
        # the same answer from the logical sequence alone (plain attention over the donor's first L tokens + the new one)
        ks = np.concatenate([k_seq[0][:L], k_new]).astype(np.uint16)
        vs = np.concatenate([v_seq[0][:L], v_new]).astype(np.uint16)
        lo = max(0, L - W + 1) if s else 0
        K, V = wl.bits_to_f64(ks[lo:, :, :]), wl.bits_to_f64(vs[lo:, :, :])
        Q = wl.bits_to_f64(q)[0]
        for hq in range(d.num_q_heads):
            kh = hq // d.group
            sc = cfg.sm_scale * (K[:, kh, :] @ Q[hq])
            w_ = np.exp(sc - sc.max())
            want = (w_[:, None] * V[:, kh, :]).sum(0) / w_.sum()
            assert np.abs(ref[0, hq] - want).max() < 1e-9
    hb.hswa_step_advance(h, 1, nb.ctx_len, nb.ring_head, None)
    hb.hswa_swa_release(h, 1, nb.ctx_len, None, new_from)
    assert new_from.cpu().numpy().tolist() == [max(0, L + 1 - (W - 1))]
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)


def test_layerwise_loadback_equals_resident_run():
    """Paper Sec. 3.1.2: the SWA state of a suspended batch lives in pinned host memory (only the W - 1 positions
    per request and layer the next token needs) and is loaded back layer by layer on a copy stream that runs ahead
    of the compute stream.  The decode step on the reloaded rings must give the same bits as on resident rings."""
    d = wl.Dims(num_q_heads=16, num_kv_heads=2, head_dim=128, page_size=64)
    W = d.window
    n_layers, B = 6, 5
    ctx = [5000, 130, 127, 64, 900]
    t = wl.make_tables(d, ctx, [1] * B, seed=90)
    h = make_handle(d, out_dtype=torch.bfloat16)
    g = torch.Generator(device="cuda")
    g.manual_seed(90)
    rings = [torch.randn((t.num_ring_pages, 2, d.num_kv_heads, d.page_size, d.head_dim), generator=g, device="cuda",
                         dtype=torch.float32).to(torch.bfloat16) for _ in range(n_layers)]
    q = torch.randn((n_layers, B, d.num_q_heads, d.head_dim), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    k = torch.randn((n_layers, B, d.num_kv_heads, d.head_dim), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn((n_layers, B, d.num_kv_heads, d.head_dim), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    b = hb.Batch(dev_i32(t.ctx_len), dev_i32(t.block_table), dev_i32(t.ring_table), dev_i32(t.ring_head), None, max_q_len=1,
                 total_q=B, max_ctx_len=max(ctx))

    def run(pools):
        out = torch.zeros((n_layers, B, d.num_q_heads, d.head_dim), dtype=torch.bfloat16, device="cuda")
        for i in range(n_layers):
            hb.hswa_decode_attn(h, hb.Layer(pools[i], True), b, q[i], k[i], v[i], out[i], None, None)
        return out

    # offload: gather every layer's windows into pinned host memory
    shape = (B, W - 1, 2, d.num_kv_heads, d.head_dim)
    host = [torch.empty(shape, dtype=torch.bfloat16).pin_memory() for _ in range(n_layers)]
    for i in range(n_layers):
        hb.hswa_swa_window_gather(h, hb.Layer(rings[i], True), b, host[i])
    torch.cuda.synchronize()
    resident = [r.clone() for r in rings]
    want = run(resident)
    # loadback into rings that hold garbage, layer by layer on a copy stream, the compute stream gated per layer
    reloaded = [torch.full_like(r, 1000.0) for r in rings]
    staging = [torch.empty(shape, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    copy_stream = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    events = []
    start = torch.cuda.Event()
    start.record(main)
    with torch.cuda.stream(copy_stream):
        copy_stream.wait_event(start)
        for i in range(n_layers):
            staging[i].copy_(host[i], non_blocking=True)
            hb.hswa_swa_window_scatter(h, hb.Layer(reloaded[i], True), b, staging[i])
            ev = torch.cuda.Event()
            ev.record(copy_stream)
            events.append(ev)
    out = torch.zeros((n_layers, B, d.num_q_heads, d.head_dim), dtype=torch.bfloat16, device="cuda")
    for i in range(n_layers):
        main.wait_event(events[i])
        hb.hswa_decode_attn(h, hb.Layer(reloaded[i], True), b, q[i], k[i], v[i], out[i], None, None)
    torch.cuda.synchronize()
    assert hb.hswa_get_async_error(h)[0] == hb.HSWA_OK, hb.hswa_get_async_error(h)
    assert torch.equal(out.view(torch.int16), want.view(torch.int16))   # same bits as the resident run
    # and right: the oracle on the resident rings (one layer)
    cfg = oracle_config(d)
    ob = orc.OracleBatch(t.ctx_len, t.block_table, t.ring_table, t.ring_head)
    ref, _ = orc.attention(cfg, orc.OracleLayer(to_host_bits(rings[2]), True), ob, to_host_bits(q[2]), to_host_bits(k[2]),
                           to_host_bits(v[2]))
    err = np.abs(out[2].float().cpu().numpy() - ref)
    assert (err <= np.maximum(TOL, np.abs(ref) * 2.0 ** -8)).all()
