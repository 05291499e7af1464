"""CPU pins of the fp64 oracle against things other than itself: brute force, a library routine,
identities, invariants, closed forms and the constants the paper prints."""
import os

import numpy as np
import pytest
import torch

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import workloads as wl
from helpers import POISON_V, brute_force_attention, build_scenario, oracle_config, poison_pool

D8 = wl.Dims(num_q_heads=4, num_kv_heads=2, head_dim=8, page_size=4, window=8)      # W=8, P=4, C=12
D16 = wl.Dims(num_q_heads=4, num_kv_heads=1, head_dim=64, page_size=16, window=128)  # config-1 dims
D64 = wl.Dims(num_q_heads=8, num_kv_heads=1, head_dim=16, page_size=64, window=128)  # G=8, P=64, C=192


def oracle_both(sc, is_swa, fused=True):
    layer = sc.layer(is_swa)
    return orc.attention(sc.cfg, layer, sc.batch(), sc.q, sc.k_new if fused else None,
                         sc.v_new if fused else None)


def ctx_sweep(d):
    W, P, C = d.window, d.page_size, d.ring_slots
    return sorted({0, 1, W - 2, W - 1, W, W + 1, P - 1, P, P + 1, C - 1, C, C + 1, 3 * C + 5})


# ---- P1: brute force ---------------------------------------------------------------------------------
@pytest.mark.parametrize("dims", [D8, D16, D64], ids=["W8P4", "W128P16", "W128P64"])
@pytest.mark.parametrize("is_swa", [False, True])
def test_p1_bruteforce_decode(dims, is_swa):
    ctx = ctx_sweep(dims)
    sc = build_scenario(dims, ctx, [1] * len(ctx), seed=11)
    out, lse = oracle_both(sc, is_swa)
    ref, ref_lse = brute_force_attention(sc, is_swa)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)
    assert np.abs(out).max() < 100.0  # no poison leaked


@pytest.mark.parametrize("dims", [D8, D16], ids=["W8P4", "W128P16"])
@pytest.mark.parametrize("is_swa", [False, True])
@pytest.mark.parametrize("n", [2, 17, 18, 64, 65])
def test_p1_bruteforce_prefill(dims, is_swa, n):
    ctx = ctx_sweep(dims)[::2]
    C = dims.ring_slots
    q_len = [n, 1, 2 * C + 3, C, C + 1, 4, 66][: len(ctx)]
    sc = build_scenario(dims, ctx, q_len, seed=12 + n)
    out, lse = oracle_both(sc, is_swa)
    ref, ref_lse = brute_force_attention(sc, is_swa)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)
    assert np.abs(out).max() < 100.0


# ---- P2: library routine ------------------------------------------------------------------------------
@pytest.mark.parametrize("is_swa", [False, True])
def test_p2_torch_sdpa(is_swa):
    d = D16
    sc = build_scenario(d, [100, 512, 0, 127], [64, 64, 5, 3], seed=21, scale=1.0)
    out, _ = oracle_both(sc, is_swa)
    t = sc.tables
    for r in range(t.batch):
        c, n = int(t.ctx_len[r]), int(t.q_len[r])
        K = torch.from_numpy(wl.bits_to_f64(sc.k_seq[r])).permute(1, 0, 2)  # [Hkv][L][D]
        V = torch.from_numpy(wl.bits_to_f64(sc.v_seq[r])).permute(1, 0, 2)
        Q = torch.from_numpy(wl.bits_to_f64(sc.q[t.q_indptr[r]: t.q_indptr[r + 1]])).permute(1, 0, 2)
        K = K.repeat_interleave(d.group, dim=0)
        V = V.repeat_interleave(d.group, dim=0)
        pq = c + torch.arange(n)[:, None]
        pk = torch.arange(c + n)[None, :]
        mask = pk <= pq
        if is_swa:
            mask = mask & (pk > pq - d.window)
        ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], attn_mask=mask[None, None],
                                                                scale=sc.cfg.sm_scale)[0]
        got = out[t.q_indptr[r]: t.q_indptr[r + 1]].transpose(1, 0, 2)
        np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=1e-12)


# ---- P3: SWA == Full while the sequence fits the window ---------------------------------------------------
def test_p3_swa_equals_full_when_short():
    d = D16
    sc = build_scenario(d, [100, 0, 27, 127], [1, 128, 101, 1], seed=31)
    full, lf = oracle_both(sc, False)
    swa, ls = oracle_both(sc, True)
    assert np.array_equal(full, swa) and np.array_equal(lf, ls)
    # one past the window they must differ
    sc2 = build_scenario(d, [128], [1], seed=32)
    a, _ = oracle_both(sc2, False)
    b, _ = oracle_both(sc2, True)
    assert not np.array_equal(a, b)


# ---- P4 + P7 + P11: ring == contiguous, chunking invariance, storage law, over a multi-step history -------
def run_history(d, chunks, seed, head0):
    """Serve one request through the given chunk sizes with append + attention + advance in the oracle.
    Returns outputs per position for both layer types and the final pools."""
    cfg = oracle_config(d)
    L = sum(chunks)
    Hkv, Hq, D = d.num_kv_heads, d.num_q_heads, d.head_dim
    K = wl.bf16_bits_normal(seed, (L, Hkv, D))
    V = wl.bf16_bits_normal(seed + 1, (L, Hkv, D))
    Q = wl.bf16_bits_normal(seed + 2, (L, Hq, D))
    t = wl.make_tables(d, [0], [L], seed)  # enough Full pages for the whole life of the request
    full = orc.OracleLayer(poison_pool(t.num_full_pages, d), False)
    swa = orc.OracleLayer(poison_pool(t.num_ring_pages, d), True)
    ctx = np.zeros(1, np.int32)
    head = np.array([head0], np.int32)
    outs = {False: [], True: []}
    ring_pages = set(int(x) for x in t.ring_table[0])
    for n in chunks:
        b = orc.OracleBatch(ctx.copy(), t.block_table, t.ring_table, head.copy(), np.array([0, n], np.int32))
        c = int(ctx[0])
        for layer in (full, swa):
            o, _ = orc.attention(cfg, layer, b, Q[c:c + n], K[c:c + n], V[c:c + n])  # pre-append state
            outs[layer.is_swa].append(o)
            before = layer.pool.copy()
            orc.kv_append(cfg, layer, b, K[c:c + n], V[c:c + n])
            if layer.is_swa:  # P11: only ring pages are ever touched
                changed = np.nonzero((before != layer.pool).reshape(before.shape[0], -1).any(axis=1))[0]
                assert set(int(x) for x in changed) <= ring_pages
        inv = (int(head[0]) - int(ctx[0])) % d.ring_slots
        orc.step_advance(cfg, ctx, head, np.array([0, n], np.int32))
        assert (int(head[0]) - int(ctx[0])) % d.ring_slots == inv  # (head - ctx) mod C is invariant
    # P11: the ring holds exactly the last min(L, C) tokens
    b = orc.OracleBatch(ctx, t.block_table, t.ring_table, head)
    C = d.ring_slots
    valid = 0
    for p in range(max(0, L - C), L):
        page, slot = orc.locate(cfg, True, b, 0, p)
        assert np.array_equal(swa.pool[page, 0, :, slot, :], K[p]) and np.array_equal(swa.pool[page, 1, :, slot, :], V[p])
        valid += 1
    poison_rows = (wl.bits_to_f64(swa.pool[:, 1]) == POISON_V).all(axis=-1).sum()
    assert poison_rows == (swa.pool.shape[0] * d.page_size - valid) * Hkv
    return {k: np.concatenate(v) for k, v in outs.items()}, (K, V, Q)


@pytest.mark.parametrize("dims,head0", [(D8, 0), (D8, 5), (D8, 11), (D16, 143), (D64, 63)])
def test_p4_p7_p11_history(dims, head0):
    C, W = dims.ring_slots, dims.window
    plans = [[3, 17, 1, 1, 64, 5, 1], [100], [C - W + 1] * 5, [1] * 40, [2 * C + 3, 1, 1], [C, C + 1, 1]]
    if dims.window > 8:
        plans = plans[:3] + [[65, 200, 1, 66]]
    for i, chunks in enumerate(plans):
        outs, (K, V, Q) = run_history(dims, chunks, seed=40 + i, head0=head0)
        L = sum(chunks)
        # single-shot brute force over the logical (contiguous) sequence
        Kd, Vd, Qd = wl.bits_to_f64(K), wl.bits_to_f64(V), wl.bits_to_f64(Q)
        pq = np.arange(L)[:, None]
        pk = np.arange(L)[None, :]
        for is_swa in (False, True):
            mask = pk <= pq
            if is_swa:
                mask = mask & (pk > pq - W)
            for h in range(dims.num_q_heads):
                S = np.where(mask, (Qd[:, h] @ Kd[:, h // dims.group].T) / np.sqrt(dims.head_dim), -np.inf)
                E = np.exp(S - S.max(axis=1, keepdims=True))
                ref = (E @ Vd[:, h // dims.group]) / E.sum(axis=1, keepdims=True)
                np.testing.assert_allclose(outs[is_swa][:, h], ref, rtol=0, atol=1e-12)


def test_append_then_attend_limit():
    """On a ring, appending first is only safe for n <= C - W + 1: one more token and the chunk overwrites
    a slot its own first query still needs."""
    for d in (D8, D16, D64):
        C, W = d.ring_slots, d.window
        for n, safe in ((C - W + 1, True), (C - W + 2, False)):
            sc = build_scenario(d, [3 * C + 5], [n], seed=50, ring_keep=C)
            ref, _ = brute_force_attention(sc, True)
            layer = sc.layer(True)
            orc.kv_append(sc.cfg, layer, sc.batch(), sc.k_new, sc.v_new)
            got, _ = orc.attention(sc.cfg, layer, sc.batch(), sc.q, None, None)  # reads everything from the ring
            assert (np.abs(got - ref).max() < 1e-12) == safe


# ---- P5: page permutation ------------------------------------------------------------------------------
@pytest.mark.parametrize("is_swa", [False, True])
def test_p5_page_permutation(is_swa):
    a = build_scenario(D16, [100, 512, 300], [64, 1, 7], seed=51, permute=True)
    b = build_scenario(D16, [100, 512, 300], [64, 1, 7], seed=51, permute=False, ring_head=a.tables.ring_head)
    assert not np.array_equal(a.tables.block_table, b.tables.block_table)
    oa, la = oracle_both(a, is_swa)
    ob, lb = oracle_both(b, is_swa)
    assert np.array_equal(oa, ob) and np.array_equal(la, lb)


# ---- P6: shared prefix -----------------------------------------------------------------------------------
def test_p6_shared_prefix():
    kw = dict(seed=61, shared_prefix_tokens=64)
    a = build_scenario(D16, [64, 100, 200], [1, 9, 1], share_pages=True, **kw)
    b = build_scenario(D16, [64, 100, 200], [1, 9, 1], share_pages=False, **kw)
    assert (a.tables.block_table[:, :4] == a.tables.block_table[0, :4]).all()
    assert len(set(b.tables.block_table[:, 0])) == 3
    assert a.tables.num_full_pages < b.tables.num_full_pages
    for is_swa in (False, True):
        oa, la = oracle_both(a, is_swa)
        ob, lb = oracle_both(b, is_swa)
        assert np.array_equal(oa, ob) and np.array_equal(la, lb)
        ref, _ = brute_force_attention(a, is_swa)
        np.testing.assert_allclose(oa, ref, rtol=0, atol=1e-12)


# ---- P8: closed forms -------------------------------------------------------------------------------------
def test_p8_closed_forms():
    d = D16
    sc = build_scenario(d, [300, 5, 0], [1, 1, 1], seed=71)
    t = sc.tables
    # q = 0  ->  uniform weights  ->  arithmetic mean of V over the visible keys; lse = ln(#keys)
    sc.q[:] = 0
    for is_swa in (False, True):
        out, lse = oracle_both(sc, is_swa)
        for r in range(3):
            L = int(t.ctx_len[r]) + 1
            lo = max(0, L - d.window) if is_swa else 0
            mean = wl.bits_to_f64(sc.v_seq[r])[lo:L, 0].mean(axis=0)
            for h in range(d.num_q_heads):
                np.testing.assert_allclose(out[r, h], mean, rtol=0, atol=1e-12)
                assert abs(lse[r, h] - np.log(L - lo)) < 1e-12
    # single key (ctx = 0, n = 1): out = v exactly, lse = score
    sc2 = build_scenario(d, [0], [1], seed=72)
    out, lse = oracle_both(sc2, True)
    v = wl.bits_to_f64(sc2.v_seq[0])[0, 0]
    k = wl.bits_to_f64(sc2.k_seq[0])[0, 0]
    for h in range(d.num_q_heads):
        assert np.array_equal(out[0, h], v)
        s = sc2.cfg.sm_scale * float(wl.bits_to_f64(sc2.q)[0, h] @ k)
        assert abs(lse[0, h] - s) < 1e-12
    # constant V -> that constant, whatever the scores
    sc3 = build_scenario(d, [200], [3], seed=73)
    const = wl.bf16_bits_const(0.375, (1,))[0]
    sc3.full_pool[:, 1] = const
    sc3.swa_pool[:, 1] = const
    sc3.v_new[:] = const
    for is_swa in (False, True):
        out, _ = oracle_both(sc3, is_swa)
        np.testing.assert_allclose(out, 0.375, rtol=0, atol=1e-13)
    # one dominant logit -> that key's V row
    sc4 = build_scenario(d, [50], [1], seed=74, sm_scale=1.0)
    big = wl.bf16_bits_const(8.0, (d.head_dim,))
    sc4.q[0, :, :] = big
    page, slot = orc.locate(sc4.cfg, False, sc4.batch(), 0, 20)
    sc4.full_pool[page, 0, 0, slot, :] = big          # score 64*64 = 4096 >> the rest
    out, _ = oracle_both(sc4, False)
    target = wl.bits_to_f64(sc4.v_seq[0])[20, 0]
    np.testing.assert_allclose(out[0, 0], target, rtol=0, atol=1e-9)


# ---- P9: the paper's ~1/7 ------------------------------------------------------------------------------
def test_p9_accounting_matches_paper():
    consts = {}
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            consts[k] = int(v)
    assert consts["full_layers"] + consts["swa_layers"] == consts["total_layers"] == 70
    cfg = oracle_config(wl.BIG)
    assert cfg.window == consts["window"]
    flags = wl.hybrid_layer_flags(consts["total_layers"])
    assert sum(flags) == consts["swa_layers"]
    from paper_2607_13095_b200 import accounting
    expect = {4096: 0.1696, 32768: 0.1462, 262144: 0.1433, 1048576: 0.1430}
    for n, ratio in expect.items():
        p = n - 1
        hybrid = sum(orc.attended_keys(cfg, f, p) for f in flags)
        assert hybrid == 10 * (p + 1) + 60 * min(p + 1, 128)
        assert hybrid == sum(int(accounting.attended_keys(f, p, 128)) for f in flags)
        assert abs(hybrid / (70 * (p + 1)) - ratio) < 5e-5
    assert abs(expect[1048576] - consts["asymptotic_ratio_num"] / consts["asymptotic_ratio_den"]) < 2e-4


# ---- P12: append exactness ----------------------------------------------------------------------------
@pytest.mark.parametrize("dims", [D8, D16])
def test_p12_append_bit_exact(dims):
    d = dims
    C, P = d.ring_slots, d.page_size
    ctx = [0, 1, P - 1, C + 1, 3 * C + 5]
    q_len = [2 * C + 3, 1, C, 17, 0]
    sc = build_scenario(d, ctx, q_len, seed=81, ring_keep=C)
    t = sc.tables
    for is_swa in (False, True):
        layer = sc.layer(is_swa)
        expect = layer.pool.copy()
        offs = orc.kv_append(sc.cfg, layer, sc.batch(), sc.k_new, sc.v_new, want_offsets=True)
        # sequential python model of the same storage rule
        exp_offs = np.zeros_like(offs)
        st = [s // 2 for s in expect.strides]
        for r in range(t.batch):
            for i in range(int(t.q_len[r])):
                tok = int(t.q_indptr[r]) + i
                p = int(t.ctx_len[r]) + i
                if is_swa:
                    s = (int(t.ring_head[r]) + i) % C
                    page, slot = int(t.ring_table[r, s // P]), s % P
                else:
                    page, slot = int(t.block_table[r, p // P]), p % P
                expect[page, 0, :, slot, :] = sc.k_new[tok]
                expect[page, 1, :, slot, :] = sc.v_new[tok]
                for kv in range(2):
                    for h in range(d.num_kv_heads):
                        exp_offs[tok, kv, h] = page * st[0] + kv * st[1] + h * st[2] + slot * st[3]
        assert np.array_equal(layer.pool, expect)
        assert np.array_equal(offs, exp_offs)
        if is_swa:  # only the last min(n, C) tokens survive
            r = 0
            n = int(t.q_len[r])
            b2 = orc.OracleBatch(t.ctx_len + t.q_len, t.block_table, t.ring_table,
                                 np.mod(t.ring_head + t.q_len, C))
            for p in range(n - C, n):
                page, slot = orc.locate(sc.cfg, True, b2, r, p)
                assert np.array_equal(layer.pool[page, 0, :, slot, :], sc.k_new[p])


def test_step_advance_and_mod():
    cfg = oracle_config(D8)
    ctx = np.array([0, 5, 100], np.int32)
    head = np.array([11, 0, 7], np.int32)
    orc.step_advance(cfg, ctx, head, np.array([0, 1, 30, 30], np.int32))
    assert ctx.tolist() == [1, 34, 100] and head.tolist() == [0, 5, 7]
    orc.step_advance(cfg, ctx, head, None)
    assert ctx.tolist() == [2, 35, 101] and head.tolist() == [1, 6, 8]
    # negative offsets use the mathematical mod
    b = orc.OracleBatch(np.array([10], np.int32), np.zeros((1, 4), np.int32), np.array([[7, 8, 9]], np.int32),
                        np.array([1], np.int32))
    assert orc.locate(cfg, True, b, 0, 8) == (9, 3)   # slot (1 - 2) mod 12 = 11 -> page index 2, slot 3


def test_locate_hand_worked_literals():
    """Position -> (page, slot) worked by hand from the two storage rules (Full: block p div P of the request's
    table, slot p mod P; SWA: ring slot (head + p - ctx) mod C, page = ring_table[slot div P]), on permuted tables,
    for both layer kinds, including wrapped rings and positions behind and ahead of the ring head."""
    cfg = oracle_config(D8)                                    # W = 8, P = 4, R = 3, C = 12
    bt = np.array([[1, 3, 7, 4], [5, 2, 9, 0]], np.int32)
    rt = np.array([[7, 8, 9], [8, 2, 5]], np.int32)
    b = orc.OracleBatch(np.array([10, 30], np.int32), bt, rt, np.array([1, 10], np.int32))
    full = {(0, 6): (3, 2), (1, 0): (5, 0), (1, 3): (5, 3), (1, 4): (2, 0), (1, 11): (9, 3), (1, 13): (0, 1)}
    for (r, p), want in full.items():
        assert orc.locate(cfg, False, b, r, p) == want, (r, p)
    swa = {
        (0, 10): (7, 1),    # the next write sits at the ring head
        (0, 9): (7, 0), (0, 8): (9, 3),     # one and two back: the second wraps to the last page
        (0, 3): (8, 2),     # (1 - 7) mod 12 = 6
        (0, 11): (7, 2), (0, 13): (8, 0),   # new tokens ahead of the head
        (1, 30): (5, 2), (1, 31): (5, 3), (1, 32): (8, 0),   # head 10: the third new token wraps to slot 0
        (1, 23): (8, 3),    # oldest key of a window of 8: (10 - 7) = 3
        (1, 25): (2, 1), (1, 19): (5, 3),   # (10 - 11) mod 12 = 11
    }
    for (r, p), want in swa.items():
        assert orc.locate(cfg, True, b, r, p) == want, (r, p)
    big = oracle_config(wl.BIG)                                # W = 128, P = 64, R = 3, C = 192
    b = orc.OracleBatch(np.array([5000], np.int32), np.array([[11, 0, 6]], np.int32), np.array([[40, 3, 17]], np.int32),
                        np.array([190], np.int32))
    assert orc.locate(big, False, b, 0, 64) == (0, 0) and orc.locate(big, False, b, 0, 191) == (6, 63)
    for p, want in {5000: (17, 62), 5001: (17, 63), 5002: (40, 0), 4873: (40, 63), 4936: (3, 62), 4999: (17, 61)}.items():
        assert orc.locate(big, True, b, 0, p) == want, p
