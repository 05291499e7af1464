"""CPU pins of the oracle's SWA-aware prefix-reuse functions (paper Sec. 3.1.3 window-safe length; Sec. 3.1.1 /
3.1.2 window-only data movement)."""
import numpy as np
import pytest

from oracle import hswa_oracle as orc
from paper_2607_13095_b200 import workloads as wl
from helpers import build_scenario, poison_pool

D8 = wl.Dims(num_q_heads=4, num_kv_heads=2, head_dim=8, page_size=4, window=8)
D16 = wl.Dims(num_q_heads=4, num_kv_heads=1, head_dim=64, page_size=16, window=128)


def brute_safe_len(m, W, valid):
    best = 0
    for L in range(0, m + 1):
        lo = max(0, L - (W - 1))
        if all(valid[lo:L]):
            best = L
    return best


def test_window_safe_len_bruteforce_and_figure():
    rng = np.random.default_rng(0)
    for W in (1, 2, 4, 8, 128):
        for _ in range(60):
            n = int(rng.integers(1, 300))
            valid = (rng.random(n) < rng.choice([0.5, 0.9, 0.99])).astype(np.uint8)
            if rng.random() < 0.5:  # typical shape: only a tail survives
                valid[: int(rng.integers(0, n))] = 0
            m = int(rng.integers(0, n + 1))
            assert orc.window_safe_len(m, W, valid) == brute_safe_len(m, W, valid)
    # the paper's figure uses a window of 4: a node whose last 3 SWA slots are valid is a full hit,
    # one with an evicted tail is clipped back to the last position whose tail is intact
    assert orc.window_safe_len(10, 4, np.array([0] * 7 + [1] * 3, np.uint8)) == 10
    assert orc.window_safe_len(10, 4, np.array([1] * 5 + [0] * 5, np.uint8)) == 5
    assert orc.window_safe_len(10, 4, np.zeros(10, np.uint8)) == 0
    assert orc.window_safe_len(2, 4, np.ones(2, np.uint8)) == 2       # shorter than the window: all cached tokens valid
    assert orc.window_safe_len(10, 1, np.zeros(10, np.uint8)) == 10   # window 1 needs no cached key


@pytest.mark.parametrize("dims", [D8, D16])
def test_window_gather_matches_logical_tail(dims):
    W, C = dims.window, dims.ring_slots
    ctx = [0, 1, W - 2, W - 1, W, C + 1, 3 * C + 5]
    sc = build_scenario(dims, ctx, [1] * len(ctx), seed=91)
    buf = orc.window_gather(sc.cfg, sc.layer(True), sc.batch())
    for r, c in enumerate(ctx):
        for j in range(W - 1):
            p = c - (W - 1) + j
            if p < 0:
                assert not buf[r, j].any()
            else:
                assert np.array_equal(buf[r, j, 0], sc.k_seq[r][p]) and np.array_equal(buf[r, j, 1], sc.v_seq[r][p])


@pytest.mark.parametrize("dims", [D8, D16])
def test_window_scatter_roundtrip_and_equals_append(dims):
    W, C = dims.window, dims.ring_slots
    ctx = [0, 3, W - 1, W + 5, 3 * C + 5]
    donor = build_scenario(dims, ctx, [1] * len(ctx), seed=92)
    buf = orc.window_gather(donor.cfg, donor.layer(True), donor.batch())
    # seed a fresh ring (different pages, different head) from the buffer
    fresh = wl.make_tables(dims, ctx, [1] * len(ctx), seed=93)
    dst = orc.OracleLayer(poison_pool(fresh.num_ring_pages, dims), True)
    db = orc.OracleBatch(fresh.ctx_len, fresh.block_table, fresh.ring_table, fresh.ring_head)
    orc.window_scatter(donor.cfg, dst, db, buf)
    assert np.array_equal(orc.window_gather(donor.cfg, dst, db), buf)            # round trip
    # the same ring contents result from appending those tokens with the ring rewound by their count
    ref = orc.OracleLayer(poison_pool(fresh.num_ring_pages, dims), True)
    keep = np.minimum(fresh.ctx_len, W - 1).astype(np.int32)
    ptr = np.zeros(len(ctx) + 1, np.int32)
    ptr[1:] = np.cumsum(keep)
    if ptr[-1]:
        k = np.concatenate([donor.k_seq[r][c - keep[r]: c] for r, c in enumerate(ctx)])
        v = np.concatenate([donor.v_seq[r][c - keep[r]: c] for r, c in enumerate(ctx)])
        rb = orc.OracleBatch(fresh.ctx_len - keep, fresh.block_table, fresh.ring_table,
                             np.mod(fresh.ring_head - keep, dims.ring_slots), ptr)
        orc.kv_append(donor.cfg, ref, rb, k, v)
    assert np.array_equal(dst.pool, ref.pool)
    # and a decode step on the seeded ring gives the donor's output
    a, _ = orc.attention(donor.cfg, donor.layer(True), donor.batch(), donor.q, donor.k_new, donor.v_new)
    b, _ = orc.attention(donor.cfg, dst, db, donor.q, donor.k_new, donor.v_new)
    assert np.array_equal(a, b)
