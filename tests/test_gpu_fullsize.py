"""Parity at the full sizes of the named workloads, in the launch configuration bench.py times (same state
builder, same calls), on sampled output rows the oracle computes one by one, plus bit-exact checks of the
appended rows and of everything the append must leave untouched."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import hswa_oracle as orc  # noqa: E402
from paper_2607_13095_b200 import binding as hb  # noqa: E402
from gpu_utils import to_host_bits  # noqa: E402

pytestmark = pytest.mark.gpu
TOL = 1e-2


def sample_rows(rng, t, Hq, n_rows, always_requests):
    reqs = list(always_requests) + list(rng.integers(0, t.batch, n_rows))
    reqs = np.array(reqs[:n_rows], dtype=np.int32)
    heads = rng.integers(0, Hq, len(reqs)).astype(np.int32)
    heads[: min(len(heads), Hq)] = np.arange(min(len(heads), Hq))  # every head at least once
    return reqs, heads


def check_decode_workload(name, n_rows_full, layers=0, batch=0):
    dev = torch.device("cuda", 0)
    w = bench.make_workload(name, layers=layers, batch=batch)
    b = bench.DecodeBench(w, 4, dev)
    t, d = b.t, w.dims
    cfg = orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages)
    ob = orc.OracleBatch(t.ctx_len, t.block_table, t.ring_table, t.ring_head)
    rng = np.random.default_rng(123)
    always = [int(np.argmax(t.ctx_len)), int(np.argmin(t.ctx_len)), 0, t.batch - 1]
    fi, si = b.full_idx[0], w.layer_is_swa.index(True)
    before = {i: to_host_bits(b.layers[i].pool) for i in (fi, si)}
    b.step()                      # the bench's own step: all layers + advance
    torch.cuda.synchronize()
    assert hb.hswa_get_async_error(b.h)[0] == hb.HSWA_OK
    out = b.out.float().cpu().numpy()
    worst = 0.0
    for i, n_rows in ((fi, n_rows_full), (si, 512)):
        is_swa = w.layer_is_swa[i]
        tok, head = sample_rows(rng, t, d.num_q_heads, n_rows, always)
        q, k, v = to_host_bits(b.q[i]), to_host_bits(b.k_new[i]), to_host_bits(b.v_new[i])
        layer = orc.OracleLayer(before[i], is_swa)
        ref, _ = orc.attention(cfg, layer, ob, q, k, v, rows=(tok, head))
        got = out[i][tok, head]
        err = float(np.abs(got - ref).max())
        worst = max(worst, err)
        assert err <= TOL, (name, "swa" if is_swa else "full", err)
        # append: the oracle's append on the host copy must reproduce the device pool byte for byte
        orc.kv_append(cfg, layer, ob, k, v)
        assert np.array_equal(to_host_bits(b.layers[i].pool), before[i]), (name, i, "pool bytes after fused append")
    # step advance
    ectx, ehead = t.ctx_len.copy(), t.ring_head.copy()
    orc.step_advance(cfg, ectx, ehead, None)
    assert np.array_equal(b.ctx.cpu().numpy(), ectx) and np.array_equal(b.head.cpu().numpy(), ehead)
    return worst


def test_config2_decode_block_fullsize():
    check_decode_workload("cfg2", 384)


def test_config4_prefix_hit_decode_fullsize():
    w = bench.make_workload("cfg4")
    assert w.tables.shared_prefix_pages == 256
    assert (w.tables.block_table[:, :256] == w.tables.block_table[0, :256]).all()
    check_decode_workload("cfg4", 384)


def test_config5_long_context_decode_fullsize_two_layers():
    # full batch and contexts (64k-256k); one Full + one SWA layer of the 70 (the others repeat them)
    check_decode_workload("cfg5", 96, layers=2)


def test_config3_chunked_prefill_fullsize():
    dev = torch.device("cuda", 0)
    w = bench.make_workload("cfg3")
    pb = bench.PrefillBench(w, dev)
    t, d = w.tables, w.dims
    cfg = orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages)
    ob = orc.OracleBatch(t.ctx_len, t.block_table, t.ring_table, t.ring_head, t.q_indptr)
    rng = np.random.default_rng(321)
    W, P, C = d.window, d.page_size, d.ring_slots
    toks = []
    for r in range(t.batch):
        n, base = int(t.q_len[r]), int(t.q_indptr[r])
        special = [0, 1, W - 2, W - 1, W, W + 1, P - 1, P, P + 1, C - 1, C, C + 1, 63, 64, 65, 127, 128, 129, n - 1, n - 2,
                   n // 2]
        # chunk-relative rows whose absolute position sits on a page boundary
        c = int(t.ctx_len[r])
        special += [((-c) % P), ((-c) % P) + 1, max(((-c) % P) - 1, 0)]
        toks += [base + i for i in special if 0 <= i < n]
    toks += list(rng.integers(0, t.total_q, 2048 - len(toks)))
    tok = np.array(toks, dtype=np.int32)
    head = rng.integers(0, d.num_q_heads, len(tok)).astype(np.int32)
    q, k, v = to_host_bits(pb.q), to_host_bits(pb.k_new), to_host_bits(pb.v_new)
    for i in (w.layer_is_swa.index(False), w.layer_is_swa.index(True)):
        is_swa = w.layer_is_swa[i]
        before = to_host_bits(pb.layers[i].pool)
        pb.out.zero_()
        pb.run_layer(i)
        torch.cuda.synchronize()
        assert hb.hswa_get_async_error(pb.h)[0] == hb.HSWA_OK
        layer = orc.OracleLayer(before, is_swa)
        ref, _ = orc.attention(cfg, layer, ob, q, k, v, rows=(tok, head))
        got = pb.out.float().cpu().numpy()[tok, head]
        err = np.abs(got - ref)
        # bf16 output: 1e-2 absolute where the value is small, one bf16 ulp (2^-8 relative) where it is large
        bound = np.maximum(TOL, np.abs(ref) * 2.0 ** -8)
        assert (err <= bound).all(), ("swa" if is_swa else "full", float(err.max()))
        orc.kv_append(cfg, layer, ob, k, v)
        assert np.array_equal(to_host_bits(pb.layers[i].pool), before), (i, "pool bytes after prefill append")


def test_config5_seventy_layer_step_late_layers():
    """The whole 70-layer step bench.py times (100 GB of pools, every layer's kernels chained on one stream), checked
    on a late Full layer (63) and the SWA layer behind it (64): sampled output rows and the appended rows of a few
    requests, whose pages are gathered on the device so that no 10 GB pool crosses to the host."""
    dev = torch.device("cuda", 0)
    free, _ = torch.cuda.mem_get_info()
    if free < 120e9:
        pytest.skip("needs 120 GB of free device memory")
    w = bench.make_workload("cfg5")
    b = bench.DecodeBench(w, 4, dev)
    t, d = b.t, w.dims
    assert len(b.layers) == 70 and not w.layer_is_swa[63] and w.layer_is_swa[64]
    cfg = orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages)
    reqs = bench.pick_requests(t, 3)
    bt, full_ids, rt, ring_ids = bench.compact_tables(t, d, reqs)
    ridx = torch.from_numpy(reqs).to(dev)
    gather = {63: torch.from_numpy(full_ids).to(dev), 64: torch.from_numpy(ring_ids).to(dev)}
    before = {i: to_host_bits(b.layers[i].pool.index_select(0, gather[i])) for i in (63, 64)}
    b.step()
    torch.cuda.synchronize()
    assert hb.hswa_get_async_error(b.h)[0] == hb.HSWA_OK
    ob = orc.OracleBatch(t.ctx_len[reqs], bt, rt, t.ring_head[reqs])
    rng = np.random.default_rng(7)
    for i, heads in ((63, rng.choice(d.num_q_heads, 12, replace=False)), (64, np.arange(d.num_q_heads))):
        is_swa = w.layer_is_swa[i]
        tok = np.repeat(np.arange(len(reqs)), len(heads)).astype(np.int32)
        head = np.tile(heads, len(reqs)).astype(np.int32)
        q, k, v = (to_host_bits(x[i].index_select(0, ridx)) for x in (b.q, b.k_new, b.v_new))
        layer = orc.OracleLayer(before[i], is_swa)
        ref, _ = orc.attention(cfg, layer, ob, q, k, v, rows=(tok, head))
        got = b.out[i].index_select(0, ridx).float().cpu().numpy()[tok, head]
        assert np.abs(got - ref).max() <= TOL, (i, float(np.abs(got - ref).max()))
        orc.kv_append(cfg, layer, ob, k, v)
        after = to_host_bits(b.layers[i].pool.index_select(0, gather[i]))
        assert np.array_equal(after, before[i]), (i, "pool bytes after the fused append")
