"""CPU checks of the bench's host-side bookkeeping: roofline numerators (logical and unique bytes), the bounded
oracle sample (request choice, compact page tables) and the oracle-timed reference arm on a tiny workload."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2607_13095_b200 import accounting  # noqa: E402
from paper_2607_13095_b200 import workloads as wl  # noqa: E402


def test_unique_bytes_count_the_shared_prefix_once():
    w = wl.config4()
    d, t = w.dims, w.tables
    logical, unique = accounting.decode_algorithmic_bytes(w), accounting.decode_unique_bytes(w)
    shared_bytes = t.shared_prefix_pages * d.page_size * d.kv_bytes_per_token
    n_full = sum(1 for s in w.layer_is_swa if not s)
    assert logical - unique == n_full * (t.batch - 1) * shared_bytes
    # hand arithmetic for this seed (128 requests x 16 384 shared tokens, suffix sum 296 899, 4096 B per token and Full
    # layer, 128 window slots per SWA layer): 10.24 GB logical, 1.72 GB unique per 7-layer step
    assert abs(logical / 1e9 - 10.24) < 0.01 and abs(unique / 1e9 - 1.72) < 0.01
    # per layer: the sum over layers reproduces the step
    per = sum(accounting.decode_layer_bytes(w, s, unique=True) for s in w.layer_is_swa)
    assert per == unique
    # no sharing: both figures agree
    w2 = wl.config2()
    assert accounting.decode_algorithmic_bytes(w2) == accounting.decode_unique_bytes(w2)
    assert abs(accounting.decode_algorithmic_bytes(w2) / 1e9 - 5.29) < 0.01
    assert abs(accounting.decode_algorithmic_bytes(wl.config5()) / 1e9 - 100.3) < 0.1


def test_prefill_compulsory_bytes_config3():
    w = wl.config3()
    assert abs(accounting.prefill_compulsory_bytes(w, True) / 1e9 - 2.42) < 0.01   # Q + O 2.15 GB + new KV 0.27 GB
    assert abs(accounting.prefill_flops(w, False) / 1e12 - 25.28) < 0.01


def test_compact_tables_keep_shared_pages_once_and_preserve_the_mapping():
    w = wl.config4(batch=6, prefix=256)
    t, d = w.tables, w.dims
    reqs = bench.pick_requests(t, 3)
    assert len(reqs) == 3 and int(np.argmax(t.ctx_len)) in reqs and int(np.argmin(t.ctx_len)) in reqs
    bt, full_ids, rt, ring_ids = bench.compact_tables(t, d, reqs)
    assert len(set(full_ids.tolist())) == len(full_ids)                      # every physical page once
    for i, r in enumerate(reqs):
        need = -(-(int(t.ctx_len[r]) + 1) // d.page_size)
        assert np.array_equal(full_ids[bt[i, :need]], t.block_table[r, :need])  # compact id -> same physical page
        assert np.array_equal(ring_ids[rt[i]], t.ring_table[r])
    shared = t.shared_prefix_pages
    assert shared == 4 and (bt[:, :shared] == bt[0, :shared]).all()            # still shared after renumbering


def test_reference_arm_prints_one_extrapolated_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg2",
                          "--batch", "3", "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["impl"] == "reference" and line["extrapolated"] is True and line["gpu_launches"] == 0
    assert line["value"] > 0 and line["measured_seconds_per_step_sample"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("cfg2") and line["config"]["batch"] == 3
