#!/usr/bin/env python
"""Benchmark of the hybrid-SWA attention hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg4|cfg5|cfg3] [--impl reference]

A "step" is one pass of the whole hot path over one synthetic batch: for every layer of the stack the fused
KV append + attention (+ split combine), then the step advance.  The default workload is the largest
single-GPU configuration: the full-stack long-context decode step (70 layers = 60 SWA + 10 Full, batch 16,
contexts U[64k, 256k], 100 GB of KV per step).  The default run also reports, under "extra", the other named
configurations, each with its own warm-up, >= 20 timed steps and clock record: the 7-layer decode block at batch 64
(one token per request, and 4 tokens per request through the multi-token entry point), the prefix-hit decode
(plain and cascade, against logical and unique bytes) and the chunked-prefill block (per-layer-kind rooflines).
One JSON line is printed by rank 0.  With N > 1 (torchrun) every rank runs its own batch (weak scaling, no
data-path collective) and the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode_attn_tokens_per_s"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg2", "cfg3", "cfg4", "cfg5", "prefix_sweep", "prefetch", "buckets"])
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (cfg5: fewer to fit)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (smaller cases for profiling)")
    ap.add_argument("--chunk", type=int, default=0, help="cfg3: override the prefill chunk length")
    ap.add_argument("--mtp", type=int, default=1, help="decode q_len per request (2-4: hswa_decode_attn_mtp)")
    ap.add_argument("--cascade", action="store_true", help="cfg4: use hswa_decode_attn_shared_prefix on the shared prefix")
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations reported under 'extra'")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="run the end-to-end step eagerly instead of as a CUDA graph")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def stored_traffic(key):
    """DRAM bytes per launch from a committed ncu capture, if one was recorded for this kernel/workload."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if os.path.exists(path):
        return json.load(open(path)).get(key)
    return None


def make_workload(name, seed_offset=0, layers=0, batch=0, chunk=0):
    from paper_2607_13095_b200 import workloads as wl
    kw = {"batch": batch} if batch else {}
    if name == "cfg2":
        return wl.config2(seed=2 + seed_offset, **kw)
    if name == "cfg3":
        if chunk:
            kw["chunk"] = chunk
        return wl.config3(seed=3 + seed_offset, **kw)
    if name == "cfg4":
        return wl.config4(seed=4 + seed_offset, **kw)
    return wl.config5(seed=5 + seed_offset, num_layers=layers or 70, **kw)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev)
                for bit, nm in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


# ---------------------------------------------------------------------------------------------------------
class DecodeBench:
    """Device-resident state of a decode workload and one-step runner."""

    def __init__(self, w, total_steps, device, cascade=False, mtp=1):
        self.shared_prefix = w.tables.shared_prefix_pages * w.dims.page_size if cascade else 0
        self.mtp = mtp
        import torch
        from paper_2607_13095_b200 import binding as hb
        from paper_2607_13095_b200 import workloads as wl
        self.torch, self.hb, self.w = torch, hb, w
        d, t0 = w.dims, w.tables
        # page ids for the contexts plus the tokens the run will append
        self.t = wl.make_tables(d, t0.ctx_len, np.full(t0.batch, total_steps + 1 + mtp), w.seed,
                                shared_prefix_tokens=t0.shared_prefix_pages * d.page_size, slack=1.0)
        t = self.t
        g = torch.Generator(device=device)
        g.manual_seed(w.seed)
        self.h = hb.Handle(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages, 0.0,
                           torch.bfloat16)
        self.layers = []
        for is_swa in w.layer_is_swa:
            n_pages = t.num_ring_pages if is_swa else t.num_full_pages
            pool = torch.empty((n_pages, 2, d.num_kv_heads, d.page_size, d.head_dim), dtype=torch.bfloat16, device=device)
            pool.normal_(generator=g)
            self.layers.append(hb.Layer(pool, is_swa))
        L, B = len(self.layers), t.batch * mtp
        self.q = torch.randn((L, B, d.num_q_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.k_new = torch.randn((L, B, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.v_new = torch.randn((L, B, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.out = torch.empty((L, B, d.num_q_heads, d.head_dim), device=device, dtype=torch.bfloat16)
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.ctx0, self.head0 = i32(t.ctx_len), i32(t.ring_head)
        self.ctx, self.head = self.ctx0.clone(), self.head0.clone()
        B = t.batch
        # bound of ctx_len over the run: one accepted token per step; the tables above cover max_ctx + mtp positions
        self.max_ctx = int(t.ctx_len.max()) + total_steps
        self.batch = hb.Batch(self.ctx, i32(t.block_table), i32(t.ring_table), self.head, None, max_q_len=1,
                              total_q=B, max_ctx_len=self.max_ctx)
        ws_bytes = hb.hswa_workspace_bytes(self.h, B, B * mtp, self.max_ctx)
        self.ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=device)
        self.full_idx = [i for i, s in enumerate(w.layer_is_swa) if not s]
        # kernels per Full layer: decode + combine (+ the shared-prefix stage); with draft tokens: append + decode + combine
        self.launches_per_step = sum(1 if s else (3 if (self.shared_prefix or mtp > 1) else 2) for s in w.layer_is_swa) + 1

    def reset(self):
        self.ctx.copy_(self.ctx0)
        self.head.copy_(self.head0)

    def step(self, events=None, layer_hook=None):
        hb = self.hb
        for i, layer in enumerate(self.layers):
            timed = events is not None and i == self.full_idx[0]
            if timed:
                events[0].record()
            if self.mtp > 1:
                hb.hswa_decode_attn_mtp(self.h, layer, self.batch, self.mtp, self.q[i], self.k_new[i], self.v_new[i],
                                        self.out[i], None, self.ws)
            elif self.shared_prefix:
                hb.hswa_decode_attn_shared_prefix(self.h, layer, self.batch, self.shared_prefix, self.q[i], self.k_new[i],
                                                  self.v_new[i], self.out[i], None, self.ws)
            else:
                hb.hswa_decode_attn(self.h, layer, self.batch, self.q[i], self.k_new[i], self.v_new[i], self.out[i], None,
                                    self.ws)
            if timed:
                events[1].record()
            if layer_hook is not None:
                layer_hook(i)
        hb.hswa_step_advance(self.h, self.t.batch, self.ctx, self.head, None)


class PrefillBench:
    def __init__(self, w, device):
        import torch
        from paper_2607_13095_b200 import binding as hb
        self.torch, self.hb, self.w = torch, hb, w
        d, t = w.dims, w.tables
        g = torch.Generator(device=device)
        g.manual_seed(w.seed)
        self.h = hb.Handle(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages, 0.0,
                           torch.bfloat16)
        self.layers = []
        for is_swa in w.layer_is_swa:
            n_pages = t.num_ring_pages if is_swa else t.num_full_pages
            pool = torch.empty((n_pages, 2, d.num_kv_heads, d.page_size, d.head_dim), dtype=torch.bfloat16, device=device)
            pool.normal_(generator=g)
            self.layers.append(hb.Layer(pool, is_swa))
        T = t.total_q
        # one set of activations shared by the layers of a kind keeps the footprint small; K/V/Q are > L2 anyway
        self.q = torch.randn((T, d.num_q_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.k_new = torch.randn((T, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.v_new = torch.randn((T, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
        self.out = torch.empty((T, d.num_q_heads, d.head_dim), device=device, dtype=torch.bfloat16)
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.batch = hb.Batch(i32(t.ctx_len), i32(t.block_table), i32(t.ring_table), i32(t.ring_head), i32(t.q_indptr),
                              max_q_len=t.max_q_len, total_q=T, max_ctx_len=t.max_ctx_len)

    def run_layer(self, i, events=None):
        """One layer: attention + KV append.  With events, the two are issued as separate calls (the library runs
        the same two kernels in the same order either way) so that the attention kernel can be timed by itself."""
        if events is None:
            self.hb.hswa_prefill_attn(self.h, self.layers[i], self.batch, self.q, self.k_new, self.v_new, True, self.out,
                                      None, None)
            return
        events[0].record()
        self.hb.hswa_prefill_attn(self.h, self.layers[i], self.batch, self.q, self.k_new, self.v_new, False, self.out,
                                  None, None)
        events[1].record()
        self.hb.hswa_kv_append(self.h, self.layers[i], self.batch, self.k_new, self.v_new)


def time_events(torch, fn, warmup, steps):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def stats(xs):
    xs = np.asarray(xs, dtype=np.float64)
    return {"mean": float(xs.mean()), "median": float(np.median(xs)), "min": float(xs.min()), "max": float(xs.max()),
            "n": int(xs.size)}


def time_launches(torch, fn, warmup, n, index):
    """n separately timed calls of fn (CUDA events on the current stream) after `warmup` untimed ones, with the SM
    clock sampled meanwhile.  Returns (per-call ms list, clock summary)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    with ClockSampler(index) as clocks:
        for a, b in ev:
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in ev], clocks.summary()


def prefill_extra(device, peaks, index=0, launches=20):
    """Chunked-prefill block (8 requests x 8192 new tokens over cached contexts U[0, 16k]): each layer kind timed
    over `launches` separately timed layer calls (attention + append) after 3 warm-ups, with its own roofline
    object and clock record.  Inputs (Q 1.07 GB, chunk K/V 0.27 GB, output 1.07 GB) are larger than L2."""
    import torch
    from paper_2607_13095_b200 import accounting
    from paper_2607_13095_b200 import binding as hb
    w = make_workload("cfg3")
    pb = PrefillBench(w, device)
    full_i = w.layer_is_swa.index(False)
    swa_i = w.layer_is_swa.index(True)
    ms_full, clk_full = time_launches(torch, lambda: pb.run_layer(full_i), 3, launches, index)
    ms_swa, clk_swa = time_launches(torch, lambda: pb.run_layer(swa_i), 3, launches, index)
    # the SWA layer again right behind a Full layer, i.e. at the clock the Full layer leaves behind (as in the block)
    ms_swa_in_block = []
    for _ in range(5):
        pb.run_layer(full_i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        pb.run_layer(swa_i)
        e1.record()
        torch.cuda.synchronize()
        ms_swa_in_block.append(e0.elapsed_time(e1))
    st = hb.hswa_get_async_error(pb.h)
    if st[0] != hb.HSWA_OK:
        raise SystemExit(f"device error word set during the prefill block: {st}")
    sf, ss = stats(ms_full), stats(ms_swa)
    f_full, f_swa = accounting.prefill_flops(w, False), accounting.prefill_flops(w, True)
    b_swa = accounting.prefill_compulsory_bytes(w, True)
    n_full = sum(1 for s in w.layer_is_swa if not s)
    n_swa = len(w.layer_is_swa) - n_full
    swa_blk = float(np.median(ms_swa_in_block))
    block_ms = n_full * sf["mean"] + n_swa * swa_blk
    tf = f_full / (sf["mean"] * 1e-3) / 1e12
    gbs = b_swa / (ss["mean"] * 1e-3) / 1e9
    return {
        "workload": w.name, "launches_timed": launches, "warmup": 3,
        "full_layer_ms": sf["mean"], "full_layer_ms_stats": sf, "swa_layer_ms": ss["mean"], "swa_layer_ms_stats": ss,
        "swa_layer_ms_behind_full_layer": swa_blk,
        "full_layer_tflops": tf, "swa_layer_tflops": f_swa / (ss["mean"] * 1e-3) / 1e12,
        "block_ms": block_ms, "block_tflops": (n_full * f_full + n_swa * f_swa) / (block_ms * 1e-3) / 1e12,
        "block_tokens_per_s": w.tables.total_q / (block_ms * 1e-3),
        "full_layer_roofline": {
            "bound": "tensor", "achieved": tf, "unit": "TFLOP/s", "peak": peaks["bf16_tflops"],
            "frac": tf / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (cuBLAS bf16 burst)",
            "frac_of_measured_sustained": tf / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": tf / 2250.0,
            "ms_per_launch": sf["mean"], "algorithmic_flops_per_launch": f_full,
            "traffic": stored_traffic("prefill_full_cfg3"),
            "kernel": "prefill_tc_kernel + append_kernel, one Full layer", "clocks": clk_full},
        "swa_layer_roofline": {
            "bound": "hbm", "achieved": gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
            "peak_source": peaks["source"], "frac_of_nominal_8TBs": gbs / 8000.0, "ms_per_launch": ss["mean"],
            "algorithmic_bytes_per_launch": b_swa, "traffic": stored_traffic("prefill_swa_cfg3"),
            "kernel": "SWA prefill kernels + append_ring_kernel, one SWA layer", "clocks": clk_swa},
    }


# ---------------------------------------------------------------------------------------------------------
def pick_requests(t, n):
    """A bounded sample of requests: the longest, the shortest and evenly spaced others (deterministic)."""
    order = np.argsort(t.ctx_len, kind="stable")
    idx = {int(order[-1]), int(order[0])}
    for k in np.linspace(0, t.batch - 1, num=max(n, 2)):
        if len(idx) >= n:
            break
        idx.add(int(order[int(round(k))]))
    return np.array(sorted(idx), dtype=np.int64)


def compact_tables(t, d, reqs):
    """Block and ring tables of the requests `reqs` renumbered onto compact pools that hold only their pages.
    Returns (block_table, full page ids in compact order, ring_table, ring page ids in compact order).  Pure
    bookkeeping: which physical page sits where; pages shared between requests are kept once."""
    need = [-(-(int(t.ctx_len[r]) + 1) // d.page_size) for r in reqs]
    full_ids, remap = [], {}
    bt = np.zeros((len(reqs), max(need)), dtype=np.int32)
    for i, r in enumerate(reqs):
        for j in range(need[i]):
            pg = int(t.block_table[r, j])
            if pg not in remap:
                remap[pg] = len(full_ids)
                full_ids.append(pg)
            bt[i, j] = remap[pg]
    ring_ids = t.ring_table[reqs].reshape(-1)
    rt = np.arange(ring_ids.size, dtype=np.int32).reshape(len(reqs), -1)
    return bt, np.array(full_ids, dtype=np.int64), rt, ring_ids.astype(np.int64)


def oracle_decode_sample(w, t, reqs, bt, full_pool, rt, ring_pool, q, k, v, heads_full=None):
    """Time the CPU oracle, as it stands, on all (or `heads_full`) query heads of the requests `reqs` for one Full
    and one SWA layer, and extrapolate to a whole step by key count.  Pools and tables are the compact ones of
    compact_tables; q, k, v hold only those requests.  Returns (estimated seconds per step, description, threads,
    measured seconds)."""
    from oracle import hswa_oracle as orc
    d = w.dims
    cfg = orc.OracleConfig(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages)
    ob = orc.OracleBatch(t.ctx_len[reqs], bt, rt, t.ring_head[reqs])
    n_full = sum(1 for s in w.layer_is_swa if not s)
    n_swa = len(w.layer_is_swa) - n_full
    est, spent, desc = 0.0, 0.0, []
    for is_swa, pool, count in ((False, full_pool, n_full), (True, ring_pool, n_swa)):
        Hq = d.num_q_heads
        heads = np.arange(Hq) if (is_swa or heads_full is None) else np.asarray(heads_full)
        tok = np.repeat(np.arange(len(reqs)), len(heads)).astype(np.int32)
        head = np.tile(heads, len(reqs)).astype(np.int32)
        keys = np.minimum(t.ctx_len.astype(np.int64) + 1, d.window) if is_swa else t.ctx_len.astype(np.int64) + 1
        total_keys = float(keys.sum()) * Hq
        sample_keys = float(keys[reqs].sum()) * len(heads)
        layer = orc.OracleLayer(pool, is_swa)
        t0 = time.perf_counter()
        orc.attention(cfg, layer, ob, q, k, v, rows=(tok, head))
        dt = time.perf_counter() - t0
        spent += dt
        est += dt * (total_keys / max(sample_keys, 1.0)) * count
        desc.append(f"{'swa' if is_swa else 'full'} layer: {len(tok)} of {t.batch * Hq} (request, head) rows "
                    f"({len(reqs)} requests x {len(heads)} heads) in {dt:.2f}s, scaled by keys "
                    f"x{total_keys / max(sample_keys, 1.0):.2f} and x{count} layers")
    return est, "; ".join(desc), orc.num_threads(), spent


def host_bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def cpu_baseline_decode(bench, n_requests=4):
    """The oracle on a bounded sample of the bench's own device state (the pages of a few requests are gathered on
    the device and copied to the host, so a 10 GB pool never crosses PCIe whole)."""
    import torch
    w, t, d = bench.w, bench.t, bench.w.dims
    fi, si = bench.full_idx[0], w.layer_is_swa.index(True)
    reqs = pick_requests(t, min(n_requests, t.batch))
    bt, full_ids, rt, ring_ids = compact_tables(t, d, reqs)
    dev = bench.layers[fi].pool.device
    full_pool = host_bits(bench.layers[fi].pool.index_select(0, torch.from_numpy(full_ids).to(dev)))
    ring_pool = host_bits(bench.layers[si].pool.index_select(0, torch.from_numpy(ring_ids).to(dev)))
    ridx = torch.from_numpy(reqs).to(dev)
    q, k, v = (host_bits(x[fi].index_select(0, ridx)) for x in (bench.q, bench.k_new, bench.v_new))
    est, desc, threads, spent = oracle_decode_sample(w, t, reqs, bt, full_pool, rt, ring_pool, q, k, v)
    return {"value": t.batch / est, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
            "extrapolated": True, "measured_seconds": spent}


# ---------------------------------------------------------------------------------------------------------
def run_reference(args):
    """The reference arm: the fp64 CPU oracle, as it stands, on the host cores.  Each step times a bounded sample
    of the workload (a few requests, a few heads of the Full layer, every head of an SWA layer) and extrapolates to
    the whole step by key count; the line says so ("extrapolated") and gives the seconds actually measured."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_13095_b200 import workloads as wl
    w = make_workload(args.workload if args.workload != "cfg3" else "cfg2", layers=args.layers, batch=args.batch)
    d, t = w.dims, w.tables
    reqs = pick_requests(t, min(3, t.batch))
    bt, full_ids, rt, ring_ids = compact_tables(t, d, reqs)

    # host-only state: compact pools filled by repeating a random 64-page block (the values do not affect time)
    def rand_pool(n_pages, seed):
        base = wl.bf16_bits_normal(seed, (min(n_pages, 64), 2, d.num_kv_heads, d.page_size, d.head_dim))
        return np.resize(base, (n_pages,) + base.shape[1:])
    full_pool, ring_pool = rand_pool(len(full_ids), 11), rand_pool(len(ring_ids), 12)
    q = wl.bf16_bits_normal(13, (len(reqs), d.num_q_heads, d.head_dim))
    k = wl.bf16_bits_normal(14, (len(reqs), d.num_kv_heads, d.head_dim))
    v = wl.bf16_bits_normal(15, (len(reqs), d.num_kv_heads, d.head_dim))
    # heads of the Full layer per step: about 5e7 (row, key) pairs, i.e. a second or two on a few cores
    keys = float((t.ctx_len[reqs].astype(np.int64) + 1).sum())
    n_heads = int(min(d.num_q_heads, max(1, round(5e7 / keys))))
    ests, spents = [], []
    desc, threads = "", 1
    for i in range(args.warmup + args.steps):
        heads = (np.arange(n_heads) * (d.num_q_heads // n_heads) + i) % d.num_q_heads
        est, desc, threads, spent = oracle_decode_sample(w, t, reqs, bt, full_pool, rt, ring_pool, q, k, v, heads_full=heads)
        if i >= args.warmup:
            ests.append(est)
            spents.append(spent)
    sec = float(np.mean(ests))
    val = t.batch / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "extrapolated": True,
        "measured_seconds_per_step_sample": float(np.mean(spents)),
        "config": workload_config(w, t, False, 1) | {
            "note": "CPU oracle timed on a bounded sample per step and extrapolated by key count; ms_per_step is that "
                    "estimate, measured_seconds_per_step_sample the time each step's sample really took"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, t, cascade, mtp):
    d = w.dims
    return {"workload": w.name, "layers": len(w.layer_is_swa), "swa_layers": int(sum(w.layer_is_swa)),
            "batch": t.batch, "num_q_heads": d.num_q_heads, "num_kv_heads": d.num_kv_heads,
            "head_dim": d.head_dim, "page_size": d.page_size, "window": d.window,
            "ctx_sum": int(t.ctx_len.astype(np.int64).sum()), "shared_prefix_tokens": t.shared_prefix_pages * d.page_size,
            "cascade": bool(cascade), "mtp_q_len": mtp, "l2": "inputs larger than L2 (Full-layer KV streamed per step "
            "exceeds 126 MB and evicts the SWA rings between reuses)", "out_dtype": "bf16"}


def run_prefix_sweep(args, torch, device, peaks):
    """Paper Sec. 5.2 (figure: relative prefill throughput vs cached sequence length with a fixed 16K compute
    chunk): one request, a 16 384-token chunk, cached prefix 0 / 64K / 256K / 1M tokens (the paper's length
    buckets), attention of one hybrid block (1 Full + 6 SWA layers) only.  Prints tokens/s per prefix and the
    throughput relative to the empty prefix."""
    from paper_2607_13095_b200 import accounting
    from paper_2607_13095_b200 import workloads as wl
    chunk = args.chunk or 16384
    rows = []
    for prefix in (0, 65536, 262144, 1048576):
        t = wl.make_tables(wl.BIG, [prefix], [chunk], seed=7, slack=1.0)
        w = wl.Workload(f"prefix{prefix}-chunk{chunk}", wl.BIG, wl.hybrid_layer_flags(7)[:2], t, 7)
        pb = PrefillBench(w, device)
        ms_full = time_events(torch, lambda: pb.run_layer(0), 1, max(1, args.steps // 10))
        ms_swa = time_events(torch, lambda: pb.run_layer(1), 2, 10)
        block_ms = ms_full + 6 * ms_swa
        rows.append({"prefix": prefix, "full_layer_ms": ms_full, "swa_layer_ms": ms_swa, "block_ms": block_ms,
                     "tokens_per_s": chunk / (block_ms * 1e-3),
                     "full_layer_tflops": accounting.prefill_flops(w, False) / (ms_full * 1e-3) / 1e12})
        del pb
        torch.cuda.empty_cache()
    base = rows[0]["tokens_per_s"]
    for r_ in rows:
        r_["relative"] = r_["tokens_per_s"] / base
    print(json.dumps({"metric": "prefill_attn_relative_throughput_vs_prefix", "unit": "x", "chunk": chunk,
                      "value": rows[-1]["relative"], "rows": rows, "n_gpus": 1, "data": "synthetic", "dtype": "bf16",
                      "note": "attention + append of one 1 Full + 6 SWA block; the paper's whole-model curve falls to "
                              "about 0.12x at a 1M prefix (unnamed GPU), attention alone falls further"}))


def run_length_buckets(args, torch, device):
    """Paper Sec. 5.3 (length bucketing): when requests whose cached prefixes differ a lot are scheduled into the
    same chunked-prefill step of one instance, its data-parallel attention ranks synchronise after every layer and
    all wait for the rank with the longest prefix.  Emulates one instance of 8 such ranks on this GPU, one rank at
    a time: a rank's work is one request's 16K-token chunk over its cached prefix through one hybrid block
    (1 Full + 6 SWA layers), and a synchronised step costs its slowest rank.  48 seeded requests (24 / 16 / 8 in
    the paper's tiers 0-64K / 64K-256K / 256K-1M) are scheduled in arrival order and with the three-tier bucketing
    (every step's 8 requests come from one tier); the balanced bound is the sum of all times / 8."""
    from paper_2607_13095_b200 import workloads as wl
    chunk, ranks = args.chunk or 16384, 8
    rng = np.random.default_rng(53)
    tiers = [(0, 65536, 24), (65536, 262144, 16), (262144, 1048576 - chunk, 8)]
    reqs = [(ti, int(rng.integers(lo, hi))) for ti, (lo, hi, n) in enumerate(tiers) for _ in range(n)]
    order = rng.permutation(len(reqs))  # arrival order
    ms = []
    for ti, prefix in reqs:
        t = wl.make_tables(wl.BIG, [prefix], [chunk], seed=7, slack=1.0)
        w = wl.Workload(f"prefix{prefix}-chunk{chunk}", wl.BIG, wl.hybrid_layer_flags(7)[:2], t, 7)
        pb = PrefillBench(w, device)
        ms_full = time_events(torch, lambda: pb.run_layer(0), 1, 1 if prefix > 262144 else 2)
        ms_swa = time_events(torch, lambda: pb.run_layer(1), 1, 3)
        ms.append(ms_full + 6 * ms_swa)
        del pb
        torch.cuda.empty_cache()
    ms = np.array(ms)

    def schedule(seq):
        return float(sum(ms[seq[i:i + ranks]].max() for i in range(0, len(seq), ranks)))

    arrival = [int(i) for i in order]
    bucketed = sorted(arrival, key=lambda i: reqs[i][0])  # stable: arrival order inside a tier
    t_mixed, t_bucket, t_bound = schedule(arrival), schedule(bucketed), float(ms.sum() / ranks)
    tokens = len(reqs) * chunk
    balance = one_launch_balance(torch, device, reqs, arrival, bucketed, ranks)
    print(json.dumps({
        "metric": "prefill_attn_tokens_per_s_bucketed_vs_arrival_order", "unit": "x", "value": t_mixed / t_bucket,
        "chunk": chunk, "ranks": ranks, "requests": len(reqs), "n_gpus": 1, "data": "synthetic", "dtype": "bf16",
        "tokens_per_s": {"arrival_order": tokens / (t_mixed * 1e-3), "three_tier_buckets": tokens / (t_bucket * 1e-3),
                         "balanced_bound": tokens / (t_bound * 1e-3)},
        "block_ms_by_tier": [float(ms[[i for i, r_ in enumerate(reqs) if r_[0] == ti]].mean()) for ti in range(3)],
        "one_launch_balance": balance,
        "note": "8 data-parallel attention ranks of one instance emulated one at a time on one GPU; a step costs its "
                "slowest rank (per-layer synchronisation before the MoE stage); attention + append of one hybrid block"}))


def one_launch_balance(torch, device, reqs, arrival, bucketed, per_batch, chunk=2048):
    """The same requests batched 8 at a time into ONE Full-layer prefill launch each (a 2048-token chunk per request
    over its cached prefix), in arrival order and bucketed by the paper's three tiers, with the blocks of a launch
    handed out request by request in batch order, longest request first (the default) and globally longest tile first.  Measured from per-block start / end stamps
    (hswa_set_block_trace): the idle tail of an SM is the time between its last block's end and the launch's end;
    reported as the mean over SMs, as a share of the launch's span, weighted by span over the launches."""
    from paper_2607_13095_b200 import binding as hb
    from paper_2607_13095_b200 import workloads as wl
    d = wl.BIG
    h = hb.Handle(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages, 0.0, torch.bfloat16)
    g = torch.Generator(device=device)
    g.manual_seed(11)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
    res = {}
    for sched_name, seq in (("arrival_order", arrival), ("three_tier_buckets", bucketed)):
        acc = {m: {"span_ms": 0.0, "idle_ms": 0.0} for m in ("by_request", "longest_request_first", "longest_tile_first")}
        for i in range(0, len(seq), per_batch):
            prefixes = [reqs[j][1] for j in seq[i:i + per_batch]]
            t = wl.make_tables(d, prefixes, [chunk] * len(prefixes), seed=7, slack=1.0)
            pool = torch.empty((t.num_full_pages, 2, d.num_kv_heads, d.page_size, d.head_dim), dtype=torch.bfloat16, device=device)
            pool.normal_(generator=g)
            layer = hb.Layer(pool, False)
            T = t.total_q
            q = torch.randn((T, d.num_q_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
            k = torch.randn((T, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
            v = torch.randn((T, d.num_kv_heads, d.head_dim), generator=g, device=device, dtype=torch.bfloat16)
            out = torch.empty((T, d.num_q_heads, d.head_dim), device=device, dtype=torch.bfloat16)
            batch = hb.Batch(i32(t.ctx_len), i32(t.block_table), i32(t.ring_table), i32(t.ring_head), i32(t.q_indptr),
                             max_q_len=t.max_q_len, total_q=T, max_ctx_len=t.max_ctx_len)
            blocks = (d.group // 2) * d.num_kv_heads * t.batch * ((chunk + 127) // 128)
            for mode_name, mode in (("by_request", hb.PREFILL_ORDER_BY_REQUEST),
                                    ("longest_request_first", hb.PREFILL_ORDER_LONGEST_REQUEST_FIRST),
                                    ("longest_tile_first", hb.PREFILL_ORDER_LONGEST_TILE_FIRST)):
                hb.hswa_set_prefill_order(h, mode)
                trace = torch.zeros((blocks, 4), dtype=torch.int64, device=device)
                hb.hswa_set_block_trace(h, trace)
                hb.hswa_prefill_attn(h, layer, batch, q, k, v, False, out, None, None)
                torch.cuda.synchronize()
                hb.hswa_set_block_trace(h, None)
                tr = trace.cpu().numpy()
                tr = tr[tr[:, 1] > 0]
                start, end = tr[:, 0].min(), tr[:, 1].max()
                last_on_sm = np.array([tr[tr[:, 2] == s_, 1].max() for s_ in np.unique(tr[:, 2])])
                acc[mode_name]["span_ms"] += float(end - start) * 1e-6
                acc[mode_name]["idle_ms"] += float((end - last_on_sm).mean()) * 1e-6
            del pool, q, k, v, out
            torch.cuda.empty_cache()
        res[sched_name] = {m: {"launch_ms_total": a_["span_ms"], "idle_tail_frac": a_["idle_ms"] / a_["span_ms"]}
                           for m, a_ in acc.items()}
    st = hb.hswa_get_async_error(h)
    if st[0] != hb.HSWA_OK:
        raise SystemExit(f"device error word set: {st}")
    res["chunk"] = chunk
    res["batch"] = per_batch
    return res


def run_layerwise_prefetch(args, torch, device):
    """Paper Sec. 3.1.2 (layerwise KVCache prefetch): the SWA state of every request lives in pinned host memory
    (W - 1 tokens per request and SWA layer: the only part a resumed request needs) and is loaded back layer by
    layer.  Times one config-5-shaped decode step (70 layers, batch 16) three ways: state already on the device;
    loadback of layer l right before layer l on the compute stream; loadback on a copy stream running ahead of
    the compute stream, gated per layer by events."""
    from paper_2607_13095_b200 import binding as hb
    w = make_workload("cfg5", layers=args.layers or 70, batch=args.batch)
    bench = DecodeBench(w, 8, device)
    d, t = w.dims, bench.t
    swa = [i for i, s_ in enumerate(w.layer_is_swa) if s_]
    shape = (t.batch, d.window - 1, 2, d.num_kv_heads, d.head_dim)
    host = {}
    for i in swa:  # offload: gather each SWA layer's windows into pinned host memory
        host[i] = torch.empty(shape, dtype=torch.bfloat16).pin_memory()
        hb.hswa_swa_window_gather(bench.h, bench.layers[i], bench.batch, host[i])
    torch.cuda.synchronize()
    copy_stream = torch.cuda.Stream(device=device, priority=-1)
    main = torch.cuda.current_stream()
    # device staging tiles: the DMA engine brings a layer's windows over PCIe, a small kernel scatters them
    staging = {i: torch.empty(shape, dtype=torch.bfloat16, device=device) for i in swa}

    def layer_call(i):
        hb.hswa_decode_attn(bench.h, bench.layers[i], bench.batch, bench.q[i], bench.k_new[i], bench.v_new[i], bench.out[i],
                            None, bench.ws)

    def step_resident():
        for i in range(len(bench.layers)):
            layer_call(i)

    def step_serial():
        for i in range(len(bench.layers)):
            if i in host:
                hb.hswa_swa_window_scatter(bench.h, bench.layers[i], bench.batch, host[i])
            layer_call(i)

    def step_overlapped():
        start = torch.cuda.Event()
        start.record(main)
        events = {}
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(start)  # the previous step has stopped reading the rings
            for i in swa:
                staging[i].copy_(host[i], non_blocking=True)
                hb.hswa_swa_window_scatter(bench.h, bench.layers[i], bench.batch, staging[i])
                events[i] = torch.cuda.Event()
                events[i].record(copy_stream)
        for i in range(len(bench.layers)):
            if i in events:
                main.wait_event(events[i])
            layer_call(i)

    res = {}
    for name, fn in (("resident", step_resident), ("loadback_serial", step_serial), ("loadback_layerwise", step_overlapped)):
        res[name + "_ms"] = time_events(torch, fn, 3, args.steps if args.steps < 50 else 10)
    st = hb.hswa_get_async_error(bench.h)
    if st[0] != hb.HSWA_OK:
        raise SystemExit(f"device error word set: {st}")
    bytes_per_step = len(swa) * int(np.prod(shape)) * 2
    print(json.dumps({"metric": "decode_step_ms_with_swa_loadback", "unit": "ms", "value": res["loadback_layerwise_ms"], **res,
                      "n_gpus": 1, "higher_is_better": False, "data": "synthetic", "dtype": "bf16",
                      "config": {"workload": w.name, "layers": len(w.layer_is_swa), "batch": t.batch},
                      "h2d_bytes_per_step": bytes_per_step,
                      "full_kv_bytes_if_not_windowed": int(t.ctx_len.astype(np.int64).sum()) * d.kv_bytes_per_token * len(swa)}))


def run_prefill_main(args, torch, dist, world, rank, local_rank, device, peaks):
    """--workload cfg3: the chunked-prefill block as the measured workload (value = attention TFLOP/s of the
    whole 1 Full + 6 SWA block, fused append included)."""
    from paper_2607_13095_b200 import accounting
    from paper_2607_13095_b200 import binding as hb
    w = make_workload("cfg3", seed_offset=rank, batch=args.batch, chunk=args.chunk)
    pb = PrefillBench(w, device)
    t, d = w.tables, w.dims
    full_i = w.layer_is_swa.index(False)
    L = len(w.layer_is_swa)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step(events=None):
        for i in range(L):
            pb.run_layer(i, events if events is not None and i == full_i else None)

    for _ in range(args.warmup):
        step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        e0.record()
        for k in range(args.steps):
            step(ev[k])
        e1.record()
        torch.cuda.synchronize()
    barrier()
    st = hb.hswa_get_async_error(pb.h)
    if st[0] != hb.HSWA_OK:
        raise SystemExit(f"device error word set during the timed region: {st}")
    tmax = torch.tensor([e0.elapsed_time(e1)], device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    ms_step = float(tmax.item()) / args.steps
    full_ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    f_full, f_swa = accounting.prefill_flops(w, False), accounting.prefill_flops(w, True)
    n_full = sum(1 for s in w.layer_is_swa if not s)
    flops_step = n_full * f_full + (L - n_full) * f_swa
    if rank != 0:
        return
    achieved = f_full / (full_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    line = {
        "metric": "prefill_attn_tflops", "value": flops_step * world / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "layers": L, "swa_layers": int(sum(w.layer_is_swa)), "batch": t.batch,
                   "chunk": int(t.q_len.max()), "ctx": [int(x) for x in t.ctx_len], "num_q_heads": d.num_q_heads,
                   "num_kv_heads": d.num_kv_heads, "head_dim": d.head_dim, "page_size": d.page_size,
                   "l2": "inputs larger than L2 (Q, K/V chunk and output tensors are 1.07 GB + 0.27 GB + 1.07 GB)"},
        "tokens_per_s": t.total_q * world / (ms_step * 1e-3),
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "traffic": stored_traffic("prefill_full_cfg3"), "kernel": "prefill_tc_kernel, one Full layer (its append_kernel, 0.09 ms, is in the step but not in this figure)",
                     "ms_per_launch": full_ms, "algorithmic_flops_per_launch": f_full, "peak_source": peaks["source"]
                     + " (sustained cuBLAS bf16; kernel timed inside a long step)",
                     "frac_of_measured_burst": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0},
        "clocks": clocks.summary(), "e2e": None, "gpu_launches": 2 * L * args.steps,
    }
    print(json.dumps(line))


def read_stream_gbs(torch, device):
    """A plain read-only stream over 4 GiB through the library's probe kernel (bulk copies into shared memory, no
    arithmetic), best of 7: what this machine's HBM gives a kernel that only reads, which is what decode attention does;
    reported beside the copy-based measured peak."""
    from paper_2607_13095_b200 import binding as hb
    from paper_2607_13095_b200 import workloads as wl
    d = wl.BIG
    h = hb.Handle(d.num_q_heads, d.num_kv_heads, d.head_dim, d.page_size, d.window, d.ring_pages, 0.0, torch.bfloat16)
    x = torch.empty(4 << 30, dtype=torch.uint8, device=device)
    x.zero_()
    best = float("inf")
    for _ in range(8):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        hb.hswa_probe_read_stream(h, x)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    if hb.hswa_get_async_error(h)[0] != hb.HSWA_OK:
        return None
    return x.numel() / (best * 1e-3) / 1e9


def measure_decode(bench, steps, warmup, index, barrier, world=1, dist=None):
    """Warm-up, then EXACTLY `steps` steps between two events (with barrier + synchronize on both sides); the first
    Full layer of every step is bracketed by its own events (the dominant kernel's launch time), every step by its
    own pair too (spread).  Returns a dict of times in ms and the clock record."""
    import torch
    from paper_2607_13095_b200 import binding as hb
    for _ in range(warmup):
        bench.step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    with ClockSampler(index) as clocks:
        marks[0].record()
        for k in range(steps):
            bench.step(ev[k])
            marks[k + 1].record()
        torch.cuda.synchronize()
    barrier()
    st = hb.hswa_get_async_error(bench.h)
    if st[0] != hb.HSWA_OK:
        raise SystemExit(f"device error word set during the timed region: {st}")
    ms_total = marks[0].elapsed_time(marks[-1])
    tmax = torch.tensor([ms_total], device=bench.ctx.device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    per_step = [marks[k].elapsed_time(marks[k + 1]) for k in range(steps)]
    full = [a.elapsed_time(b) for a, b in ev]
    n_full = len(bench.full_idx)
    n_swa = len(bench.layers) - n_full
    ms_step = float(tmax.item()) / steps
    return {"ms_per_step": ms_step, "ms_per_step_stats": stats(per_step), "full_layer_ms": float(np.mean(full)),
            "full_layer_ms_stats": stats(full),
            # what is left of a step after its Full layers, per SWA layer (includes the step advance)
            "swa_layer_ms_derived": max(ms_step - n_full * float(np.mean(full)), 0.0) / max(n_swa, 1),
            "clocks": clocks.summary()}


def decode_rooflines(w, bench, m, peaks, steps, warmup, read_gbs, traffic_key=None):
    """Roofline objects of a decode measurement: the Full-layer call against logical and unique bytes, the step."""
    from paper_2607_13095_b200 import accounting
    d, t = w.dims, bench.t
    grown = t.batch * (warmup + steps // 2) * d.kv_bytes_per_token  # context growth of the run so far (mean)
    logical = accounting.decode_layer_bytes(w, False) + grown
    unique = accounting.decode_layer_bytes(w, False, unique=True) + grown
    ms = m["full_layer_ms"]
    ach_l, ach_u = logical / (ms * 1e-3) / 1e9, unique / (ms * 1e-3) / 1e9
    shared = t.shared_prefix_pages > 0
    # a roofline is bytes that must cross the HBM interface: with a shared prefix that is the unique figure; the
    # logical figure (what a sharing-oblivious kernel asks for, partly served by L2) is reported beside it
    ach = ach_u if shared else ach_l
    roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
            "traffic": None,
            "kernel": ("append_kernel + decode_mtp_tc_kernel + combine_runs_kernel, one Full layer" if bench.mtp > 1 else
                       "decode_kernel + combine_kernel, one Full layer"
                       + (" (+ prefill_tc_kernel<prefix> with --cascade)" if bench.shared_prefix else "")),
            "ms_per_launch": ms, "algorithmic_bytes_per_launch": unique if shared else logical,
            "peak_source": peaks["source"] + " (copy: read + write bytes)", "frac_of_nominal_8TBs": ach / 8000.0,
            "frac_of_read_stream": (ach / read_gbs) if read_gbs else None, "read_stream_gbs": read_gbs}
    if shared:
        roof["bytes"] = "unique (the shared prefix counted once)"
        roof["frac_unique"] = ach_u / peaks["hbm_gbs"]
        roof["logical_gbs"] = ach_l
        roof["frac_logical"] = ach_l / peaks["hbm_gbs"]
        roof["logical_bytes_per_launch"] = logical
    per_key = stored_traffic("decode_full_dram_bytes_per_kv_byte")
    if per_key and not shared:
        roof["traffic"] = int(per_key * logical)
        roof["traffic_note"] = "ncu DRAM bytes of a small capture scaled by KV bytes (traffic is proportional to them)"
    step_l = accounting.decode_algorithmic_bytes(w)
    step_u = accounting.decode_unique_bytes(w)
    out = {"roofline": roof, "step_gbs": step_l / (m["ms_per_step"] * 1e-3) / 1e9,
           "step_frac_of_measured_hbm": (step_u if shared else step_l) / (m["ms_per_step"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    if shared:
        out["step_unique_gbs"] = step_u / (m["ms_per_step"] * 1e-3) / 1e9
        out["step_frac_logical"] = step_l / (m["ms_per_step"] * 1e-3) / 1e9 / peaks["hbm_gbs"]
    return out


def decode_extra(name, device, peaks, read_gbs, index, steps=30, warmup=5, cascade=False, mtp=1, batch=0):
    """One more decode configuration measured like the headline one (own warm-up, own clocks), as a summary dict."""
    import torch
    w = make_workload(name, batch=batch)
    bench = DecodeBench(w, 2 * (steps + warmup) + 8, device, cascade=cascade, mtp=mtp)

    def barrier():
        torch.cuda.synchronize()

    m = measure_decode(bench, steps, warmup, index, barrier)
    r = decode_rooflines(w, bench, m, peaks, steps, warmup, read_gbs)
    tokens = bench.t.batch * mtp
    res = {"workload": w.name, "cascade": bool(cascade), "mtp_q_len": mtp, "steps": steps, "warmup": warmup,
           "tokens_per_s": tokens / (m["ms_per_step"] * 1e-3), **m, **r,
           "gpu_launches": bench.launches_per_step * steps}
    del bench
    torch.cuda.empty_cache()
    return res


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2607_13095_b200 import binding as hb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    hb.load()
    peaks = measured_peaks()

    if args.workload == "prefetch":
        run_layerwise_prefetch(args, torch, device)
        return
    if args.workload == "prefix_sweep":
        run_prefix_sweep(args, torch, device, peaks)
        return
    if args.workload == "buckets":
        run_length_buckets(args, torch, device)
        return
    if args.workload == "cfg3":
        run_prefill_main(args, torch, dist, world, rank, local_rank, device, peaks)
        return
    read_gbs = read_stream_gbs(torch, device) if world == 1 else None
    with_extras = not args.no_extra and world == 1 and args.workload == "cfg5" and not args.layers and not args.batch
    # The compute-bound extra goes first: the prefill kernel runs against the board's power cap, and what clock the cap
    # leaves it depends on how warm the long memory-bound runs below have made the device.
    prefill_first = prefill_extra(device, peaks, local_rank) if with_extras else None
    torch.cuda.empty_cache()
    w = make_workload(args.workload, seed_offset=rank, layers=args.layers, batch=args.batch)
    total_steps = args.steps + args.warmup
    bench = DecodeBench(w, 2 * total_steps + 8, device, cascade=args.cascade, mtp=args.mtp)
    t, d = bench.t, w.dims

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    m = measure_decode(bench, args.steps, args.warmup, local_rank, barrier, world, dist)
    ms_step = m["ms_per_step"]
    tokens_per_step = t.batch * world * args.mtp  # with --mtp: query tokens scored per step (1 accepted + drafts)
    value = tokens_per_step / (ms_step * 1e-3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- end to end: pinned host inputs -> device, step, result -> host, every step ----
    e2e = None
    if not args.no_e2e:
        bench.reset()
        hq, hk, hv = (x.cpu().pin_memory() for x in (bench.q, bench.k_new, bench.v_new))
        hout = torch.empty_like(bench.out, device="cpu").pin_memory()

        # Three streams: the first (Full) layer's inputs go up first, the other layers' inputs follow while the Full
        # layer runs; every layer's output goes down as soon as the layer is done.  All copies of a step are inside
        # the timed region; the step ends when the last output has reached the host.
        s_up, s_down = torch.cuda.Stream(), torch.cuda.Stream()
        L = len(bench.layers)
        ev_in0, ev_in1 = torch.cuda.Event(), torch.cuda.Event()
        ev_layer = [torch.cuda.Event() for _ in range(L)]
        ev_free = torch.cuda.Event()

        def e2e_body():
            cur = torch.cuda.current_stream()
            ev_free.record(cur)  # device input buffers are free once the previous step's kernels are done
            with torch.cuda.stream(s_up):
                s_up.wait_event(ev_free)
                for x, hx in ((bench.q, hq), (bench.k_new, hk), (bench.v_new, hv)):
                    x[0].copy_(hx[0], non_blocking=True)
                ev_in0.record(s_up)
                for x, hx in ((bench.q, hq), (bench.k_new, hk), (bench.v_new, hv)):
                    x[1:].copy_(hx[1:], non_blocking=True)
                ev_in1.record(s_up)
            cur.wait_event(ev_in0)
            bench.step(layer_hook=lambda i: (ev_layer[i].record(cur), cur.wait_event(ev_in1) if i == 0 else None))
            with torch.cuda.stream(s_down):
                for i in range(L):
                    s_down.wait_event(ev_layer[i])
                    hout[i].copy_(bench.out[i], non_blocking=True)
            cur.wait_stream(s_down)

        # The step (copies, kernels, events) is captured once into a CUDA graph and replayed, which takes the
        # host's launch time out of the critical path, as a serving engine does for decode; if capture is not
        # possible the same body runs eagerly.
        e2e_mode = "eager"
        graph = None
        if not args.no_graph:
            try:
                e2e_body()  # warm the lazy initialisations outside the capture
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    e2e_body()
                e2e_mode = "cuda graph"
            except Exception as ex:  # noqa: BLE001
                sys.stderr.write(f"bench: e2e graph capture failed ({ex}); running eagerly\n")
                graph = None
                torch.cuda.synchronize()

        def e2e_step():
            if graph is not None:
                graph.replay()
            else:
                e2e_body()
            torch.cuda.synchronize()

        for _ in range(min(args.warmup, 5)):
            e2e_step()
        barrier()
        n_e2e = args.steps
        e0.record()
        for _ in range(n_e2e):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        if not torch.equal(hout.to(device), bench.out):  # the host really holds the last step's result
            raise RuntimeError("end-to-end step: host copy of the output differs from the device tensor")
        tm = torch.tensor([e0.elapsed_time(e1)], device=device, dtype=torch.float64)
        if world > 1:
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        e2e = {"value": tokens_per_step / (float(tm.item()) / n_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(sum(x.numel() * x.element_size() for x in (hq, hk, hv))),
               "d2h_bytes_per_step": int(hout.numel() * hout.element_size()),
               "mode": e2e_mode + ", per-layer copies on two side streams overlap the kernels"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: Full-layer decode (split-K partial kernel + combine) ----
    r = decode_rooflines(w, bench, m, peaks, args.steps, args.warmup, read_gbs)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "ms_per_step_stats": m["ms_per_step_stats"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, t, args.cascade, args.mtp),
        "full_layer_ms": m["full_layer_ms"], "swa_layer_ms_derived": m["swa_layer_ms_derived"],
        "step_gbs": r["step_gbs"] * world, "step_frac_of_measured_hbm": r["step_frac_of_measured_hbm"],
        "roofline": r["roofline"], "clocks": m["clocks"], "e2e": e2e,
        "gpu_launches": bench.launches_per_step * args.steps,
    }
    for key in ("step_unique_gbs", "step_frac_logical"):
        if key in r:
            line[key] = r[key]
    if not args.no_graph and world == 1:
        # The same device-resident step replayed as one CUDA graph (reported separately: the host's launch time
        # matters at small batch, where a layer's kernels are shorter than the calls that launch them).
        try:
            bench.reset()
            bench.step()
            torch.cuda.synchronize()
            g_step = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_step):
                bench.step()
            n_rep = min(args.steps, 2 * total_steps + 4)
            line["step_as_cuda_graph_ms"] = time_events(torch, g_step.replay, 3, max(1, n_rep - 3))
        except Exception as ex:  # noqa: BLE001
            sys.stderr.write(f"bench: step graph capture failed ({ex})\n")
            torch.cuda.synchronize()
    if not args.no_cpu_baseline and world == 1:
        bench.reset()
        line["cpu_baseline"] = cpu_baseline_decode(bench)
    if with_extras:
        # the other named configurations, one after the other on the freed device
        del bench
        torch.cuda.empty_cache()
        extra = {}
        extra["cfg2"] = decode_extra("cfg2", device, peaks, read_gbs, local_rank, steps=50)
        extra["mtp4"] = decode_extra("cfg2", device, peaks, read_gbs, local_rank, steps=30, mtp=4)
        extra["cfg4"] = {"plain": decode_extra("cfg4", device, peaks, read_gbs, local_rank, steps=30),
                         "cascade": decode_extra("cfg4", device, peaks, read_gbs, local_rank, steps=30, cascade=True)}
        extra["prefill"] = prefill_first
        extra["prefill"]["order"] = "measured first, before the decode configurations"
        line["extra"] = extra
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
