// Multi-token decode on Full layers with tcgen05 / TMEM / TMA (paper Sec. 6.2: a decode step carries the last
// accepted token plus up to 3 drafts per request; Sec. 2.2: decode is bound by the KV bytes it streams).
//
// The nq <= 4 new tokens x 8 query heads of one (request, KV head) are 32 rows of a 128-row MMA tile, so the
// whole group is served by one pass over the KV bytes and shared memory is read once per tile by the tensor core
// (the warp-MMA kernel reads every tile once per token and sits at the shared-memory bandwidth).
//
// Work: the 128-key tiles of all (request, KV head) streams form one flat sequence (prefix sums of the tile
// counts are computed in every block); block b takes the contiguous slice [b * per, (b + 1) * per) of it, so every
// SM streams the same number of bytes without a tail, and a slice may start and end in the middle of a stream.  A
// maximal piece of one stream inside a slice is a RUN; it ends in an unnormalised partial (m, l, o) per row, and a
// combine kernel merges the partials of a stream (runs are numbered stream index + block index, which is unique and
// contiguous per stream).
//
// Inside a block two CHAINS work on alternate tiles of the slice, each with its own K and V buffer, S / P and O
// columns of TMEM and softmax state; a chain is S = Q K^T -> softmax -> O += P V, strictly in that order, and the two
// chains overlap each other.  A Q tile in shared memory has the full 128 rows of an MMA tile, of which a TMA box fills
// the first 32 and the rest stay zero.  Chain 0's rows are TMEM lanes 0-31; chain 1's A descriptor starts 32 rows
// before the Q tile, so its rows are lanes 32-63 and the two softmax warps (warp 0 and warp 1: a warp may touch only
// the 32 lanes of its quarter) sit on different schedulers.  Warps: 0, 1 softmax; 2 TMA producer; 3, 4 MMA issuers
// (one per chain).  Every barrier is waited on, by parity, only by threads that see each of its phases in turn.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "hswa_internal.cuh"
#include "tc_primitives.cuh"

namespace {
using namespace hswa_dev;

namespace mtc {
constexpr int BN = 128;                    // keys per tile
constexpr int HD = 128;                    // head dim
constexpr int PG = 64;                     // page size
constexpr int ROWS = 32;                   // rows of a run: 4 token slots x 8 heads
constexpr int HALF_BYTES = BN * 128;       // one 64-element half of a K or V tile: [128 rows][128 B]
constexpr int TILE_BYTES = 2 * HALF_BYTES; // 32 KB
constexpr int Q_ROWS_BYTES = ROWS * 128;   // 4 KB: the rows a TMA box fills in each half of a Q tile
constexpr int Q_HALF = HALF_BYTES;         // a Q tile has the full 128 rows (the MMA reads them all); rows 32-127 stay zero
constexpr int Q_BYTES = 2 * Q_HALF;        // 32 KB
constexpr int OFF_Q = 4096;                // 4 KB of zeros in front: chain 1's A descriptor starts 32 rows early
constexpr int OFF_K = OFF_Q + 2 * Q_BYTES; // two Q tiles (runs alternate), then one K and one V tile per chain
constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;
constexpr int SMEM = OFF_V + 2 * TILE_BYTES + 1024;
// (Deeper buffering was measured and changes nothing: two K tiles or two V tiles per chain, same time; a ring of three
// tiles per chain shared by K and V, 5 % slower.  With one K and one V tile per chain the kernel already streams at the
// rate of the single-token kernel.)
constexpr int THREADS = 160;
constexpr int MAX_BATCH = 1024;            // prefix sums live in shared memory
constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t IDESC_PV = IDESC_S | (1u << 16);  // B (= V) is MN-major: [key][d] with d contiguous
// barriers; [c] = chain, [q] = Q buffer
enum { B_KFULL = 0, B_KEMPTY = 2, B_VFULL = 4, B_VEMPTY = 6, B_SFULL = 8, B_PFA = 10, B_PFB = 12, B_OFINAL = 14, B_OFREE = 16,
       B_VPATCH = 18, B_QFULL = 20, B_QFREE = 22, NBARS = 24 };

// A maximal piece of one (request, KV head) stream inside a block's slice of the flat tile sequence.
struct Run {
  int r, kh, t0, len, n0, rho;  // request, KV head, first tile of the stream, tiles, slice-local index of the first, run number
  int tiles_r;                  // tiles of the whole stream
};
struct RunIter {
  const int* cum;  // cum[r] = tiles of all streams of requests before r; cum[B] = total
  int B, Hkv, u0, u1, u, rho;
  __device__ RunIter(const int* cum_, int B_, int Hkv_, int u0_, int u1_) : cum(cum_), B(B_), Hkv(Hkv_), u0(u0_), u1(u1_), u(u0_), rho(0) {}
  __device__ bool next(Run& x) {
    if (u >= u1) return false;
    int lo = 0, hi = B;  // cum[lo] <= u < cum[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cum[mid] <= u) lo = mid; else hi = mid;
    }
    x.r = lo;
    x.tiles_r = (cum[lo + 1] - cum[lo]) / Hkv;
    const int rem = u - cum[lo];
    x.kh = rem / x.tiles_r;
    x.t0 = rem - x.kh * x.tiles_r;
    x.len = min(x.tiles_r - x.t0, u1 - u);
    x.n0 = u - u0;
    x.rho = rho++;
    u += x.len;
    return true;
  }
};
// Chain c's tiles of a run are the slice-local indices of parity c: first one, and whether there is any.
__device__ __forceinline__ int first_own(const Run& x, int c) { return x.n0 + ((c - x.n0) & 1); }
}  // namespace mtc

__global__ void __launch_bounds__(mtc::THREADS, 1)
decode_mtp_tc_kernel(const __grid_constant__ CUtensorMap tm_pool, const __grid_constant__ CUtensorMap tm_q, const DecodeParams p,
                     float* __restrict__ run_o, float2* __restrict__ run_ml, int2* __restrict__ stream_info) {
  using namespace mtc;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[NBARS];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int cum[MAX_BATCH + 1];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const ModelParams& M = p.m;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int B = p.b.B, nq = p.nq, Hkv = M.Hkv;

  // ---- tiles per request and their prefix sums (every block computes the same) ----
  // chunks of 32 requests: warp 0 scans them one after the other
  if (warp == 0) {
    int running = 0;
    for (int base = 0; base < B; base += 32) {
      const int r = base + lane;
      int t = 0;
      if (r < B) {
        const int ctx = p.b.ctx_len[r];
        if (blockIdx.x == 0 && ctx > p.max_ctx_len) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, ctx);
        t = ((min(ctx, p.max_ctx_len) + nq + BN - 1) / BN) * Hkv;
      }
      int incl = t;
#pragma unroll
      for (int sh = 1; sh < 32; sh <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += o;
      }
      if (r < B) cum[r] = running + incl - t;
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) cum[B] = running;
  }
  __syncthreads();
  const int total = cum[B];
  const int per = max(1, (total + (int)gridDim.x - 1) / (int)gridDim.x);
  const int u0 = blockIdx.x * per, u1 = min(total, u0 + per);
  if (u0 >= u1) return;
  if (*reinterpret_cast<volatile int32_t*>(p.err) != 0) return;

  auto bar = [&](int i) { return smem_u32(&bars[i]); };
  if (threadIdx.x == 0) {
    for (int i = 0; i < NBARS; ++i) mbar_init(bar(i), i >= B_QFREE ? 2 : 1);  // a Q buffer is released by both issuers
    mbar_fence_init();
  }
  // the rows of the Q tiles that no TMA box fills, and the padding in front, are read by every S MMA: zero, once
  for (int i = threadIdx.x; i < OFF_K / 16; i += THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;

  if (warp == 2) {
    // ======================= TMA producer =======================
    // Order of issue: Q of a run before its first K; K of tile n; then V of tile n - 1 (a K buffer is free as soon as
    // its S MMAs have run, a V buffer only after the PV MMAs, so K runs a tile ahead and does not queue behind V).
    tma_prefetch_desc(&tm_pool);
    tma_prefetch_desc(&tm_q);
    RunIter it(cum, B, Hkv, u0, u1);
    Run x;
    bool ok = true;
    bool pend = false;  // V of the previous tile is still to be issued
    int pend_pg0 = 0, pend_pg1 = 0, pend_n = 0, pend_kh = 0, pend_patch = 0, pend_r = 0;
    auto issue_v = [&]() {  // lane 0 only
      const int c = pend_n & 1, k = pend_n >> 1, vs = c;
      if (k >= 1 && !mbar_wait(bar(B_VEMPTY + vs), (k - 1) & 1)) {
        record_error(p.err, HSWA_ERR_TIMEOUT, pend_r, pend_n, 81);
        ok = false;
        return;
      }
      const uint32_t full = pend_patch ? bar(B_VPATCH + c) : bar(B_VFULL + vs);
      mbar_arrive_expect_tx(full, TILE_BYTES);
      const uint32_t dst = sbase + OFF_V + vs * TILE_BYTES;
      for (int q = 0; q < 2; ++q)
        for (int hf = 0; hf < 2; ++hf)
          tma_load_4d(dst + hf * HALF_BYTES + q * PG * 128, &tm_pool, full, hf * 64, 0, Hkv + pend_kh, q ? pend_pg1 : pend_pg0);
    };
    while (ok && it.next(x)) {
      const int ctx = min(p.b.ctx_len[x.r], p.max_ctx_len);
      const int kv_len = ctx + nq;
      const int n_pages = (kv_len + PG - 1) / PG;
      const int32_t* tbl = p.b.block_table + (int64_t)x.r * p.b.max_blocks;
      if (lane == 0) {
        if (x.t0 == 0) {  // this block owns the stream's first tile: tell the combine where its runs are
          const int s = x.r * Hkv + x.kh;
          const int start = cum[x.r] + x.kh * x.tiles_r;
          stream_info[s] = make_int2(s + (int)blockIdx.x, (start + x.tiles_r - 1) / per - (int)blockIdx.x + 1);
        }
        const int buf = x.rho & 1;
        if (x.rho >= 2 && !mbar_wait(bar(B_QFREE + buf), ((x.rho >> 1) - 1) & 1)) {
          record_error(p.err, HSWA_ERR_TIMEOUT, x.r, x.rho, 80);
          ok = false;
        } else {
          mbar_arrive_expect_tx(bar(B_QFULL + buf), 2 * Q_ROWS_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            tma_load_3d(sbase + OFF_Q + buf * Q_BYTES + hf * Q_HALF, &tm_q, bar(B_QFULL + buf), hf * 64, x.kh * 8, x.r * nq);
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      // page ids of the run, 32 at a time (lane i holds page first + i)
      int first = 2 * x.t0;
      int pid = first + lane < n_pages ? tbl[first + lane] : 0;
      for (int j = 0; j < x.len && ok; ++j) {
        const int t = x.t0 + j, n = x.n0 + j;
        const int i0 = 2 * t, i1 = (2 * t + 1 < n_pages) ? 2 * t + 1 : 2 * t;  // a missing page repeats its neighbour
        if (i1 >= first + 32) {
          first = i0;
          pid = first + lane < n_pages ? tbl[first + lane] : 0;
        }
        int pg0 = __shfl_sync(0xffffffffu, pid, i0 - first), pg1 = __shfl_sync(0xffffffffu, pid, i1 - first);
        if (lane == 0) {
          if (pg0 < 0 || pg0 >= p.num_pages || pg1 < 0 || pg1 >= p.num_pages) {
            record_error(p.err, HSWA_ERR_BOUNDS, x.r, i0, pg0 < 0 || pg0 >= p.num_pages ? pg0 : pg1);
            pg0 = pg1 = 0;
          }
          const int c = n & 1, k = n >> 1, ks = c;
          if (k >= 1 && !mbar_wait(bar(B_KEMPTY + ks), (k - 1) & 1)) {
            record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 82);
            ok = false;
          } else {
            mbar_arrive_expect_tx(bar(B_KFULL + ks), TILE_BYTES);
            const uint32_t dst = sbase + OFF_K + ks * TILE_BYTES;
            for (int q = 0; q < 2; ++q)
              for (int hf = 0; hf < 2; ++hf)
                tma_load_4d(dst + hf * HALF_BYTES + q * PG * 128, &tm_pool, bar(B_KFULL + ks), hf * 64, 0, x.kh, q ? pg1 : pg0);
            if (pend) issue_v();
            pend = true;
            pend_pg0 = pg0;
            pend_pg1 = pg1;
            pend_n = n;
            pend_kh = x.kh;
            pend_r = x.r;
            // the stream's last tile may end inside the tile: its V goes through the chain's softmax warp, which
            // zeroes the rows behind the last key (they may hold anything; 0 x NaN must not reach the output)
            pend_patch = (t == x.tiles_r - 1) && (kv_len & (BN - 1)) != 0;
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
      }
    }
    if (lane == 0 && ok && pend) issue_v();
  } else if (warp == 3 || warp == 4) {
    // ======================= MMA issuer of chain c =======================
    // The whole warp walks the loop converged; one elected lane issues.
    const int c = warp - 3;
    RunIter it(cum, B, Hkv, u0, u1);
    Run x;
    bool ok = true;
    int runs_done = 0;  // runs in which this chain had tiles
    const uint64_t dK = smem_desc(sbase + OFF_K + c * TILE_BYTES, 16), dV = smem_desc(sbase + OFF_V + c * TILE_BYTES, HALF_BYTES);
    const uint32_t tS = tmem + c * 128, tO = tmem + 256 + c * 128;
    while (ok && it.next(x)) {
      const int buf = x.rho & 1;
      ok = mbar_wait(bar(B_QFULL + buf), (x.rho >> 1) & 1);  // every run, so that no phase of this barrier goes unseen
      if (!ok) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, x.rho, 83);
        break;
      }
      const int n_first = first_own(x, c), n_end = x.n0 + x.len;
      if (n_first >= n_end) {
        if (lane == 0) mbar_arrive(bar(B_QFREE + buf));
        continue;
      }
      // chain 1's rows are rows 32-63 of the MMA tile: its A descriptor starts 32 rows (4 KB) before the Q buffer
      const uint64_t dQ = smem_desc(sbase + OFF_Q + buf * Q_BYTES - c * Q_ROWS_BYTES, 16);
      for (int n = n_first; n < n_end && ok; n += 2) {
        const int k = n >> 1;
        const bool first_tile = n == n_first, last_tile = n + 2 >= n_end;
        const int ks = c, vs = c;
        ok = mbar_wait(bar(B_KFULL + ks), k & 1);
        if (!ok) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 84);
          break;
        }
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < HD / 16; ++ks)
            tc_mma_ss(tS, desc_advance(dQ, (ks >> 2) * Q_HALF + (ks & 3) * 32), desc_advance(dK, (ks >> 2) * HALF_BYTES + (ks & 3) * 32),
                      IDESC_S, ks > 0);
          tc_commit(bar(B_SFULL + c));
          tc_commit(bar(B_KEMPTY + ks));
          if (last_tile) tc_commit(bar(B_QFREE + buf));
        }
        __syncwarp();
        ok = mbar_wait(bar(B_VFULL + vs), k & 1) && mbar_wait(bar(B_PFA + c), k & 1);
        // the accumulator of the chain's previous run must have been read out before this run's first PV overwrites it
        if (ok && first_tile && runs_done >= 1) ok = mbar_wait(bar(B_OFREE + c), (runs_done - 1) & 1);
        if (!ok) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 85);
          break;
        }
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int q = 0; q < 4; ++q) tc_mma_ts(tO, tS + q * 8, desc_advance(dV, q * 2048), IDESC_PV, !(first_tile && q == 0));
        }
        __syncwarp();
        ok = mbar_wait(bar(B_PFB + c), k & 1);
        if (!ok) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 86);
          break;
        }
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int q = 4; q < 8; ++q) tc_mma_ts(tO, tS + q * 8, desc_advance(dV, q * 2048), IDESC_PV, 1u);
          tc_commit(bar(B_VEMPTY + vs));
          if (last_tile) tc_commit(bar(B_OFINAL + c));
        }
        __syncwarp();
      }
      ++runs_done;
    }
  } else if (warp < 2) {
    // ======================= softmax warp of chain c: lane = row = (token, head) =======================
    const int c = warp;
    const int w = lane >> 3, g = lane & 7;
    const uint32_t lane_addr = (uint32_t)(32 * c) << 16;
    const uint32_t tS = tmem + lane_addr + c * 128, tO = tmem + lane_addr + 256 + c * 128;
    RunIter it(cum, B, Hkv, u0, u1);
    Run x;
    bool ok = true;
    int runs_done = 0, n_patched = 0;
    while (ok && it.next(x)) {
      const int run_id = x.r * Hkv + x.kh + (int)blockIdx.x;
      const int64_t prow = ((int64_t)run_id * 2 + c) * ROWS + lane;
      const int n_first = first_own(x, c), n_end = x.n0 + x.len;
      if (n_first >= n_end) {  // no tile of this run for this chain: an empty partial
        run_ml[prow] = make_float2(-INFINITY, 0.f);
        continue;
      }
      const int ctx = min(p.b.ctx_len[x.r], p.max_ctx_len);
      const int kv_len = ctx + nq;
      float m_st = -INFINITY, l_run = 0.f;
      for (int n = n_first; n < n_end; n += 2) {
        const int k = n >> 1, t = x.t0 + (n - x.n0);
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SFULL + c), k & 1));
        if (!ok) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 87);
          break;
        }
        // visible columns of this row in this tile: keys up to its own position ctx + w
        int vis = ctx + min(w, nq - 1) + 1 - t * BN;
        vis = vis < 0 ? 0 : (vis > BN ? BN : vis);
        uint32_t v[128];
        tc_fence_after();
        tmem_ld32(tS, v);
        tmem_ld32(tS + 32, v + 32);
        tmem_ld32(tS + 64, v + 64);
        tmem_ld32(tS + 96, v + 96);
        tc_wait_ld();
        if (vis < BN) {
#pragma unroll
          for (int col = 0; col < 128; ++col)
            if (col >= vis) v[col] = 0xff800000u;  // -inf
        }
        float mx8[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) mx8[q] = fmaxf(__uint_as_float(v[2 * q]), __uint_as_float(v[2 * q + 1]));
#pragma unroll
        for (int col = 16; col < 128; col += 16) {
#pragma unroll
          for (int q = 0; q < 8; ++q) mx8[q] = max3(mx8[q], __uint_as_float(v[col + 2 * q]), __uint_as_float(v[col + 2 * q + 1]));
        }
        const float mx = fmaxf(fmaxf(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[5])), fmaxf(mx8[6], mx8[7]));
        const float mx_s = mx * M.scale_log2;
        if (n == n_first) {
          m_st = mx_s;
        } else {
          // lazy rescale: only when some row's maximum grew by more than 2^8 (exact: the final normalisation uses
          // the same reference)
          const bool grow = mx_s > m_st + 8.f;
          if (__any_sync(0xffffffffu, grow)) {
            const float m_new = grow ? mx_s : m_st;
            const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m_st - m_new);
#pragma unroll 1
            for (int c16 = 0; c16 < 8; ++c16) {
              uint32_t o16[16];
              tmem_ld16(tO + c16 * 16, o16);
              tc_wait_ld();
#pragma unroll
              for (int q = 0; q < 16; ++q) o16[q] = __float_as_uint(__uint_as_float(o16[q]) * alpha);
              tmem_st16p(tO + c16 * 16, o16);
            }
            l_run *= alpha;
            m_st = m_new;
          }
        }
        const float m_use = (m_st == -INFINITY) ? 0.f : m_st;
        const float2 sc2 = make_float2(M.scale_log2, M.scale_log2), nm2 = make_float2(-m_use, -m_use);
        float2 acc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q] = make_float2(0.f, 0.f);
#pragma unroll
        for (int part = 0; part < 4; ++part) {
#pragma unroll
          for (int q = part * 16; q < part * 16 + 16; ++q) {
            const float2 xx = __ffma2_rn(make_float2(__uint_as_float(v[2 * q]), __uint_as_float(v[2 * q + 1])), sc2, nm2);
            const float2 e = make_float2(fast_exp2(xx.x), fast_exp2(xx.y));  // masked columns: 2^(-inf) = 0
            v[q] = pack_bf16x2(e.x, e.y);
            acc[q & 3] = __fadd2_rn(acc[q & 3], e);
          }
          tmem_st16p(tS + part * 16, v + part * 16);
          if (part == 1) {  // the first 64 keys of P: their PV MMAs run under the rest of the row
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_PFA + c));
          }
        }
        const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
        l_run += (a01.x + a01.y) + (a23.x + a23.y);
        tc_wait_st();
        if (t == x.tiles_r - 1 && (kv_len & (BN - 1)) != 0) {
          // the stream's last tile ends inside the tile: zero the V rows behind the last key, then release the tile
          ok = __all_sync(0xffffffffu, mbar_wait(bar(B_VPATCH + c), n_patched & 1));
          ++n_patched;
          if (!ok) {
            if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, n, 88);
            break;
          }
          const int live = kv_len - t * BN;
          const int vs = c;
          uint8_t* sV = smem + OFF_V + vs * TILE_BYTES;
          for (int idx = live * 8 + lane; idx < BN * 8; idx += 32) {  // 16-byte chunks of rows [live, 128), both halves
            const int row = idx >> 3, ch = idx & 7;
            *reinterpret_cast<uint4*>(sV + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(sV + HALF_BYTES + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_VFULL + vs));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_PFB + c));
      }
      if (!ok) break;
      // ---- the run's partial: unnormalised o with its (m, l) ----
      ok = __all_sync(0xffffffffu, mbar_wait(bar(B_OFINAL + c), runs_done & 1));
      if (!ok) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, x.r, x.rho, 89);
        break;
      }
      tc_fence_after();
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t o32[32];
        tmem_ld32(tO + c4 * 32, o32);
        tc_wait_ld();
        float4* dst = reinterpret_cast<float4*>(run_o + prow * HD + c4 * 32);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          dst[q] = make_float4(__uint_as_float(o32[4 * q]), __uint_as_float(o32[4 * q + 1]), __uint_as_float(o32[4 * q + 2]),
                               __uint_as_float(o32[4 * q + 3]));
      }
      run_ml[prow] = make_float2(m_st, l_run);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_OFREE + c));
      ++runs_done;
      (void)g;
    }
  }

  // ---- teardown ----
  if (*reinterpret_cast<volatile int32_t*>(p.err) != 0) __nanosleep(100000);  // a role gave up: outwait loads in flight
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// Merge the partials of each row's stream: out = sum_i 2^(m_i - m) o_i / sum_i 2^(m_i - m) l_i.  One warp per
// (request, token, head).
__global__ void __launch_bounds__(128) combine_runs_kernel(const DecodeParams p, const float* __restrict__ run_o,
                                                            const float2* __restrict__ run_ml, const int2* __restrict__ stream_info) {
  constexpr int D = mtc::HD;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const ModelParams& M = p.m;
  if (warp_global >= p.b.B * p.nq * M.Hq) return;
  const int h = warp_global % M.Hq, w = (warp_global / M.Hq) % p.nq, r = warp_global / (M.Hq * p.nq);
  const int2 info = stream_info[r * M.Hkv + h / M.G];
  const int row32 = w * 8 + h % M.G;
  const int n = 2 * info.y;
  const int64_t base = (int64_t)info.x * 2;
  float mm = -INFINITY;
  for (int i = lane; i < n; i += 32) mm = fmaxf(mm, run_ml[(base + i) * mtc::ROWS + row32].x);
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, sh));
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float L = 0.f;
  if (mm != -INFINITY) {
    for (int i = 0; i < n; ++i) {
      const float2 ml = run_ml[(base + i) * mtc::ROWS + row32];
      if (ml.x == -INFINITY) continue;  // an empty partial: its o was never written
      const float f = fast_exp2(ml.x - mm);
      const float4 o = *reinterpret_cast<const float4*>(run_o + ((base + i) * mtc::ROWS + row32) * D + lane * 4);
      L += f * ml.y;
      acc.x += f * o.x;
      acc.y += f * o.y;
      acc.z += f * o.z;
      acc.w += f * o.w;
    }
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  const int64_t row = warp_global;
  if (M.out_fp32)
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + row * D + lane * 4) =
        make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
  else
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + row * D + lane * 4) =
        make_uint2(pack_bf16x2(acc.x * inv, acc.y * inv), pack_bf16x2(acc.z * inv, acc.w * inv));
  if (lane == 0 && p.lse) p.lse[row] = L > 0.f ? (mm + log2f(L)) * 0.6931471805599453f : -INFINITY;
}

}  // namespace

bool hswa_decode_mtp_tc_supported(const ModelParams& m, int batch, int nq) {
  return m.D == 128 && m.P == 64 && m.G == 8 && nq >= 2 && nq <= 4 && batch <= mtc::MAX_BATCH;
}

// Scratch of the tensor-core multi-token path: run partials (o, then (m, l)) and one int2 per stream.
void hswa_decode_mtp_tc_scratch(const ModelParams& m, int batch, int num_sms, size_t* o_bytes, size_t* ml_bytes, size_t* info_bytes) {
  const size_t runs = (size_t)num_sms + (size_t)batch * m.Hkv + 1;  // run numbers are stream index + block index
  *o_bytes = (runs * 2 * mtc::ROWS * mtc::HD * sizeof(float) + 255) & ~size_t(255);
  *ml_bytes = (runs * 2 * mtc::ROWS * sizeof(float2) + 255) & ~size_t(255);
  *info_bytes = ((size_t)batch * m.Hkv * sizeof(int2) + 255) & ~size_t(255);
}

// tm_q: box {64, 8 heads, 4 tokens} over q viewed as [B * nq][Hq][D]; tm_pool: box {64, one page, 1, 1}.
cudaError_t hswa_launch_decode_mtp_tc(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const DecodeParams& p, int num_sms,
                                      void* scratch, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(decode_mtp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, mtc::SMEM);
  if (e != cudaSuccess) return e;
  size_t ob, mb, ib;
  hswa_decode_mtp_tc_scratch(p.m, p.b.B, num_sms, &ob, &mb, &ib);
  float* run_o = static_cast<float*>(scratch);
  float2* run_ml = reinterpret_cast<float2*>(static_cast<char*>(scratch) + ob);
  int2* info = reinterpret_cast<int2*>(static_cast<char*>(scratch) + ob + mb);
  decode_mtp_tc_kernel<<<num_sms, mtc::THREADS, mtc::SMEM, s>>>(tm_pool, tm_q, p, run_o, run_ml, info);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int rows = p.b.B * p.nq * p.m.Hq;
  combine_runs_kernel<<<(rows + 3) / 4, 128, 0, s>>>(p, run_o, run_ml, info);
  return cudaGetLastError();
}
