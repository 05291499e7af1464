// SWA-layer decode over the ring of pages, compact-window forms (paper Sec. 2.1: an SWA layer attends inside a window
// of W keys; Sec. 3.1.1: strictly O(W) KV per request in a ring; Sec. 6.2: a decode step may carry draft tokens).
//
// Two kernels that stage ONLY the 16-slot granules of a ring that meet the window, compactly (72 KB of K and V at
// W = 128), three blocks per SM; the streaming ring kernel (decode.cu) stages whole 64-slot tiles, two blocks per SM.
//   decode_ring_window_kernel   single-token steps on batches with more rings than the streaming kernel keeps resident
//                               (described above the kernel);
//   decode_ring_compact_kernel  multi-token steps on rings longer than the three tiles the streaming kernel can keep
//                               staged at once, any window that fits shared memory (described next).
//
// decode_ring_compact_kernel: persistent blocks walk (request, KV head) items and refill the K tiles of the next item as
// soon as the scores of the current one exist, the V tiles as soon as its output accumulators are complete.
//
// Work split inside a block (4 warps, no producer / consumer roles):
//   load      warp 0 works out the circular interval of visible slots [head - min(W - 1, ctx), head + nq - 1] and
//             issues one TMA tensor load (128-byte swizzle) per run of granules that are consecutive inside a page --
//             three runs for a window of 128 on pages of 64 -- with a tensor map per box height, K and V on a barrier
//             each.  (Issuing a tensor load costs its thread on the order of a hundred cycles whatever the box size,
//             and the copies of an SM are issued one after the other: 16-slot boxes, 36 per ring, made the issue
//             itself the bottleneck.)
//   phase 1   split by keys: warp w computes S^T[keys x heads] = K Q^T (mma.sync m16n8k16, the GQA group's 8 heads
//             are N = 8) for the 16-key blocks w, w + 4, ..., masks and scales them and publishes its partial row
//             maxima; after a barrier (K is dead from here on) it turns its scores into P = 2^(S - m), rounds them to
//             bf16 and leaves them in shared memory already in B-fragment order, with its partial row sums;
//   phase 2   split by head dims: every warp accumulates O^T[its D / 4 dims x heads] += V^T P^T over ALL keys -- one
//             8-byte load per 16 keys and token, one ldmatrix per MMA -- so no warp's result has to be merged with
//             another's, and writes its rows straight from the accumulators.
// Draft tokens (NT = 2 or 4 query tokens per request, causal among themselves) ride along as extra N columns: K and V
// fragments are loaded once and multiplied with every token's Q / P.  The new tokens' K/V rows are patched into the
// staged tiles and written to the cache here (fused append).  Rows of the staged tiles that hold slots outside every
// token's window -- stale ring slots, possibly non-finite -- never count: their scores are masked and their V
// fragments are zeroed after ldmatrix; a 16-key block wholly inside the window skips both.
#include "hswa_internal.cuh"

namespace {
using namespace hswa_dev;

constexpr int GR = HSWA_RING_GRANULE;  // slots per TMA box; divides every supported page size

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// The same m16n8k16 as mma_bf16_16816, as a pure function of its operands so that the compiler may interleave
// independent accumulation chains.
__device__ __forceinline__ void mma_pure(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Tensor maps over one pool with boxes of 16, 32, 48 and 64 slots (only the heights up to a page are used).
struct RingMaps {
  CUtensorMap m[4];
};

template <int D, int NT>
__global__ void __launch_bounds__(128, NT == 1 ? 3 : 2)
decode_ring_compact_kernel(const __grid_constant__ RingMaps maps, const DecodeParams p, const int ng_max,
                           const int k_region_bytes, const int n_items) {
  constexpr int NW = 4;           // warps
  constexpr int MT = D / 16 / NW; // 16-dim output blocks per warp
  constexpr int HALVES = D / 64;
  constexpr int KS = D / 16;      // k-steps of K Q^T
  constexpr int CHUNKS = D / 8;   // 16-byte chunks per row
  constexpr int NCOL = NT * 8;    // score columns: tokens x heads
  constexpr int KB_REG = 3;       // 16-key blocks whose scores a warp can keep in registers
  static_assert(2 * CHUNKS <= 32, "one chunk of a new K/V row per lane");

  // All shared memory is one dynamic window (no static part, so that it starts on the 1 KB boundary the swizzled
  // tiles need and three blocks fit an SM to the byte): K tiles | V tiles | P | scores (long windows) | small state.
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);

  const ModelParams& M = p.m;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.nq;
  const bool fuse = p.k_new != nullptr;
  const int rows_max = ng_max * GR;
  const int half_bytes = rows_max * 128;  // one 64-column half of K (or V)
  const uint32_t aK = smem_base, aV = smem_base + k_region_bytes;
  uint8_t* sK = smem;
  uint8_t* sV = smem + k_region_bytes;
  // Behind the V tiles: P (bf16, B-fragment order) [16-key block][NCOL][16], and for windows of more than
  // KB_REG * NW granules, whose scores cannot wait in registers, a score area S [NCOL][sstr] fp32.
  const bool s_in_regs = ng_max <= KB_REG * NW;
  uint32_t* Pb = reinterpret_cast<uint32_t*>(smem + k_region_bytes + HALVES * half_bytes);
  const int sstr = rows_max + 8;
  float* S = reinterpret_cast<float*>(smem + k_region_bytes + HALVES * half_bytes + ng_max * NCOL * 32);
  uint8_t* state = reinterpret_cast<uint8_t*>(S) + (s_in_regs ? 0 : NCOL * sstr * 4);
  uint64_t* bars = reinterpret_cast<uint64_t*>(state);                     // [2] K tiles landed, V tiles landed
  float(*pm)[NCOL] = reinterpret_cast<float(*)[NCOL]>(state + 16);         // [NW] per-warp partial row maxima
  float(*pl)[NCOL] = reinterpret_cast<float(*)[NCOL]>(state + 16 + NW * NCOL * 4);  // [NW] per-warp partial row sums
  uint32_t* s_okm = reinterpret_cast<uint32_t*>(state + 16 + 2 * NW * NCOL * 4);    // [2] per item parity: granules loaded
  int& s_abort = *reinterpret_cast<int*>(state + 16 + 2 * NW * NCOL * 4 + 8);       // a bounded wait ran out: all warps leave
  const int ring_grans = M.C / GR;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    mbar_fence_init();
    for (int i = 0; i < M.P / GR && i < 4; ++i) tma_prefetch_desc(&maps.m[i]);
    s_abort = 0;
    if (smem_base & 1023u) {  // the swizzled tile addressing below assumes a 1 KB-aligned window
      record_error(p.err, HSWA_ERR_CUDA, -1, (int)(smem_base & 1023u), 9);
      s_abort = 1;
    }
  }
  griddep_launch_dependents();  // the next kernel may begin its own cache loads (it waits before it touches q or out)
  __syncthreads();
  if (s_abort) return;

  // ---- per-item state, fetched one item ahead ----
  struct Meta {
    int ctx, head, my_page;  // lane i keeps page id i of the ring
  };
  auto load_meta = [&](int item) {  // lengths, ring head and ring table are constant during a step
    Meta m;
    const int r = item / M.Hkv;
    m.ctx = p.b.ctx_len[r];
    m.head = p.b.ring_head[r];
    m.my_page = lane < M.R ? p.b.ring_table[(int64_t)r * M.R + lane] : -1;
    return m;
  };
  // Warp 0: issue the TMA loads of one item's K (kv = 0) or V (kv = 1) tiles, one lane per granule.
  auto issue_tiles = [&](int item, const Meta& m, int kv, int par) {
    const int r = item / M.Hkv, kh = item % M.Hkv;
    const int back = min(M.W - 1, m.ctx);
    int start = m.head - back;
    if (start < 0) start += M.C;
    const int n_gran = min((start % GR + back + nq - 1) / GR + 1, ng_max);
    int gi = start / GR + lane;
    gi -= gi >= ring_grans ? ring_grans : 0;
    gi -= gi >= ring_grans ? ring_grans : 0;  // lanes beyond the ring's granules do not load
    const int slot_lo = gi * GR;
    const int gpp = M.P / GR;  // granules per page
    // a run: granules that follow each other inside one page; it starts at the interval's first granule and at every
    // page boundary (the wrap to slot 0 is one)
    const bool run_start = lane < n_gran && (lane == 0 || gi % gpp == 0);
    const unsigned starts = __ballot_sync(0xffffffffu, run_start) | (1u << n_gran);
    const int len = run_start ? __ffs(starts >> (lane + 1)) : 0;  // granules up to the next run
    const int page = __shfl_sync(0xffffffffu, m.my_page, (slot_lo / M.P) & 31);
    uint32_t okm = 0;
    if (run_start) {
      if (page < 0 || page >= p.num_pages) {
        if (kv == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, slot_lo / M.P, page);
      } else {
        okm = ((1u << len) - 1u) << lane;
      }
    }
    okm = __reduce_or_sync(0xffffffffu, okm);
    const uint32_t full_bar = smem_u32(&bars[kv]);
    if (lane == 0) {
      if (kv == 0) s_okm[par] = okm;
      if (okm == 0)
        mbar_arrive(full_bar);
      else
        mbar_arrive_expect_tx(full_bar, __popc(okm) * HALVES * GR * 128);
    }
    __syncwarp();
    if (run_start && ((okm >> lane) & 1u)) {
#pragma unroll
      for (int hf = 0; hf < HALVES; ++hf)
        tma_load_4d((kv == 0 ? aK : aV) + hf * half_bytes + lane * GR * 128, &maps.m[len - 1], full_bar, hf * 64,
                    slot_lo % M.P, kv * M.Hkv + kh, page);
    }
  };
  const int g_row = lane >> 2;  // head of this thread's B-fragment column
  const int qd = (lane & 3) * 2;
  const int mi = lane >> 3, mr = lane & 7;
  uint32_t qf[NT][KS][2];
  uint4 newrow[NT];
  auto load_q = [&](int item) {
    const int r = item / M.Hkv, kh = item % M.Hkv;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const bool live = nt < nq && g_row < M.G;
      const __nv_bfloat16* qrow = p.q + (((int64_t)r * nq + (nt < nq ? nt : 0)) * M.Hq + kh * M.G + (g_row < M.G ? g_row : 0)) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qf[nt][ks][0] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
        qf[nt][ks][1] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
      }
      if (fuse && lane < 2 * CHUNKS && nt < nq)
        newrow[nt] = *reinterpret_cast<const uint4*>((lane < CHUNKS ? p.k_new : p.v_new) +
                                                     (((int64_t)r * nq + nt) * M.Hkv + kh) * D + (lane % CHUNKS) * 8);
    }
  };

  int it = blockIdx.x;
  if (it >= n_items) return;
  Meta mt_next = load_meta(it);
  if (warp == 0) {
    issue_tiles(it, mt_next, 0, 0);
    issue_tiles(it, mt_next, 1, 0);
  }
  // q, k_new, v_new may be the previous kernel's output: nothing of them may be read before it has finished, but
  // pulling their lines towards L2 (the point of coherence) early is harmless and takes DRAM latency off the chain
  {
    const int r = it / M.Hkv, kh = it % M.Hkv;
    const char* qb = reinterpret_cast<const char*>(p.q + ((int64_t)r * nq * M.Hq + kh * M.G) * D);
    if (threadIdx.x < M.G * D * 2 / 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(qb + threadIdx.x * 128));
    if (fuse && threadIdx.x >= 64 && threadIdx.x < 64 + 2 * D * 2 / 128) {
      const int j = threadIdx.x - 64, kv = j / (D * 2 / 128), o128 = j % (D * 2 / 128);
      asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>((kv == 0 ? p.k_new : p.v_new) +
                                                                                    ((int64_t)r * nq * M.Hkv + kh) * D) + o128 * 128));
    }
  }
  griddep_wait();
  load_q(it);

  for (int k = 0; it < n_items; ++k, it += gridDim.x) {
    const int par = k & 1;
    const int r = it / M.Hkv, kh = it % M.Hkv;
    const Meta m = mt_next;
    const int nxt = it + gridDim.x;
    const bool has_next = nxt < n_items;
    if (has_next) mt_next = load_meta(nxt);
    const int ctx = m.ctx, head = m.head;
    const int back = min(M.W - 1, ctx);  // cached positions token 0 can see
    int start = head - back;             // ring slot of the oldest visible position
    if (start < 0) start += M.C;
    const int sr = start % GR;
    const int last = back + nq - 1;      // offset of the newest token's slot from `start`
    const int n_gran = min((sr + last) / GR + 1, ng_max);

    bool ok = mbar_wait(smem_u32(&bars[0]), par);
    if (!ok && lane == 0) {
      record_error(p.err, HSWA_ERR_TIMEOUT, r, kh, 8);
      *reinterpret_cast<volatile int*>(&s_abort) = 1;
    }
    const uint32_t okm = *reinterpret_cast<volatile uint32_t*>(&s_okm[par]);

    // fused append: token nt sits at offset back + nt from `start`, i.e. in compact row sr + back + nt.  Every warp
    // patches the rows (same bytes) so that it needs no block barrier before reading them; warp 0 writes the cache.
    if (fuse && ok && lane < CHUNKS) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int row = sr + back + nt;
        if (nt < nq && row < rows_max) *reinterpret_cast<uint4*>(sK + (lane >> 3) * half_bytes + swz128(row, lane & 7)) = newrow[nt];
      }
      fence_proxy_async_smem();  // a later TMA load overwrites these rows
    }
    __syncwarp();

    // In compact rows: token nt sees [row_lo(nt), row_hi(nt)], any token sees [sr, sr + last]; rows of granules that
    // were not loaded see nothing.
    auto row_lo = [&](int nt) { return sr + max(0, back + nt - (M.W - 1)); };
    auto row_hi = [&](int nt) { return sr + back + nt; };
    auto visible = [&](int j, int nt) { return ((okm >> (j / GR)) & 1u) && j >= row_lo(nt) && j <= row_hi(nt); };
    auto visible_any = [&](int j) { return ((okm >> (j / GR)) & 1u) && j >= sr && j <= sr + last; };
    // is the 16-key block kb loaded and wholly inside [lo, hi]?  (same answer in every thread)
    auto interior = [&](int kb, int lo, int hi) { return ((okm >> kb) & 1u) && kb * 16 >= lo && kb * 16 + 15 <= hi; };

    // ---------------- phase 1a: scores of this warp's 16-key blocks, partial row maxima ----------------
    float mx[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) mx[nt][0] = mx[nt][1] = -INFINITY;
    auto score_block = [&](int kb, float (&sv)[NT][4]) {
      // two accumulators per token halve the dependent MMA chain
      float e[NT][4], f[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) e[nt][c] = f[nt][c] = 0.f;
      const int key = kb * 16 + (mi & 1) * 8 + mr;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int chunk = 2 * ks + (mi >> 1);
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4(aK + (chunk >> 3) * half_bytes + swz128(key, chunk & 7), a0, a1, a2, a3);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_pure((ks & 1) ? f[nt] : e[nt], a0, a1, a2, a3, qf[nt][ks][0], qf[nt][ks][1]);
      }
      const int keyA = kb * 16 + (lane >> 2), keyB = keyA + 8;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const bool inner = nt < nq && interior(kb, row_lo(nt), row_hi(nt));
        const bool vA = inner || (nt < nq && visible(keyA, nt)), vB = inner || (nt < nq && visible(keyB, nt));
        sv[nt][0] = vA ? (e[nt][0] + f[nt][0]) * M.scale_log2 : -INFINITY;
        sv[nt][1] = vA ? (e[nt][1] + f[nt][1]) * M.scale_log2 : -INFINITY;
        sv[nt][2] = vB ? (e[nt][2] + f[nt][2]) * M.scale_log2 : -INFINITY;
        sv[nt][3] = vB ? (e[nt][3] + f[nt][3]) * M.scale_log2 : -INFINITY;
        mx[nt][0] = fmaxf(mx[nt][0], fmaxf(sv[nt][0], sv[nt][2]));
        mx[nt][1] = fmaxf(mx[nt][1], fmaxf(sv[nt][1], sv[nt][3]));
      }
    };
    float s[KB_REG][NT][4];
    if (s_in_regs) {
#pragma unroll
      for (int i = 0; i < KB_REG; ++i)
        if (warp + NW * i < n_gran && ok) score_block(warp + NW * i, s[i]);
    } else {
      for (int kb = warp; kb < n_gran && ok; kb += NW) {
        float sv[NT][4];
        score_block(kb, sv);
        const int keyA = kb * 16 + (lane >> 2);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float* row0 = S + (nt * 8 + qd) * sstr;
          row0[keyA] = sv[nt][0];
          row0[sstr + keyA] = sv[nt][1];
          row0[keyA + 8] = sv[nt][2];
          row0[sstr + keyA + 8] = sv[nt][3];
        }
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        mx[nt][0] = fmaxf(mx[nt][0], __shfl_xor_sync(0xffffffffu, mx[nt][0], sh));
        mx[nt][1] = fmaxf(mx[nt][1], __shfl_xor_sync(0xffffffffu, mx[nt][1], sh));
      }
      if (lane < 4) {
        pm[warp][nt * 8 + qd] = mx[nt][0];
        pm[warp][nt * 8 + qd + 1] = mx[nt][1];
      }
    }
    // V rows of the new tokens, needed from phase 2 on (the V tiles may still be landing while phase 1 runs)
    uint4 vrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) vrow[nt] = newrow[nt];
    int new_page[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      int s_new = head + nt;
      s_new -= s_new >= M.C ? M.C : 0;
      new_page[nt] = __shfl_sync(0xffffffffu, m.my_page, (s_new / M.P) & 31);
    }
    // the cache copy of the new rows (warp 0: K from lanes [0, CHUNKS), V from lanes [CHUNKS, 2 CHUNKS))
    if (fuse && ok && warp == 0 && lane < 2 * CHUNKS) {
      const int kv = lane / CHUNKS, ch = lane % CHUNKS;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (nt >= nq) continue;
        int s_new = head + nt;
        s_new -= s_new >= M.C ? M.C : 0;
        if (new_page[nt] < 0 || new_page[nt] >= p.num_pages) {
          if (lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, new_page[nt]);
        } else {
          *reinterpret_cast<uint4*>(p.pool + ((((int64_t)new_page[nt] * 2 + kv) * M.Hkv + kh) * M.P + s_new % M.P) * D + ch * 8) =
              newrow[nt];
        }
      }
    }
    // next item's Q and new rows: the registers are free from here on, the latency hides behind phases 1b and 2
    if (has_next) load_q(nxt);
    __syncthreads();  // every warp is done reading K and every partial maximum is published
    if (*reinterpret_cast<volatile int*>(&s_abort)) return;
    if (warp == 0 && has_next) issue_tiles(nxt, mt_next, 0, par ^ 1);  // the K tiles are dead: refill them

    // ---------------- phase 1b: P = 2^(S - m) in bf16, B-fragment order, partial row sums ----------------
    // This thread's accumulator columns are heads qd, qd + 1.  A B fragment of 16 keys x 8 columns wants, from the
    // thread with (column g, t = lane mod 4), the word pairs {P[2t], P[2t+1]} and {P[2t+8], P[2t+9]} of column g: P is
    // stored per (block, column) as 8 words in the order t0: {k0,k1},{k8,k9}; t1: {k2,k3},{k10,k11}; ... so phase 2
    // reads 8 bytes per thread.  The accumulator holds keys kq = lane / 4 and kq + 8: neighbouring key lanes (kq even /
    // odd) exchange values so that each writes one whole word.
    float m_col[NT][2], lsum[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) mm = fmaxf(mm, pm[w][nt * 8 + qd + j]);
        m_col[nt][j] = mm;
        lsum[nt][j] = 0.f;
      }
    auto emit_block = [&](int kb, const float (&sv)[NT][4]) {
      const int kq = lane >> 2;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float m0 = m_col[nt][0] == -INFINITY ? 0.f : m_col[nt][0], m1 = m_col[nt][1] == -INFINITY ? 0.f : m_col[nt][1];
        // bf16 values the tensor core will multiply; sum exactly those
        const uint32_t lo = pack_bf16x2(fast_exp2(sv[nt][0] - m0), fast_exp2(sv[nt][1] - m1));  // key kq: cols qd, qd + 1
        const uint32_t hi = pack_bf16x2(fast_exp2(sv[nt][2] - m0), fast_exp2(sv[nt][3] - m1));  // key kq + 8
        const float2 flo = unpack_bf16x2(lo), fhi = unpack_bf16x2(hi);
        lsum[nt][0] += flo.x + fhi.x;
        lsum[nt][1] += flo.y + fhi.y;
        // partner lane holds key kq ^ 1, same columns
        const uint32_t plo = __shfl_xor_sync(0xffffffffu, lo, 4), phi = __shfl_xor_sync(0xffffffffu, hi, 4);
        // even kq writes column qd, odd kq writes column qd + 1: word {P[k even][col], P[k odd][col]}
        const bool odd = kq & 1;
        const uint32_t w_lo = odd ? __byte_perm(plo, lo, 0x7632) : __byte_perm(lo, plo, 0x5410);  // keys (kq & ~1, kq | 1)
        const uint32_t w_hi = odd ? __byte_perm(phi, hi, 0x7632) : __byte_perm(hi, phi, 0x5410);  // keys + 8
        const int col = nt * 8 + qd + (odd ? 1 : 0);
        uint32_t* dst = Pb + ((size_t)(kb * NCOL + col)) * 8 + (kq >> 1) * 2;
        *reinterpret_cast<uint2*>(dst) = make_uint2(w_lo, w_hi);
      }
    };
    if (s_in_regs) {
#pragma unroll
      for (int i = 0; i < KB_REG; ++i)
        if (warp + NW * i < n_gran && ok) emit_block(warp + NW * i, s[i]);
    } else {
      for (int kb = warp; kb < n_gran && ok; kb += NW) {
        float sv[NT][4];
        const int keyA = kb * 16 + (lane >> 2);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float* row0 = S + (nt * 8 + qd) * sstr;
          sv[nt][0] = row0[keyA];
          sv[nt][1] = row0[sstr + keyA];
          sv[nt][2] = row0[keyA + 8];
          sv[nt][3] = row0[sstr + keyA + 8];
        }
        emit_block(kb, sv);
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        lsum[nt][0] += __shfl_xor_sync(0xffffffffu, lsum[nt][0], sh);
        lsum[nt][1] += __shfl_xor_sync(0xffffffffu, lsum[nt][1], sh);
      }
      if (lane < 4) {
        pl[warp][nt * 8 + qd] = lsum[nt][0];
        pl[warp][nt * 8 + qd + 1] = lsum[nt][1];
      }
    }
    // the V tiles: wait, then patch in the new tokens' rows
    if (ok && !mbar_wait(smem_u32(&bars[1]), par)) {
      ok = false;
      if (lane == 0) {
        record_error(p.err, HSWA_ERR_TIMEOUT, r, kh, 9);
        *reinterpret_cast<volatile int*>(&s_abort) = 1;
      }
    }
    if (fuse && ok && lane >= CHUNKS && lane < 2 * CHUNKS) {
      const int ch = lane - CHUNKS;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int row = sr + back + nt;
        if (nt < nq && row < rows_max) *reinterpret_cast<uint4*>(sV + (ch >> 3) * half_bytes + swz128(row, ch & 7)) = vrow[nt];
      }
      fence_proxy_async_smem();
    }
    __syncthreads();  // P and the partial sums are complete
    if (*reinterpret_cast<volatile int*>(&s_abort)) return;

    // ---------------- phase 2: O^T[this warp's dims x heads] over all keys ----------------
    float o[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
    {
      const uint32_t* pcol = Pb + (size_t)g_row * 8 + (lane & 3) * 2;
      const int krow = (mi >> 1) * 8 + mr;
      uint32_t v_addr[MT];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const int chunk = 2 * (warp * MT + mt) + (mi & 1);
        v_addr[mt] = aV + (chunk >> 3) * half_bytes + swz128(krow, chunk & 7);  // + 2 KB per 16-key block
      }
#pragma unroll 3
      for (int kb = 0; kb < n_gran; ++kb) {
        uint2 b[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) b[nt] = *reinterpret_cast<const uint2*>(pcol + ((size_t)(kb * NCOL + nt * 8)) * 8);
        // V^T fragments: a0 / a1 hold keys 16 kb + qd, qd + 1 in their halves, a2 / a3 keys 16 kb + 8 + qd, qd + 9.
        // Rows no token can see may hold anything: zero them (0 x NaN would poison the sum); interior blocks have none.
        uint32_t keep_lo = 0xffffffffu, keep_hi = 0xffffffffu;
        if (!interior(kb, sr, sr + last)) {
          const int k0 = kb * 16 + qd;
          keep_lo = (visible_any(k0) ? 0x0000ffffu : 0u) | (visible_any(k0 + 1) ? 0xffff0000u : 0u);
          keep_hi = (visible_any(k0 + 8) ? 0x0000ffffu : 0u) | (visible_any(k0 + 9) ? 0xffff0000u : 0u);
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4_trans(v_addr[mt] + kb * 2048, a0, a1, a2, a3);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            mma_pure(o[mt][nt], a0 & keep_lo, a1 & keep_lo, a2 & keep_hi, a3 & keep_hi, b[nt].x, b[nt].y);
        }
      }
    }
    // row sums and maxima of this thread's accumulator columns (heads qd, qd + 1), read before the barrier below lets
    // the next item overwrite them
    float inv[NT][2], lse_v[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) l += pl[w][nt * 8 + qd + j];
        inv[nt][j] = l > 0.f ? 1.f / l : 0.f;
        lse_v[nt][j] = (p.lse && l > 0.f) ? (m_col[nt][j] + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
    __syncthreads();  // every warp is done with the V tiles, P and the partial sums
    if (warp == 0 && has_next) issue_tiles(nxt, mt_next, 1, par ^ 1);

    // ---------------- output: straight from the accumulators ----------------
    // (thread: heads qd, qd + 1; head dims 16 (warp MT + mt) + lane / 4 and + 8)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      if (nt >= nq) continue;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (qd + j >= M.G) continue;
        const int64_t row = ((int64_t)r * nq + nt) * M.Hq + kh * M.G + qd + j;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int d0 = (warp * MT + mt) * 16 + (lane >> 2);
          const float x = o[mt][nt][j] * inv[nt][j], y = o[mt][nt][2 + j] * inv[nt][j];
          if (M.out_fp32) {
            reinterpret_cast<float*>(p.out)[row * D + d0] = x;
            reinterpret_cast<float*>(p.out)[row * D + d0 + 8] = y;
          } else {
            reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d0] = __float2bfloat16_rn(x);
            reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d0 + 8] = __float2bfloat16_rn(y);
          }
        }
        if (warp == 0 && (lane >> 2) == 0 && p.lse) p.lse[row] = lse_v[nt][j];
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------------
// Single-token steps, windows up to 128 keys: a loader warp and three compute warps per ring, compact staging.
//
// A block owns one (request, KV head) item at a time and stages ONLY the 16-slot granules that meet the window, granule
// by granule (72 KB of K and V at D = 128), so that three blocks fit an SM; persistent blocks refill their K tiles with
// the next item's as soon as the scores exist and their V tiles as soon as the output accumulators are complete.
//   staging  granule-major: a 16-slot granule is [64-column half][16 rows][128 bytes], so that ONE tensor load (5-D
//            view of the pool, 128-byte swizzle) brings a whole run of granules with both halves of every row.  Issuing
//            the three or four loads of a K (or V) window costs the issuing warp 1200-1800 cycles, which is why a warp
//            of its own does nothing else: it waits for "K tiles free" / "V tiles free" and refills them;
//   scores   split by keys: compute warp c computes S^T[keys x heads] = K Q^T (m16n8k16, the 8 heads of the group are
//            N) for granules c, c + 3, c + 6 and keeps them in registers; partial maxima meet in shared memory
//            (named barrier among the compute warps);
//   softmax  P^T reaches B-fragment order through movmatrix and is left in shared memory, 8 bytes per lane and granule,
//            for the lane of the same number in every warp; partial row sums beside it (second barrier);
//   output   split by head dims: a compute warp accumulates O^T[its dims x heads] += V^T P^T over all granules (V^T read
//            by ldmatrix.trans), so no result has to be merged, and writes its rows from the accumulators (bf16:
//            transposed once more with movmatrix so that a thread stores two neighbouring dims).
// One ldmatrix + MMA pair costs a warp about 17 cycles however the code is arranged (the tensor pipe of its scheduler
// takes one m16n8k16 per 10 cycles); a ring is 144 such pairs.  Fragment loads are issued a granule ahead of the MMAs
// that use them.
// Stale rows (slots outside the window, granules not loaded) are masked in the scores and zeroed in the V fragments.
// Second form (VE = 4, head_dim 128, between three and four rings per SM): only four V granules have a place of their
// own, the others land in the K area once every compute warp has its scores, on a barrier of their own that every warp
// waits on once per ring; 52 KB of tiles and 128 registers per thread, so four blocks fit an SM and no block walks a
// second ring.  The next ring's loads then wait for the whole ring, which is why this form is not used beyond four rings
// per SM.
__device__ __forceinline__ void mma_inorder(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3,
                                            int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
// Barrier among the three compute warps that also tells every thread whether any of them saw a wait run out, so that
// all of them leave together (a warp that left alone would leave the others at the next barrier for ever).
__device__ __forceinline__ bool compute_warps_sync_or(bool failed) {
  uint32_t any;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.u32 q, %1, 0;\n"
      "bar.red.or.pred p, 1, 96, q;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(any)
      : "r"((uint32_t)failed)
      : "memory");
  return any != 0;
}

template <int D, int VE>
__global__ void __launch_bounds__(128, VE == 9 ? 3 : 4)
decode_ring_window_kernel(const __grid_constant__ RingMaps maps, const DecodeParams p, const int n_items) {
  constexpr int NG = 9;            // granules a window of up to 128 keys can meet: (15 + 127) / 16 + 1
  // VE = V granules with a place of their own (loaded with K).  VE = NG: all of them, three blocks per SM at D = 128.
  // VE = 4: a fourth block fits; V granules VE .. NG - 1 land in the K area once the scores exist.
  constexpr bool SPLIT = VE < NG;
  constexpr int HALVES = D / 64;
  constexpr int KS = D / 16;
  constexpr int NC = 3;                     // compute warps (warps 1 .. 3; warp 0 loads)
  constexpr int MTOT = D / 16;              // 16-dim output blocks
  constexpr int MT = (MTOT + NC - 1) / NC;  // per compute warp (the last warp may have fewer)
  constexpr int KBW = NG / NC;              // granules per compute warp in the score phase
  constexpr int CHUNKS = D / 8;
  constexpr int GRAN_BYTES = HALVES * GR * 128;  // one granule of K (or V): [half][16 rows][128 B]
  constexpr int REGION = NG * GRAN_BYTES;          // K area
  constexpr int TILES = REGION + VE * GRAN_BYTES;  // K area + V area
  static_assert(2 * CHUNKS <= 32, "one chunk of the new K/V row per lane");
  static_assert(NG % NC == 0, "granules split evenly over the compute warps");
  static_assert(VE >= 1 && VE <= NG, "late V granules fit the K area");
  enum { B_KFULL = 0, B_VFULL = 1, B_KFREE = 2, B_VFREE = 3, B_V2FULL = 4 };

  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t aK = smem_base, aV = smem_base + REGION;
  uint8_t* sK = smem;
  uint8_t* sV = smem + REGION;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + TILES);                // [5]
  float(*pm)[8] = reinterpret_cast<float(*)[8]>(smem + TILES + 48);          // [NC] partial row maxima
  float(*pl)[8] = reinterpret_cast<float(*)[8]>(smem + TILES + 48 + 128);    // [NC] partial row sums
  uint2* Pb = reinterpret_cast<uint2*>(smem + TILES + 48 + 256);             // [NG][32] P^T as B fragments
  volatile int& s_abort = *reinterpret_cast<volatile int*>(smem + TILES + 48 + 256 + NG * 256);  // a wait ran out

  const ModelParams& M = p.m;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool fuse = p.k_new != nullptr;
  const int ring_grans = M.C / GR;
  const int gpp = M.P / GR;  // granules per page

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars[B_KFULL]), 1);
    mbar_init(smem_u32(&bars[B_VFULL]), 1);
    mbar_init(smem_u32(&bars[B_KFREE]), NC);
    mbar_init(smem_u32(&bars[B_VFREE]), NC);
    mbar_init(smem_u32(&bars[B_V2FULL]), 1);
    mbar_fence_init();
    for (int i = 0; i < gpp && i < 4; ++i) tma_prefetch_desc(&maps.m[i]);
    s_abort = 0;
  }
  griddep_launch_dependents();
  __syncthreads();
  if (smem_base & 1023u) {  // the swizzled tile addressing assumes a 1 KB-aligned window
    if (threadIdx.x == 0) record_error(p.err, HSWA_ERR_CUDA, -1, (int)(smem_base & 1023u), 10);
    return;
  }

  struct Meta {
    int ctx, head, my_page;  // lane i keeps page id i of the ring
  };
  auto load_meta = [&](int item) {
    Meta m;
    const int r = item / M.Hkv;
    m.ctx = p.b.ctx_len[r];
    m.head = p.b.ring_head[r];
    m.my_page = lane < M.R ? p.b.ring_table[(int64_t)r * M.R + lane] : -1;
    return m;
  };
  // A ring head outside [0, C): nothing of such a ring is loaded or written, and the page check records it.  (Applied
  // where the values are used, so that fetching them ahead does not wait for them.)
  auto checked = [&](Meta m) {
    if (m.head < 0 || m.head >= M.C) {
      m.head = 0;
      m.my_page = -1;
    }
    return m;
  };
  // The granules of an item's window: lane i looks after granule i of the visible interval; the first lane of every run
  // of granules inside one page loads the run (loader warp).  Returns the mask of granules that are (being) loaded,
  // which every warp works out for itself.  part 0: K, all granules; part 1: V granules [0, VE) into the V area; part 2:
  // V granules [VE, NG) into the K area.
  auto window_tiles = [&](int item, const Meta& m_raw, int part, bool issue) -> uint32_t {
    const int kv = part == 0 ? 0 : 1;
    const int g0 = part == 2 ? VE : 0, g1 = part == 1 ? VE : NG;
    const Meta m = checked(m_raw);
    const int r = item / M.Hkv, kh = item % M.Hkv;
    const int back = min(M.W - 1, max(m.ctx, 0));
    int start = m.head - back;
    if (start < 0) start += M.C;
    const int n_gran = min((start % GR + back) / GR + 1, NG);
    int gi = start / GR + lane;
    gi -= gi >= ring_grans ? ring_grans : 0;
    gi -= gi >= ring_grans ? ring_grans : 0;
    const int slot_lo = gi * GR;
    const int g_end = max(min(n_gran, g1), g0);
    const bool run_start = lane >= g0 && lane < g_end && (lane == g0 || gi % gpp == 0);
    const unsigned starts = __ballot_sync(0xffffffffu, run_start) | (1u << g_end);
    const int len = run_start ? __ffs(starts >> (lane + 1)) : 0;
    const int page = __shfl_sync(0xffffffffu, m.my_page, (slot_lo / M.P) & 31);
    uint32_t okm = 0;
    if (run_start) {
      if (page < 0 || page >= p.num_pages) {
        if (kv == 0 && issue) record_error(p.err, HSWA_ERR_BOUNDS, r, slot_lo / M.P, page);
      } else {
        okm = ((1u << len) - 1u) << lane;
      }
    }
    okm = __reduce_or_sync(0xffffffffu, okm);
    if (!issue) return okm;
    const uint32_t full_bar = smem_u32(&bars[part == 0 ? B_KFULL : (part == 1 ? B_VFULL : B_V2FULL)]);
    if (lane == 0) {
      if (okm == 0)
        mbar_arrive(full_bar);
      else
        mbar_arrive_expect_tx(full_bar, __popc(okm) * GRAN_BYTES);
    }
    __syncwarp();
    if (run_start && ((okm >> lane) & 1u))
      tma_load_5d((part == 1 ? aV : aK) + (lane - g0) * GRAN_BYTES, &maps.m[len - 1], full_bar, 0, 0, 0,
                  (slot_lo % M.P) / GR, (page * 2 + kv) * M.Hkv + kh);
    return okm;
  };

  const int stride = gridDim.x;
  if (blockIdx.x >= n_items) return;
  if (warp == 0) {
    // ---------------- loader warp ----------------
    int it = blockIdx.x;
    Meta m_cur = load_meta(it);
    Meta m_nxt = m_cur;
    if (it + stride < n_items) m_nxt = load_meta(it + stride);
    window_tiles(it, m_cur, 0, true);
    window_tiles(it, m_cur, 1, true);
    for (int k = 0; SPLIT || it + stride < n_items; ++k, it += stride) {
      const int par = k & 1;
      const int nxt = it + stride;
      const bool has_next = nxt < n_items;
      const Meta m_this = m_cur;
      m_cur = m_nxt;
      if (nxt + stride < n_items) m_nxt = load_meta(nxt + stride);
      // K tiles of item k are dead once every compute warp has its scores, the V tiles once it has its accumulators
      bool ok = mbar_wait(smem_u32(&bars[B_KFREE]), par);
      bool k_issued = false, v2_issued = false;
      if (ok && !s_abort) {
        if (SPLIT) {
          // the rest of this item's V granules take the K area; the next item's loads wait for the whole item
          window_tiles(it, m_this, 2, true);
          v2_issued = true;
          if (has_next) {
            ok = mbar_wait(smem_u32(&bars[B_VFREE]), par);
            if (ok && !s_abort) {
              window_tiles(nxt, m_cur, 0, true);
              k_issued = true;
              window_tiles(nxt, m_cur, 1, true);
            }
          }
        } else {
          window_tiles(nxt, m_cur, 0, true);
          k_issued = true;
          ok = mbar_wait(smem_u32(&bars[B_VFREE]), par);
          if (ok && !s_abort) window_tiles(nxt, m_cur, 1, true);
        }
      }
      if (!ok || s_abort) {
        // the compute warps gave up, or a wait of this warp ran out: leave once no load of this block is in flight
        if (!ok && lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, it / M.Hkv, it % M.Hkv, 12);
        s_abort = 1;
        mbar_wait(smem_u32(&bars[B_KFULL]), par, 2000000);
        mbar_wait(smem_u32(&bars[B_VFULL]), par, 2000000);
        if (v2_issued) mbar_wait(smem_u32(&bars[B_V2FULL]), par, 2000000);
        if (k_issued) mbar_wait(smem_u32(&bars[B_KFULL]), par ^ 1, 2000000);
        return;
      }
      if (!has_next) break;
    }
    return;
  }

  // ---------------- compute warps ----------------
  const int cw = warp - 1;
  const int g_row = lane >> 2;
  const int qd = (lane & 3) * 2;
  const int mi = lane >> 3, mr = lane & 7;
  uint32_t qf[KS][2];
  uint4 newrow = make_uint4(0, 0, 0, 0);
  auto load_q = [&](int item) {
    const int r = item / M.Hkv, kh = item % M.Hkv;
    const bool live = g_row < M.G;
    const __nv_bfloat16* qrow = p.q + ((int64_t)r * M.Hq + kh * M.G + (live ? g_row : 0)) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
      qf[ks][1] = live ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
    }
    if (fuse && lane < 2 * CHUNKS)
      newrow = *reinterpret_cast<const uint4*>((lane < CHUNKS ? p.k_new : p.v_new) + ((int64_t)r * M.Hkv + kh) * D +
                                               (lane % CHUNKS) * 8);
  };
  // Byte offset of 16-byte chunk c (0 .. CHUNKS - 1) of row jr (0 .. 15) inside a granule
  auto gran_off = [](int jr, int c) { return (uint32_t)((c >> 3) * (GR * 128)) + swz128(jr, c & 7); };
  // This thread's ldmatrix row addresses inside a granule: K fragments of k-step ks, V^T fragments of this warp's dim
  // blocks cw * MT + mt
  uint32_t k_off[KS], v_off[MT];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) k_off[ks] = gran_off((mi & 1) * 8 + mr, 2 * ks + (mi >> 1));
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) v_off[mt] = gran_off((mi >> 1) * 8 + mr, (2 * (cw * MT + mt) + (mi & 1)) % CHUNKS);
  const int n_mt = min(MT, MTOT - cw * MT);  // dim blocks of this warp (warp-uniform)

  int it = blockIdx.x;
  // lengths, ring heads and ring tables are fetched two items ahead: right behind the dependency wait such a fetch
  // takes a few thousand cycles, more than the first item's scores
  Meta mt_next = load_meta(it);
  Meta mt_next2 = mt_next;
  if (it + stride < n_items) mt_next2 = load_meta(it + stride);
  uint32_t okm_next = window_tiles(it, mt_next, 0, false);
  griddep_wait();  // q, k_new, v_new and the outputs may belong to the previous kernel until here
  load_q(it);

  bool late_failed = false;  // the wait for the late V granules ran out: told to the other warps at the next barrier
  for (int k = 0; it < n_items; ++k, it += stride) {
    const int par = k & 1;
    const int r = it / M.Hkv, kh = it % M.Hkv;
    const Meta m = checked(mt_next);
    const uint32_t okm = okm_next;
    const int nxt = it + stride;
    const bool has_next = nxt < n_items;
    mt_next = mt_next2;
    if (nxt + stride < n_items) mt_next2 = load_meta(nxt + stride);
    const int back = min(M.W - 1, max(m.ctx, 0));  // cached positions the new token can see
    int start = m.head - back;                      // ring slot of the oldest visible position
    if (start < 0) start += M.C;
    const int sr = start % GR;
    const int hi_row = sr + back;                   // compact row of the new token; visible rows are [sr, hi_row]
    const int n_gran = min(hi_row / GR + 1, NG);
    auto visible = [&](int j) { return ((okm >> (j / GR)) & 1u) && j >= sr && j <= hi_row; };
    auto interior = [&](int kb) { return ((okm >> kb) & 1u) && kb * 16 >= sr && kb * 16 + 15 <= hi_row; };

    // A wait that ran out: the warp still reaches the next barrier among the compute warps, where all of them learn
    // of it and leave (the flag tells the loader warp, which outwaits the loads the block still has in flight).
    bool failed = late_failed;
    if (!mbar_wait(smem_u32(&bars[B_KFULL]), par)) {
      failed = true;
      s_abort = 1;
      if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, kh, 10);
    }
    // every warp patches the new K row itself (same bytes), so that it needs no barrier before reading it
    if (fuse && lane < CHUNKS) {
      *reinterpret_cast<uint4*>(sK + (hi_row >> 4) * GRAN_BYTES + gran_off(hi_row & 15, lane)) = newrow;
      fence_proxy_async_smem();  // a later TMA load overwrites this row
    }
    __syncwarp();

    // ---------------- scores of granules cw, cw + NC, ... ----------------
    float s[KBW][4];
    float mx0 = -INFINITY, mx1 = -INFINITY;
    {
      // fragments of the next granule are fetched ahead of the MMAs of this one (with four blocks per SM there are no
      // registers for that: behind them)
      constexpr int KBUF = SPLIT ? 1 : 2;
      uint32_t ka[KBUF][KS][4];
      auto fetch = [&](int kb, int buf) {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          ldmatrix_x4(aK + kb * GRAN_BYTES + k_off[ks], ka[buf][ks][0], ka[buf][ks][1], ka[buf][ks][2], ka[buf][ks][3]);
      };
      if (cw < n_gran) fetch(cw, 0);
#pragma unroll
      for (int i = 0; i < KBW; ++i) {
        const int kb = cw + NC * i;
        if (kb < n_gran) {
          const bool more = i + 1 < KBW && kb + NC < n_gran;
          if (!SPLIT && more) fetch(kb + NC, (i + 1) % KBUF);
          float e[4] = {0.f, 0.f, 0.f, 0.f}, f[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) mma_inorder((ks & 1) ? f : e, ka[i % KBUF][ks], qf[ks][0], qf[ks][1]);
          if (SPLIT && more) fetch(kb + NC, 0);
          const int keyA = kb * 16 + g_row, keyB = keyA + 8;
          const bool inner = interior(kb);
          const bool vA = inner || visible(keyA), vB = inner || visible(keyB);
          s[i][0] = vA ? (e[0] + f[0]) * M.scale_log2 : -INFINITY;
          s[i][1] = vA ? (e[1] + f[1]) * M.scale_log2 : -INFINITY;
          s[i][2] = vB ? (e[2] + f[2]) * M.scale_log2 : -INFINITY;
          s[i][3] = vB ? (e[3] + f[3]) * M.scale_log2 : -INFINITY;
        } else {
          s[i][0] = s[i][1] = s[i][2] = s[i][3] = -INFINITY;
        }
        mx0 = fmaxf(mx0, fmaxf(s[i][0], s[i][2]));
        mx1 = fmaxf(mx1, fmaxf(s[i][1], s[i][3]));
      }
    }
    __syncwarp();  // every lane's K fragments are in registers
    if (lane == 0) mbar_arrive(smem_u32(&bars[B_KFREE]));
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
    }
    if (lane < 4) {
      pm[cw][qd] = mx0;
      pm[cw][qd + 1] = mx1;
    }
    // the cache copy of the new row (last compute warp: K from lanes [0, CHUNKS), V from lanes [CHUNKS, 2 CHUNKS))
    const uint4 vrow = newrow;
    const int new_page = __shfl_sync(0xffffffffu, m.my_page, (m.head / M.P) & 31);
    if (fuse && cw == NC - 1 && lane < 2 * CHUNKS && !failed) {
      const int kv = lane / CHUNKS, ch = lane % CHUNKS;
      if (new_page < 0 || new_page >= p.num_pages) {
        if (lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, new_page);
      } else {
        *reinterpret_cast<uint4*>(p.pool + ((((int64_t)new_page * 2 + kv) * M.Hkv + kh) * M.P + m.head % M.P) * D + ch * 8) =
            newrow;
      }
    }
    if (has_next) {
      load_q(nxt);  // consumed an iteration from now
      okm_next = window_tiles(nxt, mt_next, 0, false);
    }
    if (compute_warps_sync_or(failed)) return;  // barrier 1: every partial maximum is published

    // ---------------- softmax of this warp's granules: P^T as B fragments, partial row sums ----------------
    mx0 = fmaxf(fmaxf(pm[0][qd], pm[1][qd]), pm[2][qd]);
    mx1 = fmaxf(fmaxf(pm[0][qd + 1], pm[1][qd + 1]), pm[2][qd + 1]);
    const float m0 = mx0 == -INFINITY ? 0.f : mx0, m1 = mx1 == -INFINITY ? 0.f : mx1;
    float l0 = 0.f, l1 = 0.f;
#pragma unroll
    for (int i = 0; i < KBW; ++i) {
      const int kb = cw + NC * i;
      // bf16 values the tensor core will multiply; the row sums add exactly those
      const uint32_t lo = pack_bf16x2(fast_exp2(s[i][0] - m0), fast_exp2(s[i][1] - m1));  // key g_row: heads qd, qd + 1
      const uint32_t hi = pack_bf16x2(fast_exp2(s[i][2] - m0), fast_exp2(s[i][3] - m1));  // key g_row + 8
      const float2 flo = unpack_bf16x2(lo), fhi = unpack_bf16x2(hi);
      l0 += flo.x + fhi.x;
      l1 += flo.y + fhi.y;
      const uint32_t b0 = movmatrix_trans(lo);  // keys 2t, 2t + 1 of head g_row
      const uint32_t b1 = movmatrix_trans(hi);  // keys 2t + 8, 2t + 9
      Pb[kb * 32 + lane] = make_uint2(b0, b1);
    }
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
      l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
    }
    if (lane < 4) {
      pl[cw][qd] = l0;
      pl[cw][qd + 1] = l1;
    }

    // ---------------- output: this warp's head dims over all granules ----------------
    if (!mbar_wait(smem_u32(&bars[B_VFULL]), par)) {
      failed = true;
      s_abort = 1;
      if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, kh, 11);
    }
    const int g_new = hi_row >> 4;  // granule of the new token's row
    if (fuse && g_new < VE && lane >= CHUNKS && lane < 2 * CHUNKS) {
      *reinterpret_cast<uint4*>(sV + g_new * GRAN_BYTES + gran_off(hi_row & 15, lane - CHUNKS)) = vrow;
      fence_proxy_async_smem();
    }
    if (compute_warps_sync_or(failed)) return;  // barrier 2: P and the partial sums are complete
    // Granule kb of V: in the V area up to VE, behind it in the K area (where the loader puts it once the scores exist;
    // every warp waits for that once per item, whether or not the window reaches that far, so that it sees each phase)
    auto v_gran = [&](int kb) { return (kb < VE ? aV + kb * GRAN_BYTES : aK + (kb - VE) * GRAN_BYTES); };
    auto late_v_ready = [&]() {
      if (!mbar_wait(smem_u32(&bars[B_V2FULL]), par)) {
        late_failed = true;
        s_abort = 1;
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, kh, 13);
      }
      if (fuse && g_new >= VE && lane >= CHUNKS && lane < 2 * CHUNKS) {
        *reinterpret_cast<uint4*>(sK + (g_new - VE) * GRAN_BYTES + gran_off(hi_row & 15, lane - CHUNKS)) = vrow;
        fence_proxy_async_smem();
      }
      __syncwarp();
    };
    float o[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    {
      uint32_t va[2][MT][4];
      uint2 pbv[2];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
        if (mt < n_mt) ldmatrix_x4_trans(aV + v_off[mt], va[0][mt][0], va[0][mt][1], va[0][mt][2], va[0][mt][3]);
      pbv[0] = Pb[lane];
#pragma unroll
      for (int kb = 0; kb < NG; ++kb) {
        if (SPLIT && kb + 1 == VE) late_v_ready();  // before the first fragment of a late granule is fetched
        if (kb < n_gran) {
          if (kb + 1 < NG && kb + 1 < n_gran) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              if (mt < n_mt)
                ldmatrix_x4_trans(v_gran(kb + 1) + v_off[mt], va[(kb + 1) & 1][mt][0], va[(kb + 1) & 1][mt][1],
                                  va[(kb + 1) & 1][mt][2], va[(kb + 1) & 1][mt][3]);
            pbv[(kb + 1) & 1] = Pb[(kb + 1) * 32 + lane];
          }
          // V^T fragments: a0 / a1 hold keys 16 kb + qd, qd + 1 in their halves, a2 / a3 keys 16 kb + 8 + qd, qd + 9.
          // Rows outside the window may hold anything: zero them (0 x NaN would poison the sum).
          if (!interior(kb)) {
            const int k0 = kb * 16 + qd;
            const uint32_t keep_lo = (visible(k0) ? 0x0000ffffu : 0u) | (visible(k0 + 1) ? 0xffff0000u : 0u);
            const uint32_t keep_hi = (visible(k0 + 8) ? 0x0000ffffu : 0u) | (visible(k0 + 9) ? 0xffff0000u : 0u);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              va[kb & 1][mt][0] &= keep_lo;
              va[kb & 1][mt][1] &= keep_lo;
              va[kb & 1][mt][2] &= keep_hi;
              va[kb & 1][mt][3] &= keep_hi;
            }
          }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            if (mt < n_mt) mma_inorder(o[mt], va[kb & 1][mt], pbv[kb & 1].x, pbv[kb & 1].y);
        }
      }
    }
    // row sums of this thread's accumulator columns (heads qd, qd + 1), read before the next item may overwrite them
    l0 = pl[0][qd] + pl[1][qd] + pl[2][qd];
    l1 = pl[0][qd + 1] + pl[1][qd + 1] + pl[2][qd + 1];
    __syncwarp();  // this warp is done with the V tiles
    if (lane == 0) mbar_arrive(smem_u32(&bars[B_VFREE]));
    if (SPLIT && late_failed) continue;  // nothing is written for this item; everyone leaves at the next barrier

    const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
    if (M.out_fp32) {
      // thread: heads qd, qd + 1; head dims 16 (cw MT + mt) + g_row and + 8 (eight lanes fill a 32-byte sector)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (qd + j >= M.G) continue;
        const float inv = j ? inv1 : inv0;
        float* orow = reinterpret_cast<float*>(p.out) + ((int64_t)r * M.Hq + kh * M.G + qd + j) * D + cw * MT * 16 + g_row;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if (mt < n_mt) {
            orow[mt * 16] = o[mt][j] * inv;
            orow[mt * 16 + 8] = o[mt][2 + j] * inv;
          }
        }
      }
    } else {
      // transposed once more: the thread then holds head g_row, dims 16 (cw MT + mt) + qd, qd + 1 (and + 8) as bf16 pairs
      __nv_bfloat16* orow =
          reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)r * M.Hq + kh * M.G + g_row) * D + cw * MT * 16 + qd;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const uint32_t w0 = movmatrix_trans(pack_bf16x2(o[mt][0] * inv0, o[mt][1] * inv1));
        const uint32_t w1 = movmatrix_trans(pack_bf16x2(o[mt][2] * inv0, o[mt][3] * inv1));
        if (g_row < M.G && mt < n_mt) {
          *reinterpret_cast<uint32_t*>(orow + mt * 16) = w0;
          *reinterpret_cast<uint32_t*>(orow + mt * 16 + 8) = w1;
        }
      }
    }
    if (p.lse && cw == 0 && g_row == 0) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (qd + j >= M.G) continue;
        const float l = j ? l1 : l0, mm = j ? mx1 : mx0;
        p.lse[(int64_t)r * M.Hq + kh * M.G + qd + j] = l > 0.f ? (mm + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
    }
  }
}

struct CompactPlan {
  int ng_max, k_region, smem;
};

CompactPlan compact_plan(const ModelParams& m, int nq) {
  const int D = m.D, NT = nq == 1 ? 1 : (nq == 2 ? 2 : 4);
  CompactPlan c;
  c.ng_max = (GR - 1 + m.W - 1 + nq - 1) / GR + 1;
  const int rows_max = c.ng_max * GR;
  const int tile = rows_max * D * 2;                                    // K (or V) tiles
  const int p_area = c.ng_max * NT * 8 * 32;                              // P, bf16
  const int s_area = c.ng_max <= 12 ? 0 : NT * 8 * (rows_max + 8) * 4;    // fp32 scores of long windows
  c.k_region = (tile + 1023) & ~1023;
  c.smem = c.k_region + tile + p_area + s_area + 16 + 2 * 4 * NT * 8 * 4 + 16;  // + barriers, partial maxima / sums, flags
  return c;
}

// 4-D views of the pool {D, P, 2 * Hkv, num_pages} with boxes {64, 16 k, 1, 1}, k = 1 .. P / 16, 128-byte swizzle.
cudaError_t make_ring_maps(const hswa_handle* h, const DecodeParams& p, RingMaps* out) {
  const ModelParams& m = p.m;
  cuuint64_t dims[4] = {(cuuint64_t)m.D, (cuuint64_t)m.P, (cuuint64_t)(2 * m.Hkv), (cuuint64_t)p.num_pages};
  cuuint64_t strides[3] = {(cuuint64_t)m.D * 2, (cuuint64_t)m.D * 2 * m.P, (cuuint64_t)m.D * 2 * m.P * 2 * m.Hkv};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  for (int i = 0; i < 4; ++i) {
    const int rows = (i + 1) * GR <= m.P ? (i + 1) * GR : GR;  // heights above a page are never used
    cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
    if (h->encode_tiled(&out->m[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, p.pool, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  return cudaSuccess;
}

template <int D, int NT>
cudaError_t launch_compact_t(const RingMaps& tm, const DecodeParams& p, const CompactPlan& c, int sms, bool early_start,
                             cudaStream_t s) {
  auto kern = decode_ring_compact_kernel<D, NT>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, c.smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  const int n_items = p.b.B * p.m.Hkv;
  const int resident = sms * (NT == 1 && c.smem <= 75 * 1024 ? 3 : (c.smem <= 112 * 1024 ? 2 : 1));
  cfg.gridDim = dim3(n_items < resident ? n_items : resident, 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = c.smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, tm, p, c.ng_max, c.k_region, n_items);
}

}  // namespace

// Can the compact kernel serve this shape?  It needs the window's granules of one (request, KV head) in shared memory.
bool hswa_ring_compact_supported(const ModelParams& m, int nq) {
  if (m.P % GR != 0 || nq < 1 || nq > 4 || (m.D != 64 && m.D != 128)) return false;
  const CompactPlan c = compact_plan(m, nq);
  return c.ng_max <= 31 && c.smem <= 200 * 1024;
}

// 5-D views of the pool {64, 16, D / 64, P / 16, num_pages * 2 * Hkv}: a box {64, 16, D / 64, k, 1} is a run of k granules
// of one (page, K|V, head) slab, landing granule by granule with the two 64-column halves of a granule behind each other.
cudaError_t make_ring_maps5(const hswa_handle* h, const DecodeParams& p, RingMaps* out) {
  const ModelParams& m = p.m;
  const int halves = m.D / 64, gpp = m.P / GR;
  cuuint64_t dims[5] = {64, (cuuint64_t)GR, (cuuint64_t)halves, (cuuint64_t)gpp, (cuuint64_t)p.num_pages * 2 * m.Hkv};
  cuuint64_t strides[4] = {(cuuint64_t)m.D * 2, 128, (cuuint64_t)GR * m.D * 2, (cuuint64_t)m.P * m.D * 2};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 4; ++i) {
    const int k = i + 1 <= gpp ? i + 1 : 1;  // runs longer than a page do not exist
    cuuint32_t box[5] = {64, (cuuint32_t)GR, (cuuint32_t)halves, (cuuint32_t)k, 1};
    if (h->encode_tiled(&out->m[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, p.pool, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  return cudaSuccess;
}

// Can the compact single-token kernel serve this shape?  (The window's granules, at most nine, stay in registers as scores.)
bool hswa_ring_window_supported(const ModelParams& m, int nq) {
  return nq == 1 && m.W <= 128 && m.P % GR == 0 && (m.D == 64 || m.D == 128) && m.G <= 8 && m.R <= 32;
}

cudaError_t hswa_launch_decode_ring_window(const hswa_handle* h, const DecodeParams& p, bool early_start, cudaStream_t s) {
  if (p.b.B == 0) return cudaSuccess;
  RingMaps maps;
  cudaError_t e = make_ring_maps5(h, p, &maps);
  if (e != cudaSuccess) return e;
  const int D = p.m.D;
  const int n_items = p.b.B * p.m.Hkv;
  // D = 128: with every V granule staged beside K three blocks fit an SM; with four V granules beside K and the rest
  // taking K's place once the scores exist, four fit, which saves a whole round of the walk while the rings number at
  // most four per SM (and costs each later round the latency of loads that can no longer be issued ahead)
  // (measured, us per layer: 10.9 against 12.2 at 512 rings, 11.4 against 12.3 at 576; 17.2 against 13.7 at 800)
  const bool split = D == 128 && n_items > 3 * h->num_sms && n_items <= 4 * h->num_sms;
  const int ve = split ? 4 : 9;
  const int smem = (9 + ve) * (D / 64) * GR * 128 + 48 + 256 + 9 * 256 + 16;  // K and V granules, barriers, maxima / sums, P, flag
  auto kern = D == 128 ? (split ? decode_ring_window_kernel<128, 4> : decode_ring_window_kernel<128, 9>)
                       : decode_ring_window_kernel<64, 9>;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  // three blocks fit an SM only with the whole unified cache configured as shared memory
  e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  int per_sm = (228 * 1024) / (smem + 1024);
  if (per_sm > 4) per_sm = 4;
  const int resident = h->num_sms * per_sm;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_items < resident ? n_items : resident, 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, maps, p, n_items);
}

cudaError_t hswa_launch_decode_ring_compact(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p,
                                            bool early_start, cudaStream_t s) {
  if (p.b.B == 0) return cudaSuccess;
  const int D = p.m.D, nq = p.nq;
  const int NT = nq == 1 ? 1 : (nq == 2 ? 2 : 4);
  const CompactPlan c = compact_plan(p.m, nq);
  (void)tm_pool;  // the kernel uses its own maps, one per box height
  RingMaps maps;
  cudaError_t e = make_ring_maps(h, p, &maps);
  if (e != cudaSuccess) return e;
  if (D == 128 && NT == 1) return launch_compact_t<128, 1>(maps, p, c, h->num_sms, early_start, s);
  if (D == 128 && NT == 2) return launch_compact_t<128, 2>(maps, p, c, h->num_sms, early_start, s);
  if (D == 128 && NT == 4) return launch_compact_t<128, 4>(maps, p, c, h->num_sms, early_start, s);
  if (D == 64 && NT == 1) return launch_compact_t<64, 1>(maps, p, c, h->num_sms, early_start, s);
  if (D == 64 && NT == 2) return launch_compact_t<64, 2>(maps, p, c, h->num_sms, early_start, s);
  if (D == 64 && NT == 4) return launch_compact_t<64, 4>(maps, p, c, h->num_sms, early_start, s);
  return cudaErrorInvalidValue;
}

