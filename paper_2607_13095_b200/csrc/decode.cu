// Batched GQA decode attention over the hybrid KV cache (paper Sec. 2.2: decode is memory-bound, its cost is
// the KV bytes read; Sec. 3.1.1: Full layers read pages through the block table, SWA layers read a ring of
// R pages).  One thread block handles one (request, KV head, key split):
//   - a producer warp walks the block table (or ring table) and streams 64-key K/V tiles into a multi-stage
//     shared-memory ring with TMA tensor loads (128-byte swizzle), completion on mbarriers;
//   - consumer warps each take whole tiles and keep an independent online-softmax state.  Scores are
//     computed transposed on tensor cores, S^T[keys x heads] = K[keys x D] * Q^T[D x heads], so the 8 query
//     heads of a GQA group are the N = 8 of m16n8k16 with no padding; P^T is moved into B-operand layout with
//     movmatrix and O^T[D x heads] += V^T * P^T.  Row maxima are reduced with warp shuffles;
//   - the block merges its warps' states and writes either the final output (one split) or a partial
//     (m, l, o) for the combine kernel.
// The new token's K/V row is patched into the staged tile and written to the cache by the block that owns
// its position (fused append).
#include "hswa_internal.cuh"

namespace {
using namespace hswa_dev;

constexpr int TK = 64;  // keys per pipeline stage

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start while
// the previous kernel on the stream is still running; everything it does before griddep_wait() must not depend
// on that kernel.  Without the attribute both instructions do nothing.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

struct KeyRange {
  int is_swa;
  int span;   // Full: keys in this split; SWA: ring slots C
  int head;   // SWA: ring head
  int ctx;    // tokens cached before the step
  int W, C;
  // Is the key at index `idx` of this block's range visible to the query at position ctx?
  __device__ __forceinline__ bool valid(int idx) const {
    if (!is_swa) return idx < span;
    if (idx >= C) return false;
    int off = idx - head;
    if (off < 0) off += C;
    if (off == 0) return true;  // the new token itself
    const int back = C - off;   // this slot holds position ctx - back
    return back <= W - 1 && back <= ctx;
  }
};

// One consumer warp's work on a staged 64-key tile: S^T = K Q^T, online softmax for the warp's (m, l, O^T)
// state, O^T += V^T P^T.  (vm0, vm1) is the 64-bit visibility mask of the tile for this warp's query.  V rows whose
// bit in (zm0, zm1) is clear (rows no query of the block can see: stale ring slots, the tail of the last page)
// must not reach the output as 0 * (stale or non-finite).  Two ways, chosen by the caller:
//   REG_MASK = false  zero those rows in the staged tile first (a pass over shared memory plus a proxy fence, but
//                     only on tiles that have such rows: right for Full layers, where that is the last tile);
//   REG_MASK = true   zero them in the A fragments after ldmatrix (four logic ops per fragment on every tile, no
//                     pass over shared memory: right for rings, where most tiles have such rows).
template <int D, bool REG_MASK = false>
__device__ __forceinline__ void consume_tile(uint8_t* sV, uint32_t aK, uint32_t aV, uint32_t vm0, uint32_t vm1, bool wrote,
                                             const uint32_t (&qf)[D / 16][2], float scale_log2, float (&m_run)[2],
                                             float (&l_run)[2], float (&o)[D / 16][4], int lane, uint32_t zm0, uint32_t zm1) {
  constexpr int HALF_BYTES = TK * 128;
  constexpr int KS = D / 16;
  const int mi = lane >> 3, mr = lane & 7;
  if constexpr (!REG_MASK) {
  if ((zm0 & zm1) != 0xffffffffu) {
    constexpr int CHUNKS = D / 8;
    for (int idx = lane; idx < TK * CHUNKS; idx += 32) {
      const int row = idx / CHUNKS, ch = idx % CHUNKS;
      const bool v = ((row < 32 ? zm0 : zm1) >> (row & 31)) & 1u;
      if (!v) *reinterpret_cast<uint4*>(sV + (ch >> 3) * HALF_BYTES + swz128(row, ch & 7)) = make_uint4(0, 0, 0, 0);
    }
    wrote = true;
  }
  }
  if (wrote) {  // this tile was patched through the generic proxy (zeroed rows, fused append)
    fence_proxy_async_smem();
    __syncwarp();
  }

  if ((vm0 | vm1) != 0u) {
    // S^T = K Q^T for the 64 keys (four 16-key blocks)
    float s[4][4];
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      s[kb][0] = s[kb][1] = s[kb][2] = s[kb][3] = 0.f;
      const int key = kb * 16 + (mi & 1) * 8 + mr;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int chunk = 2 * ks + (mi >> 1);
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4(aK + (chunk >> 3) * HALF_BYTES + swz128(key, chunk & 7), a0, a1, a2, a3);
        mma_bf16_16816(s[kb], a0, a1, a2, a3, qf[ks][0], qf[ks][1]);
      }
    }
    // mask, scale, tile maxima per head (this thread: heads qd and qd+1; keys lane/4 + 8j)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      const int keyA = kb * 16 + (lane >> 2), keyB = keyA + 8;
      const bool vA = ((keyA < 32 ? vm0 : vm1) >> (keyA & 31)) & 1u;
      const bool vB = ((keyB < 32 ? vm0 : vm1) >> (keyB & 31)) & 1u;
      s[kb][0] = vA ? s[kb][0] * scale_log2 : -INFINITY;
      s[kb][1] = vA ? s[kb][1] * scale_log2 : -INFINITY;
      s[kb][2] = vB ? s[kb][2] * scale_log2 : -INFINITY;
      s[kb][3] = vB ? s[kb][3] * scale_log2 : -INFINITY;
      mx[0] = fmaxf(mx[0], fmaxf(s[kb][0], s[kb][2]));
      mx[1] = fmaxf(mx[1], fmaxf(s[kb][1], s[kb][3]));
    }
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], sh));
      mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], sh));
    }
    float m_use[2], alpha[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float m_new = fmaxf(m_run[j], mx[j]);
      m_use[j] = m_new == -INFINITY ? 0.f : m_new;
      alpha[j] = fast_exp2(m_run[j] - m_use[j]);
      m_run[j] = m_new;
      l_run[j] *= alpha[j];
    }
#pragma unroll
    for (int i = 0; i < KS; ++i) {
      o[i][0] *= alpha[0];
      o[i][1] *= alpha[1];
      o[i][2] *= alpha[0];
      o[i][3] *= alpha[1];
    }
    uint32_t pk[8];
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      pk[2 * kb] = pack_bf16x2(fast_exp2(s[kb][0] - m_use[0]), fast_exp2(s[kb][1] - m_use[1]));
      pk[2 * kb + 1] = pack_bf16x2(fast_exp2(s[kb][2] - m_use[0]), fast_exp2(s[kb][3] - m_use[1]));
      const float2 f0 = unpack_bf16x2(pk[2 * kb]), f1 = unpack_bf16x2(pk[2 * kb + 1]);
      l_run[0] += f0.x + f1.x;  // sum the values the tensor core will actually multiply
      l_run[1] += f0.y + f1.y;
    }
    // O^T += V^T P^T.  After the transposing load, a0 and a1 hold keys 16 kb + 2t, 2t + 1 (t = lane mod 4) in
    // their halves, a2 and a3 hold keys 16 kb + 8 + 2t, 2t + 9.
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      const uint32_t b0 = movmatrix_trans(pk[2 * kb]);
      const uint32_t b1 = movmatrix_trans(pk[2 * kb + 1]);
      const int key = kb * 16 + (mi >> 1) * 8 + mr;
      if constexpr (!REG_MASK) {
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
          const int chunk = 2 * mt + (mi & 1);
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4_trans(aV + (chunk >> 3) * HALF_BYTES + swz128(key, chunk & 7), a0, a1, a2, a3);
          mma_bf16_16816(o[mt], a0, a1, a2, a3, b0, b1);
        }
      } else {
        const uint32_t zw = kb < 2 ? zm0 : zm1;
        const int sh = (kb & 1) * 16 + (lane & 3) * 2;
        const uint32_t bits_lo = zw >> sh, bits_hi = zw >> (sh + 8);
        const uint32_t keep_lo = ((bits_lo & 1u) ? 0x0000ffffu : 0u) | ((bits_lo & 2u) ? 0xffff0000u : 0u);
        const uint32_t keep_hi = ((bits_hi & 1u) ? 0x0000ffffu : 0u) | ((bits_hi & 2u) ? 0xffff0000u : 0u);
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
          const int chunk = 2 * mt + (mi & 1);
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4_trans(aV + (chunk >> 3) * HALF_BYTES + swz128(key, chunk & 7), a0, a1, a2, a3);
          mma_bf16_16816(o[mt], a0 & keep_lo, a1 & keep_lo, a2 & keep_hi, a3 & keep_hi, b0, b1);
        }
      }
    }
  }
}

template <int D, int P, int NS, int NW>
__global__ void __launch_bounds__((NW + 1) * 32, 2)
decode_kernel(const __grid_constant__ CUtensorMap tm_pool, const DecodeParams p) {
  constexpr int HALVES = D / 64;
  constexpr int PPT = TK / P;  // pages per tile
  constexpr int HALF_BYTES = TK * 128;
  constexpr int STAGE_BYTES = 2 * HALVES * HALF_BYTES;
  constexpr int BOX_BYTES = P * 128;
  constexpr int CHUNKS = D / 8;  // 16-byte chunks per row
  constexpr int KS = D / 16;
  static_assert(TK % P == 0, "page size must divide the tile");
  // Consumer warp c takes tiles c, c + NW, ...: with NS a multiple of NW every fill of a stage is waited for by the
  // same warp, so that warp sees each phase of the stage's barrier in turn.  A parity wait tells a phase only from
  // its neighbours: a warp that skipped phases could pass a barrier that is still one fill behind.
  static_assert(NS % NW == 0, "a stage must always be consumed by the same warp");

  // All shared memory is one dynamic window (no static part, so that it starts on the 1 KB boundary the swizzled tiles
  // need without slack): the stage buffers, then the barriers.
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NS * STAGE_BYTES);  // [2 * NS]
  const uint32_t smem_base = smem_u32(smem);

  const int r = blockIdx.x, split = blockIdx.y, kh = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const ModelParams& M = p.m;
  const int ctx = p.b.ctx_len[r];
  const int kv_len = ctx + 1;
  // the grid was sized from the host's bound: a longer context would silently lose its tail
  if (threadIdx.x == 0 && split == 0 && kh == 0 && ctx > p.max_ctx_len) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, ctx);

  KeyRange kr;
  kr.is_swa = p.is_swa;
  kr.ctx = ctx;
  kr.W = M.W;
  kr.C = M.C;
  kr.head = 0;
  int k_begin = 0;
  if (!p.is_swa) {
    k_begin = p.k_start + split * p.split_len;
    if (k_begin >= kv_len) return;
    kr.span = min(kv_len, k_begin + p.split_len) - k_begin;
  } else {
    if (split > 0) return;
    kr.head = p.b.ring_head[r];
    kr.span = M.C;
  }
  const int n_tiles = (kr.span + TK - 1) / TK;
  const int idx_new = p.is_swa ? kr.head : ctx - k_begin;  // index of the new token in this block's range
  const bool fuse = p.k_new != nullptr;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(smem_u32(&bars[i]), 1);       // full: producer's arrive + TMA bytes
      mbar_init(smem_u32(&bars[NS + i]), 1);  // empty: one consumer warp per tile
    }
    mbar_fence_init();
    tma_prefetch_desc(&tm_pool);
    if (smem_base & 1023u) record_error(p.err, HSWA_ERR_CUDA, -1, (int)(smem_base & 1023u), 15);  // tiles would be misread
  }
  __syncthreads();

  // online-softmax state of a consumer warp (unused by the producer warp)
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  float o[KS][4];
#pragma unroll
  for (int i = 0; i < KS; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  const int qd = (lane & 3) * 2;  // this thread's two heads: qd, qd + 1

  if (warp == 0) {
    // ---------------- producer ----------------
    const int32_t* tbl;
    int n_pages;
    if (!p.is_swa) {
      tbl = p.b.block_table + (int64_t)r * p.b.max_blocks + k_begin / P;
      n_pages = (kr.span + P - 1) / P;
    } else {
      tbl = p.b.ring_table + (int64_t)r * M.R;
      n_pages = M.R;
    }
    int pid_next = lane < n_pages ? tbl[lane] : 0;
    int pid_cur = 0;
    for (int t = 0; t < n_tiles; ++t) {
      const int pg0 = t * PPT;
      if ((pg0 & 31) == 0) {
        pid_cur = pid_next;
        const int nx = pg0 + 32 + lane;
        pid_next = nx < n_pages ? tbl[nx] : 0;
      }
      const int stage = t % NS;
      if (t >= NS) {
        if (!mbar_wait(smem_u32(&bars[NS + stage]), ((t / NS) - 1) & 1)) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 1);
          break;
        }
      }
      uint32_t need = 0;
      int pages[PPT];
#pragma unroll
      for (int i = 0; i < PPT; ++i) {
        const int pgi = pg0 + i;
        pages[i] = __shfl_sync(0xffffffffu, pid_cur, pgi & 31);
        bool v = false;
        if (pgi < n_pages)
          for (int s = lane; s < P; s += 32) v |= kr.valid(pgi * P + s);
        if (__any_sync(0xffffffffu, v)) need |= 1u << i;
      }
      if (lane == 0) {
        uint32_t ok = 0;
#pragma unroll
        for (int i = 0; i < PPT; ++i) {
          if (!(need & (1u << i))) continue;
          if (pages[i] < 0 || pages[i] >= p.num_pages) {
            record_error(p.err, HSWA_ERR_BOUNDS, r, pg0 + i, pages[i]);
            continue;
          }
          ok |= 1u << i;
        }
        const uint32_t full_bar = smem_u32(&bars[stage]);
        if (ok == 0) {
          mbar_arrive(full_bar);
        } else {
          mbar_arrive_expect_tx(full_bar, __popc(ok) * 2 * HALVES * BOX_BYTES);
          const uint32_t sbase = smem_base + stage * STAGE_BYTES;
#pragma unroll
          for (int i = 0; i < PPT; ++i) {
            if (!(ok & (1u << i))) continue;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv)
#pragma unroll
              for (int hf = 0; hf < HALVES; ++hf)
                tma_load_4d(sbase + (kv * HALVES + hf) * HALF_BYTES + i * BOX_BYTES, &tm_pool, full_bar, hf * 64, 0,
                            kv * M.Hkv + kh, pages[i]);
          }
        }
      }
      __syncwarp();
    }
    if (!p.late_dep_wait) griddep_wait();  // this warp takes part in the output writes below
  } else {
    // ---------------- consumers ----------------
    const int cw = warp - 1;
    const int g_row = lane >> 2;  // head index used for the Q fragment (B operand column)
    uint32_t qf[KS][2];
    // q, k_new, v_new may come from the previous kernel on the stream; the batch arrays and the cache that the
    // producer warp is already streaming do not
    if (!p.late_dep_wait) griddep_wait();
    griddep_launch_dependents();
    {
      const __nv_bfloat16* qrow = p.q + ((int64_t)r * M.Hq + kh * M.G + g_row) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qf[ks][0] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
        qf[ks][1] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
      }
    }
    for (int t = cw; t < n_tiles; t += NW) {
      const int stage = t % NS;
      if (!mbar_wait(smem_u32(&bars[stage]), (t / NS) & 1)) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 2);
        break;
      }
      uint8_t* sK = smem + stage * STAGE_BYTES;
      uint8_t* sV = sK + HALVES * HALF_BYTES;
      const uint32_t aK = smem_base + stage * STAGE_BYTES;
      const uint32_t aV = aK + HALVES * HALF_BYTES;
      const int tile_lo = t * TK;
      bool wrote = false;

      // fused append: patch the new token's row into the staged tile and write it to the cache
      if (fuse && idx_new >= tile_lo && idx_new < tile_lo + TK) {
        const int row = idx_new - tile_lo;
        int page, slot;
        if (!p.is_swa) {
          page = p.b.block_table[(int64_t)r * p.b.max_blocks + ctx / P];
          slot = ctx % P;
        } else {
          page = p.b.ring_table[(int64_t)r * M.R + kr.head / P];
          slot = kr.head % P;
        }
        const bool page_ok = page >= 0 && page < p.num_pages;
        if (!page_ok && lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, page);
        for (int c = lane; c < 2 * CHUNKS; c += 32) {
          const int kv = c / CHUNKS, ch = c % CHUNKS;
          const __nv_bfloat16* src = (kv == 0 ? p.k_new : p.v_new) + ((int64_t)r * M.Hkv + kh) * D + ch * 8;
          const uint4 val = *reinterpret_cast<const uint4*>(src);
          uint8_t* dst_s = (kv == 0 ? sK : sV) + (ch >> 3) * HALF_BYTES + swz128(row, ch & 7);
          *reinterpret_cast<uint4*>(dst_s) = val;
          if (page_ok) {
            __nv_bfloat16* dst_g = p.pool + ((((int64_t)page * 2 + kv) * M.Hkv + kh) * P + slot) * D + ch * 8;
            *reinterpret_cast<uint4*>(dst_g) = val;
          }
        }
        wrote = true;
      }
      // validity of the tile's 64 keys
      const uint32_t vm0 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + lane));
      const uint32_t vm1 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + 32 + lane));
      consume_tile<D>(sV, aK, aV, vm0, vm1, wrote, qf, M.scale_log2, m_run, l_run, o, lane, vm0, vm1);
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[NS + stage]));
    }

    // per-warp row sums: lanes with equal (lane & 3) hold the same two heads
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
    }
  }
  __syncthreads();  // every tile has been consumed: the stage buffers can now hold the merge scratch
  if (warp != 0) {
    const int cw = warp - 1;
    float* sc_o = reinterpret_cast<float*>(smem);  // [NW][8][D]
    float* sc_ml = sc_o + NW * 8 * D;              // [NW][8][2]
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
      const int d0 = mt * 16 + (lane >> 2);
      sc_o[(cw * 8 + qd) * D + d0] = o[mt][0];
      sc_o[(cw * 8 + qd + 1) * D + d0] = o[mt][1];
      sc_o[(cw * 8 + qd) * D + d0 + 8] = o[mt][2];
      sc_o[(cw * 8 + qd + 1) * D + d0 + 8] = o[mt][3];
    }
    if (lane < 4) {
      sc_ml[(cw * 8 + qd) * 2 + 0] = m_run[0];
      sc_ml[(cw * 8 + qd) * 2 + 1] = l_run[0];
      sc_ml[(cw * 8 + qd + 1) * 2 + 0] = m_run[1];
      sc_ml[(cw * 8 + qd + 1) * 2 + 1] = l_run[1];
    }
  }
  __syncthreads();

  // ---------------- merge the consumer warps' states ----------------
  const float* sc_o = reinterpret_cast<const float*>(smem);
  const float* sc_ml = sc_o + NW * 8 * D;
  for (int idx = threadIdx.x; idx < M.G * D; idx += blockDim.x) {
    const int g = idx / D, d = idx % D;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) mm = fmaxf(mm, sc_ml[(w * 8 + g) * 2]);
    float L = 0.f, O = 0.f;
    if (mm != -INFINITY) {
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float f = fast_exp2(sc_ml[(w * 8 + g) * 2] - mm);
        L += f * sc_ml[(w * 8 + g) * 2 + 1];
        O += f * sc_o[(w * 8 + g) * D + d];
      }
    }
    const int64_t row = (int64_t)r * M.Hq + kh * M.G + g;
    if (p.max_splits == 1) {
      const float val = L > 0.f ? O / L : 0.f;
      if (M.out_fp32)
        reinterpret_cast<float*>(p.out)[row * D + d] = val;
      else
        reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d] = __float2bfloat16_rn(val);
      if (d == 0 && p.lse) p.lse[row] = L > 0.f ? (mm + log2f(L)) * 0.6931471805599453f : -INFINITY;
    } else {
      p.part_o[(row * p.max_splits + p.split_base + split) * D + d] = O;
      if (d == 0) p.part_ml[row * p.max_splits + p.split_base + split] = make_float2(mm, L);
    }
  }
  // Cascade decode: this grid must not be complete before the shared-prefix stage it overlapped is, because the
  // combine waits for this grid only.
  if (p.late_dep_wait) griddep_wait();
}

// Merge split-K partials: out = sum_s 2^(m_s - m) o_s / sum_s 2^(m_s - m) l_s.  One warp per (request, head).
template <int D>
__global__ void __launch_bounds__(128) combine_kernel(const DecodeParams p) {
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const ModelParams& M = p.m;
  griddep_launch_dependents();  // the next attention kernel may start its cache loads now
  griddep_wait();               // launched early behind the kernel that writes the partials
  if (warp_global >= p.b.B * p.nq * M.Hq) return;
  const int r = warp_global / (p.nq * M.Hq);
  const int64_t row = warp_global;
  const int kv_len = p.b.ctx_len[r] + p.nq;
  const int n_splits = min(p.max_splits, p.split_base + (kv_len - p.k_start + p.split_len - 1) / p.split_len);
  const float2* ml = p.part_ml + row * p.max_splits;
  const float* po = p.part_o + row * p.max_splits * D;
  float mm = -INFINITY;
  for (int s = lane; s < n_splits; s += 32) mm = fmaxf(mm, ml[s].x);
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, sh));
  constexpr int PER = D / 32;
  float acc[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) acc[i] = 0.f;
  float L = 0.f;
  if (mm != -INFINITY) {
    for (int s = 0; s < n_splits; ++s) {
      const float2 v = ml[s];
      const float f = fast_exp2(v.x - mm);
      L += f * v.y;
      if constexpr (PER == 4) {
        const float4 x = *reinterpret_cast<const float4*>(po + (int64_t)s * D + lane * 4);
        acc[0] += f * x.x;
        acc[1] += f * x.y;
        acc[2] += f * x.z;
        acc[3] += f * x.w;
      } else {
        const float2 x = *reinterpret_cast<const float2*>(po + (int64_t)s * D + lane * 2);
        acc[0] += f * x.x;
        acc[1] += f * x.y;
      }
    }
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const float val = acc[i] * inv;
    if (M.out_fp32)
      reinterpret_cast<float*>(p.out)[row * D + lane * PER + i] = val;
    else
      reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + lane * PER + i] = __float2bfloat16_rn(val);
  }
  if (lane == 0 && p.lse) p.lse[row] = L > 0.f ? (mm + log2f(L)) * 0.6931471805599453f : -INFINITY;
}

// ---------------------------------------------------------------------------------------------------------
// SWA layers: persistent variant.  A ring holds at most C slots per (request, KV head), i.e. a handful of
// tiles, so a block per ring is all latency: table reads, one TMA round trip, a short compute, a merge.
// Here a block walks many rings: the producer warp streams the tiles of ring after ring through the same
// stage buffers (metadata of the next ring fetched one ring ahead), the consumer warps prefetch the next
// ring's Q while they work, and every ring's warps merge through a small scratch area.  The loads of ring
// k + 1 thus overlap the compute, merge and output of ring k.
// TOKENS = false: one new token per request (nq = 1), three consumer warps take one tile each and merge.
// TOKENS = true: a decode step that carries draft tokens (nq = 2 .. 4): one consumer warp per token walks all the
// tiles of the ring with its own Q, mask and softmax state, so the ring is staged once for all tokens and nothing
// has to be merged.
template <int D, int P, bool TOKENS>
__global__ void __launch_bounds__(TOKENS ? 160 : 128, 2)
decode_ring_kernel(const __grid_constant__ CUtensorMap tm_pool, const DecodeParams p, const int n_items) {
  constexpr int NS = 3, NW = 3;
  constexpr int HALVES = D / 64;
  constexpr int HALF_BYTES = TK * 128;
  constexpr int STAGE_BYTES = 2 * HALVES * HALF_BYTES;
  constexpr int GR = P < HSWA_RING_GRANULE ? P : HSWA_RING_GRANULE;  // slots per TMA box
  constexpr int NG = TK / GR;                                         // granules per tile
  constexpr int CHUNKS = D / 8;
  constexpr int KS = D / 16;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * NS];
  __shared__ int s_abort;  // token mode: a warp's wait ran out; all token warps leave together at the next barrier
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  float* sc_o = reinterpret_cast<float*>(smem + NS * STAGE_BYTES);  // [NW][8][D]
  float* sc_ml = sc_o + NW * 8 * D;                                 // [NW][8][2]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const ModelParams& M = p.m;
  const int n_tiles = (M.C + TK - 1) / TK;
  const bool fuse = p.k_new != nullptr;  // the new tokens are appended here; otherwise they are in the cache already
  // Token w of a request sits at position ctx + w in slot ring_head + w, so it sees the ring exactly as a single
  // new token of a request with ctx + w cached tokens and that ring head would (later drafts lie ahead of its
  // slot, more than W - 1 slots "back" around the ring, because nq <= C - W + 1).  When the append is fused,
  // the warp of token w patches row w into the staged tile and writes it to the cache; a barrier among the
  // token warps makes all nq rows visible before any of them reads the tiles.
  const int nq = TOKENS ? p.nq : 1;
  // One token per request: consumer warp c takes tiles c, c + NW, ... of every ring.  When the tiles of a ring are a
  // multiple of NW = NS (the paper's ring: 3 tiles) or a single one, a stage is always consumed by the same warp, which
  // therefore sees each phase of the stage's barrier in turn.  Otherwise every warp waits for every tile and releases
  // it, and works only on its own: a parity wait tells a phase only from its neighbours, so a warp that skipped
  // phases could pass a barrier that is still one fill behind.
  static_assert(NS == NW, "stage ownership below assumes as many stages as consumer warps");
  const bool lockstep = !TOKENS && n_tiles != 1 && n_tiles % NW != 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(smem_u32(&bars[i]), 1);
      // consumers that release a tile: one per token; else the one warp that works on it, or all of them in lockstep
      mbar_init(smem_u32(&bars[NS + i]), TOKENS ? nq : (lockstep ? NW : 1));
    }
    mbar_fence_init();
    tma_prefetch_desc(&tm_pool);
    s_abort = 0;
  }
  __syncthreads();

  if (warp == 0) {
    // ---------------- producer ----------------
    int it = blockIdx.x;
    int ctx_n = 0, head_n = 0, pid_n = 0;
    if (it < n_items) {
      const int r = it / M.Hkv;
      ctx_n = p.b.ctx_len[r];
      head_n = p.b.ring_head[r];
      pid_n = lane < M.R ? p.b.ring_table[(int64_t)r * M.R + lane] : 0;
    }
    bool ok = true;
    for (int k = 0; it < n_items && ok; ++k, it += gridDim.x) {
      const int r = it / M.Hkv, kh = it % M.Hkv;
      KeyRange kr;
      kr.is_swa = 1;
      kr.span = M.C;
      kr.head = head_n;
      kr.ctx = ctx_n;
      kr.W = M.W;
      kr.C = M.C;
      const int pid = pid_n;
      const int nxt = it + gridDim.x;
      if (nxt < n_items) {  // next ring's metadata, one ring ahead of its first TMA
        const int rn = nxt / M.Hkv;
        ctx_n = p.b.ctx_len[rn];
        head_n = p.b.ring_head[rn];
        pid_n = lane < M.R ? p.b.ring_table[(int64_t)rn * M.R + lane] : 0;
      }
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int g = k * n_tiles + t, stage = g % NS;
        if (g >= NS && !mbar_wait(smem_u32(&bars[NS + stage]), ((g / NS) - 1) & 1)) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 3);
          ok = false;
          break;
        }
        // The tile's TK slots are loaded in granules of GR slots (a granule never straddles a page), and only
        // the granules that meet the window: the slots visible to at least one of the nq tokens form the circular
        // interval [head - min(W - 1, ctx), head + nq - 1].  Rows of granules that are not loaded keep whatever the
        // stage buffer held; the consumers never let them count (masked scores, V fragments zeroed).
        const int back = min(M.W - 1, kr.ctx);
        const int start = math_mod(kr.head - back, M.C);
        const int last = back + nq - 1;  // offset of the last visible slot from `start`
        uint32_t okm = 0;
        const int slot_lo = t * TK + (lane % NG) * GR;  // lane i < NG looks after granule i
        const int pgi = slot_lo / P;
        const int page_of = __shfl_sync(0xffffffffu, pid, pgi & 31);
        if (lane < NG) {
          if (pgi < M.R && (math_mod(slot_lo - start, M.C) <= last || math_mod(start - slot_lo, M.C) < GR)) {
            if (page_of < 0 || page_of >= p.num_pages)
              record_error(p.err, HSWA_ERR_BOUNDS, r, pgi, page_of);
            else
              okm = 1u << lane;
          }
        }
#pragma unroll
        for (int sh = 1; sh < NG; sh <<= 1) okm |= __shfl_xor_sync(0xffffffffu, okm, sh);
        const uint32_t full_bar = smem_u32(&bars[stage]);
        if (lane == 0) {
          if (okm == 0)
            mbar_arrive(full_bar);
          else
            mbar_arrive_expect_tx(full_bar, __popc(okm) * 2 * HALVES * GR * 128);
        }
        __syncwarp();
        if (lane < NG && (okm >> lane) & 1u) {
          const uint32_t sb = smem_base + stage * STAGE_BYTES + lane * GR * 128;
          const int slot_in_page = slot_lo % P;
#pragma unroll
          for (int kv = 0; kv < 2; ++kv)
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
              tma_load_4d(sb + (kv * HALVES + hf) * HALF_BYTES, &tm_pool, full_bar, hf * 64, slot_in_page, kv * M.Hkv + kh, page_of);
        }
        __syncwarp();
      }
    }
  } else if constexpr (TOKENS) {
    // ---------------- consumers: one warp per draft token ----------------
    const int w_tok = warp - 1;
    if (w_tok < nq) {
      const int g_row = lane >> 2;
      const int qd = (lane & 3) * 2;
      int it = blockIdx.x;
      uint32_t qn[KS][2];
      int ctx_n = 0, head_n = 0, pid_n = -1;
      static_assert(2 * CHUNKS <= 32, "one chunk of the new K/V row per lane");
      uint4 an = make_uint4(0, 0, 0, 0);
      auto prefetch_meta = [&](int item) {  // constant during a step: may be read before the dependency wait
        const int r = item / M.Hkv;
        ctx_n = p.b.ctx_len[r];
        head_n = p.b.ring_head[r];
        pid_n = lane < M.R ? p.b.ring_table[(int64_t)r * M.R + lane] : -1;
      };
      auto prefetch_qkv = [&](int item) {
        const int r = item / M.Hkv, kh = item % M.Hkv;
        const __nv_bfloat16* qrow = p.q + (((int64_t)r * nq + w_tok) * M.Hq + kh * M.G + g_row) * D;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          qn[ks][0] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
          qn[ks][1] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
        }
        if (fuse && lane < 2 * CHUNKS)
          an = *reinterpret_cast<const uint4*>((lane < CHUNKS ? p.k_new : p.v_new) +
                                               (((int64_t)r * nq + w_tok) * M.Hkv + kh) * D + (lane % CHUNKS) * 8);
      };
      if (it < n_items) prefetch_meta(it);
      griddep_wait();  // q, k_new, v_new and out may belong to the previous kernel on the stream
      griddep_launch_dependents();
      if (it < n_items) prefetch_qkv(it);
      for (int k = 0; it < n_items; ++k, it += gridDim.x) {
        const int r = it / M.Hkv, kh = it % M.Hkv;
        uint32_t qf[KS][2];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          qf[ks][0] = qn[ks][0];
          qf[ks][1] = qn[ks][1];
        }
        KeyRange kr;
        kr.is_swa = 1;
        kr.span = M.C;
        kr.head = math_mod(head_n + w_tok, M.C);
        kr.ctx = ctx_n + w_tok;
        kr.W = M.W;
        kr.C = M.C;
        const uint4 a_cur = an;
        const int pid_cur = pid_n;
        if (it + gridDim.x < n_items) {
          prefetch_meta(it + gridDim.x);
          prefetch_qkv(it + gridDim.x);
        }
        // every tile of the ring is staged before this token's row is patched in and before anything is read
        bool ok = true;
        for (int t = 0; t < n_tiles; ++t) {
          const int g = k * n_tiles + t;
          if (!mbar_wait(smem_u32(&bars[g % NS]), (g / NS) & 1)) {
            if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 4);
            ok = false;
            break;
          }
        }
        if (!ok && lane == 0) *reinterpret_cast<volatile int*>(&s_abort) = 1;
        if (fuse && ok) {
          const int t_new = kr.head / TK, row = kr.head % TK;
          uint8_t* sK = smem + ((k * n_tiles + t_new) % NS) * STAGE_BYTES;
          uint8_t* sV = sK + HALVES * HALF_BYTES;
          const int page = __shfl_sync(0xffffffffu, pid_cur, kr.head / P);
          const bool page_ok = page >= 0 && page < p.num_pages;
          if (!page_ok && lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, page);
          if (lane < 2 * CHUNKS) {
            const int kv = lane / CHUNKS, ch = lane % CHUNKS;
            *reinterpret_cast<uint4*>((kv == 0 ? sK : sV) + (ch >> 3) * HALF_BYTES + swz128(row, ch & 7)) = a_cur;
            if (page_ok)
              *reinterpret_cast<uint4*>(p.pool + ((((int64_t)page * 2 + kv) * M.Hkv + kh) * P + kr.head % P) * D + ch * 8) = a_cur;
          }
          fence_proxy_async_smem();
        }
        asm volatile("bar.sync 1, %0;" ::"r"(nq * 32) : "memory");  // all nq rows are in the tiles now
        if (*reinterpret_cast<volatile int*>(&s_abort)) break;  // same value in every token warp: they stop together
        float m_run[2] = {-INFINITY, -INFINITY};
        float l_run[2] = {0.f, 0.f};
        float o[KS][4];
#pragma unroll
        for (int i = 0; i < KS; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
          const int stage = (k * n_tiles + t) % NS;
          if (ok) {
            uint8_t* sV = smem + stage * STAGE_BYTES + HALVES * HALF_BYTES;
            const uint32_t aK = smem_base + stage * STAGE_BYTES;
            const uint32_t aV = aK + HALVES * HALF_BYTES;
            const int tile_lo = t * TK;
            const uint32_t vm0 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + lane));
            const uint32_t vm1 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + 32 + lane));
            consume_tile<D, true>(sV, aK, aV, vm0, vm1, false, qf, M.scale_log2, m_run, l_run, o, lane, vm0, vm1);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bars[NS + stage]));
        }
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
          l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
          l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
        }
        // this warp owns the whole result of its token: straight from the accumulator fragments to the output
        // (thread: heads qd, qd + 1; head dims 16 mt + lane / 4 and + 8)
        if (ok) {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (qd + j >= M.G) continue;
            const float inv = l_run[j] > 0.f ? 1.f / l_run[j] : 0.f;
            const int64_t row = ((int64_t)r * nq + w_tok) * M.Hq + kh * M.G + qd + j;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
              const int d0 = mt * 16 + (lane >> 2);
              if (M.out_fp32) {
                reinterpret_cast<float*>(p.out)[row * D + d0] = o[mt][j] * inv;
                reinterpret_cast<float*>(p.out)[row * D + d0 + 8] = o[mt][2 + j] * inv;
              } else {
                reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d0] = __float2bfloat16_rn(o[mt][j] * inv);
                reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d0 + 8] = __float2bfloat16_rn(o[mt][2 + j] * inv);
              }
            }
            if ((lane >> 2) == 0 && p.lse)
              p.lse[row] = l_run[j] > 0.f ? (m_run[j] + log2f(l_run[j])) * 0.6931471805599453f : -INFINITY;
          }
        }
      }
    }
  } else {
    // ---------------- consumers ----------------
    const int cw = warp - 1;
    const int g_row = lane >> 2;
    const int qd = (lane & 3) * 2;
    int it = blockIdx.x;
    uint32_t qn[KS][2];
    int ctx_n = 0, head_n = 0, pid_n = -1;
    // fused append: the K (lanes [0, CHUNKS)) and V (lanes [CHUNKS, 2 CHUNKS)) row of the next token, one 16-byte
    // chunk per lane, fetched one pass ahead like Q
    static_assert(2 * CHUNKS <= 32, "one chunk of the new K/V row per lane");
    uint4 an = make_uint4(0, 0, 0, 0);
    // lengths, ring head and ring table do not change during a step: they may be read before the previous
    // kernel on the stream has finished (lane i keeps page id i of the ring)
    auto prefetch_meta = [&](int item) {
      const int r = item / M.Hkv;
      ctx_n = p.b.ctx_len[r];
      head_n = p.b.ring_head[r];
      pid_n = lane < M.R ? p.b.ring_table[(int64_t)r * M.R + lane] : -1;
    };
    auto prefetch_qkv = [&](int item, int w) {
      const int r = item / M.Hkv, kh = item % M.Hkv;
      const __nv_bfloat16* qrow = p.q + (((int64_t)r * nq + w) * M.Hq + kh * M.G + g_row) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qn[ks][0] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
        qn[ks][1] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
      }
      if (fuse && lane < 2 * CHUNKS)
        an = *reinterpret_cast<const uint4*>((lane < CHUNKS ? p.k_new : p.v_new) + (((int64_t)r * nq + w) * M.Hkv + kh) * D +
                                             (lane % CHUNKS) * 8);
    };
    if (it < n_items) prefetch_meta(it);
    griddep_wait();  // q, k_new, v_new and out may belong to the previous kernel on the stream
    griddep_launch_dependents();
    if (it < n_items) prefetch_qkv(it, 0);
    for (int k = 0; it < n_items; ++k, it += gridDim.x) {
      const int r = it / M.Hkv, kh = it % M.Hkv;
      const int ctx0 = ctx_n, head0 = head_n, pid_cur = pid_n;
      if (it + gridDim.x < n_items) prefetch_meta(it + gridDim.x);
      constexpr int w_tok = 0;  // this path serves one new token per request
      uint32_t qf[KS][2];
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qf[ks][0] = qn[ks][0];
        qf[ks][1] = qn[ks][1];
      }
      KeyRange kr;
      kr.is_swa = 1;
      kr.span = M.C;
      kr.head = math_mod(head0 + w_tok, M.C);
      kr.ctx = ctx0 + w_tok;
      kr.W = M.W;
      kr.C = M.C;
      const int ctx = kr.ctx;
      const uint4 a_cur = an;
      if (it + gridDim.x < n_items) prefetch_qkv(it + gridDim.x, 0);

      float m_run[2] = {-INFINITY, -INFINITY};
      float l_run[2] = {0.f, 0.f};
      float o[KS][4];
#pragma unroll
      for (int i = 0; i < KS; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
      bool ok = true;
      for (int t = lockstep ? 0 : cw; t < n_tiles; t += lockstep ? 1 : NW) {
        const int g = k * n_tiles + t, stage = g % NS;
        if (!mbar_wait(smem_u32(&bars[stage]), (g / NS) & 1)) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 4);
          ok = false;
          break;
        }
        if (lockstep && t % NW != cw) {
          if (lane == 0) mbar_arrive(smem_u32(&bars[NS + stage]));
          continue;
        }
        uint8_t* sK = smem + stage * STAGE_BYTES;
        uint8_t* sV = sK + HALVES * HALF_BYTES;
        const uint32_t aK = smem_base + stage * STAGE_BYTES;
        const uint32_t aV = aK + HALVES * HALF_BYTES;
        const int tile_lo = t * TK;
        bool wrote = false;
        if (fuse && kr.head >= tile_lo && kr.head < tile_lo + TK) {
          // fused append: this pass's token goes to its ring slot, in the staged tile and in the cache
          const int row = kr.head - tile_lo;
          const int page = __shfl_sync(0xffffffffu, pid_cur, kr.head / P);
          const int slot = kr.head % P;
          const bool page_ok = page >= 0 && page < p.num_pages;
          if (!page_ok && lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, page);
          if (lane < 2 * CHUNKS) {
            const int kv = lane / CHUNKS, ch = lane % CHUNKS;
            *reinterpret_cast<uint4*>((kv == 0 ? sK : sV) + (ch >> 3) * HALF_BYTES + swz128(row, ch & 7)) = a_cur;
            if (page_ok)
              *reinterpret_cast<uint4*>(p.pool + ((((int64_t)page * 2 + kv) * M.Hkv + kh) * P + slot) * D + ch * 8) = a_cur;
          }
          wrote = true;
        }
        const uint32_t vm0 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + lane));
        const uint32_t vm1 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + 32 + lane));
        consume_tile<D, true>(sV, aK, aV, vm0, vm1, wrote, qf, M.scale_log2, m_run, l_run, o, lane, vm0, vm1);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars[NS + stage]));
      }
      (void)ok;
      (void)ctx;
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
      }
      // merge the three warps' states through the scratch area and write the ring's output
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        const int d0 = mt * 16 + (lane >> 2);
        sc_o[(cw * 8 + qd) * D + d0] = o[mt][0];
        sc_o[(cw * 8 + qd + 1) * D + d0] = o[mt][1];
        sc_o[(cw * 8 + qd) * D + d0 + 8] = o[mt][2];
        sc_o[(cw * 8 + qd + 1) * D + d0 + 8] = o[mt][3];
      }
      if (lane < 4) {
        sc_ml[(cw * 8 + qd) * 2 + 0] = m_run[0];
        sc_ml[(cw * 8 + qd) * 2 + 1] = l_run[0];
        sc_ml[(cw * 8 + qd + 1) * 2 + 0] = m_run[1];
        sc_ml[(cw * 8 + qd + 1) * 2 + 1] = l_run[1];
      }
      asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
      for (int idx = threadIdx.x - 32; idx < M.G * (D / 4); idx += NW * 32) {
        const int g = idx / (D / 4), d = (idx % (D / 4)) * 4;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) mm = fmaxf(mm, sc_ml[(w * 8 + g) * 2]);
        float L = 0.f;
        float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mm != -INFINITY) {
#pragma unroll
          for (int w = 0; w < NW; ++w) {
            const float f = fast_exp2(sc_ml[(w * 8 + g) * 2] - mm);
            const float4 x = *reinterpret_cast<const float4*>(&sc_o[(w * 8 + g) * D + d]);
            L += f * sc_ml[(w * 8 + g) * 2 + 1];
            O.x += f * x.x;
            O.y += f * x.y;
            O.z += f * x.z;
            O.w += f * x.w;
          }
        }
        const int64_t row = ((int64_t)r * nq + w_tok) * M.Hq + kh * M.G + g;
        const float inv = L > 0.f ? 1.f / L : 0.f;
        if (M.out_fp32)
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + row * D + d) = make_float4(O.x * inv, O.y * inv, O.z * inv, O.w * inv);
        else
          *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + row * D + d) =
              make_uint2(pack_bf16x2(O.x * inv, O.y * inv), pack_bf16x2(O.z * inv, O.w * inv));
        if (d == 0 && p.lse) p.lse[row] = L > 0.f ? (mm + log2f(L)) * 0.6931471805599453f : -INFINITY;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");  // scratch may be rewritten
    }
  }
}

template <int D, int P>
cudaError_t launch_ring_t(const hswa_handle* h, const CUtensorMap& tm, const DecodeParams& p, bool early_start, cudaStream_t s) {
  constexpr int STAGE_BYTES = 2 * (D / 64) * TK * 128;
  constexpr int SMEM = 3 * STAGE_BYTES + 3 * 8 * D * 4 + 3 * 8 * 2 * 4 + 1024;
  const bool tokens = p.nq > 1;
  auto kern = tokens ? decode_ring_kernel<D, P, true> : decode_ring_kernel<D, P, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  const int n_items = p.b.B * p.m.Hkv;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_items < 2 * h->num_sms ? n_items : 2 * h->num_sms, 1, 1);
  cfg.blockDim = dim3(tokens ? 160 : 128, 1, 1);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, tm, p, n_items);
}


// ---------------------------------------------------------------------------------------------------------
// Multi-token decode on Full layers (paper Sec. 6.2: the model drafts with 3 MTP layers, so a decode step
// carries the last accepted token plus up to 3 drafts per request).  The nq new tokens are already in the cache
// (the append runs first on the stream).  One consumer warp per draft token: every warp walks every staged tile
// with its own Q, its own causal mask and its own softmax state, so the KV bytes are streamed from HBM once for
// all nq tokens and no cross-warp merge is needed.  The layer takes 0.055 ms more per extra token on config 2
// whatever the split of the work (two tokens per warp sharing the K / V fragments: same time; two warps per
// token, 32 keys each: 5 % slower): that is the m16n8k16 work itself (64 MMAs per token and tile, N = 8), which
// only partly hides under the HBM stream.  On SWA layers a multi-token step runs through the ring kernel, one
// work item per ring and token.
struct KeyRangeMulti {
  int span, k_begin, ctx;
  // key idx of this split visible to draft token w (absolute position ctx + w)?
  __device__ __forceinline__ bool valid(int idx, int w) const { return idx < span && k_begin + idx <= ctx + w; }
  // visible to at least one of the nq tokens?
  __device__ __forceinline__ bool any(int idx) const { return idx < span; }
};

template <int D, int P, int NS>
__global__ void __launch_bounds__(160, 3)
decode_mtp_kernel(const __grid_constant__ CUtensorMap tm_pool, const DecodeParams p) {
  constexpr int HALVES = D / 64;
  constexpr int PPT = TK / P;
  constexpr int HALF_BYTES = TK * 128;
  constexpr int STAGE_BYTES = 2 * HALVES * HALF_BYTES;
  constexpr int BOX_BYTES = P * 128;
  constexpr int KS = D / 16;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * NS];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);

  const int r = blockIdx.x, split = blockIdx.y, kh = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const ModelParams& M = p.m;
  const int nq = p.nq;
  const int ctx = p.b.ctx_len[r];
  const int kv_len = ctx + nq;
  if (threadIdx.x == 0 && split == 0 && kh == 0 && ctx > p.max_ctx_len) record_error(p.err, HSWA_ERR_BOUNDS, r, -1, ctx);

  KeyRangeMulti kr;
  kr.ctx = ctx;
  kr.k_begin = split * p.split_len;
  if (kr.k_begin >= kv_len) return;
  kr.span = min(kv_len, kr.k_begin + p.split_len) - kr.k_begin;
  const int n_tiles = (kr.span + TK - 1) / TK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(smem_u32(&bars[i]), 1);        // full: producer's arrive + TMA bytes
      mbar_init(smem_u32(&bars[NS + i]), nq);  // empty: every consumer warp reads every tile
    }
    mbar_fence_init();
    tma_prefetch_desc(&tm_pool);
  }
  __syncthreads();

  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  float o[KS][4];
#pragma unroll
  for (int i = 0; i < KS; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  const int qd = (lane & 3) * 2;

  if (warp == 0) {
    const int32_t* tbl = p.b.block_table + (int64_t)r * p.b.max_blocks + kr.k_begin / P;
    const int n_pages = (kr.span + P - 1) / P;
    int pid_next = lane < n_pages ? tbl[lane] : 0;
    int pid_cur = 0;
    for (int t = 0; t < n_tiles; ++t) {
      const int pg0 = t * PPT;
      if ((pg0 & 31) == 0) {
        pid_cur = pid_next;
        const int nx = pg0 + 32 + lane;
        pid_next = nx < n_pages ? tbl[nx] : 0;
      }
      const int stage = t % NS;
      if (t >= NS && !mbar_wait(smem_u32(&bars[NS + stage]), ((t / NS) - 1) & 1)) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 5);
        break;
      }
      uint32_t need = 0;
      int pages[PPT];
#pragma unroll
      for (int i = 0; i < PPT; ++i) {
        const int pgi = pg0 + i;
        pages[i] = __shfl_sync(0xffffffffu, pid_cur, pgi & 31);
        bool v = false;
        if (pgi < n_pages)
          for (int s = lane; s < P; s += 32) v |= kr.any(pgi * P + s);
        if (__any_sync(0xffffffffu, v)) need |= 1u << i;
      }
      if (lane == 0) {
        uint32_t ok = 0;
#pragma unroll
        for (int i = 0; i < PPT; ++i) {
          if (!(need & (1u << i))) continue;
          if (pages[i] < 0 || pages[i] >= p.num_pages) {
            record_error(p.err, HSWA_ERR_BOUNDS, r, pg0 + i, pages[i]);
            continue;
          }
          ok |= 1u << i;
        }
        const uint32_t full_bar = smem_u32(&bars[stage]);
        if (ok == 0) {
          mbar_arrive(full_bar);
        } else {
          mbar_arrive_expect_tx(full_bar, __popc(ok) * 2 * HALVES * BOX_BYTES);
          const uint32_t sb = smem_base + stage * STAGE_BYTES;
#pragma unroll
          for (int i = 0; i < PPT; ++i) {
            if (!(ok & (1u << i))) continue;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv)
#pragma unroll
              for (int hf = 0; hf < HALVES; ++hf)
                tma_load_4d(sb + (kv * HALVES + hf) * HALF_BYTES + i * BOX_BYTES, &tm_pool, full_bar, hf * 64, 0,
                            kv * M.Hkv + kh, pages[i]);
          }
        }
      }
      __syncwarp();
    }
  } else if (warp <= nq) {
    const int w = warp - 1;  // draft token
    const int g_row = lane >> 2;
    uint32_t qf[KS][2];
    {
      const __nv_bfloat16* qrow = p.q + (((int64_t)r * nq + w) * M.Hq + kh * M.G + g_row) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qf[ks][0] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd) : 0u;
        qf[ks][1] = g_row < M.G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + qd + 8) : 0u;
      }
    }
    for (int t = 0; t < n_tiles; ++t) {
      const int stage = t % NS;
      if (!mbar_wait(smem_u32(&bars[stage]), (t / NS) & 1)) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, t, 6);
        break;
      }
      uint8_t* sV = smem + stage * STAGE_BYTES + HALVES * HALF_BYTES;
      const uint32_t aK = smem_base + stage * STAGE_BYTES;
      const uint32_t aV = aK + HALVES * HALF_BYTES;
      const int tile_lo = t * TK;
      const uint32_t vm0 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + lane, w));
      const uint32_t vm1 = __ballot_sync(0xffffffffu, kr.valid(tile_lo + 32 + lane, w));
      const uint32_t zm0 = __ballot_sync(0xffffffffu, kr.any(tile_lo + lane));
      const uint32_t zm1 = __ballot_sync(0xffffffffu, kr.any(tile_lo + 32 + lane));
      consume_tile<D>(sV, aK, aV, vm0, vm1, false, qf, M.scale_log2, m_run, l_run, o, lane, zm0, zm1);
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[NS + stage]));
    }
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
    }
  }
  __syncthreads();  // every tile has been consumed: the stage buffers now hold the per-token results
  float* sc_o = reinterpret_cast<float*>(smem);  // [nq][8][D]
  float* sc_ml = sc_o + 4 * 8 * D;               // [nq][8][2]
  if (warp >= 1 && warp <= nq) {
    const int w = warp - 1;
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
      const int d0 = mt * 16 + (lane >> 2);
      sc_o[(w * 8 + qd) * D + d0] = o[mt][0];
      sc_o[(w * 8 + qd + 1) * D + d0] = o[mt][1];
      sc_o[(w * 8 + qd) * D + d0 + 8] = o[mt][2];
      sc_o[(w * 8 + qd + 1) * D + d0 + 8] = o[mt][3];
    }
    if (lane < 4) {
      sc_ml[(w * 8 + qd) * 2 + 0] = m_run[0];
      sc_ml[(w * 8 + qd) * 2 + 1] = l_run[0];
      sc_ml[(w * 8 + qd + 1) * 2 + 0] = m_run[1];
      sc_ml[(w * 8 + qd + 1) * 2 + 1] = l_run[1];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nq * M.G * D; idx += blockDim.x) {
    const int w = idx / (M.G * D), g = (idx / D) % M.G, d = idx % D;
    const float mm = sc_ml[(w * 8 + g) * 2], L = sc_ml[(w * 8 + g) * 2 + 1], O = sc_o[(w * 8 + g) * D + d];
    const int64_t row = ((int64_t)r * nq + w) * M.Hq + kh * M.G + g;
    if (p.max_splits == 1) {
      const float val = L > 0.f ? O / L : 0.f;
      if (M.out_fp32)
        reinterpret_cast<float*>(p.out)[row * D + d] = val;
      else
        reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d] = __float2bfloat16_rn(val);
      if (d == 0 && p.lse) p.lse[row] = L > 0.f ? (mm + log2f(L)) * 0.6931471805599453f : -INFINITY;
    } else {
      p.part_o[(row * p.max_splits + split) * D + d] = O;
      if (d == 0) p.part_ml[row * p.max_splits + split] = make_float2(mm, L);
    }
  }
}

template <int D, int P, int NS>
cudaError_t launch_mtp_t(const CUtensorMap& tm, const DecodeParams& p, cudaStream_t s) {
  constexpr int STAGE_BYTES = 2 * (D / 64) * TK * 128;
  constexpr int SMEM = NS * STAGE_BYTES + 1024;
  static_assert(4 * 8 * D * 4 + 4 * 64 <= NS * STAGE_BYTES, "per-token results must fit the stage buffers");
  auto kern = decode_mtp_kernel<D, P, NS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  dim3 grid(p.b.B, p.grid_splits, p.m.Hkv);
  kern<<<grid, (p.nq + 1) * 32, SMEM, s>>>(tm, p);
  return cudaGetLastError();
}

template <int D, int P, int NS, int NW>
cudaError_t launch_decode_t(const CUtensorMap& tm, const DecodeParams& p, bool early_start, cudaStream_t s) {
  constexpr int STAGE_BYTES = 2 * (D / 64) * TK * 128;
  constexpr int SMEM = NS * STAGE_BYTES + 2 * NS * 8 + 16;  // stage buffers, barriers
  static_assert(NW * 8 * D * 4 + NW * 64 <= NS * STAGE_BYTES, "merge scratch must fit the stage buffers");
  auto kern = decode_kernel<D, P, NS, NW>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.b.B, p.grid_splits, p.m.Hkv);
  cfg.blockDim = dim3((NW + 1) * 32, 1, 1);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, tm, p);
}

}  // namespace

cudaError_t hswa_launch_decode(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p, bool early_start,
                               cudaStream_t s) {
  if (p.b.B == 0) return cudaSuccess;
  const int D = p.m.D, P = p.m.P;
  if (p.is_swa) {
    // persistent blocks streaming whole 64-slot ring tiles; a multi-token step needs the whole ring staged in the three
    // stage buffers at once, so longer rings take the compact-window kernel
    if (p.nq > 1 && (p.m.C + TK - 1) / TK > 3) return hswa_launch_decode_ring_compact(h, tm_pool, p, early_start, s);
    // single-token steps with more rings than the streaming kernel keeps resident (two blocks per SM): the compact
    // kernel holds three or four rings per SM and loses a round of the walk (17 vs 21 us per layer at batch 128, 10.9 vs
    // 12.5 at batch 64; on fewer rings the streaming kernel's shorter path per ring wins, 5.3 vs 5.6 us at batch 16)
    if (p.b.B * p.m.Hkv > 2 * h->num_sms && hswa_ring_window_supported(p.m, p.nq))
      return hswa_launch_decode_ring_window(h, p, early_start, s);
    if (D == 128 && P == 64) return launch_ring_t<128, 64>(h, tm_pool, p, early_start, s);
    if (D == 128 && P == 32) return launch_ring_t<128, 32>(h, tm_pool, p, early_start, s);
    if (D == 128 && P == 16) return launch_ring_t<128, 16>(h, tm_pool, p, early_start, s);
    if (D == 64 && P == 64) return launch_ring_t<64, 64>(h, tm_pool, p, early_start, s);
    if (D == 64 && P == 32) return launch_ring_t<64, 32>(h, tm_pool, p, early_start, s);
    if (D == 64 && P == 16) return launch_ring_t<64, 16>(h, tm_pool, p, early_start, s);
    return cudaErrorInvalidValue;
  }
  if (D == 128 && P == 64) return launch_decode_t<128, 64, 3, 3>(tm_pool, p, early_start, s);
  if (D == 128 && P == 32) return launch_decode_t<128, 32, 3, 3>(tm_pool, p, early_start, s);
  if (D == 128 && P == 16) return launch_decode_t<128, 16, 3, 3>(tm_pool, p, early_start, s);
  if (D == 64 && P == 64) return launch_decode_t<64, 64, 3, 3>(tm_pool, p, early_start, s);
  if (D == 64 && P == 32) return launch_decode_t<64, 32, 3, 3>(tm_pool, p, early_start, s);
  if (D == 64 && P == 16) return launch_decode_t<64, 16, 3, 3>(tm_pool, p, early_start, s);
  return cudaErrorInvalidValue;
}

cudaError_t hswa_launch_combine(const DecodeParams& p, cudaStream_t s) {
  const int rows = p.b.B * p.nq * p.m.Hq;
  if (rows == 0) return cudaSuccess;
  const int blocks = (rows * 32 + 127) / 128;
  // programmatic dependent launch: the blocks are resident (and wait) by the time the partials are complete
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks, 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return p.m.D == 128 ? cudaLaunchKernelEx(&cfg, combine_kernel<128>, p) : cudaLaunchKernelEx(&cfg, combine_kernel<64>, p);
}

cudaError_t hswa_launch_decode_mtp(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p, bool early_start,
                                   cudaStream_t s) {
  if (p.b.B == 0) return cudaSuccess;
  if (p.nq < 1 || p.nq > 4) return cudaErrorInvalidValue;
  if (p.is_swa) return hswa_launch_decode(h, tm_pool, p, early_start, s);  // rings: one work item per (ring, token)
  const int D = p.m.D, P = p.m.P;
  if (D == 128 && P == 64) return launch_mtp_t<128, 64, 2>(tm_pool, p, s);
  if (D == 128 && P == 32) return launch_mtp_t<128, 32, 2>(tm_pool, p, s);
  if (D == 128 && P == 16) return launch_mtp_t<128, 16, 2>(tm_pool, p, s);
  if (D == 64 && P == 64) return launch_mtp_t<64, 64, 4>(tm_pool, p, s);
  if (D == 64 && P == 32) return launch_mtp_t<64, 32, 4>(tm_pool, p, s);
  if (D == 64 && P == 16) return launch_mtp_t<64, 16, 4>(tm_pool, p, s);
  return cudaErrorInvalidValue;
}
