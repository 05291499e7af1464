// Chunked prefill attention, general tile kernel on warp-level tensor-core MMA (paper Sec. 2.1: prefill is
// compute-bound and an SWA layer only attends inside its window; Sec. 3.1.1: Full layers read pages, SWA
// layers a ring).  It handles every supported shape and both layer kinds, and is the path for shapes the
// tcgen05 kernel does not cover.
//
// One thread block = 64 query rows of one (request, query head).  Key tiles of 64 absolute positions are
// gathered row by row with cp.async: a position below ctx comes from the cache as it is before this chunk's
// append (block table, or ring slot (ring_head + j - ctx) mod C), a position at or above ctx from the chunk's
// own K/V tensors.  Tiles wholly above the causal diagonal or wholly below the window are never loaded.
#include "hswa_internal.cuh"

namespace {
using namespace hswa_dev;

constexpr int BM = 64;
constexpr int BN = 64;

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool pred) {
  const int sz = pred ? 16 : 0;  // size 0 zero-fills the destination
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int D>
__global__ void __launch_bounds__(128, 2) prefill_mma_kernel(const PrefillParams p) {
  constexpr int HALVES = D / 64;
  constexpr int HALF_BYTES = BN * 128;
  constexpr int TILE_BYTES = HALVES * HALF_BYTES;  // one K or V or Q tile
  constexpr int CHUNKS = D / 8;
  constexpr int KS = D / 16;
  constexpr int NT_O = D / 8;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sKV = sQ + TILE_BYTES;  // [2 buffers][K, V][TILE_BYTES]

  const ModelParams& M = p.m;
  const int r = blockIdx.z, h = blockIdx.y;
  const int kh = h / M.G;
  const int t0 = p.b.q_indptr ? p.b.q_indptr[r] : r;
  const int n = p.b.q_indptr ? p.b.q_indptr[r + 1] - t0 : 1;
  const int q_tiles = (n + BM - 1) / BM;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;  // longest tiles first
  if (qt >= q_tiles) return;
  const int i0 = qt * BM;
  const int ctx = p.b.ctx_len[r];
  const int head = p.is_swa ? p.b.ring_head[r] : 0;
  const int rows = min(BM, n - i0);
  const int p_first = ctx + i0, p_last = ctx + i0 + rows - 1;
  const int j_lo = p.is_swa ? max(0, p_first - M.W + 1) : 0;
  const int tile_lo = j_lo / BN, tile_hi = p_last / BN;  // inclusive

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- Q tile -> shared (rows past the request's end are zero) ----
  for (int idx = tid; idx < BM * CHUNKS; idx += 128) {
    const int row = idx / CHUNKS, ch = idx % CHUNKS;
    const bool ok = row < rows;
    const __nv_bfloat16* src = p.q + ((int64_t)(t0 + i0 + (ok ? row : 0)) * M.Hq + h) * D + ch * 8;
    cp_async_16(sQ + (ch >> 3) * HALF_BYTES + swz128(row, ch & 7), src, ok);
  }
  cp_async_commit();

  auto load_kv = [&](int tile, int buf) {
    const int j0 = tile * BN;
    const uint32_t sK = sKV + buf * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
    for (int idx = tid; idx < BN * CHUNKS; idx += 128) {
      const int row = idx / CHUNKS, ch = idx % CHUNKS;
      const int j = j0 + row;
      const __nv_bfloat16 *ks = p.k_new, *vs = p.v_new;
      bool ok = j >= j_lo && j <= p_last;
      if (ok) {
        if (j < ctx) {
          int page, slot;
          if (!p.is_swa) {
            page = p.b.block_table[(int64_t)r * p.b.max_blocks + j / M.P];
            slot = j % M.P;
          } else {
            const int s = math_mod(head + (j - ctx), M.C);
            page = p.b.ring_table[(int64_t)r * M.R + s / M.P];
            slot = s % M.P;
          }
          if (page < 0 || page >= p.num_pages) {
            ok = false;
          } else {
            ks = p.pool + ((((int64_t)page * 2 + 0) * M.Hkv + kh) * M.P + slot) * D + ch * 8;
            vs = p.pool + ((((int64_t)page * 2 + 1) * M.Hkv + kh) * M.P + slot) * D + ch * 8;
          }
        } else {
          const int64_t off = ((int64_t)(t0 + j - ctx) * M.Hkv + kh) * D + ch * 8;
          ks = p.k_new + off;
          vs = p.v_new + off;
        }
      }
      const uint32_t o = (ch >> 3) * HALF_BYTES + swz128(row, ch & 7);
      cp_async_16(sK + o, ks, ok);
      cp_async_16(sV + o, vs, ok);
    }
    cp_async_commit();
  };

  load_kv(tile_lo, 0);

  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o[NT_O][4];
#pragma unroll
  for (int i = 0; i < NT_O; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  uint32_t qf[KS][4];
  const int mi = lane >> 3, mr = lane & 7;
  const int prow0 = p_first + warp * 16 + (lane >> 2);  // absolute position of this thread's first row

  for (int tile = tile_lo; tile <= tile_hi; ++tile) {
    const int buf = (tile - tile_lo) & 1;
    if (tile < tile_hi) {
      load_kv(tile + 1, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (tile == tile_lo) {
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int row = warp * 16 + (mi & 1) * 8 + mr;
        const int chunk = 2 * ks + (mi >> 1);
        ldmatrix_x4(sQ + (chunk >> 3) * HALF_BYTES + swz128(row, chunk & 7), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t sK = sKV + buf * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
    const int j0 = tile * BN;

    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      const int key = np * 16 + (mi >> 1) * 8 + mr;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int chunk = 2 * ks + (mi & 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(sK + (chunk >> 3) * HALF_BYTES + swz128(key, chunk & 7), b0, b1, b2, b3);
        mma_bf16_16816(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
        mma_bf16_16816(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
      }
    }
    // scale and mask
    const bool need_mask = (j0 + BN - 1 > p_first) || (p.is_swa && j0 < p_last - M.W + 1);
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[nt][e] * M.scale_log2;
        if (need_mask) {
          const int j = j0 + nt * 8 + (lane & 3) * 2 + (e & 1);
          const int pr = prow0 + (e >> 1) * 8;
          const bool ok = j <= pr && (!p.is_swa || j > pr - M.W);
          v = ok ? v : -INFINITY;
        }
        s[nt][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float m_use[2], alpha[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 1));
      mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 2));
      const float m_new = fmaxf(m_run[j], mx[j]);
      m_use[j] = m_new == -INFINITY ? 0.f : m_new;
      alpha[j] = fast_exp2(m_run[j] - m_use[j]);
      m_run[j] = m_new;
      l_run[j] *= alpha[j];
    }
#pragma unroll
    for (int i = 0; i < NT_O; ++i) {
      o[i][0] *= alpha[0];
      o[i][1] *= alpha[0];
      o[i][2] *= alpha[1];
      o[i][3] *= alpha[1];
    }
    uint32_t pa[4][4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int nt = 2 * kk + half;
        const uint32_t lo = pack_bf16x2(fast_exp2(s[nt][0] - m_use[0]), fast_exp2(s[nt][1] - m_use[0]));
        const uint32_t hi = pack_bf16x2(fast_exp2(s[nt][2] - m_use[1]), fast_exp2(s[nt][3] - m_use[1]));
        const float2 f0 = unpack_bf16x2(lo), f1 = unpack_bf16x2(hi);
        l_run[0] += f0.x + f0.y;
        l_run[1] += f1.x + f1.y;
        pa[kk][half * 2 + 0] = lo;
        pa[kk][half * 2 + 1] = hi;
      }
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const int key = kk * 16 + (mi & 1) * 8 + mr;
#pragma unroll
      for (int dp = 0; dp < D / 16; ++dp) {
        const int chunk = 2 * dp + (mi >> 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(sV + (chunk >> 3) * HALF_BYTES + swz128(key, chunk & 7), b0, b1, b2, b3);
        mma_bf16_16816(o[2 * dp], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], b0, b1);
        mma_bf16_16816(o[2 * dp + 1], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], b2, b3);
      }
    }
    __syncthreads();
  }

  // ---- epilogue ----
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 1);
    l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 2);
  }
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int row = warp * 16 + (lane >> 2) + half * 8;
    if (row >= rows) continue;
    const float L = l_run[half];
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const int64_t orow = ((int64_t)(t0 + i0 + row) * M.Hq + h);
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt) {
      const int d = nt * 8 + (lane & 3) * 2;
      const float x = o[nt][half * 2] * inv, y = o[nt][half * 2 + 1] * inv;
      if (M.out_fp32)
        *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.out) + orow * D + d) = make_float2(x, y);
      else
        *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow * D + d) =
            __floats2bfloat162_rn(x, y);
    }
    if ((lane & 3) == 0 && p.lse)
      p.lse[orow] = L > 0.f ? (m_run[half] + log2f(L)) * 0.6931471805599453f : -INFINITY;
  }
}

template <int D>
cudaError_t launch_t(const PrefillParams& p, cudaStream_t s) {
  constexpr int SMEM = 5 * (D / 64) * BN * 128 + 1024;
  auto kern = prefill_mma_kernel<D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  dim3 grid((p.max_q_len + BM - 1) / BM, p.m.Hq, p.b.B);
  kern<<<grid, 128, SMEM, s>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t hswa_launch_prefill_mma(const PrefillParams& p, cudaStream_t s) {
  if (p.b.B == 0 || p.total_q == 0 || p.max_q_len == 0) return cudaSuccess;
  if (p.m.D == 128) return launch_t<128>(p, s);
  if (p.m.D == 64) return launch_t<64>(p, s);
  return cudaErrorInvalidValue;
}
