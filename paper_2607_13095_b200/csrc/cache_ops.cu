// Cache bookkeeping kernels: KV append into pages / ring slots (paper Sec. 3.1.1 dual pools; Sec. 3.1.3: an
// SWA pool stays at window magnitude), step advance of (ctx_len, ring_head), and the debug validator.
#include "hswa_internal.cuh"

namespace {
using namespace hswa_dev;

// Request owning new-token row t: largest r with q_indptr[r] <= t (q_indptr null: r = t).
__device__ __forceinline__ int find_request(const BatchParams& b, int t) {
  if (b.q_indptr == nullptr) return t;
  int lo = 0, hi = b.B;  // invariant: q_indptr[lo] <= t < q_indptr[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (b.q_indptr[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// Full layer: one warp moves the K (or V) rows of one token, all KV heads: Hkv * D * 2 bytes, up to four
// 16-byte chunks per lane in flight at once.
__global__ void __launch_bounds__(256) append_kernel(const AppendParams p) {
  const ModelParams& M = p.m;
  const int chunks_per_row = M.D / 8;
  const int chunks = M.Hkv * chunks_per_row;  // 16-byte chunks of one token's K (or V)
  const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (int64_t)p.total_q * 2) return;
  const int t = (int)(wid >> 1), kv = (int)(wid & 1);
  const int r = p.uniform_n > 0 ? t / p.uniform_n : find_request(p.b, t);
  const int t0 = p.uniform_n > 0 ? r * p.uniform_n : (p.b.q_indptr ? p.b.q_indptr[r] : r);
  const int pos = p.b.ctx_len[r] + (t - t0);
  const int blk = pos / M.P;
  if (pos < 0 || blk >= p.b.max_blocks) {  // the block table does not cover this position: skip the write
    if (lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, -3, blk);
    return;
  }
  const int page = p.b.block_table[(int64_t)r * p.b.max_blocks + blk];
  const int slot = pos % M.P;
  if (page < 0 || page >= p.num_pages) {
    if (lane == 0) record_error(p.err, HSWA_ERR_BOUNDS, r, blk, page);
    return;
  }
  const __nv_bfloat16* src = (kv == 0 ? p.k_new : p.v_new) + (int64_t)t * M.Hkv * M.D;
  __nv_bfloat16* dst = p.pool + (((int64_t)page * 2 + kv) * M.Hkv * M.P + slot) * M.D;  // head 0 of this (page, K|V)
  for (int c0 = lane; c0 < chunks; c0 += 128) {
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + 32 * u;
      if (c < chunks) v[u] = *reinterpret_cast<const uint4*>(src + c * 8);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + 32 * u;
      if (c < chunks) {
        const int kh = c / chunks_per_row, ch = c % chunks_per_row;
        *reinterpret_cast<uint4*>(dst + (int64_t)kh * M.P * M.D + ch * 8) = v[u];
      }
    }
  }
}

// SWA layer: only the last min(n, C) tokens of a request survive on its ring (later writes win), so the grid
// covers C tokens per request (blockIdx.y = request) instead of the whole chunk.
__global__ void __launch_bounds__(256) append_ring_kernel(const AppendParams p) {
  const ModelParams& M = p.m;
  const int chunks_per_row = M.D / 8;
  const int chunks_per_tok = 2 * M.Hkv * chunks_per_row;
  const int r = blockIdx.y;
  const int t0 = p.uniform_n > 0 ? r * p.uniform_n : (p.b.q_indptr ? p.b.q_indptr[r] : r);
  const int n = p.uniform_n > 0 ? p.uniform_n : (p.b.q_indptr ? p.b.q_indptr[r + 1] - t0 : 1);
  const int keep = min(n, M.C);
  const int gid = blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= keep * chunks_per_tok) return;
  const int i = n - keep + gid / chunks_per_tok;  // chunk-relative token
  int c = gid % chunks_per_tok;
  const int kv = c / (M.Hkv * chunks_per_row);
  c -= kv * M.Hkv * chunks_per_row;
  const int kh = c / chunks_per_row;
  const int ch = c % chunks_per_row;
  const int s = math_mod(p.b.ring_head[r] + (i % M.C), M.C);
  const int page = p.b.ring_table[(int64_t)r * M.R + s / M.P];
  const int slot = s % M.P;
  if (page < 0 || page >= p.num_pages) {
    record_error(p.err, HSWA_ERR_BOUNDS, r, s / M.P, page);
    return;
  }
  const __nv_bfloat16* src = (kv == 0 ? p.k_new : p.v_new) + ((int64_t)(t0 + i) * M.Hkv + kh) * M.D + ch * 8;
  __nv_bfloat16* dst = p.pool + ((((int64_t)page * 2 + kv) * M.Hkv + kh) * M.P + slot) * M.D + ch * 8;
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}

// Window-only data movement (paper Sec. 3.1.1 "cross-tier transfers move only valid window data", Sec. 3.1.2
// layerwise loadback, Sec. 3.1.3 ring seeding after a prefix hit): the W - 1 cached positions the next token's
// window needs, between a request's ring and a compact buffer [B][W-1][2][Hkv][D].  GATHER: ring -> buffer
// (positions below 0 become zeros); otherwise buffer -> ring (positions below 0 are skipped).  One thread per
// 16-byte chunk; blockIdx.y = request.  The buffer may be device memory or pinned host memory.
template <bool GATHER>
__global__ void __launch_bounds__(256) window_move_kernel(ModelParams M, BatchParams b, __nv_bfloat16* pool, int64_t num_pages,
                                                          __nv_bfloat16* buf, int32_t* err) {
  const int chunks_per_row = M.D / 8;
  const int chunks_per_tok = 2 * M.Hkv * chunks_per_row;
  const int Wm = M.W - 1;
  const int r = blockIdx.y;
  const int gid = blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= Wm * chunks_per_tok) return;
  const int j = gid / chunks_per_tok;
  int c = gid % chunks_per_tok;
  const int kv = c / (M.Hkv * chunks_per_row);
  c -= kv * M.Hkv * chunks_per_row;
  const int kh = c / chunks_per_row;
  const int ch = c % chunks_per_row;
  const int pos = b.ctx_len[r] - Wm + j;
  uint4* slot_in_buf = reinterpret_cast<uint4*>(buf + ((((int64_t)r * Wm + j) * 2 + kv) * M.Hkv + kh) * M.D + ch * 8);
  if (pos < 0) {
    if (GATHER) *slot_in_buf = make_uint4(0, 0, 0, 0);
    return;
  }
  const int s = math_mod(b.ring_head[r] - Wm + j, M.C);
  const int page = b.ring_table[(int64_t)r * M.R + s / M.P];
  if (page < 0 || page >= num_pages) {
    record_error(err, HSWA_ERR_BOUNDS, r, s / M.P, page);
    return;
  }
  uint4* in_pool = reinterpret_cast<uint4*>(pool + ((((int64_t)page * 2 + kv) * M.Hkv + kh) * M.P + s % M.P) * M.D + ch * 8);
  if (GATHER)
    *slot_in_buf = *in_pool;
  else
    *in_pool = *slot_in_buf;
}

__global__ void advance_kernel(ModelParams M, int B, int32_t* ctx_len, int32_t* ring_head, const int32_t* q_indptr) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= B) return;
  const int n = q_indptr ? q_indptr[r + 1] - q_indptr[r] : 1;
  ctx_len[r] += n;
  ring_head[r] = math_mod(ring_head[r] + (n % M.C), M.C);
}

// One block per request; threads scan the table entries the step would touch.
__global__ void __launch_bounds__(128) validate_kernel(ModelParams M, BatchParams b, int is_swa, int64_t num_pages,
                                                       int max_ctx_len, int max_q_len, int32_t* err) {
  const int r = blockIdx.x;
  const int ctx = b.ctx_len[r];
  const int n = b.q_indptr ? b.q_indptr[r + 1] - b.q_indptr[r] : 1;
  if (threadIdx.x == 0) {
    // the launch geometry of every kernel is planned from the host's bounds: a longer request would lose keys
    if (ctx < 0 || ctx > max_ctx_len) record_error(err, HSWA_ERR_BOUNDS, r, -1, ctx);
    if (n < 0 || n > max_q_len) record_error(err, HSWA_ERR_BOUNDS, r, -2, n);
  }
  if (ctx < 0 || n < 0) return;
  if (!is_swa) {
    const int64_t need = ((int64_t)ctx + n + M.P - 1) / M.P;
    if (need > b.max_blocks) {
      if (threadIdx.x == 0) record_error(err, HSWA_ERR_BOUNDS, r, -3, (int)need);
      return;
    }
    for (int i = threadIdx.x; i < need; i += blockDim.x) {
      const int pg = b.block_table[(int64_t)r * b.max_blocks + i];
      if (pg < 0 || pg >= num_pages) record_error(err, HSWA_ERR_BOUNDS, r, i, pg);
    }
  } else {
    if (threadIdx.x == 0) {
      const int hd = b.ring_head[r];
      if (hd < 0 || hd >= M.C) record_error(err, HSWA_ERR_BOUNDS, r, -4, hd);
    }
    for (int i = threadIdx.x; i < M.R; i += blockDim.x) {
      const int pg = b.ring_table[(int64_t)r * M.R + i];
      if (pg < 0 || pg >= num_pages) record_error(err, HSWA_ERR_BOUNDS, r, i, pg);
    }
  }
}

// Out-of-window SWA release bookkeeping (paper Sec. 3.1.3 item 2).  swa_valid_from[r] is the first cached position
// of request r whose SWA KV is still valid; the valid positions of a live request are the suffix
// [swa_valid_from, ctx).  The ring overwrites everything older than C positions; a release (chunk end, request end,
// every N decoded tokens: the caller's flags) drops everything the next token's window cannot reach.
__global__ void swa_release_kernel(ModelParams M, int B, const int32_t* ctx_len, const uint8_t* release, int32_t* valid_from) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= B) return;
  const int len = ctx_len[r];
  int from = valid_from[r];
  from = max(from, len - M.C);
  if (release == nullptr || release[r]) from = max(from, len - (M.W - 1));
  valid_from[r] = max(from, 0);
}

// Per-position SWA status: mask[r][p] = 1 iff swa_valid_from[r] <= p < ctx_len[r], 0 up to `stride`.  One thread
// per 16 positions; blockIdx.y = request.  `mask` may be device memory or pinned host memory.
__global__ void __launch_bounds__(256) swa_valid_mask_kernel(const int32_t* ctx_len, const int32_t* valid_from, int64_t stride,
                                                             uint8_t* mask) {
  const int r = blockIdx.y;
  const int64_t p0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
  if (p0 >= stride) return;
  const int64_t lo = valid_from[r], hi = ctx_len[r];
  uint8_t* row = mask + (int64_t)r * stride;
  if (p0 + 16 <= stride && ((reinterpret_cast<uintptr_t>(row + p0) & 15) == 0)) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t v = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int64_t p = p0 + j * 4 + b;
        v |= (uint32_t)(p >= lo && p < hi) << (8 * b);
      }
      w[j] = v;
    }
    *reinterpret_cast<uint4*>(row + p0) = make_uint4(w[0], w[1], w[2], w[3]);
  } else {
    for (int64_t p = p0; p < min(p0 + 16, stride); ++p) row[p] = (p >= lo && p < hi) ? 1 : 0;
  }
}

// Read-bandwidth probe: the memory side of the Full-layer decode kernel without its arithmetic.  Persistent blocks
// (two per SM, one warp each) stream their share of a buffer through a three-stage shared-memory ring with 32 KB bulk
// copies completing on mbarriers; nobody looks at the bytes.  What this reaches is the practical ceiling for a kernel
// that only reads HBM through TMA, which a copy-based peak (reads + writes) understates.
constexpr int PROBE_CHUNK = 32 * 1024, PROBE_STAGES = 3;
__global__ void __launch_bounds__(32) read_probe_kernel(const uint8_t* buf, long long chunks, int32_t* err) {
  extern __shared__ __align__(128) uint8_t probe_smem[];
  __shared__ __align__(8) uint64_t bars[PROBE_STAGES];
  if (threadIdx.x != 0) return;
  for (int i = 0; i < PROBE_STAGES; ++i) mbar_init(smem_u32(&bars[i]), 1);
  mbar_fence_init();
  long long k = 0;
  for (long long c = blockIdx.x; c < chunks; c += gridDim.x, ++k) {
    const int stage = (int)(k % PROBE_STAGES);
    const uint32_t bar = smem_u32(&bars[stage]);
    if (k >= PROBE_STAGES && !mbar_wait(bar, (uint32_t)((k / PROBE_STAGES - 1) & 1))) {  // the copy that used this stage
      record_error(err, HSWA_ERR_TIMEOUT, -1, stage, 11);
      return;
    }
    mbar_arrive_expect_tx(bar, PROBE_CHUNK);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(probe_smem + stage * PROBE_CHUNK)),
                 "l"(buf + c * PROBE_CHUNK), "r"(PROBE_CHUNK), "r"(bar)
                 : "memory");
  }
  // drain: no copy may be in flight when the block leaves
  for (long long j = k > PROBE_STAGES ? k - PROBE_STAGES : 0; j < k; ++j) {
    const int stage = (int)(j % PROBE_STAGES);
    if (!mbar_wait(smem_u32(&bars[stage]), (uint32_t)((j / PROBE_STAGES) & 1))) {
      record_error(err, HSWA_ERR_TIMEOUT, -1, stage, 12);
      return;
    }
  }
}

// Self-test of the bounded-wait path every pipeline kernel relies on: warp 1 waits, with the given limit, on an
// mbarrier that warp 0 (the would-be producer) never arms.  The wait runs out, the waiter records
// HSWA_ERR_TIMEOUT in the error word exactly as the pipeline kernels do, and the block returns normally:
// nothing spins past the limit and nothing is left in flight.
__global__ void __launch_bounds__(64) wait_selftest_kernel(long long limit_clocks, int32_t* err) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if ((threadIdx.x >> 5) == 1) {
    const bool ok = mbar_wait(smem_u32(&bar), 0, limit_clocks);
    if (!ok && (threadIdx.x & 31) == 0) record_error(err, HSWA_ERR_TIMEOUT, -1, 0, 7);
  }
}

}  // namespace

cudaError_t hswa_launch_append(const AppendParams& p, cudaStream_t s) {
  const int chunks_per_tok = 2 * p.m.Hkv * (p.m.D / 8);
  if (p.total_q == 0 || p.b.B == 0) return cudaSuccess;
  if (p.is_swa) {
    const int per_req = min(p.max_q_len, p.m.C) * chunks_per_tok;
    if (per_req == 0) return cudaSuccess;
    dim3 grid((per_req + 255) / 256, p.b.B);
    append_ring_kernel<<<grid, 256, 0, s>>>(p);
  } else {
    const int64_t warps = (int64_t)p.total_q * 2;
    append_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, s>>>(p);
  }
  return cudaGetLastError();
}

cudaError_t hswa_launch_advance(const ModelParams& m, int32_t B, int32_t* ctx_len, int32_t* ring_head,
                                const int32_t* q_indptr, cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  advance_kernel<<<(B + 127) / 128, 128, 0, s>>>(m, B, ctx_len, ring_head, q_indptr);
  return cudaGetLastError();
}

cudaError_t hswa_launch_validate(const ModelParams& m, const BatchParams& b, int32_t is_swa, int64_t num_pages,
                                 int32_t max_ctx_len, int32_t max_q_len, int32_t* err, cudaStream_t s) {
  if (b.B == 0) return cudaSuccess;
  validate_kernel<<<b.B, 128, 0, s>>>(m, b, is_swa, num_pages, max_ctx_len, max_q_len, err);
  return cudaGetLastError();
}

cudaError_t hswa_launch_swa_release(const ModelParams& m, int32_t B, const int32_t* ctx_len, const uint8_t* release,
                                    int32_t* valid_from, cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  swa_release_kernel<<<(B + 127) / 128, 128, 0, s>>>(m, B, ctx_len, release, valid_from);
  return cudaGetLastError();
}

cudaError_t hswa_launch_swa_valid_mask(int32_t B, const int32_t* ctx_len, const int32_t* valid_from, int64_t stride,
                                       uint8_t* mask, cudaStream_t s) {
  if (B == 0 || stride == 0) return cudaSuccess;
  const int64_t threads = (stride + 15) / 16;
  dim3 grid((unsigned)((threads + 255) / 256), B);
  swa_valid_mask_kernel<<<grid, 256, 0, s>>>(ctx_len, valid_from, stride, mask);
  return cudaGetLastError();
}

cudaError_t hswa_launch_read_probe(const void* buf, size_t bytes, int num_sms, int32_t* err, cudaStream_t s) {
  const long long chunks = (long long)(bytes / PROBE_CHUNK);
  if (chunks == 0) return cudaSuccess;
  const int smem = PROBE_STAGES * PROBE_CHUNK;
  cudaError_t e = cudaFuncSetAttribute(read_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  const long long want = 2LL * num_sms;
  read_probe_kernel<<<(unsigned)(chunks < want ? chunks : want), 32, smem, s>>>(static_cast<const uint8_t*>(buf), chunks, err);
  return cudaGetLastError();
}

cudaError_t hswa_launch_wait_selftest(int64_t limit_clocks, int32_t* err, cudaStream_t s) {
  wait_selftest_kernel<<<1, 64, 0, s>>>((long long)limit_clocks, err);
  return cudaGetLastError();
}

cudaError_t hswa_launch_window_move(const ModelParams& m, const BatchParams& b, __nv_bfloat16* pool, int64_t num_pages,
                                    __nv_bfloat16* buf, int gather, int32_t* err, cudaStream_t s) {
  const int per_req = (m.W - 1) * 2 * m.Hkv * (m.D / 8);
  if (b.B == 0 || per_req == 0) return cudaSuccess;
  dim3 grid((per_req + 255) / 256, b.B);
  if (gather)
    window_move_kernel<true><<<grid, 256, 0, s>>>(m, b, pool, num_pages, buf, err);
  else
    window_move_kernel<false><<<grid, 256, 0, s>>>(m, b, pool, num_pages, buf, err);
  return cudaGetLastError();
}
