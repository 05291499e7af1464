// Internal declarations shared by the library's translation units: handle, kernel parameter blocks and
// the sm_100a device primitives (mbarrier, TMA, ldmatrix, mma) the kernels are written with.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hswa.h"

typedef CUresult (*hswa_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                         const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                         CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                         CUtensorMapFloatOOBfill);

struct hswa_handle {
  hswa_config cfg;  // ring_pages and sm_scale resolved
  int32_t ring_slots;  // C
  int32_t group;       // G
  int32_t device;
  int32_t num_sms;
  int32_t* err;  // device int32[4]
  hswa_encode_tiled_fn encode_tiled;
  // Early-start bookkeeping: the last call through this handle was a fused decode on this stream and batch, so
  // the next fused decode may overlap its prologue and cache loads with that kernel's tail.
  void* chain_stream;
  const void* chain_ctx;
  const void* chain_pool;  // pool of the previous fused decode: a kernel must not start early on the pool its predecessor writes
  int32_t chain_ok;
  int32_t overlap_enabled;  // hswa_set_overlap
  int32_t prefill_order;    // hswa_set_prefill_order
  long long* trace;         // hswa_set_block_trace: device int64 [trace_cap][4] or null
  int64_t trace_cap;
};

// Model constants every kernel needs.
struct ModelParams {
  int32_t Hq, Hkv, G, D, P, W, R, C;
  float scale_log2;  // sm_scale * log2(e)
  int32_t out_fp32;
};

// The batch arrays as the kernels see them (device pointers).
struct BatchParams {
  int32_t B;
  const int32_t* ctx_len;
  const int32_t* q_indptr;
  const int32_t* block_table;
  int32_t max_blocks;
  const int32_t* ring_table;
  const int32_t* ring_head;
};

struct DecodeParams {
  ModelParams m;
  BatchParams b;
  __nv_bfloat16* pool;
  int64_t num_pages;
  int32_t is_swa;
  const __nv_bfloat16* q;      // [B][Hq][D]
  const __nv_bfloat16* k_new;  // [B][Hkv][D] or null
  const __nv_bfloat16* v_new;
  void* out;   // [B][Hq][D]
  float* lse;  // [B][Hq] or null
  int32_t split_len;   // keys per split (multiple of 64)
  int32_t max_splits;  // partial slots per row; 1 = write final output directly
  int32_t k_start;     // first key position this launch covers (cascade decode: the shared prefix length), else 0
  int32_t split_base;  // partial slot of this launch's split 0
  int32_t grid_splits; // splits this launch covers (grid extent)
  int32_t nq;          // new tokens per request (1; 2-4 for multi-token decode)
  int32_t max_ctx_len; // host-known bound of ctx_len the launch geometry was planned for
  int32_t late_dep_wait;  // cascade decode: the dependency wait moves to the end of the block (see decode_kernel)
  float* part_o;       // [B*Hq][max_splits][D]
  float2* part_ml;     // [B*Hq][max_splits] (m in log2 units, l)
  int32_t* err;
};

struct AppendParams {
  ModelParams m;
  BatchParams b;
  __nv_bfloat16* pool;
  int64_t num_pages;
  int32_t is_swa;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  int32_t total_q;
  int32_t max_q_len;  // host-known bound of new tokens per request
  int32_t uniform_n;  // > 0: every request has exactly this many new tokens and q_indptr is ignored
  int32_t* err;       // device error word: out-of-range block index or page id is recorded, the write skipped
};

struct PrefillParams {
  ModelParams m;
  BatchParams b;
  __nv_bfloat16* pool;
  int64_t num_pages;
  int32_t is_swa;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  void* out;
  float* lse;
  int32_t total_q;
  int32_t max_q_len;
  int32_t* err;
  int32_t order_mode;    // block order of the Full-layer tile kernel (hswa_set_prefill_order)
  long long* trace;      // per-block {start ns, end ns, SM id, request << 32 | tile} (hswa_set_block_trace) or null
  int64_t trace_cap;
  // shared-prefix stage of cascade decode only
  int32_t prefix_len;              // shared tokens (multiple of the page size)
  int32_t prefix_tiles_per_split;  // 128-key tiles per prefix slice
  int32_t max_splits;              // partial slots per (request, head) row
  float* part_o;
  float2* part_ml;
};

// Launchers implemented in the kernel translation units.
cudaError_t hswa_launch_append(const AppendParams& p, cudaStream_t s);
// Slots per TMA box of the persistent ring decode kernel (its tensor map is built with this box height).
#define HSWA_RING_GRANULE 16
cudaError_t hswa_launch_decode(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p, bool early_start,
                               cudaStream_t s);
cudaError_t hswa_launch_combine(const DecodeParams& p, cudaStream_t s);
// SWA layers whose window fits shared memory: one block per (request, KV head) over a compact copy of the window
bool hswa_ring_compact_supported(const ModelParams& m, int nq);
cudaError_t hswa_launch_decode_ring_compact(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p,
                                            bool early_start, cudaStream_t s);
// SWA layers, one new token, windows up to 128 keys: one autonomous warp per (request, KV head)
bool hswa_ring_window_supported(const ModelParams& m, int nq);
cudaError_t hswa_launch_decode_ring_window(const hswa_handle* h, const DecodeParams& p, bool early_start, cudaStream_t s);
cudaError_t hswa_launch_decode_mtp(const hswa_handle* h, const CUtensorMap& tm_pool, const DecodeParams& p,
                                   bool early_start, cudaStream_t s);
// Multi-token decode on Full layers on the tensor cores (group of 8, head_dim 128, page 64, 2-4 tokens per request)
bool hswa_decode_mtp_tc_supported(const ModelParams& m, int batch, int nq);
void hswa_decode_mtp_tc_scratch(const ModelParams& m, int batch, int num_sms, size_t* o_bytes, size_t* ml_bytes, size_t* info_bytes);
cudaError_t hswa_launch_decode_mtp_tc(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const DecodeParams& p, int num_sms,
                                      void* scratch, cudaStream_t s);
cudaError_t hswa_launch_prefill_mma(const PrefillParams& p, cudaStream_t s);
bool hswa_prefill_tc_supported(const ModelParams& m);
cudaError_t hswa_launch_prefill_tc(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                   const CUtensorMap& tm_v, const PrefillParams& p, int tile_limit, cudaStream_t s);
void hswa_prefill_packed_geometry(int G, int* tq, int* nkeys);
cudaError_t hswa_launch_decode_prefix(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const PrefillParams& p, int n_slices,
                                      cudaStream_t s);
cudaError_t hswa_launch_prefill_swa_stream(const CUtensorMap& tm_q, const CUtensorMap& tm_k16, const CUtensorMap& tm_v16,
                                           const CUtensorMap& tm_out, int tma_out, const PrefillParams& p, int num_sms,
                                           cudaStream_t s);
cudaError_t hswa_launch_prefill_swa_packed(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                           const PrefillParams& p, int first_tok, cudaStream_t s);
cudaError_t hswa_launch_advance(const ModelParams& m, int32_t B, int32_t* ctx_len, int32_t* ring_head,
                                const int32_t* q_indptr, cudaStream_t s);
cudaError_t hswa_launch_window_move(const ModelParams& m, const BatchParams& b, __nv_bfloat16* pool, int64_t num_pages,
                                    __nv_bfloat16* buf, int gather, int32_t* err, cudaStream_t s);
cudaError_t hswa_launch_validate(const ModelParams& m, const BatchParams& b, int32_t is_swa, int64_t num_pages,
                                 int32_t max_ctx_len, int32_t max_q_len, int32_t* err, cudaStream_t s);
cudaError_t hswa_launch_swa_release(const ModelParams& m, int32_t B, const int32_t* ctx_len, const uint8_t* release,
                                    int32_t* valid_from, cudaStream_t s);
cudaError_t hswa_launch_swa_valid_mask(int32_t B, const int32_t* ctx_len, const int32_t* valid_from, int64_t stride,
                                       uint8_t* mask, cudaStream_t s);
cudaError_t hswa_launch_read_probe(const void* buf, size_t bytes, int num_sms, int32_t* err, cudaStream_t s);
cudaError_t hswa_launch_wait_selftest(int64_t limit_clocks, int32_t* err, cudaStream_t s);

#ifdef __CUDACC__
namespace hswa_dev {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void record_error(int32_t* err, int code, int a, int b, int c) {
  if (atomicCAS(err, 0, code) == 0) {
    err[1] = a;
    err[2] = b;
    err[3] = c;
  }
}

// ---- mbarrier -----------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a phase.  try_wait above may suspend the thread for a hardware-chosen time when the phase
// has not completed, which is right for a thread with one thing to wait for; a thread that polls several barriers
// in turn (whichever is ready first) must use this one, or it sleeps on one barrier while another completes.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` SM clocks (default: about two seconds) and reports false.
constexpr long long kWaitLimitClocks = 4000000000LL;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit = kWaitLimitClocks) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- TMA (tiled tensor loads into shared memory, completion on an mbarrier) ---------------------------
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// ---- warp-level matrix primitives ---------------------------------------------------------------------
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t u) {
  __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&u);
  return __bfloat1622float2(v);
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a tile of 128-byte rows written by TMA
// with the 128-byte swizzle (the tile base is 1024-byte aligned).
__device__ __forceinline__ uint32_t swz128(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ int math_mod(int a, int m) {
  int r = a % m;
  return r < 0 ? r + m : r;
}

}  // namespace hswa_dev
#endif  // __CUDACC__
