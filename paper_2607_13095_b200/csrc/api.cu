// Host side of the C ABI: argument validation, launch planning, TMA descriptor construction, dispatch.
#include <cmath>
#include <cstring>
#include <new>

#include "hswa_internal.cuh"

namespace {

constexpr int kMinSplitLen = 256;
constexpr int kMaxSplitLen = 4096;  // measured on configs 2, 4 and 5: 4096-8192 beat 2048 (fewer block prologues) and 16384 (tail)

ModelParams model_params(const hswa_handle* h) {
  ModelParams m;
  m.Hq = h->cfg.num_q_heads;
  m.Hkv = h->cfg.num_kv_heads;
  m.G = h->group;
  m.D = h->cfg.head_dim;
  m.P = h->cfg.page_size;
  m.W = h->cfg.window;
  m.R = h->cfg.ring_pages;
  m.C = h->ring_slots;
  m.scale_log2 = h->cfg.sm_scale * 1.4426950408889634f;
  m.out_fp32 = h->cfg.out_dtype;
  return m;
}

BatchParams batch_params(const hswa_batch* b) {
  BatchParams o;
  o.B = b->batch;
  o.ctx_len = b->ctx_len;
  o.q_indptr = b->q_indptr;
  o.block_table = b->block_table;
  o.max_blocks = b->max_blocks;
  o.ring_table = b->ring_table;
  o.ring_head = b->ring_head;
  return o;
}

// Checks every host-visible field of a (layer, batch) pair.
hswa_status check_common(const hswa_handle* h, const hswa_layer* layer, const hswa_batch* b) {
  if (!h || !layer || !b) return HSWA_ERR_INVALID_ARG;
  if (b->batch < 0 || b->total_q < 0 || b->max_q_len < 0 || b->max_ctx_len < 0) return HSWA_ERR_INVALID_ARG;
  if (b->batch == 0) return HSWA_OK;
  if (!layer->pool || layer->num_pages <= 0) return HSWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(layer->pool) & 255) != 0) return HSWA_ERR_INVALID_ARG;
  if (layer->num_pages > (int64_t)INT32_MAX) return HSWA_ERR_UNSUPPORTED;
  if (!b->ctx_len) return HSWA_ERR_INVALID_ARG;
  if (layer->is_swa) {
    if (!b->ring_table || !b->ring_head) return HSWA_ERR_INVALID_ARG;
  } else {
    if (!b->block_table || b->max_blocks <= 0) return HSWA_ERR_INVALID_ARG;
  }
  if (b->q_indptr == nullptr && (b->total_q != b->batch || b->max_q_len != 1)) return HSWA_ERR_INVALID_ARG;
  if (b->max_q_len > b->total_q) return HSWA_ERR_INVALID_ARG;
  return HSWA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Keys per split for Full-layer decode: long enough that the partial (m, l, o) traffic stays below one
// percent of the KV bytes, short enough that the grid fills the machine.
int plan_split_len(const hswa_handle* h, int batch, int max_ctx_len) {
  const long long kv_len = (long long)max_ctx_len + 1;
  int len = kMaxSplitLen;
  const long long want = 4LL * h->num_sms;
  while (len > kMinSplitLen && (long long)batch * h->cfg.num_kv_heads * ((kv_len + len - 1) / len) < want) len >>= 1;
  return len;
}

int plan_max_splits(int split_len, int max_ctx_len) {
  const long long kv_len = (long long)max_ctx_len + 1;
  return (int)((kv_len + split_len - 1) / split_len);
}

// Everything the host decides about one decode call from host-known values only (so that results do not depend
// on where pages sit): whether the shared-prefix stage runs and in how many slices, the split length of the
// streaming kernel, the partial slots per (request, token, head) row and the scratch bytes they take.
struct DecodePlan {
  bool cascade;
  int prefix_slices, prefix_tps;  // shared-prefix stage: slices and 128-key tiles per slice
  int k_start, split_base;        // first key and first partial slot of the streaming kernel
  int split_len, grid_splits, max_splits;
  size_t o_bytes, ml_bytes;       // scratch: o partials, then (m, l) pairs; 0 when rows are written directly
  bool tc;                        // multi-token decode on the tensor cores: run partials and one int2 per stream
  size_t info_bytes;
};

bool plan_decode(const hswa_handle* h, int is_swa, int batch, int max_ctx_len, int shared_prefix_len, int q_len,
                 DecodePlan* pl) {
  DecodePlan d = {};
  d.cascade = !is_swa && q_len == 1 && shared_prefix_len >= 128 && h->cfg.head_dim == 128 && h->cfg.page_size == 64 &&
              h->group == 8;
  d.tc = !is_swa && q_len >= 2 && hswa_decode_mtp_tc_supported(model_params(h), batch, q_len);
  if (is_swa) {
    d.split_len = ((h->ring_slots + 63) / 64) * 64;
    d.grid_splits = d.max_splits = 1;
  } else if (d.tc) {
    d.split_len = 128;
    d.grid_splits = 1;
    d.max_splits = 2;
    hswa_decode_mtp_tc_scratch(model_params(h), batch, h->num_sms, &d.o_bytes, &d.ml_bytes, &d.info_bytes);
  } else {
    if (d.cascade) {
      const int tiles = (shared_prefix_len + 127) / 128;
      const int base = ((batch + 31) / 32) * h->cfg.num_kv_heads;
      // Slices of the prefix: a whole wave of blocks.  (Measured on the prefix-hit workload, Full layer: giving the
      // stage 25 / 45 / 70 % of the SMs so that the suffix stream runs beside it on the others: 0.403 / 0.306 / 0.286 ms
      // against 0.280 ms for the whole wave -- the stage is tensor-bound and slows down next to the stream.)
      int want = h->num_sms / base;
      want = want < 1 ? 1 : (want > tiles ? tiles : want);
      d.prefix_tps = (tiles + want - 1) / want;
      d.prefix_slices = (tiles + d.prefix_tps - 1) / d.prefix_tps;  // no slice is empty
      d.k_start = shared_prefix_len;
      d.split_base = d.prefix_slices;
    }
    const int last = max_ctx_len + q_len - 1 - d.k_start;  // highest key position the streaming kernel covers, relative
    d.split_len = plan_split_len(h, batch, last);
    d.grid_splits = plan_max_splits(d.split_len, last);
    d.max_splits = d.split_base + d.grid_splits;
    if (d.grid_splits > 65535) return false;
    if (d.max_splits > 1) {
      const size_t rows = (size_t)batch * q_len * h->cfg.num_q_heads;
      d.o_bytes = (rows * d.max_splits * h->cfg.head_dim * sizeof(float) + 255) & ~size_t(255);
      d.ml_bytes = (rows * d.max_splits * sizeof(float2) + 255) & ~size_t(255);
    }
  }
  *pl = d;
  return true;
}

// 4-D view of a pool for TMA: {D, P, 2 * Hkv, num_pages}, box {64, box_slots, 1, 1} (0: a whole page),
// 128-byte swizzle.
hswa_status make_pool_map(const hswa_handle* h, const hswa_layer* layer, CUtensorMap* tm, int box_slots = 0) {
  const hswa_config& c = h->cfg;
  cuuint64_t dims[4] = {(cuuint64_t)c.head_dim, (cuuint64_t)c.page_size, (cuuint64_t)(2 * c.num_kv_heads),
                        (cuuint64_t)layer->num_pages};
  cuuint64_t strides[3] = {(cuuint64_t)c.head_dim * 2, (cuuint64_t)c.head_dim * 2 * c.page_size,
                           (cuuint64_t)c.head_dim * 2 * c.page_size * 2 * c.num_kv_heads};
  cuuint32_t box[4] = {64, (cuuint32_t)(box_slots > 0 ? box_slots : c.page_size), 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = h->encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, layer->pool, dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? HSWA_OK : HSWA_ERR_CUDA;
}

// 3-D view of a [T][heads][D] activation tensor for TMA: box {64, 1, box_rows}, 128-byte swizzle.
hswa_status make_rows_map(const hswa_handle* h, const void* ptr, int heads, int64_t rows, int box_rows, CUtensorMap* tm,
                          int box_heads = 1) {
  const cuuint64_t D = (cuuint64_t)h->cfg.head_dim;
  cuuint64_t dims[3] = {D, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {D * 2, D * 2 * (cuuint64_t)heads};
  cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult rc = h->encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? HSWA_OK : HSWA_ERR_CUDA;
}

}  // namespace

extern "C" {

const char* hswa_status_string(hswa_status s) {
  switch (s) {
    case HSWA_OK: return "ok";
    case HSWA_ERR_INVALID_ARG: return "invalid argument";
    case HSWA_ERR_UNSUPPORTED: return "unsupported shape";
    case HSWA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case HSWA_ERR_CUDA: return "CUDA call failed";
    case HSWA_ERR_BOUNDS: return "device-side bounds violation";
    case HSWA_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
  }
  return "unknown status";
}

hswa_status hswa_create(const hswa_config* cfg, hswa_handle** out) {
  if (!cfg || !out) return HSWA_ERR_INVALID_ARG;
  *out = nullptr;
  hswa_config c = *cfg;
  if (c.num_q_heads <= 0 || c.num_kv_heads <= 0 || c.num_q_heads % c.num_kv_heads != 0) return HSWA_ERR_INVALID_ARG;
  if (c.window <= 0 || c.page_size <= 0 || c.ring_pages < 0) return HSWA_ERR_INVALID_ARG;
  if (c.out_dtype != 0 && c.out_dtype != 1) return HSWA_ERR_INVALID_ARG;
  if (!(c.sm_scale >= 0.f) || std::isinf(c.sm_scale)) return HSWA_ERR_INVALID_ARG;
  if (c.head_dim != 64 && c.head_dim != 128) return HSWA_ERR_UNSUPPORTED;
  if (c.page_size != 16 && c.page_size != 32 && c.page_size != 64) return HSWA_ERR_UNSUPPORTED;
  const int group = c.num_q_heads / c.num_kv_heads;
  if (group > 8) return HSWA_ERR_UNSUPPORTED;
  if (c.ring_pages == 0) c.ring_pages = (c.window + c.page_size - 1) / c.page_size + 1;
  if ((int64_t)c.ring_pages * c.page_size < (int64_t)c.window + 1) return HSWA_ERR_INVALID_ARG;
  if ((int64_t)c.ring_pages * c.page_size > (1 << 20)) return HSWA_ERR_UNSUPPORTED;
  if (c.sm_scale == 0.f) c.sm_scale = 1.0f / std::sqrt((float)c.head_dim);

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HSWA_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return HSWA_ERR_CUDA;
  if (prop.major != 10) return HSWA_ERR_CUDA;  // kernels are built for sm_100a only

  hswa_handle* h = new (std::nothrow) hswa_handle();
  if (!h) return HSWA_ERR_INVALID_ARG;
  h->cfg = c;
  h->ring_slots = c.ring_pages * c.page_size;
  h->group = group;
  h->device = dev;
  h->num_sms = prop.multiProcessorCount;
  h->err = nullptr;
  h->encode_tiled = nullptr;
  h->chain_stream = nullptr;
  h->chain_ctx = nullptr;
  h->chain_pool = nullptr;
  h->chain_ok = 0;
  h->overlap_enabled = 1;
  h->prefill_order = 2;
  h->trace = nullptr;
  h->trace_cap = 0;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete h;
    return HSWA_ERR_CUDA;
  }
  h->encode_tiled = reinterpret_cast<hswa_encode_tiled_fn>(fn);
  if (cudaMalloc(&h->err, 4 * sizeof(int32_t)) != cudaSuccess || cudaMemset(h->err, 0, 4 * sizeof(int32_t)) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    if (h->err) cudaFree(h->err);
    delete h;
    return HSWA_ERR_CUDA;
  }
  *out = h;
  return HSWA_OK;
}

void hswa_destroy(hswa_handle* h) {
  if (!h) return;
  cudaDeviceSynchronize();
  if (h->err) cudaFree(h->err);
  delete h;
}

size_t hswa_workspace_bytes(const hswa_handle* h, int32_t max_batch, int32_t max_total_q, int32_t max_ctx_len) {
  if (!h || max_batch <= 0 || max_ctx_len < 0) return 0;
  // multi-token decode has max_total_q = batch x q_len rows; prefill needs no scratch
  if (max_total_q > max_batch && max_total_q <= 4 * max_batch) max_batch = max_total_q;
  // Upper bound of rows * splits over every batch <= max_batch and context <= max_ctx_len under
  // plan_split_len: at the longest split length a row has ceil(kv / 4096) splits; a shorter length is only
  // chosen while batch * Hkv * splits stays below twice the fill target.
  const size_t kv = (size_t)max_ctx_len + 1;
  const size_t long_splits = (kv + kMaxSplitLen - 1) / kMaxSplitLen + 2;
  const size_t want = 4 * (size_t)h->num_sms;
  // (+ the shared-prefix slices of cascade decode: at most num_sms / (groups of 32 requests x Hkv) per row)
  const size_t row_splits = (size_t)h->cfg.num_q_heads * max_batch * long_splits + 2 * want * h->group +
                            (size_t)32 * h->group * h->num_sms;
  const size_t o_bytes = row_splits * h->cfg.head_dim * sizeof(float);
  const size_t ml_bytes = row_splits * sizeof(float2);
  size_t need = ((o_bytes + 255) & ~size_t(255)) + ((ml_bytes + 255) & ~size_t(255));
  // the tensor-core multi-token path keeps partials per run (streams + blocks of them), not per row and split
  size_t tc_o, tc_ml, tc_info;
  hswa_decode_mtp_tc_scratch(model_params(h), max_batch, h->num_sms, &tc_o, &tc_ml, &tc_info);
  if (need < tc_o + tc_ml + tc_info) need = tc_o + tc_ml + tc_info;
  return need;
}

size_t hswa_decode_workspace_need(const hswa_handle* h, int32_t is_swa, int32_t batch, int32_t max_ctx_len,
                                  int32_t shared_prefix_len, int32_t q_len) {
  if (!h || batch <= 0 || max_ctx_len < 0 || shared_prefix_len < 0 || shared_prefix_len > max_ctx_len || q_len < 1 || q_len > 4)
    return 0;
  DecodePlan pl;
  if (!plan_decode(h, is_swa, batch, max_ctx_len, shared_prefix_len, q_len, &pl)) return 0;
  return pl.o_bytes + pl.ml_bytes + pl.info_bytes;
}

hswa_status hswa_set_overlap(hswa_handle* h, int32_t enabled) {
  if (!h) return HSWA_ERR_INVALID_ARG;
  h->overlap_enabled = enabled != 0;
  h->chain_ok = 0;
  return HSWA_OK;
}

hswa_status hswa_set_prefill_order(hswa_handle* h, int32_t mode) {
  if (!h || mode < 0 || mode > 3) return HSWA_ERR_INVALID_ARG;
  h->prefill_order = mode;
  return HSWA_OK;
}

hswa_status hswa_set_block_trace(hswa_handle* h, int64_t* buf, int64_t capacity_blocks) {
  if (!h || capacity_blocks < 0 || (buf == nullptr) != (capacity_blocks == 0)) return HSWA_ERR_INVALID_ARG;
  h->trace = reinterpret_cast<long long*>(buf);
  h->trace_cap = capacity_blocks;
  return HSWA_OK;
}

hswa_status hswa_probe_read_stream(hswa_handle* h, const void* buf, size_t bytes, void* stream) {
  if (!h || !buf || (reinterpret_cast<uintptr_t>(buf) & 127) != 0 || bytes % (32 * 1024) != 0) return HSWA_ERR_INVALID_ARG;
  h->chain_ok = 0;
  return hswa_launch_read_probe(buf, bytes, h->num_sms, h->err, (cudaStream_t)stream) == cudaSuccess ? HSWA_OK : HSWA_ERR_CUDA;
}

hswa_status hswa_selftest_wait_timeout(hswa_handle* h, int64_t limit_clocks, void* stream) {
  if (!h || limit_clocks < 1 || limit_clocks > 2000000000LL) return HSWA_ERR_INVALID_ARG;
  h->chain_ok = 0;
  if (cudaSetDevice(h->device) != cudaSuccess) return HSWA_ERR_CUDA;
  return hswa_launch_wait_selftest(limit_clocks, h->err, (cudaStream_t)stream) == cudaSuccess ? HSWA_OK : HSWA_ERR_CUDA;
}

hswa_status hswa_validate_batch(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, void* stream) {
  if (h) h->chain_ok = 0;
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  if (cudaSetDevice(h->device) != cudaSuccess) return HSWA_ERR_CUDA;
  cudaError_t e = hswa_launch_validate(model_params(h), batch_params(b), layer->is_swa, layer->num_pages, b->max_ctx_len,
                                       b->max_q_len, h->err, (cudaStream_t)stream);
  return e == cudaSuccess ? HSWA_OK : HSWA_ERR_CUDA;
}

hswa_status hswa_kv_append(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, const void* k_new,
                           const void* v_new, void* stream) {
  if (h) h->chain_ok = 0;
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  if (b->batch == 0 || b->total_q == 0) return HSWA_OK;
  if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return HSWA_ERR_INVALID_ARG;
  AppendParams p;
  p.m = model_params(h);
  p.b = batch_params(b);
  p.pool = static_cast<__nv_bfloat16*>(layer->pool);
  p.num_pages = layer->num_pages;
  p.is_swa = layer->is_swa;
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.total_q = b->total_q;
  p.max_q_len = b->max_q_len;
  p.uniform_n = 0;
  p.err = h->err;
  return hswa_launch_append(p, (cudaStream_t)stream) == cudaSuccess ? HSWA_OK : HSWA_ERR_CUDA;
}

static hswa_status decode_impl(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, int32_t shared_prefix_len,
                               const void* q, const void* k_new, const void* v_new, void* out, float* lse, void* workspace,
                               size_t workspace_bytes, void* stream) {
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  if (b->q_indptr != nullptr) return HSWA_ERR_INVALID_ARG;
  if (b->batch == 0) return HSWA_OK;
  if (!q || !out || !aligned16(q) || !aligned16(out)) return HSWA_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return HSWA_ERR_INVALID_ARG;
  if (k_new && (!aligned16(k_new) || !aligned16(v_new))) return HSWA_ERR_INVALID_ARG;
  // the block table must cover every position the host bound allows (position max_ctx_len is the new token's)
  if (!layer->is_swa && (int64_t)b->max_ctx_len + 1 > (int64_t)b->max_blocks * h->cfg.page_size) return HSWA_ERR_INVALID_ARG;

  DecodeParams p;
  p.m = model_params(h);
  p.b = batch_params(b);
  p.pool = static_cast<__nv_bfloat16*>(layer->pool);
  p.num_pages = layer->num_pages;
  p.is_swa = layer->is_swa;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.out = out;
  p.lse = lse;
  p.err = h->err;
  p.part_o = nullptr;
  p.part_ml = nullptr;
  p.k_start = 0;
  p.split_base = 0;
  p.nq = 1;
  p.max_ctx_len = b->max_ctx_len;
  p.late_dep_wait = 0;
  // Cascade decode: the shared prefix is attended once per group of requests on the tensor cores, the
  // per-request suffixes by the streaming kernel; both leave partials for the combine.
  DecodePlan pl;
  if (!plan_decode(h, layer->is_swa, b->batch, b->max_ctx_len, shared_prefix_len, 1, &pl)) return HSWA_ERR_UNSUPPORTED;
  const bool cascade = pl.cascade;
  const int prefix_slices = pl.prefix_slices, prefix_tps = pl.prefix_tps;
  p.k_start = pl.k_start;
  p.split_base = pl.split_base;
  p.split_len = pl.split_len;
  p.grid_splits = pl.grid_splits;
  p.max_splits = pl.max_splits;
  if (p.max_splits > 1) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 || workspace_bytes < pl.o_bytes + pl.ml_bytes)
      return HSWA_ERR_WORKSPACE;
    p.part_o = static_cast<float*>(workspace);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(workspace) + pl.o_bytes);
  }
  CUtensorMap tm;
  // SWA layers: the ring kernel loads 16-slot granules, only those that meet the window
  st = make_pool_map(h, layer, &tm, layer->is_swa ? (h->cfg.page_size < HSWA_RING_GRANULE ? h->cfg.page_size : HSWA_RING_GRANULE) : 0);
  if (st != HSWA_OK) return st;
  // A fused decode that directly follows another fused decode of the same step (same handle, stream and batch
  // arrays) may start early: those kernels never write the batch arrays or another layer's pool.
  // The previous kernel appends to its own layer's pool, so a call on that same pool waits for it to finish.
  const bool early = h->overlap_enabled && h->chain_ok && k_new != nullptr && h->chain_stream == stream && h->chain_ctx == (const void*)b->ctx_len &&
                     h->chain_pool != (const void*)layer->pool;
  h->chain_ok = 0;
  if (cascade) {
    PrefillParams pp = {};
    pp.m = p.m;
    pp.b = p.b;
    pp.pool = p.pool;
    pp.num_pages = p.num_pages;
    pp.is_swa = 0;
    pp.q = p.q;
    pp.err = h->err;
    pp.prefix_len = shared_prefix_len;
    pp.prefix_tiles_per_split = prefix_tps;
    pp.max_splits = p.max_splits;
    pp.part_o = p.part_o;
    pp.part_ml = p.part_ml;
    CUtensorMap tq;
    if ((st = make_rows_map(h, q, h->cfg.num_q_heads, b->batch, 16, &tq, 8)) != HSWA_OK) return st;
    if (hswa_launch_decode_prefix(tm, tq, pp, prefix_slices, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  }
  // Behind the shared-prefix stage the suffix kernel always starts early, and it does not wait for that stage before
  // it computes: the stage was launched in plain stream order (everything older is complete), reads only q and the
  // shared pages and writes only its own partial slots.  The suffix blocks wait for it just before they exit, so
  // that the combine, which waits for the suffix kernel, finds both sets of partials complete.
  p.late_dep_wait = cascade ? 1 : 0;
  if (hswa_launch_decode(h, tm, p, early || cascade, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  if (p.max_splits > 1 && hswa_launch_combine(p, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  if (k_new != nullptr) {
    h->chain_ok = 1;
    h->chain_stream = stream;
    h->chain_ctx = (const void*)b->ctx_len;
    h->chain_pool = (const void*)layer->pool;
  }
  return HSWA_OK;
}

hswa_status hswa_decode_attn(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, const void* q,
                             const void* k_new, const void* v_new, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream) {
  return decode_impl(h, layer, b, 0, q, k_new, v_new, out, lse, workspace, workspace_bytes, stream);
}

hswa_status hswa_decode_attn_mtp(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, int32_t q_len, const void* q,
                                 const void* k_new, const void* v_new, void* out, float* lse, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  if (q_len == 1) return decode_impl(h, layer, b, 0, q, k_new, v_new, out, lse, workspace, workspace_bytes, stream);
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  // a ring kernel with the append fused may start early behind another fused decode kernel of the same step
  const bool early = h->overlap_enabled && layer->is_swa && h->chain_ok && h->chain_stream == stream && h->chain_ctx == (const void*)b->ctx_len &&
                     h->chain_pool != (const void*)layer->pool;
  h->chain_ok = 0;
  if (b->q_indptr != nullptr || q_len < 1 || q_len > 4) return HSWA_ERR_INVALID_ARG;
  if (b->batch == 0) return HSWA_OK;
  if (!q || !out || !k_new || !v_new) return HSWA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new)) return HSWA_ERR_INVALID_ARG;
  if (layer->is_swa && q_len > h->ring_slots - h->cfg.window + 1) return HSWA_ERR_INVALID_ARG;  // append-then-attend limit
  // The streaming ring kernel's token mode keeps a whole ring staged (three 64-slot buffers) while its warps patch and
  // read it; longer rings take the compact-window kernel, which needs the window itself to fit shared memory
  if (layer->is_swa && (h->ring_slots + 63) / 64 > 3 && !hswa_ring_compact_supported(model_params(h), q_len))
    return HSWA_ERR_UNSUPPORTED;
  if (!layer->is_swa && (int64_t)b->max_ctx_len + q_len > (int64_t)b->max_blocks * h->cfg.page_size) return HSWA_ERR_INVALID_ARG;

  AppendParams a;
  a.m = model_params(h);
  a.b = batch_params(b);
  a.pool = static_cast<__nv_bfloat16*>(layer->pool);
  a.num_pages = layer->num_pages;
  a.is_swa = layer->is_swa;
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.v_new = static_cast<const __nv_bfloat16*>(v_new);
  a.total_q = b->batch * q_len;
  a.max_q_len = q_len;
  a.uniform_n = q_len;
  a.err = h->err;

  DecodeParams p;
  p.m = a.m;
  p.b = a.b;
  p.pool = a.pool;
  p.num_pages = a.num_pages;
  p.is_swa = layer->is_swa;
  p.q = static_cast<const __nv_bfloat16*>(q);
  // Full layers: the tokens are in the cache by the time the attention kernel runs (append kernel first); rings:
  // the ring kernel appends them itself
  p.k_new = layer->is_swa ? a.k_new : nullptr;
  p.v_new = layer->is_swa ? a.v_new : nullptr;
  p.out = out;
  p.lse = lse;
  p.err = h->err;
  p.part_o = nullptr;
  p.part_ml = nullptr;
  p.k_start = 0;
  p.split_base = 0;
  p.nq = q_len;
  p.max_ctx_len = b->max_ctx_len;
  p.late_dep_wait = 0;
  DecodePlan pl;
  if (!plan_decode(h, layer->is_swa, b->batch, b->max_ctx_len, 0, q_len, &pl)) return HSWA_ERR_UNSUPPORTED;
  p.split_len = pl.split_len;
  p.grid_splits = pl.grid_splits;
  p.max_splits = pl.max_splits;
  if (p.max_splits > 1) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 ||
        workspace_bytes < pl.o_bytes + pl.ml_bytes + pl.info_bytes)
      return HSWA_ERR_WORKSPACE;
    p.part_o = static_cast<float*>(workspace);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(workspace) + pl.o_bytes);
  }
  CUtensorMap tm;
  const int granule = h->cfg.page_size < HSWA_RING_GRANULE ? h->cfg.page_size : HSWA_RING_GRANULE;
  if ((st = make_pool_map(h, layer, &tm, layer->is_swa ? granule : 0)) != HSWA_OK) return st;
  if (!layer->is_swa && hswa_launch_append(a, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  if (pl.tc) {
    // tensor-core path: the rows of a request (tokens x heads) share one pass over its KV bytes
    CUtensorMap tm_q;
    if ((st = make_rows_map(h, q, h->cfg.num_q_heads, (int64_t)b->batch * q_len, 4, &tm_q, 8)) != HSWA_OK) return st;
    if (hswa_launch_decode_mtp_tc(tm, tm_q, p, h->num_sms, workspace, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  } else {
    if (hswa_launch_decode_mtp(h, tm, p, early, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
    if (p.max_splits > 1 && hswa_launch_combine(p, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  }
  h->chain_ok = 1;  // none of these kernels writes the batch arrays or another layer's pool
  h->chain_stream = stream;
  h->chain_ctx = (const void*)b->ctx_len;
  h->chain_pool = (const void*)layer->pool;
  return HSWA_OK;
}

hswa_status hswa_decode_attn_shared_prefix(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b,
                                           int32_t shared_prefix_len, const void* q, const void* k_new, const void* v_new,
                                           void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
  if (!h || shared_prefix_len < 0 || shared_prefix_len % h->cfg.page_size != 0) return HSWA_ERR_INVALID_ARG;
  if (b && shared_prefix_len > b->max_ctx_len) return HSWA_ERR_INVALID_ARG;
  return decode_impl(h, layer, b, shared_prefix_len, q, k_new, v_new, out, lse, workspace, workspace_bytes, stream);
}

hswa_status hswa_prefill_attn(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, const void* q,
                              const void* k_new, const void* v_new, int32_t fuse_append, void* out, float* lse,
                              void* workspace, size_t workspace_bytes, void* stream) {
  if (h) h->chain_ok = 0;
  (void)workspace;
  (void)workspace_bytes;
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  if (b->batch == 0 || b->total_q == 0) return HSWA_OK;
  if (!q || !out || !k_new || !v_new) return HSWA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new)) return HSWA_ERR_INVALID_ARG;
  PrefillParams p;
  p.m = model_params(h);
  p.b = batch_params(b);
  p.pool = static_cast<__nv_bfloat16*>(layer->pool);
  p.num_pages = layer->num_pages;
  p.is_swa = layer->is_swa;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.out = out;
  p.lse = lse;
  p.total_q = b->total_q;
  p.max_q_len = b->max_q_len;
  p.err = h->err;
  p.order_mode = h->prefill_order;
  p.trace = h->trace;
  p.trace_cap = h->trace_cap;
  const int64_t tc_tiles = (int64_t)b->batch * ((b->max_q_len + 127) / 128);
  if (hswa_prefill_tc_supported(p.m) && b->q_indptr != nullptr && tc_tiles <= 65535) {
    // tcgen05 / TMEM / TMA tile kernel
    CUtensorMap tm_pool, tm_q, tm_k, tm_v;
    if ((st = make_pool_map(h, layer, &tm_pool)) != HSWA_OK) return st;
    if ((st = make_rows_map(h, q, h->cfg.num_q_heads, b->total_q, 128, &tm_q)) != HSWA_OK) return st;
    if ((st = make_rows_map(h, k_new, h->cfg.num_kv_heads, b->total_q, 128, &tm_k)) != HSWA_OK) return st;
    if ((st = make_rows_map(h, v_new, h->cfg.num_kv_heads, b->total_q, 128, &tm_v)) != HSWA_OK) return st;
    // SWA layers: tokens whose whole window lies inside the chunk go to the GQA-packed kernel; the first
    // tokens (which also read the ring) stay on the general tile kernel.
    int tq = 0, nkeys = 0;
    hswa_prefill_packed_geometry(h->group, &tq, &nkeys);
    const int split_tiles = (h->cfg.window - 1 + 127) / 128;  // 128-token tiles that can reach below the chunk
    const bool packed = layer->is_swa && tq > 0 && h->cfg.window <= 128 && b->max_q_len > split_tiles * 128;
    if (hswa_launch_prefill_tc(tm_pool, tm_q, tm_k, tm_v, p, packed ? split_tiles : 0, (cudaStream_t)stream) != cudaSuccess)
      return HSWA_ERR_CUDA;
    if (packed) {
      CUtensorMap pq, pk, pv;
      if ((st = make_rows_map(h, q, h->cfg.num_q_heads, b->total_q, tq, &pq, h->group)) != HSWA_OK) return st;
      if (h->group == 8 && h->cfg.window == 128) {
        // streaming kernel (its mask shortcuts assume the paper's W = 128): K/V arrive in 16-row pieces
        CUtensorMap po = pq, k16, v16;
        const int tma_out = h->cfg.out_dtype == 0;  // bf16 output leaves through a TMA tensor store
        if (tma_out && (st = make_rows_map(h, out, h->cfg.num_q_heads, b->total_q, tq, &po, h->group)) != HSWA_OK) return st;
        if ((st = make_rows_map(h, k_new, h->cfg.num_kv_heads, b->total_q, 16, &k16)) != HSWA_OK) return st;
        if ((st = make_rows_map(h, v_new, h->cfg.num_kv_heads, b->total_q, 16, &v16)) != HSWA_OK) return st;
        if (hswa_launch_prefill_swa_stream(pq, k16, v16, po, tma_out, p, h->num_sms, (cudaStream_t)stream) != cudaSuccess)
          return HSWA_ERR_CUDA;
      } else {
        if ((st = make_rows_map(h, k_new, h->cfg.num_kv_heads, b->total_q, nkeys, &pk)) != HSWA_OK) return st;
        if ((st = make_rows_map(h, v_new, h->cfg.num_kv_heads, b->total_q, nkeys, &pv)) != HSWA_OK) return st;
        if (hswa_launch_prefill_swa_packed(pq, pk, pv, p, split_tiles * 128, (cudaStream_t)stream) != cudaSuccess)
          return HSWA_ERR_CUDA;
      }
    }
  } else {
    if (hswa_launch_prefill_mma(p, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  }
  if (fuse_append) {
    // stream order puts the append after every read of the pre-append ring contents
    AppendParams a;
    a.m = p.m;
    a.b = p.b;
    a.pool = p.pool;
    a.num_pages = p.num_pages;
    a.is_swa = p.is_swa;
    a.k_new = p.k_new;
    a.v_new = p.v_new;
    a.total_q = p.total_q;
    a.max_q_len = p.max_q_len;
    a.uniform_n = 0;
    a.err = h->err;
    if (hswa_launch_append(a, (cudaStream_t)stream) != cudaSuccess) return HSWA_ERR_CUDA;
  }
  return HSWA_OK;
}

static hswa_status window_move(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, void* buf, int gather,
                               void* stream) {
  hswa_status st = check_common(h, layer, b);
  if (st != HSWA_OK) return st;
  h->chain_ok = 0;
  if (!layer->is_swa) return HSWA_ERR_INVALID_ARG;
  if (b->batch == 0 || h->cfg.window <= 1) return HSWA_OK;
  if (!buf || !aligned16(buf)) return HSWA_ERR_INVALID_ARG;
  return hswa_launch_window_move(model_params(h), batch_params(b), static_cast<__nv_bfloat16*>(layer->pool), layer->num_pages,
                                 static_cast<__nv_bfloat16*>(buf), gather, h->err, (cudaStream_t)stream) == cudaSuccess
             ? HSWA_OK
             : HSWA_ERR_CUDA;
}

hswa_status hswa_swa_window_gather(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, void* buf, void* stream) {
  return window_move(h, layer, b, buf, 1, stream);
}

hswa_status hswa_swa_window_scatter(hswa_handle* h, const hswa_layer* layer, const hswa_batch* b, const void* buf,
                                    void* stream) {
  return window_move(h, layer, b, const_cast<void*>(buf), 0, stream);
}

int64_t hswa_window_safe_len(int64_t match_len, int32_t window, const uint8_t* swa_valid) {
  if (match_len <= 0 || window <= 1 || !swa_valid) return match_len > 0 && window <= 1 ? match_len : 0;
  // run[i] = number of consecutive valid positions ending at i; L is safe iff run[L - 1] >= min(L, W - 1)
  int64_t best = 0, run = 0;
  for (int64_t i = 0; i < match_len; ++i) {
    run = swa_valid[i] ? run + 1 : 0;
    const int64_t L = i + 1, need = L < window - 1 ? L : window - 1;
    if (run >= need) best = L;
  }
  return best;
}

int64_t hswa_prefix_hit_len(int64_t match_len, int32_t window, const uint8_t* full_valid, const uint8_t* swa_valid) {
  if (match_len <= 0 || window < 1 || !full_valid) return 0;
  // Full layers read every position below the hit length: the hit cannot pass the first token without Full KV
  int64_t limit = 0;
  while (limit < match_len && full_valid[limit]) ++limit;
  if (window <= 1) return limit;
  return hswa_window_safe_len(limit, window, swa_valid);
}

hswa_status hswa_swa_release(hswa_handle* h, int32_t batch, const int32_t* ctx_len, const uint8_t* release,
                             int32_t* swa_valid_from, void* stream) {
  if (h) h->chain_ok = 0;
  if (!h || batch < 0) return HSWA_ERR_INVALID_ARG;
  if (batch == 0) return HSWA_OK;
  if (!ctx_len || !swa_valid_from) return HSWA_ERR_INVALID_ARG;
  return hswa_launch_swa_release(model_params(h), batch, ctx_len, release, swa_valid_from, (cudaStream_t)stream) == cudaSuccess
             ? HSWA_OK
             : HSWA_ERR_CUDA;
}

hswa_status hswa_swa_valid_mask(hswa_handle* h, int32_t batch, const int32_t* ctx_len, const int32_t* swa_valid_from,
                                int64_t mask_stride, uint8_t* mask, void* stream) {
  if (h) h->chain_ok = 0;
  if (!h || batch < 0 || mask_stride < 0) return HSWA_ERR_INVALID_ARG;
  if (batch == 0 || mask_stride == 0) return HSWA_OK;
  if (!ctx_len || !swa_valid_from || !mask) return HSWA_ERR_INVALID_ARG;
  return hswa_launch_swa_valid_mask(batch, ctx_len, swa_valid_from, mask_stride, mask, (cudaStream_t)stream) == cudaSuccess
             ? HSWA_OK
             : HSWA_ERR_CUDA;
}

hswa_status hswa_step_advance(hswa_handle* h, int32_t batch, int32_t* ctx_len, int32_t* ring_head,
                              const int32_t* q_indptr, void* stream) {
  if (h) h->chain_ok = 0;
  if (!h || batch < 0) return HSWA_ERR_INVALID_ARG;
  if (batch == 0) return HSWA_OK;
  if (!ctx_len || !ring_head) return HSWA_ERR_INVALID_ARG;
  return hswa_launch_advance(model_params(h), batch, ctx_len, ring_head, q_indptr, (cudaStream_t)stream) == cudaSuccess
             ? HSWA_OK
             : HSWA_ERR_CUDA;
}

hswa_status hswa_get_async_error(hswa_handle* h, void* stream, int32_t info[4]) {
  if (h) h->chain_ok = 0;
  if (!h || !info) return HSWA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(info, h->err, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess) return HSWA_ERR_CUDA;
  if (cudaMemsetAsync(h->err, 0, 4 * sizeof(int32_t), s) != cudaSuccess) return HSWA_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return HSWA_ERR_CUDA;
  return (hswa_status)info[0];
}

}  // extern "C"
