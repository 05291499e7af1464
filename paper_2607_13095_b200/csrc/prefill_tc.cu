// Chunked prefill attention on 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands
// staged by TMA) for head_dim 128, page size 64 and an even GQA group.  Paper Sec. 2.1: prefill is
// compute-bound, Full layers attend to the whole prefix, SWA layers only inside the window; Sec. 3.1.1: Full
// layers read pages through the block table, SWA layers a ring (as it is before this chunk's append).
//
// One thread block = 128 query tokens x 2 query heads of one GQA group (two 128-row Q tiles that share every
// K/V tile and every mask).  Warp roles:
//   warps 0-3   softmax for Q tile 0: TMEM lane = row = thread; a thread holds the 128 scores of its row in
//               registers, so row maxima and sums need no exchange
//   warps 4-7   softmax for Q tile 1
//   warp  8     TMA producer: Q once, then 128-key K and V tiles through two 2-stage rings whose slots are
//               released separately (K right after the S MMAs, V after both tiles' PV MMAs)
//   warps 9,10  MMA issuers, one per Q tile: S_i = Q_i K^T (SS form), O_i += P_i V (TS form, P read from TMEM
//               where it overwrites S_i).  They take turns, [PV0(j), S0(j+1)] [PV1(j), S1(j+1)] ..., so that one
//               tile's softmax overlaps the other tile's MMAs; while one holds the turn, the other polls the
//               mbarriers of its next group (an mbarrier poll costs 100-200 cycles while the tensor cores
//               saturate shared memory, and a single issuer spent a third of its time in them)
// TMEM columns: S0 0-127, S1 128-255, O0 256-383, O1 384-511 (all fp32; P_i = bf16 pairs in the first 64
// columns of S_i).  O is rescaled lazily: only when a row maximum grows by more than 2^8.
//
// Key tiles: phase A covers cached positions (Full: pages 2a, 2a+1 of the block table; SWA: the ring pages,
// only for the first tokens of the chunk), phase B covers the chunk's own K/V in chunk-relative 128-token
// tiles, so every tile has a single source and masks take care of ragged edges.  Tiles wholly above the
// diagonal or wholly below the window are never loaded or multiplied.
#include "hswa_internal.cuh"
#include "tc_primitives.cuh"

namespace {
using namespace hswa_dev;

constexpr int BM = 128;               // query rows per Q tile
constexpr int BN = 128;               // keys per tile
constexpr int HD = 128;               // head dim
constexpr int PG = 64;                // page size
constexpr int HALF_BYTES = 128 * 128; // [128 rows][128 B]: one 64-element half of a 128-row tile
constexpr int TILE_BYTES = 2 * HALF_BYTES;
constexpr int KV_STAGES = 2;
constexpr int NUM_THREADS = 384;  // 8 softmax warps + producer + one MMA issuer per Q tile + the patch warp
// Registers per thread after the roles have split; the sum over the block must not pass what the launch gave
// (384 x 168), or the softmax warps' request would never be granted: checked against the compiled kernel before launch.
constexpr int REGS_SERVICE = 56, REGS_SOFTMAX = 224;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                  // 2 Q tiles
constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;             // the K ring, then the V ring (both `stages` tiles deep)
constexpr int tile_kernel_smem(int stages) { return OFF_K + 2 * stages * TILE_BYTES + 256; }  // + barriers and flags

constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
constexpr uint32_t IDESC_PV = IDESC_S | (1u << 16);  // B (= V) is MN-major: [key][d] with d contiguous

// barrier indices
enum { BAR_Q = 0, BAR_KFULL = 1, BAR_KEMPTY = 3, BAR_VFULL = 5, BAR_VEMPTY = 7, BAR_SFULL = 9,
       BAR_PFULL = 11 /* [Q tile][half of the key columns] */, BAR_OFINAL = 15 /* [Q tile] */,
       BAR_VPATCH = 17 /* [stage]: a V tile whose dead rows are zeroed before the MMA issuers see it */, NUM_BARS = 19 };

constexpr int P_PARTS = 2;  // P is posted to the MMA issuer in two halves of 64 keys

// The sequence of key tiles one block walks: nA cached tiles, then chunk tiles c_lo .. c_lo + nB - 1.
struct TileSeq {
  int nA, c_lo, nB;
  __device__ __forceinline__ int total() const { return nA + nB; }
};
__device__ __forceinline__ TileSeq tile_seq(int is_swa, int ctx, int b, int W, int R) {
  TileSeq s;
  if (!is_swa) {
    s.nA = (ctx + BN - 1) / BN;
    s.c_lo = 0;
  } else {
    const bool ring = ctx > 0 && b * BM < W - 1;  // some row of this tile reaches below the chunk
    s.nA = ring ? (R + 1) / 2 : 0;
    const int low = b * BM - W + 1;  // lowest chunk-relative key any row needs
    s.c_lo = low > 0 ? low / BN : 0;
  }
  s.nB = b - s.c_lo + 1;
  return s;
}

// Global longest-first order of the (request, 128-token tile) pairs of a Full-layer prefill batch (paper Sec. 5.3:
// mixed prefix lengths leave whoever got the long ones running last).  Tile b of request r walks
// work(r, b) = ceil(ctx_r / 128) + b + 1 key tiles.  Pair number idx in descending order of work (ties: ascending
// request) is found without sorting: count_ge(w), the number of pairs with work >= w, is a sum over requests of
// clamped linear terms and falls with w, so a binary search finds the work value w* of pair idx, and idx minus
// count_ge(w* + 1) says which of the requests that own a tile of exactly that work it is.  One warp, lanes strided
// over requests; false when idx is beyond the last pair.
__device__ __forceinline__ bool pick_longest_first(const BatchParams& bp, int idx, int lane, int* r_out, int* b_out) {
  auto tiles_of = [&](int r, int& cr, int& nt) {
    cr = (bp.ctx_len[r] + BN - 1) / BN;
    nt = (bp.q_indptr[r + 1] - bp.q_indptr[r] + BM - 1) / BM;
  };
  auto count_ge = [&](int w) {
    int c = 0;
    for (int r = lane; r < bp.B; r += 32) {
      int cr, nt;
      tiles_of(r, cr, nt);
      c += min(max(cr + nt - w + 1, 0), nt);
    }
#pragma unroll
    for (int sh = 16; sh; sh >>= 1) c += __shfl_xor_sync(0xffffffffu, c, sh);
    return c;
  };
  int w_max = 0;
  for (int r = lane; r < bp.B; r += 32) {
    int cr, nt;
    tiles_of(r, cr, nt);
    w_max = max(w_max, nt > 0 ? cr + nt : 0);
  }
#pragma unroll
  for (int sh = 16; sh; sh >>= 1) w_max = max(w_max, __shfl_xor_sync(0xffffffffu, w_max, sh));
  if (count_ge(1) <= idx) return false;
  int lo = 1, hi = w_max + 1, above = 0;  // count_ge(lo) > idx >= count_ge(hi) = above
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    const int c = count_ge(mid);
    if (c > idx) {
      lo = mid;
    } else {
      hi = mid;
      above = c;
    }
  }
  int k = idx - above;  // rank among the pairs of work exactly lo
  for (int base = 0; base < bp.B; base += 32) {
    const int r = base + lane;
    int cr = 0, nt = 0;
    if (r < bp.B) tiles_of(r, cr, nt);
    const unsigned has = __ballot_sync(0xffffffffu, r < bp.B && lo >= cr + 1 && lo <= cr + nt);
    const int cnt = __popc(has);
    if (k < cnt) {
      const int sel = __fns(has, 0, k + 1);
      *r_out = base + sel;
      *b_out = lo - 1 - __shfl_sync(0xffffffffu, cr, sel);
      return true;
    }
    k -= cnt;
  }
  return false;
}

// Longest REQUEST first: the tiles of a request stay together (their blocks walk the same K/V pages at the same
// time, which keeps them in L2 and measured 4 % faster on the chunked-prefill workload than any order that
// interleaves requests), requests are taken in descending order of their longest tile's work, ceil(ctx_r / 128) +
// tiles_r (ties: ascending request), and inside a request the longest tile goes first, so that the launch ends on the
// shortest tiles of the shortest request.  Same search as above on T(w) = number of tiles of all requests whose key
// is >= w.
__device__ __forceinline__ bool pick_longest_request_first(const BatchParams& bp, int idx, int lane, int* r_out, int* b_out) {
  auto tiles_of = [&](int r, int& key, int& nt) {
    nt = (bp.q_indptr[r + 1] - bp.q_indptr[r] + BM - 1) / BM;
    key = nt > 0 ? (bp.ctx_len[r] + BN - 1) / BN + nt : 0;
  };
  auto tiles_ge = [&](int w) {
    int c = 0;
    for (int r = lane; r < bp.B; r += 32) {
      int key, nt;
      tiles_of(r, key, nt);
      c += key >= w ? nt : 0;
    }
#pragma unroll
    for (int sh = 16; sh; sh >>= 1) c += __shfl_xor_sync(0xffffffffu, c, sh);
    return c;
  };
  int w_max = 0;
  for (int r = lane; r < bp.B; r += 32) {
    int key, nt;
    tiles_of(r, key, nt);
    w_max = max(w_max, key);
  }
#pragma unroll
  for (int sh = 16; sh; sh >>= 1) w_max = max(w_max, __shfl_xor_sync(0xffffffffu, w_max, sh));
  if (tiles_ge(1) <= idx) return false;
  int lo = 1, hi = w_max + 1, above = 0;  // tiles_ge(lo) > idx >= tiles_ge(hi) = above
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    const int c = tiles_ge(mid);
    if (c > idx) {
      lo = mid;
    } else {
      hi = mid;
      above = c;
    }
  }
  int k = idx - above;  // tile index among the requests whose key is exactly lo, taken in ascending request order
  for (int base = 0; base < bp.B; base += 32) {
    const int r = base + lane;
    int key = 0, nt = 0;
    if (r < bp.B) tiles_of(r, key, nt);
    const int mine = key == lo ? nt : 0;
    int incl = mine;  // inclusive prefix sum over the lanes
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, sh);
      if (lane >= sh) incl += v;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (k < total) {
      const unsigned hit = __ballot_sync(0xffffffffu, mine > 0 && k >= incl - mine && k < incl);
      const int sel = __ffs(hit) - 1;
      const int before = __shfl_sync(0xffffffffu, incl - mine, sel), ntile = __shfl_sync(0xffffffffu, nt, sel);
      *r_out = base + sel;
      *b_out = ntile - 1 - (k - before);  // longest tile first
      return true;
    }
    k -= total;
  }
  return false;
}

__device__ __forceinline__ long long global_timer_ns() {
  long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Called by every thread on its way out.  A role that gave up (a wait ran out, an error was recorded) leaves its
// loop while TMA loads that nobody will wait for may still be in flight towards this block's shared memory; a block
// must not exit, and hand its shared memory to the next block, before they have landed.  No barrier says when that
// is once the protocol is broken, so the error path simply outwaits them (0.1 ms, far above any TMA latency).
__device__ __forceinline__ void linger_after_error(const int32_t* err) {
  if (*reinterpret_cast<const volatile int32_t*>(err) != 0) __nanosleep(100000);
}

// PREFIX = true turns the same pipeline into the shared-prefix stage of batched decode (paper Sec. 3.1.3 /
// 3.1.4: requests that share a system prompt share its pages): the 128 rows of a Q tile are 16 requests x
// the 8 query heads of one KV head, the keys are a slice of the shared prefix pages, nothing is masked, and
// the block writes an unnormalised (m, l, o) partial per row for the split-K combine instead of an output.
// Does cached tile j (of nA) of a request with ctx cached tokens hold rows that no row of the block can see?  On a
// Full layer: the last tile when ctx ends inside it.  On an SWA layer: every ring tile (slots older than the window,
// never written, or past the ring's last page).
__device__ __forceinline__ bool v_tile_needs_patch(int is_swa, int ctx, int j) { return is_swa || ctx - j * BN < BN; }

// STAGES = depth of the K and of the V tile ring: 2 for prefill; 1 for the shared-prefix stage, whose block then leaves
// room on its SM for a block of the suffix decode kernel that streams beside it.
template <bool PREFIX, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_pool, const __grid_constant__ CUtensorMap tm_q,
                  const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const PrefillParams p, const int max_tiles) {  // tiles b < max_tiles only
  // All shared memory is one dynamic window (no static part, so that it starts on the 1 KB boundary the swizzled tiles
  // need without slack): Q tiles | K ring | V ring | barriers and flags.
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr int OFF_V = OFF_K + STAGES * TILE_BYTES;
  constexpr int OFF_STATE = OFF_V + STAGES * TILE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_STATE);                     // [NUM_BARS]
  uint32_t& tmem_base_slot = *reinterpret_cast<uint32_t*>(smem + OFF_STATE + 160);
  int& mma_abort = *reinterpret_cast<int*>(smem + OFF_STATE + 164);  // set by an MMA issuer that gave up, read by the other
  int* picked = reinterpret_cast<int*>(smem + OFF_STATE + 168);      // [2] (request, tile) under the longest-first order
  static_assert(NUM_BARS * 8 <= 160, "barriers fit their slot");
  const uint32_t sbase = smem_u32(smem);
  const ModelParams& M = p.m;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pair = blockIdx.x, kh = blockIdx.y;
  int r, b, t0, n, ctx, head, h0, page_off = 0;
  TileSeq seq;
  if constexpr (PREFIX) {
    // the suffix decode kernel that follows on the stream reads nothing this kernel writes before its own
    // dependency wait: let it start its table reads and loads now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // blockIdx.x = slice of the prefix, blockIdx.z = group of 32 requests (16 per Q tile)
    r = blockIdx.z * 32;
    if (r >= p.b.B) return;
    b = 0;
    t0 = r;
    n = p.b.B - r;  // requests left from r on
    head = 0;
    h0 = kh * M.G;
    const int tiles_total = (p.prefix_len + BN - 1) / BN;
    const int tile_begin = blockIdx.x * p.prefix_tiles_per_split;
    seq.nA = min(p.prefix_tiles_per_split, tiles_total - tile_begin);
    seq.c_lo = 0;
    seq.nB = 0;
    page_off = 2 * tile_begin;
    ctx = p.prefix_len - tile_begin * BN;  // keys from this slice's first tile to the end of the prefix
    if (seq.nA <= 0) return;               // the host plans slices so that none is empty
  } else {
    if (p.order_mode >= 2 && !p.is_swa) {
      // longest request first (2) or globally longest tile first (3); on SWA layers every tile costs the same and the
      // order does not matter
      if (warp == 0) {
        int pr = -1, pb = 0;
        const bool got = p.order_mode == 2 ? pick_longest_request_first(p.b, (int)blockIdx.z, lane, &pr, &pb)
                                           : pick_longest_first(p.b, (int)blockIdx.z, lane, &pr, &pb);
        if (!got) pr = -1;
        if (lane == 0) {
          picked[0] = pr;
          picked[1] = pb;
        }
      }
      __syncthreads();
      r = picked[0];
      b = picked[1];
      if (r < 0) return;  // uniform for the block
    } else if (p.order_mode == 0) {
      r = blockIdx.z / max_tiles;  // request by request, tiles ascending
      b = blockIdx.z % max_tiles;
    } else {
      r = blockIdx.z % p.b.B;
      b = max_tiles - 1 - (int)(blockIdx.z / p.b.B);  // every request's last (longest) tile first
    }
    t0 = p.b.q_indptr[r];
    n = p.b.q_indptr[r + 1] - t0;
    if (b * BM >= n) return;  // uniform for the block
    ctx = p.b.ctx_len[r];
    head = p.is_swa ? p.b.ring_head[r] : 0;
    h0 = kh * M.G + pair * 2;
    seq = tile_seq(p.is_swa, ctx, b, M.W, M.R);
  }
  // An earlier block gave up: do not queue behind it.  One thread reads the error word so that the whole block
  // takes the same decision (the MMA issuers below wait for each other on counted barriers).
  if (threadIdx.x == 0) {
    mma_abort = *reinterpret_cast<volatile int32_t*>(p.err) != 0;
    if (sbase & 1023u) {  // the swizzled tile addressing assumes a 1 KB-aligned window
      record_error(p.err, HSWA_ERR_CUDA, -1, (int)(sbase & 1023u), 14);
      mma_abort = 1;
    }
  }
  __syncthreads();
  if (mma_abort) return;
  const int n_tiles = seq.total();
  const int64_t trace_slot = blockIdx.x + (int64_t)gridDim.x * (blockIdx.y + (int64_t)gridDim.y * blockIdx.z);
  const bool traced = p.trace != nullptr && trace_slot < p.trace_cap;
  if (traced && threadIdx.x == 0) p.trace[trace_slot * 4] = global_timer_ns();

  auto bar = [&](int i) { return smem_u32(&bars[i]); };

  if (threadIdx.x == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar(BAR_KFULL + s), 1);
      mbar_init(bar(BAR_KEMPTY + s), 2);  // one commit per MMA issuer
      mbar_init(bar(BAR_VFULL + s), 1);
      mbar_init(bar(BAR_VEMPTY + s), 2);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_SFULL + i), 1);
      for (int q = 0; q < P_PARTS; ++q) mbar_init(bar(BAR_PFULL + P_PARTS * i + q), 4);  // one arrival per softmax warp
    }
    mbar_init(bar(BAR_OFINAL), 1);
    mbar_init(bar(BAR_OFINAL + 1), 1);
    static_assert(STAGES <= 2, "one patch barrier per V stage");
    mbar_init(bar(BAR_VPATCH), 1);
    mbar_init(bar(BAR_VPATCH + 1), 1);
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;

  // Registers move from the service warps (one warpgroup: producer, two MMA issuers and the patch warp; the
  // exchange is made by whole warpgroups) to the softmax warps, whose threads hold a row of 128 scores:
  // 8 x 32 x 224 + 4 x 32 x 56 = 384 x 168.  Each role's branch changes its own allotment.
  if (warp == 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= TMA producer =======================
    if (lane == 0) {
      tma_prefetch_desc(&tm_pool);
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      mbar_arrive_expect_tx(bar(BAR_Q), 2 * TILE_BYTES);
      for (int i = 0; i < 2; ++i)
        for (int hf = 0; hf < 2; ++hf) {
          if constexpr (PREFIX)  // box {64, 8 heads, 16 requests} over q [B][Hq][D]
            tma_load_3d(sbase + OFF_Q + i * TILE_BYTES + hf * HALF_BYTES, &tm_q, bar(BAR_Q), hf * 64, h0, r + 16 * i);
          else
            tma_load_3d(sbase + OFF_Q + i * TILE_BYTES + hf * HALF_BYTES, &tm_q, bar(BAR_Q), hf * 64, h0 + i, t0 + b * BM);
        }
    }
    // page ids of the cached tiles, 32 at a time
    const int32_t* tbl = p.is_swa ? p.b.ring_table + (int64_t)r * M.R : p.b.block_table + (int64_t)r * p.b.max_blocks + page_off;
    const int n_pages = p.is_swa ? M.R : (ctx + PG - 1) / PG;
    int pid_next = lane < n_pages ? tbl[lane] : 0;
    int pid_cur = 0;
    bool ok = true;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int stage = j % STAGES;
      int pg[2] = {0, 0};
      // Rows of a cached tile that no row of this block can see (the tail of the last page of a Full layer; ring
      // slots never written, past the ring's last page, or older than the first row's window, which a ring seeded
      // with a window only never filled) may hold anything, patterns of NaN included.  Their probabilities are exactly
      // 0, but 0 x NaN would still reach the output through the PV MMA (paper Sec. 3.1.3: attention must not be
      // affected by invalid slots).  The V half of such a tile lands on a barrier that the patch warp (warp 11)
      // waits on; that warp zeroes the dead rows and only then hands the tile to the MMA issuers.
      const bool patch = !PREFIX && j < seq.nA && v_tile_needs_patch(p.is_swa, ctx, j);
      if (j < seq.nA) {
        if (((2 * j) & 31) == 0) {
          pid_cur = pid_next;
          const int nx = 2 * j + 32 + lane;
          pid_next = nx < n_pages ? tbl[nx] : 0;
        }
        const int i0 = 2 * j, i1 = (2 * j + 1 < n_pages) ? 2 * j + 1 : 2 * j;  // a missing page repeats its neighbour
        pg[0] = __shfl_sync(0xffffffffu, pid_cur, i0 & 31);
        pg[1] = __shfl_sync(0xffffffffu, pid_cur, i1 & 31);
      }
      if (lane == 0) {
        // K and V slots are released separately (K right after the S MMAs that read it, V only after both tiles'
        // PV MMAs), so each load waits for its own slot: the K tile is on its way a whole step earlier.
        const uint32_t par = ((j / STAGES) - 1) & 1;
        const uint32_t dK = sbase + OFF_K + stage * TILE_BYTES, dV = sbase + OFF_V + stage * TILE_BYTES;
        for (int kv = 0; kv < 2 && ok; ++kv) {
          const uint32_t full_mma = bar((kv ? BAR_VFULL : BAR_KFULL) + stage);
          if (j >= STAGES && !mbar_wait(bar((kv ? BAR_VEMPTY : BAR_KEMPTY) + stage), par)) {
            record_error(p.err, HSWA_ERR_TIMEOUT, r, j, 10 + kv);
            ok = false;
            break;
          }
          const uint32_t full = (kv && patch) ? bar(BAR_VPATCH + stage) : full_mma;
          mbar_arrive_expect_tx(full, TILE_BYTES);
          const uint32_t dst = kv ? dV : dK;
          if (j < seq.nA) {
            for (int q = 0; q < 2; ++q) {
              int page = pg[q];
              if (page < 0 || page >= p.num_pages) {
                record_error(p.err, HSWA_ERR_BOUNDS, r, 2 * j + q, page);
                page = 0;
              }
              for (int hf = 0; hf < 2; ++hf)
                tma_load_4d(dst + hf * HALF_BYTES + q * PG * 128, &tm_pool, full, hf * 64, 0, kv * M.Hkv + kh, page);
            }
          } else {
            const int tok = t0 + (seq.c_lo + (j - seq.nA)) * BN;
            for (int hf = 0; hf < 2; ++hf) tma_load_3d(dst + hf * HALF_BYTES, kv ? &tm_v : &tm_k, full, hf * 64, kh, tok);
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
    }
  } else if (warp == 9 || warp == 10) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= MMA issuer =======================
    // The whole warp walks the loop converged (waits, descriptor arithmetic); one elected lane issues.
    {
      bool ok = mbar_wait(bar(BAR_Q), 0);
      const uint64_t dQ0 = smem_desc(sbase + OFF_Q, 16), dQ1 = smem_desc(sbase + OFF_Q + TILE_BYTES, 16);
      const uint64_t dK0 = smem_desc(sbase + OFF_K, 16), dV0 = smem_desc(sbase + OFF_V, HALF_BYTES);
      auto issue_S = [&](int i, int stage) {
        tc_fence_after();
        const uint64_t dq = i ? dQ1 : dQ0, dk = desc_advance(dK0, stage * TILE_BYTES);
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < HD / 16; ++ks) {
            const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
            tc_mma_ss(tmem + i * 128, desc_advance(dq, off), desc_advance(dk, off), IDESC_S, ks > 0);
          }
          tc_commit(bar(BAR_SFULL + i));
        }
        __syncwarp();
      };
      // PV k-steps of one part of the keys, issued as soon as its P columns are posted
      constexpr int KSTEPS = 8 / P_PARTS;
      auto issue_PV = [&](int i, int stage, int part, bool first) {
        tc_fence_after();
        const uint64_t dv = desc_advance(dV0, stage * TILE_BYTES + part * KSTEPS * 2048);
        const uint32_t tp = tmem + i * 128 + part * KSTEPS * 8;
        if (elect_one()) {
#pragma unroll
          for (int q = 0; q < KSTEPS; ++q)
            tc_mma_ts(tmem + 256 + i * 128, tp + q * 8, desc_advance(dv, q * 2048), IDESC_PV, !(first && part == 0 && q == 0));
        }
        __syncwarp();
      };
      // One issuer per Q tile, taking turns: [PV0(j), S0(j+1)] [PV1(j), S1(j+1)] [PV0(j+1), ...].  The turn is a
      // token passed through two named barriers (hardware barriers: no shared-memory round trip), so the order in
      // the tensor queue is the one that keeps the tiles half a step apart, while each issuer polls the
      // mbarriers of its next group during the other issuer's turn.  A warp leaves the loop only right after
      // passing the token, and passes it whenever it finds the abort flag set, so neither can wait forever.
      const int i = warp - 9;
      const int tok_in = i == 0 ? 2 : 1, tok_out = i == 0 ? 1 : 2;
      auto token_wait = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(tok_in) : "memory"); };
      auto token_pass = [&]() {
        __threadfence_block();  // the abort flag, if set, is visible to the warp this releases
        asm volatile("bar.arrive %0, 64;" ::"r"(tok_out) : "memory");
      };
      volatile int* abort_flag = &mma_abort;
      if (ok) ok = mbar_wait(bar(BAR_KFULL + 0), 0);
      if (i == 1) token_wait();
      if (!ok) *abort_flag = 1;
      if (ok && *abort_flag == 0) {
        issue_S(i, 0);
        if (elect_one()) tc_commit(bar(BAR_KEMPTY + 0));
        __syncwarp();
      }
      token_pass();
      bool done = !ok || *abort_flag != 0;
      for (int j = 0; j < n_tiles && !done; ++j) {
        const int stage = j % STAGES, nstage = (j + 1) % STAGES;
        const bool more = j + 1 < n_tiles;
        // polled during the other issuer's turn
        ok = mbar_wait(bar(BAR_VFULL + stage), (j / STAGES) & 1) && mbar_wait(bar(BAR_PFULL + P_PARTS * i), j & 1);
        if (ok && more) ok = mbar_wait(bar(BAR_KFULL + nstage), ((j + 1) / STAGES) & 1);
        token_wait();
        if (!ok) *abort_flag = 1;
        if (*abort_flag != 0) {
          token_pass();
          break;
        }
#pragma unroll
        for (int q = 0; q < P_PARTS; ++q) {
          if (q > 0 && ok) ok = mbar_wait(bar(BAR_PFULL + P_PARTS * i + q), j & 1);
          if (ok) issue_PV(i, stage, q, j == 0);
        }
        if (ok) {
          if (elect_one()) tc_commit(bar(BAR_VEMPTY + stage));
          __syncwarp();
          if (more) {
            issue_S(i, nstage);
            if (elect_one()) tc_commit(bar(BAR_KEMPTY + nstage));
            __syncwarp();
          }
        } else {
          *abort_flag = 1;
          done = true;
        }
        token_pass();
      }
      if (!ok && lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, b, 20 + i);
      if (elect_one()) tc_commit(bar(BAR_OFINAL + i));
      __syncwarp();
    }
  } else if (warp == 11) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= patch warp =======================
    // (see the producer: dead rows of a cached V tile are zeroed between the tile's arrival and its hand-over)
    if constexpr (!PREFIX) {
      uint32_t n_patched = 0;  // bit s: parity of the next patch of stage s
      for (int j = 0; j < seq.nA; ++j) {
        if (!v_tile_needs_patch(p.is_swa, ctx, j)) continue;
        const int stage = j % STAGES;
        // the producer arms this barrier once per patched tile of the stage, after the stage's previous tile has been
        // consumed: this warp sees each of its phases in turn
        if (!mbar_wait(bar(BAR_VPATCH + stage), (n_patched >> stage) & 1u)) {
          if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, j, 12);
          break;
        }
        n_patched ^= 1u << stage;
        uint8_t* sV = smem + OFF_V + stage * TILE_BYTES;
        for (int idx = lane; idx < BN * 16; idx += 32) {  // 16-byte chunks: 128 rows x 2 halves x 8
          const int row = (idx >> 3) & (BN - 1), hf = idx >> 10, ch = idx & 7;
          bool live;
          if (!p.is_swa) {
            live = row < ctx - j * BN;
          } else {
            const int slot = j * BN + row;  // ring slot; it holds position kpos = ctx - C + ((slot - head) mod C)
            int off = slot - head;
            if (off < 0) off += M.C;
            const int kpos = ctx - M.C + off;
            live = slot < M.C && kpos >= 0 && kpos > ctx + b * BM - M.W;  // visible to the block's first row at least
          }
          if (!live) *reinterpret_cast<uint4*>(sV + hf * HALF_BYTES + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_VFULL + stage));
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX) : "memory");
    // ======================= softmax warps =======================
    // 4 warps per Q tile: TMEM lane = row = thread, which holds all 128 scores of its row in registers, so row
    // maxima and sums need no exchange.  P is written to TMEM in four quarters of 32 keys and posted to the MMA
    // issuer in two halves; the first half is posted once the third quarter's exponentials are under way,
    // which hides the TMEM store latency.
    const int i = warp >> 2;                    // Q tile
    const int quad = warp & 3;
    const int rr = quad * 32 + lane;            // row in the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t tS = tmem + lane_addr + i * 128;
    const uint32_t tO = tmem + lane_addr + 256 + i * 128;
    const int ri = b * BM + rr;                 // chunk-relative row
    const int pos = ctx + ri;                   // absolute position
    float m_st = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SFULL + i), j & 1));  // warp-uniform: TMEM ops are warp-wide
      if (!ok) {
        if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, j, 30 + i);
        break;
      }
      // visible column interval [lo, hi) of this row in this tile; ring tiles are decided per column
      int lo = 0, hi = BN;
      bool ring_tile = false, masked = false;
      if (j < seq.nA) {
        if (!p.is_swa) {
          hi = min(BN, ctx - j * BN);
          masked = hi < BN;
        } else {
          ring_tile = true;
          masked = true;
        }
      } else {
        const int c = seq.c_lo + (j - seq.nA);
        hi = ri - c * BN + 1;
        hi = hi < 0 ? 0 : (hi > BN ? BN : hi);
        if (p.is_swa) {
          lo = ri - M.W + 1 - c * BN;
          lo = lo < 0 ? 0 : lo;
        }
        masked = (c == b) || p.is_swa;
      }
      // bit k of vm[w] = column 32 w + k is visible to this row
      uint32_t vm[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
      if (masked) {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint64_t m64 = 0;
          if (!ring_tile) {
            int c0 = lo - hf * 64, c1 = hi - hf * 64;
            c0 = c0 < 0 ? 0 : (c0 > 64 ? 64 : c0);
            c1 = c1 < 0 ? 0 : (c1 > 64 ? 64 : c1);
            const uint64_t below_c1 = c1 >= 64 ? ~0ull : ((1ull << c1) - 1);
            const uint64_t below_c0 = c0 >= 64 ? ~0ull : ((1ull << c0) - 1);
            m64 = c1 > c0 ? (below_c1 & ~below_c0) : 0ull;
          } else {
            // ring tile: ring page 2j + hf; slot -> position it held before the chunk's append
            const int page_in_ring = 2 * j + hf;
            if (page_in_ring < M.R) {
#pragma unroll 1
              for (int k = 0; k < 64; ++k) {
                int off = page_in_ring * PG + k - head;
                if (off < 0) off += M.C;
                const int kpos = ctx - M.C + off;
                if (kpos >= 0 && kpos > pos - M.W) m64 |= 1ull << k;
              }
            }
          }
          vm[2 * hf] = (uint32_t)m64;
          vm[2 * hf + 1] = (uint32_t)(m64 >> 32);
        }
      }
      // this thread's 128 scores: one round trip to TMEM
      uint32_t v[128];
      tc_fence_after();
      tmem_ld32(tS, v);
      tmem_ld32(tS + 32, v + 32);
      tmem_ld32(tS + 64, v + 64);
      tmem_ld32(tS + 96, v + 96);
      tc_wait_ld();
      if (masked) {
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4)
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (!((vm[w4] >> k) & 1u)) v[32 * w4 + k] = 0xff800000u;  // -inf
      }
      float mx8[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) mx8[c] = fmaxf(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]));
#pragma unroll
      for (int k = 16; k < 128; k += 16) {
#pragma unroll
        for (int c = 0; c < 8; ++c) mx8[c] = max3(mx8[c], __uint_as_float(v[k + 2 * c]), __uint_as_float(v[k + 2 * c + 1]));
      }
      const float mx = fmaxf(fmaxf(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[5])), fmaxf(mx8[6], mx8[7]));
      const float mx_s = mx * M.scale_log2;
      if (j == 0) {
        m_st = mx_s;
      } else {
        const bool grow = mx_s > m_st + 8.f;
        if (__any_sync(0xffffffffu, grow)) {
          const float m_new = grow ? mx_s : m_st;
          const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m_st - m_new);
#pragma unroll 1
          for (int c16 = 0; c16 < 8; ++c16) {
            uint32_t w[16];
            tmem_ld16(tO + c16 * 16, w);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 16; ++k) w[k] = __float_as_uint(__uint_as_float(w[k]) * alpha);
            tmem_st16p(tO + c16 * 16, w);
          }
          l_run *= alpha;
          m_st = m_new;
        }
      }
      const float m_use = (m_st == -INFINITY) ? 0.f : m_st;
      // probabilities -> bf16 pairs written over the first 64 columns of S (packed two-wide fp32 math)
      const float2 sc2 = make_float2(M.scale_log2, M.scale_log2), nm2 = make_float2(-m_use, -m_use);
      float2 acc[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[c] = make_float2(0.f, 0.f);
      constexpr int QPP = 4 / P_PARTS;  // 32-key quarters per posted part
#pragma unroll
      for (int part = 0; part < 4; ++part) {
#pragma unroll
        for (int k = part * 16; k < part * 16 + 16; ++k) {
          const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[2 * k]), __uint_as_float(v[2 * k + 1])), sc2, nm2);
          const float2 e = make_float2(fast_exp2(x.x), fast_exp2(x.y));
          v[k] = pack_bf16x2(e.x, e.y);
          // the row sum takes the fp32 values before their rounding to bf16 (summing the rounded ones instead
          // costs one more ALU op per key and 7-8 % of the kernel's time; the difference shows only for nearly
          // one-hot rows, where it is bounded by 2^-9 max|v|)
          acc[k & 3] = __fadd2_rn(acc[k & 3], e);
          if (part > 0 && (part % QPP) == 0 && k == part * 16 + 7) {
            // post the previous half: its TMEM stores have landed by now, so the wait costs nothing
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_PFULL + P_PARTS * i + part / QPP - 1));  // one arrival per warp
          }
        }
        tmem_st16p(tS + part * 16, v + part * 16);
        if (part == 3) {
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(BAR_PFULL + P_PARTS * i + P_PARTS - 1));
        }
      }
      const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
      l_run += (a01.x + a01.y) + (a23.x + a23.y);
    }
    // ---- epilogue: O / l -> global ----
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_OFINAL + i), 0));
    if (!ok && lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, r, b, 40 + i);
    tc_fence_after();
    const float l_tot = l_run;
    if constexpr (PREFIX) {
      // partial for the split-K combine: row = (request, head), unnormalised o with its (m, l)
      const int rq = r + 16 * i + (rr >> 3);
      const bool row_ok = ok && rq < p.b.B;
      const int64_t prow = ((int64_t)rq * M.Hq + kh * M.G + (rr & 7)) * p.max_splits + blockIdx.x;
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t w[32];
        tmem_ld32(tO + c4 * 32, w);
        tc_wait_ld();
        if (row_ok) {
          float4* dst = reinterpret_cast<float4*>(p.part_o + prow * HD + c4 * 32);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            dst[k] = make_float4(__uint_as_float(w[4 * k]), __uint_as_float(w[4 * k + 1]), __uint_as_float(w[4 * k + 2]),
                                 __uint_as_float(w[4 * k + 3]));
        }
      }
      if (row_ok) p.part_ml[prow] = make_float2(m_st, l_tot);
    } else {
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      const bool row_ok = ok && ri < n;
      const int64_t orow = ((int64_t)(t0 + ri) * M.Hq + (h0 + i));
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t w[32];
        tmem_ld32(tO + c4 * 32, w);
        tc_wait_ld();
        if (row_ok) {
          const int col0 = c4 * 32;
          if (M.out_fp32) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow * HD + col0);
#pragma unroll
            for (int k = 0; k < 8; ++k)
              dst[k] = make_float4(__uint_as_float(w[4 * k]) * inv, __uint_as_float(w[4 * k + 1]) * inv,
                                   __uint_as_float(w[4 * k + 2]) * inv, __uint_as_float(w[4 * k + 3]) * inv);
          } else {
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow * HD + col0);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              uint4 u;
              u.x = pack_bf16x2(__uint_as_float(w[8 * k]) * inv, __uint_as_float(w[8 * k + 1]) * inv);
              u.y = pack_bf16x2(__uint_as_float(w[8 * k + 2]) * inv, __uint_as_float(w[8 * k + 3]) * inv);
              u.z = pack_bf16x2(__uint_as_float(w[8 * k + 4]) * inv, __uint_as_float(w[8 * k + 5]) * inv);
              u.w = pack_bf16x2(__uint_as_float(w[8 * k + 6]) * inv, __uint_as_float(w[8 * k + 7]) * inv);
              dst[k] = u;
            }
          }
        }
      }
      if (row_ok && p.lse) p.lse[orow] = l_tot > 0.f ? (m_st + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    }
  }

  // ---- teardown: everyone is done with TMEM before it is released ----
  linger_after_error(p.err);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
  if (traced && threadIdx.x == 0) {
    unsigned sm;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
    p.trace[trace_slot * 4 + 1] = global_timer_ns();
    p.trace[trace_slot * 4 + 2] = sm;
    p.trace[trace_slot * 4 + 3] = ((long long)r << 32) | (unsigned)b;
  }
}



// ---------------------------------------------------------------------------------------------------------
// SWA layers, tokens whose whole window lies inside the chunk (paper Sec. 2.1: an SWA layer attends to W keys
// only, so the work per token is constant and the layer is bound by moving Q and the output, not by the
// tensor cores).  GQA-packed: one block = TQ = 128 / G consecutive tokens x the G query heads of one KV head
// (128 rows), against the TQ + W - 1 keys those tokens can see, rounded up to N.  One S MMA group, one
// softmax, one PV MMA group; K and V are loaded once for all G heads.  TMEM: S in columns [0, N), P over its
// first N / 2 columns, O in columns [128, 256) (it overlaps the tail of S, which is dead by then), 256 columns
// per block so that two blocks share an SM and hide each other's load and hand-off latencies.
template <int G>
struct PackedCfg {
  static constexpr int TQ = 128 / G;                          // tokens per block
  static constexpr int N = ((TQ + 128 - 1 + 15) / 16) * 16;   // keys per block for W <= 128
  static constexpr int KV_HALF = N * 128;                     // bytes of one 64-element half of the K or V tile
  static constexpr int KV_BYTES = 2 * KV_HALF;
  static constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = OFF_K + KV_BYTES;
  static constexpr int SMEM = OFF_V + KV_BYTES + 1024;
  static constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
};

template <int G>
__global__ void __launch_bounds__(192, 2)
prefill_swa_packed_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, const PrefillParams p, const int first_tok) {
  using C = PackedCfg<G>;
  constexpr int TQ = C::TQ, N = C::N;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[6];
  __shared__ uint32_t tmem_base_slot;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const ModelParams& M = p.m;
  enum { B_Q = 0, B_K = 1, B_V = 2, B_S = 3, B_P = 4, B_O = 5 };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kh = blockIdx.x, r = blockIdx.z;
  const int t0 = p.b.q_indptr[r];
  const int n = p.b.q_indptr[r + 1] - t0;
  const int i0 = first_tok + (int)blockIdx.y * TQ;  // first chunk-relative token of this block
  if (i0 >= n) return;
  if (*reinterpret_cast<volatile int32_t*>(p.err) != 0) return;
  const int key0 = i0 - (M.W - 1);  // chunk-relative index of key column 0 (>= 0 by construction)

  auto bar = [&](int i) { return smem_u32(&bars[i]); };
  if (threadIdx.x == 0) {
    mbar_init(bar(B_Q), 1);
    mbar_init(bar(B_K), 1);
    mbar_init(bar(B_V), 1);
    mbar_init(bar(B_S), 1);
    mbar_init(bar(B_P), 4);
    mbar_init(bar(B_O), 1);
    mbar_fence_init();
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(256)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;

  if (warp == 4) {
    if (lane == 0) {
      mbar_arrive_expect_tx(bar(B_Q), TILE_BYTES);
      mbar_arrive_expect_tx(bar(B_K), C::KV_BYTES);
      mbar_arrive_expect_tx(bar(B_V), C::KV_BYTES);
      for (int hf = 0; hf < 2; ++hf) {
        tma_load_3d(sbase + C::OFF_Q + hf * HALF_BYTES, &tm_q, bar(B_Q), hf * 64, kh * G, t0 + i0);
        tma_load_3d(sbase + C::OFF_K + hf * C::KV_HALF, &tm_k, bar(B_K), hf * 64, kh, t0 + key0);
      }
      for (int hf = 0; hf < 2; ++hf) tma_load_3d(sbase + C::OFF_V + hf * C::KV_HALF, &tm_v, bar(B_V), hf * 64, kh, t0 + key0);
    }
  } else if (warp == 5) {
    if (lane == 0) {
      bool ok = mbar_wait(bar(B_Q), 0) && mbar_wait(bar(B_K), 0);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint32_t qoff = (ks >> 2) * HALF_BYTES + (ks & 3) * 32, koff = (ks >> 2) * C::KV_HALF + (ks & 3) * 32;
          tc_mma_ss(tmem, smem_desc(sbase + C::OFF_Q + qoff, 16), smem_desc(sbase + C::OFF_K + koff, 16), C::IDESC_S, ks > 0);
        }
        tc_commit(bar(B_S));
        ok = mbar_wait(bar(B_V), 0) && mbar_wait(bar(B_P), 0);
      }
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < N / 16; ++kk)
          tc_mma_ts(tmem + 128, tmem + kk * 8, smem_desc(sbase + C::OFF_V + kk * 2048, C::KV_HALF), IDESC_PV, kk > 0);
      } else {
        record_error(p.err, HSWA_ERR_TIMEOUT, r, i0, 50);
      }
      tc_commit(bar(B_O));
    }
  } else {
    const int rr = warp * 32 + lane;             // row = TMEM lane
    const int tl = rr / G, g = rr % G;           // local token, head in group
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    const uint32_t tS = tmem + lane_addr, tO = tmem + lane_addr + 128;
    const int lo = tl, hi = tl + M.W;            // visible key columns [lo, hi)
    bool ok = __all_sync(0xffffffffu, mbar_wait(bar(B_S), 0));
    float mx = -INFINITY, l_run = 0.f, m_use = 0.f;
    if (ok) {
      tc_fence_after();
      // two passes over the N score columns in chunks of 32 (the last chunk is 16 or 32 wide)
      constexpr int CH = (N + 31) / 32;
#pragma unroll 1
      for (int c = 0; c < CH; ++c) {
        uint32_t v[32];
        const bool wide = (c + 1) * 32 <= N;
        if (wide) tmem_ld32(tS + c * 32, v); else tmem_ld16(tS + c * 32, v);
        tc_wait_ld();
        const int cnt = wide ? 32 : 16;
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          const int col = c * 32 + k;
          if (k < cnt && col >= lo && col < hi) mx = fmaxf(mx, __uint_as_float(v[k]));
        }
      }
      m_use = mx == -INFINITY ? 0.f : mx * M.scale_log2;
#pragma unroll 1
      for (int c = 0; c < CH; ++c) {
        uint32_t v[32];
        const bool wide = (c + 1) * 32 <= N;
        if (wide) tmem_ld32(tS + c * 32, v); else tmem_ld16(tS + c * 32, v);
        tc_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int col = c * 32 + 2 * k;
          float p0 = fast_exp2(__uint_as_float(v[2 * k]) * M.scale_log2 - m_use);
          float p1 = fast_exp2(__uint_as_float(v[2 * k + 1]) * M.scale_log2 - m_use);
          p0 = (col >= lo && col < hi) ? p0 : 0.f;
          p1 = (col + 1 >= lo && col + 1 < hi) ? p1 : 0.f;
          pk[k] = pack_bf16x2(p0, p1);
          if (wide || k < 8) l_run += p0 + p1;
        }
        if (wide) tmem_st16p(tS + c * 16, pk); else tmem_st8(tS + c * 16, pk);
      }
      tc_wait_st();
    } else if (lane == 0) {
      record_error(p.err, HSWA_ERR_TIMEOUT, r, i0, 51);
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(B_P));
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_O), 0));
    tc_fence_after();
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    const bool row_ok = ok && (i0 + tl) < n;
    const int64_t orow = (int64_t)(t0 + i0 + tl) * M.Hq + kh * G + g;
#pragma unroll 1
    for (int c4 = 0; c4 < 4; ++c4) {
      uint32_t v[32];
      tmem_ld32(tO + c4 * 32, v);
      tc_wait_ld();
      if (row_ok) {
        if (M.out_fp32) {
          float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow * HD + c4 * 32);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            dst[k] = make_float4(__uint_as_float(v[4 * k]) * inv, __uint_as_float(v[4 * k + 1]) * inv,
                                 __uint_as_float(v[4 * k + 2]) * inv, __uint_as_float(v[4 * k + 3]) * inv);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow * HD + c4 * 32);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(v[8 * k]) * inv, __uint_as_float(v[8 * k + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(v[8 * k + 2]) * inv, __uint_as_float(v[8 * k + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(v[8 * k + 4]) * inv, __uint_as_float(v[8 * k + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(v[8 * k + 6]) * inv, __uint_as_float(v[8 * k + 7]) * inv);
            dst[k] = w;
          }
        }
      }
    }
    if (row_ok && p.lse) p.lse[orow] = l_run > 0.f ? (m_use + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
  }
}

template <int G>
cudaError_t launch_packed(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const PrefillParams& p,
                          int first_tok, cudaStream_t s) {
  using C = PackedCfg<G>;
  auto kern = prefill_swa_packed_kernel<G>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return e;
  const int tiles = (p.max_q_len - first_tok + C::TQ - 1) / C::TQ;
  dim3 grid(p.m.Hkv, tiles, p.b.B);
  kern<<<grid, 192, C::SMEM, s>>>(tm_q, tm_k, tm_v, p, first_tok);
  return cudaGetLastError();
}


// ---------------------------------------------------------------------------------------------------------
// SWA layers, GQA group of 8, window 128, tokens whose whole window lies inside the chunk: streaming kernel.
// Persistent blocks walk long runs of 16-token sub-tiles of one (request, KV head) stream.  A sub-tile is 16
// tokens x 8 heads (128 rows) against the 144 keys its tokens can see (16 + 127, rounded up to 16).  K and V live
// in a CIRCULAR buffer of 256 key rows (16 slots of 16): sub-tile s (tokens [i, i + 16), i = 128 + 16 s) needs
// keys [i - 128, i + 16), of which only [i, i + 16) are new, so every sub-tile loads its Q tile (32 KB), ONE
// 16-key piece of K and of V (4 KB each) into the slot of the keys that fell out of every window eight sub-tiles
// ago, and stores 32 KB: each key is read once per stream.  The 144-key slice starts at row (i - 128) mod 256 and
// may wrap: the S MMA is then issued as two groups (N1 + N2 keys, adjacent TMEM columns), and the PV k-steps take
// their 16 rows from wherever they are.
// Roles: warps 0-3 and 4-7 are two softmax warpgroups that alternate sub-tiles, each with its own Q buffer and its
// own 256 TMEM columns (S in [0, 144), P over its first 72 columns, O in [128, 256)); warp 8 issues the TMA loads,
// warp 9 the S MMAs, warp 11 the PV MMAs, warp 10 the TMA stores of staged output tiles.  All of them count
// sub-tiles with one per-block counter g, so the Q load, the S MMA, the softmax, the PV MMA and the store of
// neighbouring sub-tiles overlap.
namespace stream {
constexpr int SUB = 16;                         // tokens per sub-tile
constexpr int N = 144;                          // keys per sub-tile
constexpr int KV_ROWS = 256;
constexpr int KV_HALF = KV_ROWS * 128;          // bytes of one 64-element half
constexpr int KV_BYTES = 2 * KV_HALF;           // 64 KB
constexpr int QBUF = 2;                         // Q tiles in flight (a buffer is free as soon as its S MMA has run)
constexpr int OFF_Q = 0, OFF_K = QBUF * TILE_BYTES, OFF_V = OFF_K + KV_BYTES, OFF_STAGE = OFF_V + KV_BYTES;
constexpr int SMEM = OFF_STAGE + TILE_BYTES + 1024;   // 225 KB: Q 64, K 64, V 64, output staging 32
constexpr int SLOTS = 16;
constexpr int THREADS = 384;  // 8 softmax warps + producer + S issuer + output store warp + PV issuer
// (registers move between the roles as in the tile kernel: REGS_SERVICE, REGS_SOFTMAX)
enum { B_QFULL = 0, B_QEMPTY = 2, B_SFULL = 4, B_PFULL = 6, B_OFULL = 8, B_OFREE = 10, B_STAGED = 12,
       B_PHALF = 13 /* the first 64 keys of P posted */, B_DRAIN = 15 /* every MMA of a finished stream has run */,
       B_STGFREE = 16 /* two: staged tiles use them in turn */, B_KP = 18, B_VP = 18 + SLOTS, NBARS = 18 + 2 * SLOTS };
// instruction descriptor of an S MMA over n keys (a multiple of 16)
__device__ __forceinline__ uint32_t idesc_s(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// The sub-tiles a block walks: units [u, u_end) of the flattened (stream, sub-tile) space, empty ones skipped.
struct Walker {
  const int32_t* q_indptr;
  int Hkv, ns_max, u, u_end, st, sidx, cur_stream, r_cur, kh_cur, t0, n, ns;
  bool fresh;  // the sub-tile returned last is the first this block takes from its stream
  __device__ Walker(const PrefillParams& p_, int ns_max_, int u0, int u1)
      : q_indptr(p_.b.q_indptr), Hkv(p_.m.Hkv), ns_max(ns_max_), u(u0), u_end(u1), st(u0 / ns_max_), sidx(u0 % ns_max_),
        cur_stream(-1), r_cur(0), kh_cur(0), t0(0), n(0), ns(0), fresh(false) {}
  // next non-empty sub-tile: request r, KV head kh, first chunk-relative token i; false when the range is used up
  __device__ bool next(int& r, int& kh, int& i) {
    while (u < u_end) {
      bool changed = false;
      if (st != cur_stream) {
        cur_stream = st;
        r_cur = st / Hkv;
        kh_cur = st - r_cur * Hkv;
        t0 = q_indptr[r_cur];
        n = q_indptr[r_cur + 1] - t0;
        ns = n > 128 ? (n - 128 + SUB - 1) / SUB : 0;
        changed = true;
      }
      if (sidx >= ns) {  // nothing (left) in this stream: jump to the next one
        u += ns_max - sidx;
        ++st;
        sidx = 0;
        continue;
      }
      r = r_cur;
      kh = kh_cur;
      i = 128 + sidx * SUB;
      fresh = changed;
      ++u;
      if (++sidx == ns_max) {
        ++st;
        sidx = 0;
      }
      return true;
    }
    return false;
  }
};
// Number of non-empty sub-tiles among units [u0, u1).
__device__ inline int count_sub_tiles(const PrefillParams& p, int ns_max, int u0, int u1) {
  int total = 0;
  for (int st = u0 / ns_max; st * ns_max < u1; ++st) {
    const int r = st / p.m.Hkv, n = p.b.q_indptr[r + 1] - p.b.q_indptr[r];
    const int ns = n > 128 ? (n - 128 + SUB - 1) / SUB : 0;
    const int lo = max(u0, st * ns_max), hi = min(u1, st * ns_max + ns);
    total += max(0, hi - lo);
  }
  return total;
}
}  // namespace stream

__global__ void __launch_bounds__(stream::THREADS, 1)
prefill_swa_stream_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k16,
                          const __grid_constant__ CUtensorMap tm_v16, const __grid_constant__ CUtensorMap tm_out,
                          const PrefillParams p, const int ns_max, const int units_per_block, const int tma_out) {
  using namespace stream;
  constexpr int G = 8;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[NBARS];
  __shared__ uint32_t tmem_base_slot;
  // what the softmax warps need to know about a sub-tile, written by the producer when it issues the Q load:
  // {first token (row of q / out), valid tokens, KV head, index among the staged tiles or -1}
  __shared__ int4 tile_info[4];
  __shared__ int blk_abort;  // a wait of a softmax warp ran out: both warpgroups stop at their next sub-tile
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const ModelParams& M = p.m;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_units = p.b.B * M.Hkv * ns_max;
  const int u0 = blockIdx.x * units_per_block, u1 = min(u0 + units_per_block, total_units);
  if (u0 >= u1) return;
  if (*reinterpret_cast<volatile int32_t*>(p.err) != 0) return;

  auto bar = [&](int i) { return smem_u32(&bars[i]); };
  if (threadIdx.x == 0) {
    blk_abort = 0;
    mbar_init(bar(B_STAGED), 4);
    mbar_init(bar(B_STGFREE), 1);
    mbar_init(bar(B_STGFREE + 1), 1);
    mbar_init(bar(B_DRAIN), 1);
    for (int q = 0; q < QBUF; ++q) {
      mbar_init(bar(B_QFULL + q), 1);
      mbar_init(bar(B_QEMPTY + q), 1);
    }
    for (int u = 0; u < 2; ++u) {
      mbar_init(bar(B_SFULL + u), 1);
      mbar_init(bar(B_PFULL + u), 4);
      mbar_init(bar(B_PHALF + u), 4);
      mbar_init(bar(B_OFULL + u), 1);
      mbar_init(bar(B_OFREE + u), 4);
    }
    for (int j = 0; j < SLOTS; ++j) {
      mbar_init(bar(B_KP + j), 1);
      mbar_init(bar(B_VP + j), 1);
    }
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;

  // Registers move from the four service warps (one warpgroup) to the two softmax warpgroups, whose threads hold a
  // whole row of 144 scores plus its exponentials' state: 8 x 32 x 224 + 4 x 32 x 56 = 384 x 168.
  // (each role's branch changes its own allotment: the compiler budgets a branch by the instruction that dominates it)
  if (warp == 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= TMA producer =======================
    if (lane == 0) {
      Walker w(p, ns_max, u0, u1);
      int r, kh, i, n_staged = 0, n_switch = 0;
      bool ok = true;
      // one 16-key piece (keys [key, key + 16) of the chunk) of K and of V into its slot
      auto load_piece = [&](int t0, int kh_, int key) {
        const int slot = (key / SUB) % SLOTS;
        mbar_arrive_expect_tx(bar(B_KP + slot), 2 * SUB * 128);
        mbar_arrive_expect_tx(bar(B_VP + slot), 2 * SUB * 128);
        for (int hf = 0; hf < 2; ++hf) {
          tma_load_3d(sbase + stream::OFF_K + hf * KV_HALF + slot * SUB * 128, &tm_k16, bar(B_KP + slot), hf * 64, kh_, t0 + key);
          tma_load_3d(sbase + stream::OFF_V + hf * KV_HALF + slot * SUB * 128, &tm_v16, bar(B_VP + slot), hf * 64, kh_, t0 + key);
        }
      };
      for (int g = 0; ok && w.next(r, kh, i); ++g) {
        const int qb = g % QBUF;
        // Q buffer qb is free once S(g - 2) has run; in-order MMA execution then also has S(g - 8) and PV(g - 8)
        // behind it, which were the last readers of the slot this sub-tile's piece goes to
        if (g >= QBUF && !mbar_wait(bar(B_QEMPTY + qb), ((g / QBUF) - 1) & 1)) {
          record_error(p.err, HSWA_ERR_TIMEOUT, r, g, 70);
          ok = false;
          break;
        }
        if (w.fresh) {
          // a new stream: its first eight pieces go to slots the previous stream's last sub-tiles may still be reading.
          // The PV issuer commits to a barrier of its own at every such switch, so this thread sees each of that
          // barrier's phases in turn.  (The per-sub-tile barriers will not do: a parity wait tells a phase only from its
          // neighbours, and this thread may be one phase behind or two ahead of them.)
          if (g > 0 && !mbar_wait(bar(B_DRAIN), n_switch++ & 1)) {
            record_error(p.err, HSWA_ERR_TIMEOUT, r, g, 71);
            ok = false;
            break;
          }
          for (int key = i - 128; key < i; key += SUB) load_piece(w.t0, kh, key);
        }
        // entry g & 3 was last read for sub-tile g - 4, whose accumulator S(g - 2) has waited for
        {
          const bool staged_tile = tma_out && i + SUB <= w.n;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(&tile_info[g & 3])), "r"(w.t0 + i),
                       "r"(min(SUB, w.n - i)), "r"(kh), "r"(staged_tile ? n_staged : -1)
                       : "memory");
          if (staged_tile) ++n_staged;
          __threadfence_block();
        }
        mbar_arrive_expect_tx(bar(B_QFULL + qb), TILE_BYTES);
        for (int hf = 0; hf < 2; ++hf)
          tma_load_3d(sbase + stream::OFF_Q + qb * TILE_BYTES + hf * HALF_BYTES, &tm_q, bar(B_QFULL + qb), hf * 64, kh * G, w.t0 + i);
        load_piece(w.t0, kh, i);
      }
    }
  } else if (warp == 9) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= MMA issuers =======================
    // Warp 9 issues the S MMAs, warp 11 the PV MMAs.  Each has one chain of barriers to wait for, in order, so it can
    // sleep in the wait; a single thread that polls both chains in turn spends more time polling (a test of a
    // completed mbarrier costs 100-250 clocks while the tensor cores use shared memory) than issuing.  The whole
    // warp walks the loop converged (waits, descriptor arithmetic); one elected lane issues.  Descriptors are
    // built once and advanced by additions.  The tensor pipe runs the two warps' MMAs in the order they arrive;
    // every dependence between them goes through a barrier (P posted, accumulator read out).
    Walker w(p, ns_max, u0, u1);
    uint32_t par = 0;  // per slot: parity of the fill to wait for next
    int r, kh, i;
    bool ok = true;
    const uint64_t dQ0 = smem_desc(sbase + stream::OFF_Q, 16), dQ1 = smem_desc(sbase + stream::OFF_Q + TILE_BYTES, 16);
    const uint64_t dK0 = smem_desc(sbase + stream::OFF_K, 16);
    auto wait_piece = [&](int key) {
      const int slot = (key / SUB) % SLOTS;
      const bool got = mbar_wait(bar(B_KP + slot), (par >> slot) & 1u);
      par ^= 1u << slot;
      return got;
    };
    for (int g = 0; ok && w.next(r, kh, i); ++g) {
      const int u = g & 1, start = (i - 128) & (SLOTS * SUB - 1);  // first row of the slice in the circular buffer
      const int n1 = min(N, SLOTS * SUB - start), n2 = N - n1;
      const uint64_t dq = (g % QBUF) ? dQ1 : dQ0, dk = desc_advance(dK0, start * 128);
      const uint32_t id1 = idesc_s(n1), id2 = idesc_s(n2);
      // the accumulator of sub-tile g - 2 read out, Q(g) in shared memory, the keys: this sub-tile's own piece and,
      // for the first sub-tile of a stream, the eight before it
      if (g >= 2) ok = mbar_wait(bar(B_OFREE + u), ((g >> 1) - 1) & 1);
      if (ok) ok = mbar_wait(bar(B_QFULL + g % QBUF), (g / QBUF) & 1);
      if (w.fresh)
        for (int key = i - 128; key < i && ok; key += SUB) ok = wait_piece(key);
      if (ok) ok = wait_piece(i);
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks)
          tc_mma_ss(tmem + u * 256, desc_advance(dq, (ks >> 2) * HALF_BYTES + (ks & 3) * 32),
                    desc_advance(dk, (ks >> 2) * KV_HALF + (ks & 3) * 32), id1, ks > 0);
        if (n2 > 0) {  // the slice wraps: its last n2 keys are the buffer's first rows
#pragma unroll
          for (int ks = 0; ks < HD / 16; ++ks)
            tc_mma_ss(tmem + u * 256 + n1, desc_advance(dq, (ks >> 2) * HALF_BYTES + (ks & 3) * 32),
                      desc_advance(dK0, (ks >> 2) * KV_HALF + (ks & 3) * 32), id2, ks > 0);
        }
        tc_commit(bar(B_SFULL + u));
        tc_commit(bar(B_QEMPTY + g % QBUF));  // Q(g) has been consumed once these MMAs are done
      }
      __syncwarp();
    }
    if (!ok && lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, blockIdx.x, 0, 72);
  } else if (warp == 11) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    Walker w(p, ns_max, u0, u1);
    uint32_t par = 0;
    int r, kh, i;
    bool ok = true;
    const uint64_t dV0 = smem_desc(sbase + stream::OFF_V, KV_HALF);
    auto wait_piece = [&](int key) {
      const int slot = (key / SUB) % SLOTS;
      const bool got = mbar_wait(bar(B_VP + slot), (par >> slot) & 1u);
      par ^= 1u << slot;
      return got;
    };
    for (int g = 0; ok && w.next(r, kh, i); ++g) {
      const int u = g & 1, start = (i - 128) & (SLOTS * SUB - 1);
      if (w.fresh) {
        if (g > 0) {  // every MMA of the stream that has just ended: the producer waits for this before it reuses slots
          if (elect_one()) tc_commit(bar(B_DRAIN));
          __syncwarp();
        }
        for (int key = i - 128; key < i && ok; key += SUB) ok = wait_piece(key);
      }
      // the first 64 keys of P are posted while the rest of the row's exponentials run
      if (ok) ok = mbar_wait(bar(B_PHALF + u), (g >> 1) & 1);
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int row = (start + kk * 16) & (SLOTS * SUB - 1);
          tc_mma_ts(tmem + u * 256 + 128, tmem + u * 256 + kk * 8, desc_advance(dV0, row * 128), IDESC_PV, kk > 0);
        }
      }
      __syncwarp();
      ok = wait_piece(i);
      if (ok) ok = mbar_wait(bar(B_PFULL + u), (g >> 1) & 1);
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kk = 4; kk < N / 16; ++kk) {
          const int row = (start + kk * 16) & (SLOTS * SUB - 1);
          tc_mma_ts(tmem + u * 256 + 128, tmem + u * 256 + kk * 8, desc_advance(dV0, row * 128), IDESC_PV, 1u);
        }
        tc_commit(bar(B_OFULL + u));
      }
      __syncwarp();
    }
    if (!ok && lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, blockIdx.x, 1, 72);
  } else if (warp == 10) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE) : "memory");
    // ======================= output store warp =======================
    if (lane == 0 && tma_out) {
      Walker w(p, ns_max, u0, u1);
      int r, kh, i, n_staged = 0;
      bool ok = true;
      for (int g = 0; ok && w.next(r, kh, i); ++g) {
        if (i + SUB > w.n) continue;  // a ragged last sub-tile is stored directly by its warpgroup
        ok = mbar_wait(bar(B_STAGED), n_staged & 1);
        if (!ok) break;
        for (int hf = 0; hf < 2; ++hf)
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_out),
                       "r"(sbase + stream::OFF_STAGE + hf * HALF_BYTES), "r"(hf * 64), "r"(kh * G), "r"(w.t0 + i)
                       : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // shared memory has been read
        mbar_arrive(bar(B_STGFREE + (n_staged & 1)));
        ++n_staged;
      }
      if (!ok) record_error(p.err, HSWA_ERR_TIMEOUT, blockIdx.x, n_staged, 73);
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores have landed
    }
  } else {
    // ======================= softmax warpgroups: warps 0-3 take even sub-tiles, 4-7 odd =======================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX) : "memory");
    const int u = warp >> 2;
    const int rr = (warp & 3) * 32 + lane;  // row = TMEM lane
    const int tl = rr / G, gh = rr % G;     // token within the sub-tile, head within the group
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_addr + u * 256, tO = tS + 128;
    const int lo = tl + 129 - M.W, hi = tl + 129;  // visible key columns [lo, hi) of the 144-key slice
    const int n_total = count_sub_tiles(p, ns_max, u0, u1);
    for (int g = u; g < n_total && *reinterpret_cast<volatile int*>(&blk_abort) == 0; g += 2) {
      const uint32_t par = (g >> 1) & 1;
      bool ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SFULL + u), par));
      float l_run = 0.f, m_use = 0.f;
      if (ok) {
        tc_fence_after();
        // the row's 144 scores in one round trip to TMEM; only columns [0, 32) and [128, 144) can be masked
        uint32_t v[N];
        tmem_ld32(tS, v);
        tmem_ld32(tS + 32, v + 32);
        tmem_ld32(tS + 64, v + 64);
        tmem_ld32(tS + 96, v + 96);
        tmem_ld16(tS + 128, v + 128);
        tc_wait_ld();
        {
          const uint32_t head_mask = lo >= 32 ? 0u : (0xffffffffu << (lo < 0 ? 0 : lo));     // columns 0-31: col >= lo
          const int t = hi - 128;                                                               // columns 128-143: col < hi
          const uint32_t tail_mask = t >= 16 ? 0xffffu : (t <= 0 ? 0u : ((1u << t) - 1u));
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (!((head_mask >> k) & 1u)) v[k] = 0xff800000u;
#pragma unroll
          for (int k = 0; k < 16; ++k)
            if (!((tail_mask >> k) & 1u)) v[128 + k] = 0xff800000u;
        }
        float mx4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) mx4[c] = fmaxf(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]));
#pragma unroll
        for (int k = 8; k < N; k += 8) {
#pragma unroll
          for (int c = 0; c < 4; ++c) mx4[c] = max3(mx4[c], __uint_as_float(v[k + 2 * c]), __uint_as_float(v[k + 2 * c + 1]));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        m_use = mx == -INFINITY ? 0.f : mx * M.scale_log2;
        const float2 sc2 = make_float2(M.scale_log2, M.scale_log2), nm2 = make_float2(-m_use, -m_use);
        float2 acc[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[c] = make_float2(0.f, 0.f);
        auto exps = [&](int k0, int k1) {
#pragma unroll
          for (int k = k0; k < k1; ++k) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[2 * k]), __uint_as_float(v[2 * k + 1])), sc2, nm2);
            const float2 e = make_float2(fast_exp2(x.x), fast_exp2(x.y));  // masked columns: 2^(-inf) = 0
            v[k] = pack_bf16x2(e.x, e.y);
            acc[k & 3] = __fadd2_rn(acc[k & 3], e);  // row sum of the fp32 values, not of the rounded ones
          }
        };
        // P of the first 64 keys is stored while the next exponentials run and posted on its own, so that the PV
        // MMAs of those keys run under the rest of the row
        exps(0, 32);
        tmem_st32(tS, v);
        exps(32, 44);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_PHALF + u));
        exps(44, N / 2);
        const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
        l_run = (a01.x + a01.y) + (a23.x + a23.y);
        tmem_st32(tS + 32, v + 32);
        tmem_st8(tS + 64, v + 64);
        tc_wait_st();
      } else {
        if (lane == 0) {
          record_error(p.err, HSWA_ERR_TIMEOUT, blockIdx.x, g, 74);
          mbar_arrive(bar(B_PHALF + u));
          *reinterpret_cast<volatile int*>(&blk_abort) = 1;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL + u));
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_OFULL + u), par));
      tc_fence_after();
      // (the producer wrote the entry before it issued this sub-tile's Q load, which S(g) has consumed)
      int4 info;
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(info.x), "=r"(info.y), "=r"(info.z), "=r"(info.w)
                   : "r"(smem_u32(&tile_info[g & 3]))
                   : "memory");
      const int my_stage_idx = info.w;
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      const bool row_ok = ok && tl < info.y;
      const int64_t orow = (int64_t)(info.x + tl) * M.Hq + info.z * G + gh;
      const bool staged = my_stage_idx >= 0 && ok;
      uint8_t* stage = smem + stream::OFF_STAGE;
      {
        uint32_t wv[128];  // the whole accumulator row in one round trip
        tmem_ld32(tO, wv);
        tmem_ld32(tO + 32, wv + 32);
        tmem_ld32(tO + 64, wv + 64);
        tmem_ld32(tO + 96, wv + 96);
        tc_wait_ld();
        // the accumulator has been read out: the MMA warp may reuse this TMEM buffer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_OFREE + u));
        if (staged) {
          // staged sub-tiles use the single staging tile in order: wait until the previous one's store has read it
          // (the row is scaled and packed first: that work needs no staging tile)
#pragma unroll
          for (int c = 0; c < 64; ++c) wv[c] = pack_bf16x2(__uint_as_float(wv[2 * c]) * inv, __uint_as_float(wv[2 * c + 1]) * inv);
          // Staged tile k waits until the store of tile k - 1 has read the staging tile.  The two warpgroups mostly
          // alternate, so this warpgroup saw the barrier of tile k - 2 at best: with ONE barrier it would wait for
          // a phase without having seen the one before, and a parity wait passes at once when the barrier is a
          // whole phase behind (a late store warp: corrupted tiles, miscounted arrivals).  With two barriers used
          // in turn, the phase before the awaited one belongs to tile k - 3, whose store this warpgroup's own
          // earlier wait (for k - 3 or k - 2) has already covered.
          if (my_stage_idx > 0 &&
              !__all_sync(0xffffffffu, mbar_wait(bar(B_STGFREE + ((my_stage_idx - 1) & 1)), ((my_stage_idx - 1) >> 1) & 1))) {
            if (lane == 0) record_error(p.err, HSWA_ERR_TIMEOUT, blockIdx.x, g, 75);
          }
#pragma unroll
          for (int chunk = 0; chunk < 16; ++chunk)  // 16-byte chunks of the 256-byte bf16 row
            *reinterpret_cast<uint4*>(stage + (chunk >> 3) * HALF_BYTES + swz128(rr, chunk & 7)) =
                make_uint4(wv[4 * chunk], wv[4 * chunk + 1], wv[4 * chunk + 2], wv[4 * chunk + 3]);
        } else if (row_ok) {
          if (M.out_fp32) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow * HD);
#pragma unroll
            for (int k = 0; k < 32; ++k)
              dst[k] = make_float4(__uint_as_float(wv[4 * k]) * inv, __uint_as_float(wv[4 * k + 1]) * inv,
                                   __uint_as_float(wv[4 * k + 2]) * inv, __uint_as_float(wv[4 * k + 3]) * inv);
          } else {
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow * HD);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              uint4 x;
              x.x = pack_bf16x2(__uint_as_float(wv[8 * k]) * inv, __uint_as_float(wv[8 * k + 1]) * inv);
              x.y = pack_bf16x2(__uint_as_float(wv[8 * k + 2]) * inv, __uint_as_float(wv[8 * k + 3]) * inv);
              x.z = pack_bf16x2(__uint_as_float(wv[8 * k + 4]) * inv, __uint_as_float(wv[8 * k + 5]) * inv);
              x.w = pack_bf16x2(__uint_as_float(wv[8 * k + 6]) * inv, __uint_as_float(wv[8 * k + 7]) * inv);
              dst[k] = x;
            }
          }
        }
      }
      if (row_ok && p.lse) p.lse[orow] = l_run > 0.f ? (m_use + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
      // hand the staged tile to the store warp
      if (staged) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_STAGED));
      }
    }
  }
  linger_after_error(p.err);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// The role split asks for 8 x 32 x REGS_SOFTMAX + 4 x 32 x REGS_SERVICE registers; a block that was launched with
// fewer would wait for them for ever.
template <typename Kernel>
cudaError_t check_register_budget(Kernel kernel, int threads) {
  cudaFuncAttributes attr;
  cudaError_t e = cudaFuncGetAttributes(&attr, kernel);
  if (e != cudaSuccess) return e;
  return attr.numRegs * threads < 128 * REGS_SERVICE + 256 * REGS_SOFTMAX ? cudaErrorLaunchOutOfResources : cudaSuccess;
}

cudaError_t launch_stream(const CUtensorMap& tm_q, const CUtensorMap& tm_k16, const CUtensorMap& tm_v16, const CUtensorMap& tm_out,
                          int tma_out, const PrefillParams& p, int num_sms, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(prefill_swa_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, stream::SMEM);
  if (e != cudaSuccess) return e;
  static const cudaError_t budget = check_register_budget(prefill_swa_stream_kernel, stream::THREADS);
  if (budget != cudaSuccess) return budget;
  const int ns_max = (p.max_q_len - 128 + stream::SUB - 1) / stream::SUB;
  if (ns_max <= 0) return cudaSuccess;
  const long long units = (long long)p.b.B * p.m.Hkv * ns_max;
  const int blocks = (int)(units < num_sms ? units : num_sms);
  const int per = (int)((units + blocks - 1) / blocks);
  prefill_swa_stream_kernel<<<blocks, stream::THREADS, stream::SMEM, s>>>(tm_q, tm_k16, tm_v16, tm_out, p, ns_max, per, tma_out);
  return cudaGetLastError();
}

}  // namespace

bool hswa_prefill_tc_supported(const ModelParams& m) { return m.D == 128 && m.P == 64 && (m.G % 2) == 0; }

// Geometry of the GQA-packed SWA kernel for group size G: tokens per block and keys per block (0 = unsupported).
void hswa_prefill_packed_geometry(int G, int* tq, int* nkeys) {
  *tq = 0;
  *nkeys = 0;
  if (G == 8) { *tq = PackedCfg<8>::TQ; *nkeys = PackedCfg<8>::N; }
  if (G == 4) { *tq = PackedCfg<4>::TQ; *nkeys = PackedCfg<4>::N; }
}

cudaError_t hswa_launch_prefill_swa_packed(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                           const PrefillParams& p, int first_tok, cudaStream_t s) {
  if (p.b.B == 0 || p.max_q_len <= first_tok) return cudaSuccess;
  if (p.m.G == 8) return launch_packed<8>(tm_q, tm_k, tm_v, p, first_tok, s);
  if (p.m.G == 4) return launch_packed<4>(tm_q, tm_k, tm_v, p, first_tok, s);
  return cudaErrorInvalidValue;
}

cudaError_t hswa_launch_prefill_tc(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                   const CUtensorMap& tm_v, const PrefillParams& p, int tile_limit, cudaStream_t s) {
  if (p.b.B == 0 || p.total_q == 0 || p.max_q_len == 0) return cudaSuccess;
  constexpr int SMEM_BYTES = tile_kernel_smem(KV_STAGES);
  auto kern = prefill_tc_kernel<false, KV_STAGES>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  static const cudaError_t budget = check_register_budget(kern, NUM_THREADS);
  if (budget != cudaSuccess) return budget;
  int max_tiles = (p.max_q_len + BM - 1) / BM;
  if (tile_limit > 0 && tile_limit < max_tiles) max_tiles = tile_limit;
  dim3 grid(p.m.G / 2, p.m.Hkv, (unsigned)(p.b.B * max_tiles));
  kern<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(tm_pool, tm_q, tm_k, tm_v, p, max_tiles);
  return cudaGetLastError();
}

// Shared-prefix stage of cascade decode: grid (prefix slices, KV heads, groups of 32 requests).  tm_q is the
// packed map (box {64, 8 heads, 16 requests}) over q [B][Hq][D]; p carries prefix_len, the slice plan and the
// partial buffers.
cudaError_t hswa_launch_decode_prefix(const CUtensorMap& tm_pool, const CUtensorMap& tm_q, const PrefillParams& p,
                                      int n_slices, cudaStream_t s) {
  if (p.b.B == 0 || n_slices <= 0) return cudaSuccess;
  constexpr int PREFIX_STAGES = KV_STAGES;
  constexpr int SMEM_BYTES = tile_kernel_smem(PREFIX_STAGES);
  auto kern = prefill_tc_kernel<true, PREFIX_STAGES>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  static const cudaError_t budget = check_register_budget(kern, NUM_THREADS);
  if (budget != cudaSuccess) return budget;
  dim3 grid(n_slices, p.m.Hkv, (p.b.B + 31) / 32);
  kern<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(tm_pool, tm_q, tm_pool, tm_pool, p, 1);
  return cudaGetLastError();
}

// Streaming SWA kernel (GQA group of 8, window 128): every token from the 129th of each request on.  tm_q has box
// {64, 8 heads, 16 tokens}, tm_k16 / tm_v16 have box {64, 1, 16 rows}; tm_out is tm_q's twin over a bf16 output
// tensor (used when tma_out != 0).
cudaError_t hswa_launch_prefill_swa_stream(const CUtensorMap& tm_q, const CUtensorMap& tm_k16, const CUtensorMap& tm_v16,
                                           const CUtensorMap& tm_out, int tma_out, const PrefillParams& p, int num_sms,
                                           cudaStream_t s) {
  return launch_stream(tm_q, tm_k16, tm_v16, tm_out, tma_out, p, num_sms, s);
}
