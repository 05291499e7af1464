/*
 * hswa.h -- C ABI of the hybrid sliding-window / full attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the attention hot path of a layer stack that interleaves Sliding Window Attention
 * layers (window W, 128 in the paper) with Full Attention layers (paper Sec. 2.1), over the dual-pool KV
 * cache of paper Sec. 3.1.1: Full layers keep the whole sequence in pages reached through a per-request
 * block table (equal prefixes may share physical pages, Sec. 3.1.3); SWA layers keep strictly O(W) KV per
 * request in a ring of R pages reached through a ring table and a ring head.
 *
 * Conventions
 *   - "device" pointers are CUDA device addresses on the current device; "host" pointers are ordinary
 *     host memory.  Every array is caller-owned; the library never frees or keeps caller memory.
 *   - Every call that takes `stream` (a cudaStream_t passed as void*) is asynchronous on that stream and
 *     returns after the launches are queued.  No call synchronises except hswa_get_async_error,
 *     hswa_create and hswa_destroy.
 *   - The library allocates exactly one 16-byte device error word per handle (hswa_create) and nothing
 *     else; scratch memory is a caller-provided workspace (hswa_workspace_bytes).
 *   - Host-detectable misuse returns a status at once and launches nothing.  Device-detectable misuse
 *     (hswa_validate_batch; bounded waits inside kernels) is recorded in the error word, the offending
 *     access is skipped, and the kernel returns normally: nothing traps, asserts or spins without bound.
 *   - Within a step the library may overlap consecutive fused decode calls issued through one handle on one
 *     stream (programmatic dependent launch): a later kernel reads the batch arrays and its layer's pool while
 *     the earlier one drains, and waits before touching q, k_new, v_new or its outputs.  This relies on the
 *     contract below that the batch arrays are constant during a step and that only this library, through this
 *     handle, writes the pools; any other call on the handle (append, prefill, advance, error read) ends the
 *     overlap, and two consecutive calls on the same pool never overlap.  A caller that writes a pool itself
 *     between two decode calls of a step, or shares pools between handles, switches the overlap off with
 *     hswa_set_overlap(h, 0).
 *   - No global mutable state except the static scratch of hswa_decode_attn_static_ws; a handle may be used
 *     from one thread at a time.
 *
 * Symbols (bf16 everywhere KV or Q are stored):
 *   Hq, Hkv query / KV heads, G = Hq / Hkv (query head h uses KV head h / G), D head_dim, P page_size,
 *   W window, R ring_pages, C = R * P ring slots, B batch, ctx[r] tokens cached before the step,
 *   n[r] new tokens of request r in the step, T = sum n[r], p = ctx[r] + i the absolute position of the
 *   i-th new token.
 *
 * Pool layout (one pool per layer): bf16 [num_pages][2][Hkv][P][D], index 1 being 0 = K, 1 = V, so a
 * (page, K|V, head) slab is P * D contiguous elements.  The pool base must be 256-byte aligned (TMA
 * descriptors are built over it); q, k_new, v_new and out must be 16-byte aligned.
 *
 * Position -> storage (Sec. 3.1.1, "Full index authoritative, Full -> SWA mapping"):
 *   Full layer: page = block_table[r][p / P], slot = p % P.
 *   SWA  layer: s = (ring_head[r] + (p - ctx[r])) mod C (mathematical mod),
 *               page = ring_table[r][s / P], slot = s % P.
 * Attention (plain softmax attention over the logical sequence; the cache is only storage):
 *   keys j in [lo, p], lo = 0 on a Full layer and max(0, p - W + 1) on an SWA layer (W keys including the
 *   query's own position); out = softmax(sm_scale * q K^T) V with fp32 accumulation, lse = natural-log
 *   log-sum-exp of the scaled scores.
 *   Slots that hold no key of [lo, p] (page tails behind the cached context, ring slots older than the window or
 *   never written, pages no request refers to) may contain anything, bit patterns of NaN and infinity included:
 *   no decode or prefill call lets them change a result (Sec. 3.1.3: attention must not read invalid or
 *   overwritten slots).
 *
 * Supported shapes: D in {64, 128}; P in {16, 32, 64}; 1 <= G <= 8; W >= 1; R * P >= W + 1.
 */
#ifndef HSWA_H_
#define HSWA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hswa_handle hswa_handle; /* opaque */

typedef enum {
  HSWA_OK = 0,
  HSWA_ERR_INVALID_ARG = 1, /* null pointer, negative size, inconsistent fields */
  HSWA_ERR_UNSUPPORTED = 2, /* shape outside the supported set */
  HSWA_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  HSWA_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed, or no sm_100 device */
  HSWA_ERR_BOUNDS = 5,      /* device-side validation found an out-of-range id or length */
  HSWA_ERR_TIMEOUT = 6      /* a bounded wait inside a kernel ran out */
} hswa_status;

/* Immutable per model. */
typedef struct {
  int32_t num_q_heads;  /* Hq */
  int32_t num_kv_heads; /* Hkv, divides Hq */
  int32_t head_dim;     /* D */
  int32_t page_size;    /* P */
  int32_t window;       /* W (paper: 128) */
  int32_t ring_pages;   /* R; 0 selects ceil(W / P) + 1 */
  float sm_scale;       /* 0 selects 1 / sqrt(D) */
  int32_t out_dtype;    /* 0 = bf16 output, 1 = fp32 output */
} hswa_config;

/* One layer's cache.  `pool` is a device pointer, caller-owned, layout above. */
typedef struct {
  void* pool;
  int64_t num_pages;
  int32_t is_swa; /* per-layer flag: 1 = SWA layer (ring storage, window mask), 0 = Full layer */
} hswa_layer;

/* One step's batch.  All arrays are DEVICE pointers, caller-owned, constant during the step (every layer
 * of the step reuses them); only hswa_step_advance changes ctx_len / ring_head. */
typedef struct {
  int32_t batch;              /* B >= 0 */
  const int32_t* ctx_len;     /* [B] tokens cached before this step */
  const int32_t* q_indptr;    /* [B+1] prefix sums of n[r]; NULL means n[r] = 1 for all r (decode) */
  const int32_t* block_table; /* [B][max_blocks] page ids valid in every Full layer's pool */
  int32_t max_blocks;
  const int32_t* ring_table; /* [B][R] page ids valid in every SWA layer's pool */
  const int32_t* ring_head;  /* [B] ring slot in [0, C) of position ctx_len[r] (the next write) */
  int32_t max_q_len;         /* host-known upper bound of n[r]   (launch geometry only) */
  int32_t total_q;           /* T, host-known                      */
  int32_t max_ctx_len;       /* host-known upper bound of ctx_len[r] (launch geometry only) */
} hswa_batch;

/* Create / destroy a handle on the current CUDA device.  hswa_create validates the config (status
 * UNSUPPORTED / INVALID_ARG), checks the device is compute capability 10.x and allocates the error word.
 * Both calls synchronise the device.  `cfg` is a host pointer and is copied. */
hswa_status hswa_create(const hswa_config* cfg, hswa_handle** out);
void hswa_destroy(hswa_handle* h);

/* Switches the overlap of consecutive fused decode calls (see Conventions) on (default) or off for this handle.
 * Off, every kernel waits for all earlier work on the stream before it reads anything.  (No paper counterpart:
 * a scheduling knob of this library.) */
hswa_status hswa_set_overlap(hswa_handle* h, int32_t enabled);

/* Bytes of workspace (device memory, 256-byte aligned, caller-owned) that is enough for every decode call
 * (hswa_decode_attn, _shared_prefix, _mtp with max_total_q = max_batch * q_len) on batches bounded by the three
 * arguments; hswa_prefill_attn needs none.  An upper bound over all smaller batches and contexts.  Pure host
 * arithmetic. */
size_t hswa_workspace_bytes(const hswa_handle* h, int32_t max_batch, int32_t max_total_q, int32_t max_ctx_len);

/* Exact bytes of workspace ONE decode call needs (split-K partials of paper Sec. 2.2's memory-bound decode: the
 * key range of a Full layer is cut into splits whose (m, l, o) partials live in the workspace): the call on a
 * layer of the given kind with batch->batch = batch, batch->max_ctx_len = max_ctx_len, the given
 * shared_prefix_len (0 for hswa_decode_attn) and q_len (1, or 2-4 for hswa_decode_attn_mtp).  A call is accepted
 * iff its workspace_bytes is at least this.  0 for SWA layers, for calls that need no split, and for arguments
 * out of range.  Pure host arithmetic. */
size_t hswa_decode_workspace_need(const hswa_handle* h, int32_t is_swa, int32_t batch, int32_t max_ctx_len,
                                  int32_t shared_prefix_len, int32_t q_len);

/* Debug aid (paper Sec. 3.1.3: attention must never read invalid or overwritten slots): checks on the device,
 * for the given layer kind, that every id and length the step would use is in range (0 <= ctx <= max_ctx_len,
 * 0 <= n <= max_q_len, block-table coverage of ctx + n, page ids < num_pages, ring_head in [0, C)).  The first
 * violation is recorded in the error word as {HSWA_ERR_BOUNDS, request, index, value}; index -1 / -2 / -3 / -4
 * name ctx, n, block-table coverage and ring head. */
hswa_status hswa_validate_batch(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, void* stream);

/* KV append (Sec. 3.1.1 pools; Sec. 3.1.3: an SWA pool stays at window magnitude).
 * k_new, v_new: device, bf16 [T][Hkv][D].  Token i of request r is written at the storage location of
 * position ctx[r] + i.  On an SWA layer later tokens overwrite earlier ones, so only the last min(n, C)
 * tokens of a request are written.  Nothing else in the pool changes.
 * Caller guarantees that pages receiving an append are not shared with another request.
 * A position the block table does not cover, or a page id outside the pool, is recorded in the error word
 * (HSWA_ERR_BOUNDS) and that row is not written. */
hswa_status hswa_kv_append(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, const void* k_new,
                           const void* v_new, void* stream);

/* Batched GQA decode attention, one new token per request (batch->q_indptr must be NULL).  Paper Sec. 2.2:
 * decode is memory-bound and its cost is the KV bytes read -- every cached token on a Full layer, the last W
 * on an SWA layer (Sec. 2.1), found through the block table / ring of Sec. 3.1.1.
 * q: device bf16 [B][Hq][D].  out: device [B][Hq][D] in cfg.out_dtype.  lse: device fp32 [B][Hq] or NULL.
 * k_new, v_new: device bf16 [B][Hkv][D], or both NULL.
 *   non-NULL: the new token's K/V are appended (fused into the attention kernel) and attended to.
 *   NULL:     the caller already ran hswa_kv_append with the same un-advanced batch; position ctx[r] is
 *             read from the cache.
 * Full layers split the key range over thread blocks (split-K) and merge the partial results; partials
 * live in `workspace` (hswa_decode_workspace_need bytes; too few: HSWA_ERR_WORKSPACE, nothing launched).
 * On a Full layer the block table must cover position max_ctx_len (max_blocks * P > max_ctx_len), else
 * HSWA_ERR_INVALID_ARG; a request whose ctx_len exceeds max_ctx_len is recorded as HSWA_ERR_BOUNDS. */
hswa_status hswa_decode_attn(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, const void* q,
                             const void* k_new, const void* v_new, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream);

/* Cascade decode for batches whose requests all share a cached prefix (paper Sec. 3.1.3: equal token prefixes
 * share KV pages; Sec. 3.1.4: multi-user shared system prompts).  Same arguments and results as
 * hswa_decode_attn plus shared_prefix_len: the caller (its prefix tree) guarantees that the first
 * shared_prefix_len tokens of EVERY request in the batch map to the same physical pages, i.e. the leading
 * shared_prefix_len / P block-table entries are identical across requests, that shared_prefix_len is a multiple
 * of P and that shared_prefix_len <= ctx_len[r] for all r.  On Full layers the shared keys are then attended
 * once per group of requests as a dense tensor-core problem (rows = requests x heads) instead of being streamed
 * once per request, and merged with the per-request suffixes in the split combine.  SWA layers, shapes the
 * tensor-core stage does not cover (it needs D = 128, P = 64, G = 8) and prefixes shorter than 128 tokens take
 * the hswa_decode_attn path; results are the same up to fp32 rounding order.  shared_prefix_len = 0 is
 * hswa_decode_attn.  Not a multiple of P, negative or above max_ctx_len: HSWA_ERR_INVALID_ARG. */
hswa_status hswa_decode_attn_shared_prefix(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch,
                                           int32_t shared_prefix_len, const void* q, const void* k_new,
                                           const void* v_new, void* out, float* lse, void* workspace,
                                           size_t workspace_bytes, void* stream);

/* Multi-token decode (paper Sec. 6.2: the models draft with 3 MTP layers, so a decode step verifies the last
 * accepted token plus up to 3 drafts).  Every request has exactly q_len new tokens, 1 <= q_len <= 4;
 * batch->q_indptr must be NULL, batch->total_q = B and batch->max_q_len = 1 as for hswa_decode_attn.
 * q: device bf16 [B][q_len][Hq][D]; k_new, v_new: device bf16 [B][q_len][Hkv][D] (required); out: device
 * [B][q_len][Hq][D]; lse: device fp32 [B][q_len][Hq] or NULL.  Token i of request r has position ctx[r] + i
 * and attends causally (to the cache and to new tokens 0..i; on SWA layers inside its own window).  The q_len
 * tokens end up appended (on a ring that requires q_len <= C - W + 1, checked: HSWA_ERR_INVALID_ARG): on Full
 * layers by an append launch ahead of one kernel that streams the KV once for all q_len tokens, on SWA layers
 * inside the attention kernel, which stages the ring (or, for rings of more than 192 slots, just the window) once
 * for all tokens; a window of more than about 500 tokens on such a ring does not fit one block's shared memory:
 * HSWA_ERR_UNSUPPORTED.  Workspace: as
 * hswa_decode_attn with max_total_q = max_batch * q_len.
 * After the step call hswa_step_advance with a q_indptr describing the ACCEPTED tokens per request. */
hswa_status hswa_decode_attn_mtp(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, int32_t q_len,
                                 const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* Decode attention for callers that cannot allocate device memory.  (The paper has no counterpart of this
 * call; it exists for deployment reasons only.)
 * Same arguments, results and errors as hswa_decode_attn, minus the workspace: the split-K partials go to a
 * fixed array of HSWA_STATIC_WS_BYTES bytes that is part of the library's device image, so this call performs
 * no cudaMalloc / cudaFree and calls no allocating routine.  It serves code that runs under a fixed memory
 * budget, or inside a section where an allocation (and the device-wide synchronisation it implies) is not
 * allowed, and that therefore has no workspace to offer.
 *   - Limit: a batch whose partials need more than HSWA_STATIC_WS_BYTES (roughly B * Hq * ceil((max_ctx_len
 *     + 1) / 4096) * (4 * D + 8) bytes on a Full layer, more for small batches, which get shorter splits;
 *     SWA layers need none) is rejected with
 *     HSWA_ERR_WORKSPACE and nothing is launched.
 *   - Every GPU that loads the library holds the array until the process exits.
 *   - The first call on a device looks up the array's device address (with that device current, which must be
 *     the handle's device); make that first call before any stream capture begins.
 *   - All calls on a device share the one array and it keeps whatever the last call left there.  No part of
 *     it has to start at zero: each call writes every partial it later reads.  Two calls that overlap on the
 *     GPU (different streams, or different handles) race on it; issue them on one stream. */
#define HSWA_STATIC_WS_BYTES (64u << 20)
hswa_status hswa_decode_attn_static_ws(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch,
                                       const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                                       void* stream);

/* Chunked prefill attention: request r extends its cached context by n[r] new tokens.  Paper Sec. 2.1:
 * prefill is compute-bound; a Full layer attends the whole prefix plus the chunk causally, an SWA layer only
 * inside its window of W keys, which is where the roughly 1/7 cost of the hybrid stack comes from; Sec. 5.2:
 * fixed-size chunks against a growing cached prefix.
 * q: device bf16 [T][Hq][D]; k_new, v_new: device bf16 [T][Hkv][D] (required); out: device [T][Hq][D];
 * lse: device fp32 [T][Hq] or NULL.
 * Keys j < ctx[r] are read from the cache AS IT IS BEFORE THIS CHUNK'S APPEND (pages on a Full layer; the
 * ring on an SWA layer), keys j >= ctx[r] from k_new / v_new.  Causal mask on Full layers, causal + window
 * mask on SWA layers; key tiles wholly outside the mask are skipped.
 * fuse_append != 0: the chunk's K/V are also appended to the cache by a second launch (the append kernel of
 * hswa_kv_append) queued on `stream` right behind the attention kernels, i.e. ordered after every read of the
 * old ring contents (an SWA chunk longer than C - W + 1 tokens overwrites ring slots its own first queries
 * need, so "append, then attend" is not available on SWA layers).  The append is fused into the call, not into
 * the attention kernel. */
hswa_status hswa_prefill_attn(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, const void* q,
                              const void* k_new, const void* v_new, int32_t fuse_append, void* out, float* lse,
                              void* workspace, size_t workspace_bytes, void* stream);

/* SWA-aware prefix reuse helpers (paper Sec. 3.1.3 "SWA-Aware Prefix Cache Tree", Sec. 3.1.1 "Data movement",
 * Sec. 3.1.2 layerwise prefetch).
 *
 * hswa_window_safe_len: pure host arithmetic.  A donor matches a new request on its first match_len tokens; its
 * SWA KV survives only where swa_valid[i] != 0 (host array of at least match_len bytes).  Returns the largest hit
 * length L <= match_len such that every position in [max(0, L - (W - 1)), L) is valid, i.e. the cached keys the
 * next token's window needs are all there (0 is always safe; a NULL mask means nothing is valid).
 *
 * hswa_swa_window_gather / _scatter: move ONLY the W - 1 cached positions the next token's window needs between
 * the rings of an SWA layer and a compact buffer bf16 [B][W-1][2 (K,V)][Hkv][D]; entry j of request r is position
 * ctx_len[r] - (W - 1) + j.  Gather reads the rings (positions below 0 become zeros); scatter writes the ring
 * slots those positions map to under batch->ring_head / ring_table (positions below 0 are skipped) and touches
 * nothing else.  `buf` is device memory or pinned host memory (16-byte aligned): gather + scatter with a host
 * buffer is the offload / loadback of a request's SWA state, scatter into a fresh ring seeds it after a prefix
 * hit.  (W - 1) * 4 * Hkv * D bytes per request and layer move instead of the whole context.  Layer must be an
 * SWA layer (HSWA_ERR_INVALID_ARG otherwise); asynchronous on `stream`, so a copy stream can load layer l + 1
 * while layer l computes. */
int64_t hswa_window_safe_len(int64_t match_len, int32_t window, const uint8_t* swa_valid);
hswa_status hswa_swa_window_gather(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, void* buf,
                                   void* stream);
hswa_status hswa_swa_window_scatter(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch, const void* buf,
                                    void* stream);

/* Out-of-window SWA release bookkeeping and dual-index matching (paper Sec. 3.1.3 items 2 and 3).
 *
 * State: swa_valid_from[r] (device int32 [B], caller-owned, starts at 0 for a fresh request, or at
 * max(0, ctx - (W - 1)) for a ring seeded with hswa_swa_window_scatter) is the first cached position of request
 * r whose SWA KV is still valid; the valid SWA positions of a live request are the suffix [swa_valid_from, ctx).
 *
 * hswa_swa_release, once per step AFTER hswa_step_advance: moves the boundary forward to ctx - C (the ring has
 * overwritten everything older) and, for requests with release[r] != 0 (device uint8 [B]; NULL: all), to
 * ctx - (W - 1): the paper's release events -- a prefill chunk completed, the request terminated, every N tokens
 * generated in decode -- drop everything the next token's window cannot reach, which keeps SWA use at window
 * magnitude.  Which event fired is the scheduler's knowledge, hence the flags.  The boundary never moves back.
 *
 * hswa_swa_valid_mask: the per-position SWA status a prefix-tree node records: mask[r][p] = 1 iff
 * swa_valid_from[r] <= p < ctx_len[r], for p < mask_stride (0 beyond ctx); mask is uint8 [B][mask_stride] in
 * device memory or pinned host memory.
 *
 * hswa_prefix_hit_len: pure host arithmetic.  A cached prefix matches a new request on its first match_len tokens;
 * its nodes carry per-token Full status (full_valid, host uint8, NULL: nothing valid) and SWA status (swa_valid, as
 * for hswa_window_safe_len).  Returns the largest L <= match_len such that every position in [0, L) has Full KV
 * (Full layers read all of them) and every position in [max(0, L - (W - 1)), L) has SWA KV.  Evicting the SWA part
 * of old segments on its own therefore keeps the prefix reusable; evicting a whole segment ends it there. */
hswa_status hswa_swa_release(hswa_handle* h, int32_t batch, const int32_t* ctx_len, const uint8_t* release,
                             int32_t* swa_valid_from, void* stream);
hswa_status hswa_swa_valid_mask(hswa_handle* h, int32_t batch, const int32_t* ctx_len, const int32_t* swa_valid_from,
                                int64_t mask_stride, uint8_t* mask, void* stream);
int64_t hswa_prefix_hit_len(int64_t match_len, int32_t window, const uint8_t* full_valid, const uint8_t* swa_valid);

/* Step advance, once per step after all layers (paper Sec. 3.1.1: one logical view over both pools -- every
 * layer of a step maps positions with the same lengths and ring heads, so they move once, after the last
 * layer): ctx_len[r] += n[r], ring_head[r] = (ring_head[r] + n[r]) mod C.  ctx_len, ring_head: device int32 [B], updated in place.  q_indptr: device or NULL (n = 1). */
hswa_status hswa_step_advance(hswa_handle* h, int32_t batch, int32_t* ctx_len, int32_t* ring_head,
                              const int32_t* q_indptr, void* stream);

/* Synchronises `stream`, copies the error word to info[4] = {status, request, index, value} (host), clears
 * it, and returns info[0] as a status (HSWA_OK when nothing was recorded). */
hswa_status hswa_get_async_error(hswa_handle* h, void* stream, int32_t info[4]);

const char* hswa_status_string(hswa_status s);

/* Work balance of mixed-length prefill batches (paper Sec. 5.3: requests whose cached prefixes differ a lot make
 * the ranks / blocks that got the long ones finish last; the paper buckets by length, inside one launch the
 * equivalent is the order in which blocks are handed out).
 *
 * hswa_set_prefill_order: order in which the Full-layer tile kernel of hswa_prefill_attn takes the (request,
 * 128-token tile) pairs of a batch.  Tile b of request r walks ceil(ctx[r] / 128) + b + 1 key tiles.
 *   0: request by request in batch order, tiles ascending;
 *   1: every request's last tile first, requests interleaved;
 *   2 (default): longest request first -- requests in descending order of their longest tile's work, the tiles of a
 *      request together (their blocks share K/V pages in L2) and longest first, so that the launch ends on the
 *      shortest tiles of the shortest request;
 *   3: globally longest tile first, whatever its request.
 * Orders 2 and 3 are computed on the device from ctx_len and q_indptr.  Results do not depend on the order.
 *
 * hswa_set_block_trace: debug aid.  With a device buffer int64 [capacity_blocks][4] set (NULL, 0 switches it off),
 * every non-empty block of that kernel writes {start, end (nanoseconds of the GPU's global timer), SM id,
 * request << 32 | tile} at its linear block index (x + gridDim.x * (y + gridDim.y * z)); blocks beyond the capacity write nothing.  The caller
 * zeroes the buffer first and reads it after synchronising: the idle tail of every SM follows from it. */
hswa_status hswa_set_prefill_order(hswa_handle* h, int32_t mode);
hswa_status hswa_set_block_trace(hswa_handle* h, int64_t* buf, int64_t capacity_blocks);

/* Read-bandwidth probe (no paper counterpart; a measuring aid).  Streams `bytes` of device memory at `buf`
 * (128-byte aligned, a multiple of 32 KB) through shared memory with the same kind of bulk copies the decode
 * kernels use and does nothing with them; timed by the caller with events, bytes / time is the practical ceiling
 * for a read-only HBM stream on this GPU, which the roofline of paper Sec. 2.2's memory-bound decode is judged
 * against next to the copy-based peak.  Asynchronous on `stream`. */
hswa_status hswa_probe_read_stream(hswa_handle* h, const void* buf, size_t bytes, void* stream);

/* Self-test of the bounded waits (no paper counterpart; failure detection of the library itself).  Every wait
 * on a pipeline barrier inside the kernels gives up after a fixed number of SM clocks, records
 * HSWA_ERR_TIMEOUT in the error word and lets the block finish.  This call launches a one-block kernel whose
 * consumer warp waits, with a limit of limit_clocks (1 .. 2e9), on a barrier that its producer never arms: the
 * wait runs out, the kernel returns normally, and hswa_get_async_error then reports {HSWA_ERR_TIMEOUT, -1, 0, 7}.
 * Nothing traps, nothing is left in flight, and the context stays usable. */
hswa_status hswa_selftest_wait_timeout(hswa_handle* h, int64_t limit_clocks, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HSWA_H_ */
