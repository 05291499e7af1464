/*
 * hswa_oracle.c -- plain, slow, fp64 CPU statement of hybrid sliding-window / full attention over a
 * hybrid KV cache.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the checker the CUDA library is compared against; it is not part
 * of the product and nothing in the product path may include, link or call it.  It shares no code, header,
 * table or helper with the CUDA sources.
 *
 * What it states (paper sections in brackets):
 *   - a layer stack interleaves Sliding Window Attention layers (window W, 128 in the paper) with Full
 *     Attention layers [Sec. 2.1 "Compute Analysis"];
 *   - Full layers keep the KV of the whole sequence, SWA layers only the KV inside the window, in two
 *     separate pools with one logical sequence view on top, the Full index being authoritative and a
 *     Full -> SWA mapping giving the SWA location [Sec. 3.1.1 "KVCache Dual-Pool Design"];
 *   - equal token prefixes share KV storage [Sec. 3.1.3 "SWA-Aware Prefix Cache Tree"], which here means
 *     two requests may name the same physical page in their block tables;
 *   - attention must never read a slot that is invalid or overwritten [Sec. 3.1.3].
 *
 * The paper gives no attention formula: the method computes exactly plain causal (Full) or causal +
 * windowed (SWA) softmax attention over the logical token sequence, the cache being only a storage scheme.
 * So this file is that definition written out, plus an explicit storage model (pages reached through a
 * block table; a ring of pages reached through a ring table and a ring head) that predicts every byte of
 * the pools.  Readings taken where the paper is silent (all listed in the design notes of the repository):
 *   window = W keys including the query's own position; GQA query head h uses KV head h / (Hq/Hkv);
 *   ring slot of position p is (ring_head + (p - ctx)) mod C with C = R * P, mathematical mod;
 *   a prefill chunk on an SWA layer sees the ring as it was BEFORE the chunk's append plus the chunk's own
 *   K/V tensors; zero visible keys gives out = 0 and lse = -inf.
 *
 * Arithmetic: bf16 inputs are widened exactly to double; scores, softmax and the weighted sum are double,
 * two-pass (max first, then sums in ascending key order), exp/log from libm.  No blocking, no online
 * softmax, no reordering.  OpenMP is used only across independent (token, head) output rows.
 *
 * Parity pins (tests/test_oracle_*.py, all CPU): brute-force dense softmax with an explicit boolean mask,
 * torch scaled_dot_product_attention in fp64, SWA == Full while length <= W, ring == contiguous cache,
 * page-permutation invariance, shared-prefix equivalence, chunking invariance, closed forms (uniform
 * weights, constant V, single key, dominant logit), the paper's ~1/7 accounting ratio, ring storage law,
 * sequential-overwrite append exactness; window-safe length against a brute-force scan, window gather / scatter
 * against the logical sequences, a round trip and an equivalent append.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG 1
#define ORC_ERR_RANGE 2

typedef struct {
  int32_t num_q_heads;  /* Hq */
  int32_t num_kv_heads; /* Hkv */
  int32_t head_dim;     /* D */
  int32_t page_size;    /* P, tokens per page */
  int32_t window;       /* W */
  int32_t ring_pages;   /* R, pages per request in an SWA pool; ring capacity C = R * P slots */
  double sm_scale;
} orc_config;

/* One layer's pool.  Element (page, kv, head, slot, d) lives at
 *   pool[page*stride_page + kv*stride_kv + head*stride_head + slot*stride_slot + d*stride_d]
 * (strides in elements, kv = 0 for K and 1 for V), so no memory layout is baked in here. */
typedef struct {
  uint16_t* pool; /* bf16 bit patterns */
  int64_t num_pages;
  int32_t is_swa;
  int64_t stride_page, stride_kv, stride_head, stride_slot, stride_d;
} orc_layer;

typedef struct {
  int32_t batch;
  const int32_t* ctx_len;     /* [B] tokens cached before the step */
  const int32_t* q_indptr;    /* [B+1] prefix sums of new tokens, or NULL = one new token per request */
  const int32_t* block_table; /* [B][max_blocks] */
  int32_t max_blocks;
  const int32_t* ring_table; /* [B][R] */
  const int32_t* ring_head;  /* [B] ring slot of position ctx_len[r] */
} orc_batch;

static double bf16_to_double(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static int64_t math_mod(int64_t a, int64_t m) {
  int64_t r = a % m;
  return r < 0 ? r + m : r;
}

static int32_t new_tokens_begin(const orc_batch* b, int32_t r) { return b->q_indptr ? b->q_indptr[r] : r; }
static int32_t new_tokens_end(const orc_batch* b, int32_t r) { return b->q_indptr ? b->q_indptr[r + 1] : r + 1; }

/* Position -> (page, slot) [Sec. 3.1.1: Full index authoritative, Full -> SWA mapping].
 * Full layer: logical block p / P of the request's block table, slot p mod P.
 * SWA layer: ring slot s = (ring_head + (p - ctx)) mod C, then page = ring_table[s / P], slot = s mod P. */
int orc_locate(const orc_config* cfg, int32_t is_swa, const orc_batch* b, int32_t r, int64_t p, int64_t* page,
               int32_t* slot) {
  if (r < 0 || r >= b->batch || p < 0) return ORC_ERR_ARG;
  const int64_t P = cfg->page_size;
  if (!is_swa) {
    int64_t blk = p / P;
    if (blk >= b->max_blocks) return ORC_ERR_RANGE;
    *page = b->block_table[(int64_t)r * b->max_blocks + blk];
    *slot = (int32_t)(p % P);
  } else {
    const int64_t C = (int64_t)cfg->ring_pages * P;
    int64_t s = math_mod((int64_t)b->ring_head[r] + (p - (int64_t)b->ctx_len[r]), C);
    *page = b->ring_table[(int64_t)r * cfg->ring_pages + s / P];
    *slot = (int32_t)(s % P);
  }
  return ORC_OK;
}

static int64_t elem_offset(const orc_layer* L, int64_t page, int kv, int head, int slot) {
  return page * L->stride_page + kv * L->stride_kv + head * L->stride_head + slot * L->stride_slot;
}

/* KV append [Sec. 3.1.1 pools; Sec. 3.1.3 item 2: SWA pool use stays at window magnitude].
 * For every request and every new token IN ORDER, the token's K and V rows (bf16 bits, copied verbatim)
 * are written at the location orc_locate gives for position ctx + i.  On a ring later tokens overwrite
 * earlier ones, so only the last min(n, C) tokens of a request survive; nothing else in the pool changes.
 * k_new / v_new: [T][Hkv][D] bf16 bits.  If offsets_out != NULL it receives, for token t, kv and head,
 * offsets_out[(t*2 + kv)*Hkv + head] = element offset of that row's d = 0 in the pool. */
int orc_kv_append(const orc_config* cfg, const orc_layer* L, const orc_batch* b, const uint16_t* k_new,
                  const uint16_t* v_new, int64_t* offsets_out) {
  const int Hkv = cfg->num_kv_heads, D = cfg->head_dim;
  for (int32_t r = 0; r < b->batch; ++r) {
    int32_t t0 = new_tokens_begin(b, r), t1 = new_tokens_end(b, r);
    for (int32_t t = t0; t < t1; ++t) {
      int64_t p = (int64_t)b->ctx_len[r] + (t - t0);
      int64_t page;
      int32_t slot;
      int rc = orc_locate(cfg, L->is_swa, b, r, p, &page, &slot);
      if (rc != ORC_OK) return rc;
      if (page < 0 || page >= L->num_pages) return ORC_ERR_RANGE;
      for (int kv = 0; kv < 2; ++kv) {
        const uint16_t* src = kv == 0 ? k_new : v_new;
        for (int h = 0; h < Hkv; ++h) {
          int64_t off = elem_offset(L, page, kv, h, slot);
          if (offsets_out) offsets_out[((int64_t)t * 2 + kv) * Hkv + h] = off;
          for (int d = 0; d < D; ++d) L->pool[off + d * L->stride_d] = src[((int64_t)t * Hkv + h) * D + d];
        }
      }
    }
  }
  return ORC_OK;
}

/* Fetch key/value row of logical position j for request r, KV head kh, as doubles.
 * j < ctx comes from the cache (pages, or the ring as it is now); j >= ctx comes from the step's own
 * k_new / v_new tensors when they are given, else from the cache (the caller appended already). */
static int fetch_kv(const orc_config* cfg, const orc_layer* L, const orc_batch* b, int32_t r, int64_t j, int kh,
                    const uint16_t* k_new, const uint16_t* v_new, double* krow, double* vrow) {
  const int D = cfg->head_dim, Hkv = cfg->num_kv_heads;
  const int64_t ctx = b->ctx_len[r];
  if (j >= ctx && k_new != NULL) {
    int64_t t = new_tokens_begin(b, r) + (j - ctx);
    if (t >= new_tokens_end(b, r)) return ORC_ERR_RANGE;
    for (int d = 0; d < D; ++d) {
      krow[d] = bf16_to_double(k_new[(t * Hkv + kh) * D + d]);
      vrow[d] = bf16_to_double(v_new[(t * Hkv + kh) * D + d]);
    }
    return ORC_OK;
  }
  int64_t page;
  int32_t slot;
  int rc = orc_locate(cfg, L->is_swa, b, r, j, &page, &slot);
  if (rc != ORC_OK) return rc;
  if (page < 0 || page >= L->num_pages) return ORC_ERR_RANGE;
  int64_t ok = elem_offset(L, page, 0, kh, slot), ov = elem_offset(L, page, 1, kh, slot);
  for (int d = 0; d < D; ++d) {
    krow[d] = bf16_to_double(L->pool[ok + d * L->stride_d]);
    vrow[d] = bf16_to_double(L->pool[ov + d * L->stride_d]);
  }
  return ORC_OK;
}

/* Attention for a list of output rows [Sec. 2.1: SWA layers attend inside the window, Full layers keep a
 * global view].  Row x is (token row_tok[x], query head row_head[x]); with row_tok == NULL all T * Hq rows
 * are computed in (token, head) order and n_rows must be T * Hq.
 * For token t of request r: i = t - q_indptr[r], p = ctx + i, kh = h / G,
 *   lo = is_swa ? max(0, p - W + 1) : 0,  keys j = lo .. p,
 *   s_j = sm_scale * sum_d q[d] K_j[d];  m = max_j s_j;  w_j = exp(s_j - m);
 *   out[d] = sum_j w_j V_j[d] / sum_j w_j;  lse = m + ln sum_j w_j.
 * q: [T][Hq][D] bf16 bits.  out: [n_rows][D] doubles, lse: [n_rows] doubles.
 * The pool is only read; "pre-append" state is whatever the caller passes in. */
int orc_attention(const orc_config* cfg, const orc_layer* L, const orc_batch* b, const uint16_t* q,
                  const uint16_t* k_new, const uint16_t* v_new, int64_t n_rows, const int32_t* row_tok,
                  const int32_t* row_head, double* out, double* lse) {
  const int Hq = cfg->num_q_heads, Hkv = cfg->num_kv_heads, D = cfg->head_dim;
  if (Hkv <= 0 || Hq % Hkv != 0) return ORC_ERR_ARG;
  const int G = Hq / Hkv;
  const int32_t T = new_tokens_end(b, b->batch - 1);
  if (row_tok == NULL && n_rows != (int64_t)T * Hq) return ORC_ERR_ARG;
  int status = ORC_OK;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t x = 0; x < n_rows; ++x) {
    int32_t t = row_tok ? row_tok[x] : (int32_t)(x / Hq);
    int32_t h = row_tok ? row_head[x] : (int32_t)(x % Hq);
    if (t < 0 || t >= T || h < 0 || h >= Hq) {
#pragma omp atomic write
      status = ORC_ERR_ARG;
      continue;
    }
    int32_t r = 0;
    while (r < b->batch && !(new_tokens_begin(b, r) <= t && t < new_tokens_end(b, r))) ++r;
    if (r >= b->batch) {
#pragma omp atomic write
      status = ORC_ERR_ARG;
      continue;
    }
    const int64_t ctx = b->ctx_len[r];
    const int64_t p = ctx + (t - new_tokens_begin(b, r));
    const int kh = h / G;
    int64_t lo = 0;
    if (L->is_swa && p - cfg->window + 1 > 0) lo = p - cfg->window + 1;
    const int64_t nk = p - lo + 1;
    double* s = (double*)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
    double* vbuf = (double*)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1) * D);
    double* krow = (double*)malloc(sizeof(double) * D);
    double* qrow = (double*)malloc(sizeof(double) * D);
    for (int d = 0; d < D; ++d) qrow[d] = bf16_to_double(q[((int64_t)t * Hq + h) * D + d]);
    int bad = 0;
    double m = -INFINITY;
    for (int64_t j = lo; j <= p; ++j) {
      if (fetch_kv(cfg, L, b, r, j, kh, k_new, v_new, krow, vbuf + (j - lo) * D) != ORC_OK) {
        bad = 1;
        break;
      }
      double acc = 0.0;
      for (int d = 0; d < D; ++d) acc += qrow[d] * krow[d];
      s[j - lo] = cfg->sm_scale * acc;
      if (s[j - lo] > m) m = s[j - lo];
    }
    double* o = out + x * D;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (bad) {
#pragma omp atomic write
      status = ORC_ERR_RANGE;
    } else if (nk <= 0) {
      lse[x] = -INFINITY;
    } else {
      double denom = 0.0;
      for (int64_t j = 0; j < nk; ++j) {
        double w = exp(s[j] - m);
        denom += w;
        for (int d = 0; d < D; ++d) o[d] += w * vbuf[j * D + d];
      }
      for (int d = 0; d < D; ++d) o[d] /= denom;
      lse[x] = m + log(denom);
    }
    free(s);
    free(vbuf);
    free(krow);
    free(qrow);
  }
  return status;
}

/* Step advance, once per step after all layers: ctx += n, ring_head = (ring_head + n) mod C, so that
 * (ring_head - ctx) mod C stays constant for the life of a request. */
int orc_step_advance(const orc_config* cfg, int32_t batch, int32_t* ctx_len, int32_t* ring_head,
                     const int32_t* q_indptr) {
  const int64_t C = (int64_t)cfg->ring_pages * cfg->page_size;
  for (int32_t r = 0; r < batch; ++r) {
    int64_t n = q_indptr ? (int64_t)q_indptr[r + 1] - q_indptr[r] : 1;
    ctx_len[r] = (int32_t)(ctx_len[r] + n);
    ring_head[r] = (int32_t)math_mod((int64_t)ring_head[r] + n, C);
  }
  return ORC_OK;
}

/* Number of keys the query at absolute position p attends to on one layer (for work accounting,
 * Sec. 2.1: the hybrid stack costs about 1/7 of an all-Full stack at long lengths). */
int64_t orc_attended_keys(const orc_config* cfg, int32_t is_swa, int64_t p) {
  int64_t full = p + 1;
  if (!is_swa) return full;
  return full < cfg->window ? full : (int64_t)cfg->window;
}

/* ---------------------------------------------------------------------------------------------------------
 * SWA-aware prefix reuse (paper Sec. 3.1.3, "SWA-Aware Prefix Cache Tree", and Sec. 3.1.1 "Data movement").
 *
 * Window-safe length (item 1 of Sec. 3.1.3): a donor node matches the new request on its first match_len
 * tokens; its Full KV is complete, but its SWA KV survives only where swa_valid[i] != 0.  A hit of length L is
 * usable only if the tail of the hit that the next token's window needs still has valid SWA slots.  Reading
 * taken (the paper says "the tail W tokens"; with the window including the query's own position the next
 * token at position L needs exactly the W - 1 cached positions [L - W + 1, L)): L is safe iff every position
 * in [max(0, L - (W - 1)), L) is valid.  Returns the largest safe L <= match_len (0 is always safe). */
int64_t orc_window_safe_len(int64_t match_len, int32_t window, const uint8_t* swa_valid) {
  for (int64_t L = match_len; L > 0; --L) {
    int64_t lo = L - (window - 1);
    if (lo < 0) lo = 0;
    int ok = 1;
    for (int64_t i = lo; i < L; ++i)
      if (!swa_valid[i]) {
        ok = 0;
        break;
      }
    if (ok) return L;
  }
  return 0;
}

/* Window gather / scatter (Sec. 3.1.1: cross-tier transfers move only valid window data; Sec. 3.1.2: layerwise
 * loadback).  The compact buffer holds, for request r, the W - 1 cached positions the next token's window needs:
 * buf[((r * (W - 1) + j) * 2 + kv) * Hkv * D + h * D + d] for j = 0 .. W - 2, position ctx[r] - (W - 1) + j.
 * Positions below 0 are zero in the buffer (gather) and skipped (scatter).  Gather reads the ring as it is;
 * scatter writes the ring slots those positions map to under the batch's ring_head / ring_table. */
int orc_window_gather(const orc_config* cfg, const orc_layer* L, const orc_batch* b, uint16_t* buf) {
  const int Hkv = cfg->num_kv_heads, D = cfg->head_dim, Wm = cfg->window - 1;
  for (int32_t r = 0; r < b->batch; ++r)
    for (int j = 0; j < Wm; ++j) {
      const int64_t p = (int64_t)b->ctx_len[r] - Wm + j;
      for (int kv = 0; kv < 2; ++kv)
        for (int h = 0; h < Hkv; ++h) {
          uint16_t* dst = buf + ((((int64_t)r * Wm + j) * 2 + kv) * Hkv + h) * D;
          if (p < 0) {
            for (int d = 0; d < D; ++d) dst[d] = 0;
            continue;
          }
          int64_t page;
          int32_t slot;
          int rc = orc_locate(cfg, 1, b, r, p, &page, &slot);
          if (rc != ORC_OK) return rc;
          if (page < 0 || page >= L->num_pages) return ORC_ERR_RANGE;
          const int64_t off = elem_offset(L, page, kv, h, slot);
          for (int d = 0; d < D; ++d) dst[d] = L->pool[off + d * L->stride_d];
        }
    }
  return ORC_OK;
}

int orc_window_scatter(const orc_config* cfg, const orc_layer* L, const orc_batch* b, const uint16_t* buf) {
  const int Hkv = cfg->num_kv_heads, D = cfg->head_dim, Wm = cfg->window - 1;
  for (int32_t r = 0; r < b->batch; ++r)
    for (int j = 0; j < Wm; ++j) {
      const int64_t p = (int64_t)b->ctx_len[r] - Wm + j;
      if (p < 0) continue;
      int64_t page;
      int32_t slot;
      int rc = orc_locate(cfg, 1, b, r, p, &page, &slot);
      if (rc != ORC_OK) return rc;
      if (page < 0 || page >= L->num_pages) return ORC_ERR_RANGE;
      for (int kv = 0; kv < 2; ++kv)
        for (int h = 0; h < Hkv; ++h) {
          const uint16_t* src = buf + ((((int64_t)r * Wm + j) * 2 + kv) * Hkv + h) * D;
          const int64_t off = elem_offset(L, page, kv, h, slot);
          for (int d = 0; d < D; ++d) L->pool[off + d * L->stride_d] = src[d];
        }
    }
  return ORC_OK;
}

/* ---------------------------------------------------------------------------------------------------------
 * Out-of-window SWA release and dual-index matching (paper Sec. 3.1.3 items 2 and 3).
 *
 * State per live request: swa_valid_from[r], the first cached position whose SWA KV is still valid.  The valid
 * SWA positions of a live request are always the suffix [swa_valid_from, len): KV is written in position order
 * and only ever dropped from the old end.  Two things move the boundary forward:
 *   storage   a ring of C slots holds the last C positions at most, later writes win (Sec. 3.1.1 "strictly
 *             O(W)"): after any append, swa_valid_from >= len - C;
 *   release   on the paper's three events -- a prefill chunk completes, the request terminates, every N tokens
 *             generated during decode -- everything outside the window is released.  The next token, at position
 *             len, reads the W - 1 cached positions [len - (W - 1), len) (the window includes the query itself),
 *             so a release sets swa_valid_from >= len - (W - 1).
 * ctx_len holds the lengths AFTER the step's advance; release[r] != 0 marks the requests whose event fired
 * (NULL: all of them).  The boundary never moves back and never goes below 0. */
int orc_swa_release(const orc_config* cfg, int32_t batch, const int32_t* ctx_len, const uint8_t* release,
                    int32_t* swa_valid_from) {
  const int64_t C = (int64_t)cfg->ring_pages * cfg->page_size;
  const int64_t W = cfg->window;
  for (int32_t r = 0; r < batch; ++r) {
    int64_t from = swa_valid_from[r];
    const int64_t len = ctx_len[r];
    if (len - C > from) from = len - C;                                  /* overwritten by the ring */
    if ((release == NULL || release[r]) && len - (W - 1) > from) from = len - (W - 1); /* released */
    if (from < 0) from = 0;
    swa_valid_from[r] = (int32_t)from;
  }
  return ORC_OK;
}

/* Does a release fire?  kind 0: a prefill chunk has completed; kind 1: the request has terminated; kind 2: a
 * token has been generated in decode, `decoded` tokens so far including this one, release every every_n. */
int orc_release_due(int32_t kind, int64_t decoded, int64_t every_n) {
  if (kind == 0 || kind == 1) return 1;
  if (kind == 2) return every_n > 0 && decoded > 0 && decoded % every_n == 0;
  return 0;
}

/* Per-position SWA status of a request of length len: mask[p] = 1 iff swa_valid_from <= p < len. */
int orc_swa_valid_mask(int64_t len, int64_t swa_valid_from, uint8_t* mask) {
  for (int64_t p = 0; p < len; ++p) mask[p] = p >= swa_valid_from ? 1 : 0;
  return ORC_OK;
}

/* Usable hit length on a cached prefix whose nodes carry dual indices (item 3): per token a Full Attention
 * status and an SWA status.  A Full layer of the continuing request reads every position [0, L), so all of them
 * need Full KV; an SWA layer reads the W - 1 positions before L, so those need SWA KV (item 1).  Evicting the
 * SWA part of an old segment therefore costs nothing as long as the tail is intact, while a hole in the Full
 * part ends the usable prefix there.  Returns the largest such L <= match_len. */
int64_t orc_prefix_hit_len(int64_t match_len, int32_t window, const uint8_t* full_valid, const uint8_t* swa_valid) {
  for (int64_t L = match_len; L > 0; --L) {
    int ok = 1;
    for (int64_t i = 0; i < L && ok; ++i)
      if (!full_valid[i]) ok = 0;
    int64_t lo = L - (window - 1);
    if (lo < 0) lo = 0;
    for (int64_t i = lo; i < L && ok; ++i)
      if (!swa_valid[i]) ok = 0;
    if (ok) return L;
  }
  return 0;
}
