/*
 * codecomp.h - C ABI of the CodeComp per-layer KV-cache compression step on one B200.
 *
 * The step runs once per transformer layer after prefill; every layer is compressed on its own
 * (Section 4.5):
 *
 *   score   u_h(j) = sum over the window rows t and the query heads g of KV head h of
 *           softmax_j( q_{g,t} . k_j / sqrt(d) )                       (Section 4.5)
 *   pool    1-D sliding-window pooling of u along the token axis   (Appendix, "Compression settings")
 *   fuse    f(j) = alpha * pooled(j) + beta * prior(j); tokens whose structural prior
 *           reaches a threshold are protected                 (Section 4.4, "Span scoring",
 *                                                              "Token-level protection")
 *   select  protected tokens first, then the top-ranked f, until the budget B is full
 *                                                              (Sections 4.4 and 4.5)
 *   compact gather the retained K/V rows, in original order, into a new cache
 *                                                              (Section 4.6: positions are kept)
 *
 * Conventions
 *  - Every function returns CC_OK (0) or a negative CC_ERR_* code; cc_last_error() gives a
 *    text for the last failure of a context.  Nothing is thrown, nothing aborts.
 *  - "device" pointers are CUDA device memory of the context's GPU, "host" pointers are
 *    ordinary memory.  The caller owns every buffer.  The library allocates nothing per
 *    call, never synchronises the device, and only enqueues work on the given stream
 *    (a cudaStream_t passed as void*; NULL is the default stream).  Results are valid
 *    once that stream has reached the end of the enqueued work.
 *  - A cc_layer_desc is host memory and is read during the call only.
 *  - bf16 tensors have head_dim contiguous; the other strides are given in elements.
 *  - One cc_ctx must not be used from two threads at once.
 *
 * Layout of a batch.  num_seqs == 0 means one sequence of `n` tokens and budget `budget`.
 * num_seqs >= 1 (at most CC_MAX_SEQS) means a ragged batch described by the host arrays
 * seq_lens / budgets.  With tok_off[s] = sum of earlier n_s, item_off[s] = sum of earlier
 * ceil(n_s / chunk) and idx_off[s] = sum of earlier budgets B_s:
 *    q_win   bf16 [S][w][H_q][d]          strides q_stride_seq / q_stride_row / q_stride_head
 *    k, v    bf16 page_size == 0: token j of sequence s is row tok_off[s] + j of
 *                 [N_tot][H_kv][d] (strides kv_stride_tok / kv_stride_head);
 *                 page_size > 0: it is row page_table[s][j / page_size] * page_size +
 *                 j % page_size of the same kind of array (the page pool)
 *    prior   f32  [N_tot]                 sequence s at tok_off[s]
 *    scores  f32  [H_kv][N_tot]           sequence s at column tok_off[s]
 *    lse     f32  [S][H_q][w]             natural-log sum of exp of the scaled logits
 *    fused   f32  [H_kv][M_tot]           one value per item (token, or chunk if chunk_size > 1)
 *    idx     i32  [H_kv][B_tot]           sequence s at column idx_off[s]; token indices within
 *                                         the sequence, ascending; entries past count are -1
 *    count   i32  [S][H_kv]               min(B_s, n_s)
 *    k_out, v_out  page_size == 0: slot i of sequence s is row idx_off[s] + i of
 *                 [B_tot][H_kv][d] (strides out_stride_tok / out_stride_head, 0 = dense);
 *                 page_size > 0: it is row out_page_table[s][i / page_size] * page_size +
 *                 i % page_size of the pool given as k_out / v_out (same strides as k, v).
 */
#ifndef CODECOMP_H_
#define CODECOMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CC_OK                0
#define CC_ERR_INVALID_ARG  (-1)  /* NULL pointer, negative size, inconsistent descriptor */
#define CC_ERR_UNSUPPORTED  (-2)  /* head_dim != 128, w*G > 512, even pool width, wrong GPU ... */
#define CC_ERR_WORKSPACE    (-3)  /* workspace NULL, misaligned or smaller than cc_workspace_bytes */
#define CC_ERR_CUDA         (-4)  /* a CUDA runtime/driver call failed; see cc_last_error */
#define CC_ERR_TIMEOUT      (-5)  /* device status only: a bounded wait inside a kernel ran out */
#define CC_ERR_DEVICE_FLAG  (-6)  /* device status only: a kernel met an invalid page id or index */

#define CC_BF16        1
#define CC_F32         2   /* logits of cc_ppl_chunk_scores only */
#define CC_MODE_BF16   0   /* tensor-core scores: bf16 operands, fp32 accumulate and softmax */
#define CC_MODE_FP32   1   /* verification mode: every product and sum in fp32 on CUDA cores */
#define CC_POOL_NONE   0
#define CC_POOL_MAX    1
#define CC_POOL_AVG    2
#define CC_MAX_SEQS    64
#define CC_FILL_ATTENTION 0 /* budget left by the protected tokens: top-ranked fused scores (Section 4.5) */
#define CC_FILL_NEAREST   1 /* ... or the tokens nearest to a protected token (Section 4.4, last sentence of
                               "Token-level protection") */

typedef struct cc_ctx cc_ctx;

typedef struct cc_layer_desc {
  int32_t n_heads_q;        /* H_q, a multiple of n_heads_kv */
  int32_t n_heads_kv;       /* H_kv */
  int32_t head_dim;         /* d, must be 128 */
  int32_t window;           /* w: rows of the observation window (Section 4.5, W) */
  int32_t dtype;            /* CC_BF16 */
  int32_t compute_mode;     /* CC_MODE_BF16 or CC_MODE_FP32 */
  int32_t pool_kind;        /* CC_POOL_* */
  int32_t pool_size;        /* odd width k <= 63, centred, stride 1 */
  int32_t chunk_size;       /* <= 1: token level; c > 1: rank fixed chunks of c tokens (no pooling) */
  float   alpha, beta;      /* f = alpha * pooled + beta * prior */
  float   force_threshold;  /* prior >= threshold => protected; +INFINITY disables protection */
  double  span_ratio;       /* rho_span; <= 0: no cap on protected tokens.  > 0: protected tokens
                               are limited to B_span = min(B, max(span_min, floor(rho * B))),
                               taken by (prior descending, index ascending)  (Section 4.4) */
  int32_t span_min;         /* B_min */
  int32_t n;                /* single sequence: prefix length (L_c in Section 4.5) */
  int32_t budget;           /* single sequence: B, tokens kept per KV head */
  int64_t q_stride_seq, q_stride_row, q_stride_head;   /* elements */
  int64_t kv_stride_tok, kv_stride_head;               /* elements */
  int64_t out_stride_tok, out_stride_head;             /* elements; 0 = dense [.][H_kv][d] */
  int32_t num_seqs;         /* 0 = single sequence */
  int32_t page_size;        /* 0 = contiguous; else 8, 16, 32, 64 or 128 tokens per page */
  const int32_t* seq_lens;  /* HOST [num_seqs] */
  const int32_t* budgets;   /* HOST [num_seqs] */
  const int32_t* page_table;/* DEVICE [num_seqs][page_table_stride], used when page_size > 0 */
  int32_t page_table_stride;
  int32_t pool_pages;       /* pages in the K/V pool (page ids must be < pool_pages) when page_size > 0 */
  int32_t out_page_table_stride; /* row length of out_page_table (>= ceil(B_s / page_size)) */
  int32_t causal;           /* 0: the window follows the scored keys and every row attends to all
                               n_s of them (Section 4.5).  1 (no counterpart in the paper): the
                               window is the last w tokens of the sequence itself; row t sits at
                               position n_s - w + t and attends to keys j <= n_s - w + t only.
                               Needs n_s >= w for every non-empty sequence. */
  int32_t fill_mode;        /* CC_FILL_ATTENTION (default) or CC_FILL_NEAREST: the value that ranks the
                               unprotected tokens is minus the distance, in token positions, to the
                               closest token with prior >= force_threshold (equal distances: lower
                               index first; no such token: the first tokens of the sequence).  The
                               attention scores then play no part in the selection and
                               cc_compress_layer does not compute them.  Token level only. */
} cc_layer_desc;

/* Creates a context on CUDA device `device` (must be compute capability 10.x).  Allocates a
 * few KB of device and pinned host memory (status word, scratch of the probe); the only
 * allocation the library ever makes.  *out is untouched on failure. */
int cc_create(cc_ctx** out, int device);
/* Frees the context.  The caller must have synchronised every stream that used it. */
int cc_destroy(cc_ctx* ctx);
/* Static text for a status code. */
const char* cc_status_string(int status);
/* Text describing the last failure recorded on `ctx` (empty string if none). */
const char* cc_last_error(const cc_ctx* ctx);
/* Synchronises `stream`, then reports and clears the device-side status word: CC_OK, or
 * CC_ERR_TIMEOUT / CC_ERR_DEVICE_FLAG if a kernel gave up a bounded wait or skipped an
 * invalid page id.  Outputs of a call that reported an error are unspecified. */
int cc_poll_status(cc_ctx* ctx, void* stream, int* device_status);

/* Bytes of device workspace (256-byte aligned) that any entry point below needs for `desc`.
 * Returns 0 if the descriptor is invalid. */
size_t cc_workspace_bytes(const cc_ctx* ctx, const cc_layer_desc* desc);

/* A1 - window attention scores (Section 4.5, the equation for A and u(j)), summed over the
 * query heads of each KV head.  q_win, k: device bf16.  scores: device f32 [H_kv][N_tot],
 * fully overwritten.  lse: device f32 [S][H_q][w] or NULL.  ws: device workspace. */
int cc_score_window(cc_ctx* ctx, const cc_layer_desc* desc, const void* q_win, const void* k,
                    float* scores, float* lse, void* ws, size_t ws_bytes, void* stream);

/* A2+A3 - pooling (Appendix "Compression settings") and prior fusion (Section 4.4 "Span
 * scoring").  Token level: fused[h][j] = alpha * pool(scores[h])[j] + beta * prior[j], every
 * operation rounded to f32, average pooling = left-to-right sum of the k zero-padded taps
 * divided by k, max pooling over the valid taps.  With fill_mode == CC_FILL_NEAREST the value is
 * minus the distance to the closest protected token instead (scores may be NULL).  Chunk level (chunk_size > 1): the item
 * value is the in-order f32 sum of the chunk's scores and the prior is the chunk's maximum.
 * scores, prior, fused: device f32.  Needs no workspace. */
int cc_fuse_prior_pool(cc_ctx* ctx, const cc_layer_desc* desc, const float* scores,
                       const float* prior, float* fused, void* stream);

/* A4 - selection under the budget (Section 4.4 "Token-level protection", "Span selection
 * under budget"; Section 4.5).  Items are ranked: protected first (in sequence order), then
 * larger fused value, then lower index; items are taken in rank order until min(B_s, n_s)
 * tokens are kept (a chunk that crosses the budget keeps its first tokens).  idx receives the
 * retained token indices of each head in ascending order, -1 beyond count; count receives
 * min(B_s, n_s).  fused: device f32 [H_kv][M_tot]; prior: device f32 [N_tot]. */
int cc_topk_select(cc_ctx* ctx, const cc_layer_desc* desc, const float* fused,
                   const float* prior, int32_t* idx, int32_t* count,
                   void* ws, size_t ws_bytes, void* stream);

/* (No counterpart in the paper.)  The same selection as cc_topk_select for callers that cannot
 * hand the library a workspace because they cannot allocate device memory at that point: a
 * serving process whose memory pool already owns the whole device, or a step of a request
 * loop where cudaMalloc - which may block until the device is idle - is not acceptable.  The
 * one scratch array the kernel needs (a flag byte per head and item) lives in a fixed array
 * inside the library's device image: CC_STATIC_SELECT_MAX_ITEMS bytes on every GPU that loads
 * the library, held until the process exits.  Calls with n_heads_kv * (total items of the
 * batch) above that limit fail with CC_ERR_UNSUPPORTED and enqueue nothing.  The call
 * allocates and frees nothing.  The context's device must be the current device on every call
 * (CC_ERR_INVALID_ARG otherwise).  Its first use on a device looks up the array's device
 * address; make that first call outside any stream capture.  All calls, from every context and stream, share the one array: two calls whose
 * kernels may run at the same time on the GPU race, so keep them ordered (one stream, or
 * events).  Nothing needs clearing between calls: every flag is written before it is read.
 * Inputs and outputs are exactly those of cc_topk_select. */
#define CC_STATIC_SELECT_MAX_ITEMS (1 << 20)
int cc_topk_select_static(cc_ctx* ctx, const cc_layer_desc* desc, const float* fused,
                          const float* prior, int32_t* idx, int32_t* count, void* stream);

/* A5 - compaction: k_out[slot i of head h] = k[token idx[h][i] of head h], same for v, as
 * bit copies.  Paged layout: sequence s receives ceil(min(B_s, n_s) / page_size) page ids,
 * taken in order from free_pages (device i32, sequences served in order), written to
 * out_page_table[s][.] (device i32, -1 padded).  k_out/v_out must not alias k/v rows that
 * are still to be read; in-place compaction is rejected when the pointers are equal and
 * the layout is contiguous.  k and v are only read here, 256 bytes per retained row: either may
 * be page-locked host memory that the device can address (cudaHostAlloc, cudaHostRegister) instead
 * of device memory, in which case only the retained rows cross the bus.  The same holds for v of
 * cc_compress_layer and cc_compress_layers (k is read by the scoring and belongs on the device). */
int cc_compact_kv(cc_ctx* ctx, const cc_layer_desc* desc, const void* k, const void* v,
                  const int32_t* idx, void* k_out, void* v_out,
                  const int32_t* free_pages, int32_t* out_page_table, void* stream);

/* A8 - the whole step: score, pool, fuse, select, compact, enqueued back to back with the
 * intermediates (scores, fused values) in the workspace and no host synchronisation. */
int cc_compress_layer(cc_ctx* ctx, const cc_layer_desc* desc, const void* q_win, const void* k,
                      const void* v, const float* prior, void* k_out, void* v_out,
                      int32_t* idx, int32_t* count, const int32_t* free_pages,
                      int32_t* out_page_table, void* ws, size_t ws_bytes, void* stream);

/* The same step for n_layers layers of one batch, enqueued back to back (Section 4.5: every layer
 * is compressed on its own, with the same geometry and the same prior).  q_win, k, v, k_out,
 * v_out, idx, count (and, for the paged layout, free_pages and out_page_table; NULL otherwise)
 * are HOST arrays of n_layers device pointers, entry l being what cc_compress_layer takes for
 * layer l.  The descriptor is checked and the workspace carved once; the layers share the
 * workspace (they run one after the other on the stream), so the intermediates left in it are
 * those of the last layer.  Results are those of n_layers separate calls, bit for bit. */
int cc_compress_layers(cc_ctx* ctx, const cc_layer_desc* desc, int32_t n_layers,
                       const void* const* q_win, const void* const* k, const void* const* v,
                       const float* prior, void* const* k_out, void* const* v_out,
                       int32_t* const* idx, int32_t* const* count,
                       const int32_t* const* free_pages, int32_t* const* out_page_table,
                       void* ws, size_t ws_bytes, void* stream);

/* Str. Score (Section 5.3, caption of the bug-localization table): the share of the structurally
 * critical tokens that survives compression, which the paper averages over layers and chunks.
 * For every sequence s and
 * KV head h: score[s][h] = |{i : prior[idx[h][i]] >= threshold}| / |{j : prior[j] >= threshold}|,
 * 1 when the sequence has no such token; the average over layers and chunks is the caller's.
 * idx: device i32 [H_kv][B_tot] as written by cc_topk_select / cc_compress_layer (entries < 0
 * are skipped); prior: device f32 [N_tot]; score: device f32 [num_seqs][H_kv]; counts: NULL or
 * device i32 [num_seqs][H_kv][2] receiving (retained critical tokens, critical tokens).
 * Needs no workspace.  A NaN threshold is CC_ERR_INVALID_ARG; sequences of 2^24 tokens or more
 * are CC_ERR_UNSUPPORTED (the counts would no longer convert to f32 exactly). */
int cc_structural_score(cc_ctx* ctx, const cc_layer_desc* desc, const int32_t* idx,
                        const float* prior, float threshold, float* score, int32_t* counts,
                        void* stream);

/* Chunk selection (Section 4.1 "Query-Conditioned Chunk Selection").  logits holds, for every
 * candidate chunk i and query position t, the model's V next-token logits given prefix + C_i and
 * the earlier query tokens: element (i, t, v) at logits[i * stride_chunk + t * stride_token + v]
 * (device, CC_BF16 or CC_F32; strides in elements; rows that all start on 16-byte boundaries
 * are read with vector loads, others value by value, several times slower); targets: device
 * i32 [num_tokens], the query tokens q_t.  nll: device f32 [num_chunks][num_tokens] receives
 * -log p(q_t | ...) = logsumexp(row) - row[q_t]; score: device f32 [num_chunks] receives their
 * mean s_i^ppl.  A token id outside [0, V) gives NaN and CC_ERR_DEVICE_FLAG in the status word.
 * Needs no workspace. */
int cc_ppl_chunk_scores(cc_ctx* ctx, const void* logits, int32_t logits_dtype, int32_t num_chunks,
                        int32_t num_tokens, int32_t vocab, int64_t stride_chunk,
                        int64_t stride_token, const int32_t* targets, float* nll, float* score,
                        void* stream);

/* The min(k, num_chunks) chunks with the lowest score (same section: TopK of -s^ppl), written to
 * chosen (device i32 [k]) best first; equal scores: lower index first; NaN ranks last.
 * num_chunks <= CC_MAX_CHUNKS. */
#define CC_MAX_CHUNKS 8192
int cc_select_chunks(cc_ctx* ctx, const float* score, int32_t num_chunks, int32_t k,
                     int32_t* chosen, void* stream);

/* ---- host-side planning (no GPU work, no context; all pointers are HOST memory) ----------- */

/* Section 4.3 "Structure-Aware Budget Allocation", with the appendix's multiplier range
 * [0.5, 1.5] as the usual m_min, m_max. */
typedef struct cc_budget_params {
  double r;        /* base compression ratio */
  double r_max;    /* cap on a chunk's ratio */
  double m_min;    /* capacity multiplier of the structurally least important chunk */
  double m_max;    /* ... of the most important one (>= m_min) */
  double eps;      /* floor of the score spread in the normalisation (> 0) */
} cc_budget_params;

/* Per-chunk budgets from the chunk-level structural scores sigma_i:
 *   s~_i = 0.5 if all sigma are equal, else (sigma_i - min) / max(eps, max - min);
 *   m_i = m_min + (m_max - m_min) * clip(s~_i, 0, 1);
 *   budgets[i] = floor(lens[i] * min(r_max, r * m_i)), never above lens[i];
 * evaluated in double precision in this order.  multipliers (nullable) receives m_i.
 * The budgets are what cc_layer_desc.budgets takes when every chunk is a sequence of a batch.
 * NaN scores, negative lengths or parameters out of range: CC_ERR_INVALID_ARG. */
int cc_plan_budgets(const double* sigma, const int32_t* lens, int32_t num_chunks,
                    const cc_budget_params* p, int32_t* budgets, double* multipliers);

/* Section 4.4 "Span selection under budget" for one chunk of n tokens with budget B: spans are
 * half-open token ranges [starts[i], ends[i]); all protected spans (signatures, query-matched)
 * are taken; the others follow in rank order (score descending, then earlier start, then lower
 * index), each taken whole, while fewer than B_span = min(B, max(span_min, floor(span_ratio *
 * B))) tokens are covered (span_ratio <= 0: B_span = B).  prior_mask [n] receives 1.0 for the
 * covered tokens and 0.0 elsewhere: given as `prior` with force_threshold <= 1 it makes them the
 * protected set P_i of the selection ("Token-level protection").  taken (nullable, room for
 * num_spans) receives the indices of the spans in the order taken, num_taken their number. */
int cc_select_spans(const int32_t* starts, const int32_t* ends, const float* scores,
                    const uint8_t* is_protected, int32_t num_spans, int32_t n, int32_t budget,
                    double span_ratio, int32_t span_min, float* prior_mask, int32_t* taken,
                    int32_t* num_taken);

/* (No counterpart in the paper: a measurement aid.)  Throughput of the inner loop that bounds
 * cc_score_window - acc += 2^(v * c + off), two pairs of values in three on the special-function
 * unit and one on the FMA pipe - with sixteen warps per SM doing nothing else for `iters` rounds of
 * 32 values per thread: values held in registers (from_tmem == 0) or read from tensor memory the
 * way the kernel reads its accumulators (from_tmem != 0).  *per_clock_per_sm (HOST) receives the
 * mean over the SMs of values per SM clock.  Multiplied by the SM count and the SM clock it is
 * the exponential ceiling of the score stage, which evaluates 2 * w * G exponentials per (key,
 * KV head).  Uses a few KB of device memory owned by the context; synchronises `stream`. */
int cc_exp_rate_probe(cc_ctx* ctx, int32_t from_tmem, int32_t iters, double* per_clock_per_sm,
                      void* stream);

/* Device pointers, inside the workspace last given to cc_compress_layer for `desc`, of the
 * intermediate scores [H_kv][N_tot] and fused values [H_kv][M_tot] (for inspection). */
int cc_workspace_views(const cc_ctx* ctx, const cc_layer_desc* desc, void* ws,
                       float** scores, float** fused);

#ifdef __cplusplus
}
#endif
#endif  /* CODECOMP_H_ */
