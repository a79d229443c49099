// C-ABI layer of libcodecomp: argument checks, batch geometry, workspace carving, launches.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "cc_internal.cuh"

struct cc_ctx {
  int device;
  int sm_count;
  cc::DeviceStatus* d_status;
  cc::DeviceStatus* h_status;   // pinned
  long long* d_probe;           // scratch of cc_exp_rate_probe: two words per SM
  void* encode_tiled;           // cuTensorMapEncodeTiled, resolved through the runtime
  char err[256];
};

namespace {

using namespace cc;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

int fail(cc_ctx* ctx, int code, const char* fmt, ...) __attribute__((format(printf, 3, 4)));
int fail(cc_ctx* ctx, int code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

int cuda_fail(cc_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, CC_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

struct Plan {
  BatchTable bt;
  Geometry g;
  // workspace layout (byte offsets)
  size_t off_scores, off_fused, off_score_ws, off_select_ws, total;
};

// B^span = min(B, max(B_min, floor(rho * B)))  (Section 4.4, "Span selection under budget")
int span_cap(int budget, double ratio, int span_min) {
  if (!(ratio > 0.0)) return -1;
  long long fl = (long long)floor(ratio * (double)budget + 1e-9);
  long long cap = fl > span_min ? fl : span_min;
  if (cap > budget) cap = budget;
  if (cap < 0) cap = 0;
  return (int)cap;
}

int build_plan(cc_ctx* ctx, const cc_layer_desc* d, Plan* p) {
  if (!ctx) return CC_ERR_INVALID_ARG;
  if (!d) return fail(ctx, CC_ERR_INVALID_ARG, "descriptor is NULL");
  if (d->n_heads_q <= 0 || d->n_heads_kv <= 0 || d->n_heads_q % d->n_heads_kv != 0)
    return fail(ctx, CC_ERR_INVALID_ARG, "n_heads_q must be a positive multiple of n_heads_kv");
  if (d->head_dim != kHeadDim) return fail(ctx, CC_ERR_UNSUPPORTED, "head_dim must be 128");
  if (d->dtype != CC_BF16) return fail(ctx, CC_ERR_UNSUPPORTED, "dtype must be CC_BF16");
  if (d->compute_mode != CC_MODE_BF16 && d->compute_mode != CC_MODE_FP32)
    return fail(ctx, CC_ERR_INVALID_ARG, "unknown compute_mode");
  if (d->window <= 0) return fail(ctx, CC_ERR_INVALID_ARG, "window must be positive");
  const int group = d->n_heads_q / d->n_heads_kv;
  if ((long long)group * d->window > kMaxRows)
    return fail(ctx, CC_ERR_UNSUPPORTED, "window * group exceeds %d rows", kMaxRows);
  if (d->window > 256 || group > 256)
    return fail(ctx, CC_ERR_UNSUPPORTED, "window and group are limited to 256 each");
  if (d->pool_kind < CC_POOL_NONE || d->pool_kind > CC_POOL_AVG)
    return fail(ctx, CC_ERR_INVALID_ARG, "unknown pool_kind");
  if (d->pool_kind != CC_POOL_NONE && (d->pool_size < 1 || d->pool_size % 2 == 0 || d->pool_size > 63))
    return fail(ctx, CC_ERR_UNSUPPORTED, "pool_size must be odd and at most 63");
  if (d->chunk_size > 1 && d->pool_kind != CC_POOL_NONE && d->pool_size > 1)
    return fail(ctx, CC_ERR_UNSUPPORTED, "chunk-level ranking takes no pooling");
  if (d->fill_mode != CC_FILL_ATTENTION && d->fill_mode != CC_FILL_NEAREST)
    return fail(ctx, CC_ERR_INVALID_ARG, "unknown fill_mode");
  if (d->fill_mode == CC_FILL_NEAREST && d->chunk_size > 1)
    return fail(ctx, CC_ERR_UNSUPPORTED, "the nearest-token fill is token level only");
  if (isnan(d->alpha) || isnan(d->beta) || isnan(d->force_threshold))
    return fail(ctx, CC_ERR_INVALID_ARG, "alpha, beta and force_threshold must not be NaN");
  if (d->num_seqs < 0 || d->num_seqs > CC_MAX_SEQS)
    return fail(ctx, CC_ERR_UNSUPPORTED, "num_seqs must be in [0, %d]", CC_MAX_SEQS);
  const int ps = d->page_size;
  if (!(ps == 0 || ps == 8 || ps == 16 || ps == 32 || ps == 64 || ps == 128))
    return fail(ctx, CC_ERR_UNSUPPORTED, "page_size must be 0, 8, 16, 32, 64 or 128");
  if (d->num_seqs > 0 && (!d->seq_lens || !d->budgets))
    return fail(ctx, CC_ERR_INVALID_ARG, "seq_lens / budgets are NULL");
  if (ps > 0 && (!d->page_table || d->page_table_stride <= 0 || d->pool_pages <= 0))
    return fail(ctx, CC_ERR_INVALID_ARG, "paged layout needs page_table, its stride and pool_pages");
  if (d->q_stride_head % 8 || d->q_stride_row % 8 || d->q_stride_seq % 8 || d->kv_stride_tok % 8 ||
      d->kv_stride_head % 8 || d->out_stride_tok % 8 || d->out_stride_head % 8)
    return fail(ctx, CC_ERR_UNSUPPORTED, "strides must be multiples of 8 elements (16 bytes)");
  if (d->q_stride_head < kHeadDim || d->q_stride_row < kHeadDim || d->kv_stride_head < kHeadDim ||
      d->kv_stride_tok < kHeadDim)
    return fail(ctx, CC_ERR_INVALID_ARG, "strides smaller than head_dim");

  memset(p, 0, sizeof(*p));
  BatchTable& bt = p->bt;
  Geometry& g = p->g;
  bt.num_seqs = d->num_seqs > 0 ? d->num_seqs : 1;
  bt.page_size = ps;
  bt.chunk = d->chunk_size > 1 ? d->chunk_size : 1;
  long long tok = 0, item = 0, slot = 0, tile = 0, page = 0;
  for (int s = 0; s < bt.num_seqs; ++s) {
    const int n = d->num_seqs > 0 ? d->seq_lens[s] : d->n;
    const int b = d->num_seqs > 0 ? d->budgets[s] : d->budget;
    if (n < 0 || b < 0) return fail(ctx, CC_ERR_INVALID_ARG, "negative length or budget");
    if (d->causal && n > 0 && n < d->window)
      return fail(ctx, CC_ERR_INVALID_ARG, "a causal window needs n >= window (sequence %d)", s);
    SeqInfo& q = bt.seq[s];
    q.n = n;
    q.budget = b;
    q.keep = b < n ? b : n;
    q.n_items = (n + bt.chunk - 1) / bt.chunk;
    q.tok_off = (int)tok;
    q.item_off = (int)item;
    q.idx_off = (int)slot;
    q.tile_off = (int)tile;
    q.n_tiles = (n + kTileKeys - 1) / kTileKeys;
    q.out_page_off = (int)page;
    q.span_cap = span_cap(b, d->span_ratio, d->span_min);
    tok += n;
    item += q.n_items;
    slot += b;
    tile += q.n_tiles;
    if (ps > 0) {
      page += (q.keep + ps - 1) / ps;
      if ((n + ps - 1) / ps > d->page_table_stride)
        return fail(ctx, CC_ERR_INVALID_ARG, "page_table_stride too small for sequence %d", s);
    }
    if (q.n_items > bt.max_items) bt.max_items = q.n_items;
    if (tok > 0x7fffffffLL || slot > 0x7fffffffLL)
      return fail(ctx, CC_ERR_UNSUPPORTED, "batch exceeds 2^31 tokens");
  }
  bt.n_tot = (int)tok;
  bt.m_tot = (int)item;
  bt.b_tot = (int)slot;
  bt.tiles_per_head = (int)tile;

  g.hq = d->n_heads_q;
  g.hkv = d->n_heads_kv;
  g.group = group;
  g.window = d->window;
  g.causal = d->causal != 0;
  g.rows = group * d->window;
  g.q_stride_seq = d->q_stride_seq;
  g.q_stride_row = d->q_stride_row;
  g.q_stride_head = d->q_stride_head;
  g.kv_stride_tok = d->kv_stride_tok;
  g.kv_stride_head = d->kv_stride_head;
  g.out_stride_tok = d->out_stride_tok ? d->out_stride_tok : (int64_t)d->n_heads_kv * kHeadDim;
  g.out_stride_head = d->out_stride_head ? d->out_stride_head : kHeadDim;
  g.page_table = d->page_table;
  g.page_table_stride = d->page_table_stride;
  g.out_page_table_stride = d->out_page_table_stride;
  g.pool_pages = d->pool_pages;

  size_t off = 0;
  p->off_scores = off;    off += align256((size_t)g.hkv * bt.n_tot * sizeof(float));
  p->off_fused = off;     off += align256((size_t)g.hkv * bt.m_tot * sizeof(float));
  p->off_score_ws = off;
  const size_t sw = d->compute_mode == CC_MODE_FP32 ? score_simt_ws_bytes(bt, g, ctx->sm_count)
                                                    : score_tc_ws_bytes(bt, g, ctx->sm_count);
  off += align256(sw);
  p->off_select_ws = off; off += align256(select_ws_bytes(bt, g));
  p->total = off > 256 ? off : 256;
  return CC_OK;
}

int check_ws(cc_ctx* ctx, const Plan& p, void* ws, size_t ws_bytes) {
  if (!ws) return fail(ctx, CC_ERR_WORKSPACE, "workspace is NULL");
  if ((uintptr_t)ws % 256) return fail(ctx, CC_ERR_WORKSPACE, "workspace is not 256-byte aligned");
  if (ws_bytes < p.total)
    return fail(ctx, CC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", ws_bytes, p.total);
  return CC_OK;
}

Launch make_launch(cc_ctx* ctx, void* stream) {
  Launch L;
  L.stream = (cudaStream_t)stream;
  L.status = ctx->d_status;
  L.sm_count = ctx->sm_count;
  return L;
}

int run_score(cc_ctx* ctx, const cc_layer_desc* d, const Plan& p, const void* q, const void* k,
              float* scores, float* lse, char* ws, void* stream) {
  if (p.bt.n_tot == 0) return CC_OK;
  const Launch L = make_launch(ctx, stream);
  if (d->compute_mode == CC_MODE_FP32) {
    cudaError_t e = launch_score_simt(L, p.bt, p.g, q, k, scores, lse, ws + p.off_score_ws);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "score (fp32 mode) launch");
    return CC_OK;
  }
  int drv = 0;
  cudaError_t e = launch_score_tc(L, p.bt, p.g, q, k, scores, lse, ws + p.off_score_ws,
                                  ctx->encode_tiled, (int64_t)d->pool_pages * d->page_size, &drv);
  if (drv != 0) return fail(ctx, CC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", drv);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "score (tensor-core) launch");
  return CC_OK;
}

int run_fuse(cc_ctx* ctx, const cc_layer_desc* d, const Plan& p, const float* scores,
             const float* prior, float* fused, void* stream) {
  if (p.bt.m_tot == 0) return CC_OK;
  if (d->fill_mode == CC_FILL_NEAREST) {
    cudaError_t e = launch_nearest_fill(make_launch(ctx, stream), p.bt, p.g, d->force_threshold, prior, fused);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "nearest-fill launch");
    return CC_OK;
  }
  cudaError_t e = launch_fuse_pool(make_launch(ctx, stream), p.bt, p.g, d->pool_kind, d->pool_size,
                                   d->alpha, d->beta, scores, prior, fused);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "fuse/pool launch");
  return CC_OK;
}

int run_select(cc_ctx* ctx, const cc_layer_desc* d, const Plan& p, const float* fused,
               const float* prior, int32_t* idx, int32_t* count, char* ws, void* stream) {
  const int cluster = select_cluster_size(p.bt, p.g.hkv);
  cudaError_t e;
  if (cluster > 0)
    e = launch_select_cluster(make_launch(ctx, stream), p.bt, p.g, d->force_threshold, false,
                              d->pool_kind, d->pool_size, d->alpha, d->beta, nullptr,
                              const_cast<float*>(fused), prior, idx, count, cluster);
  else
    e = launch_select(make_launch(ctx, stream), p.bt, p.g, d->force_threshold, fused, prior, idx,
                      count, ws + p.off_select_ws);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "select launch");
  return CC_OK;
}

// pooling + prior fusion + selection in one launch (items of every sequence fit a cluster)
int run_fuse_select(cc_ctx* ctx, const cc_layer_desc* d, const Plan& p, int cluster,
                    const float* scores, const float* prior, float* fused, int32_t* idx,
                    int32_t* count, void* stream) {
  cudaError_t e = launch_select_cluster(make_launch(ctx, stream), p.bt, p.g, d->force_threshold,
                                        true, d->pool_kind, d->pool_size, d->alpha, d->beta,
                                        scores, fused, prior, idx, count, cluster);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "fuse + select launch");
  return CC_OK;
}

int run_compact(cc_ctx* ctx, const cc_layer_desc* d, const Plan& p, const void* k, const void* v,
                const int32_t* idx, void* k_out, void* v_out, const int32_t* free_pages,
                int32_t* out_page_table, void* stream) {
  if (p.bt.page_size > 0) {
    if (!free_pages || !out_page_table)
      return fail(ctx, CC_ERR_INVALID_ARG, "paged compaction needs free_pages and out_page_table");
    for (int s = 0; s < p.bt.num_seqs; ++s) {
      const int used = (p.bt.seq[s].keep + p.bt.page_size - 1) / p.bt.page_size;
      if (used > d->out_page_table_stride)
        return fail(ctx, CC_ERR_INVALID_ARG, "out_page_table_stride too small for sequence %d", s);
    }
  } else if (k_out == k || v_out == v) {
    return fail(ctx, CC_ERR_INVALID_ARG, "in-place compaction is not supported");
  }
  cudaError_t e = launch_compact(make_launch(ctx, stream), p.bt, p.g, k, v, idx, k_out, v_out,
                                 free_pages, out_page_table);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "compact launch");
  return CC_OK;
}

}  // namespace

extern "C" {

int cc_create(cc_ctx** out, int device) {
  if (!out) return CC_ERR_INVALID_ARG;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count)
    return CC_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return CC_ERR_CUDA;
  if (prop.major != 10) return CC_ERR_UNSUPPORTED;
  int prev = 0;
  cudaGetDevice(&prev);
  if (cudaSetDevice(device) != cudaSuccess) return CC_ERR_CUDA;
  cc_ctx* ctx = new (std::nothrow) cc_ctx();
  if (!ctx) return CC_ERR_CUDA;
  memset(ctx, 0, sizeof(*ctx));
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  bool ok = cudaMalloc(&ctx->d_status, sizeof(cc::DeviceStatus)) == cudaSuccess &&
            cudaMemset(ctx->d_status, 0, sizeof(cc::DeviceStatus)) == cudaSuccess &&
            cudaMalloc(&ctx->d_probe, 2 * 256 * sizeof(long long)) == cudaSuccess &&
            cudaMallocHost(&ctx->h_status, sizeof(cc::DeviceStatus)) == cudaSuccess;
  if (ok) {
    cudaDriverEntryPointQueryResult qres;
    ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault,
                                 &qres) == cudaSuccess &&
         qres == cudaDriverEntryPointSuccess && ctx->encode_tiled != nullptr;
  }
  cudaSetDevice(prev);
  if (!ok) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_probe) cudaFree(ctx->d_probe);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    delete ctx;
    return CC_ERR_CUDA;
  }
  *out = ctx;
  return CC_OK;
}

int cc_destroy(cc_ctx* ctx) {
  if (!ctx) return CC_ERR_INVALID_ARG;
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_probe);
  cudaFreeHost(ctx->h_status);
  delete ctx;
  return CC_OK;
}

const char* cc_status_string(int status) {
  switch (status) {
    case CC_OK: return "ok";
    case CC_ERR_INVALID_ARG: return "invalid argument";
    case CC_ERR_UNSUPPORTED: return "unsupported configuration";
    case CC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CC_ERR_CUDA: return "CUDA call failed";
    case CC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case CC_ERR_DEVICE_FLAG: return "a kernel skipped an invalid page id or index";
    default: return "unknown status";
  }
}

const char* cc_last_error(const cc_ctx* ctx) { return ctx ? ctx->err : ""; }

int cc_poll_status(cc_ctx* ctx, void* stream, int* device_status) {
  if (!ctx || !device_status) return CC_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(cc::DeviceStatus),
                                  cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(cc::DeviceStatus), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "status poll");
  *device_status = ctx->h_status->code;
  if (ctx->h_status->code != 0)
    snprintf(ctx->err, sizeof(ctx->err), "device status %d (%s), detail %d", ctx->h_status->code,
             cc_status_string(ctx->h_status->code), ctx->h_status->detail);
  return CC_OK;
}

size_t cc_workspace_bytes(const cc_ctx* ctx, const cc_layer_desc* desc) {
  Plan p;
  if (build_plan(const_cast<cc_ctx*>(ctx), desc, &p) != CC_OK) return 0;
  return p.total;
}

int cc_score_window(cc_ctx* ctx, const cc_layer_desc* desc, const void* q_win, const void* k,
                    float* scores, float* lse, void* ws, size_t ws_bytes, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (!q_win || !k || !scores) return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if ((uintptr_t)q_win % 16 || (uintptr_t)k % 16)
    return fail(ctx, CC_ERR_INVALID_ARG, "q_win and k must be 16-byte aligned");
  if ((rc = check_ws(ctx, p, ws, ws_bytes)) != CC_OK) return rc;
  return run_score(ctx, desc, p, q_win, k, scores, lse, (char*)ws, stream);
}

int cc_fuse_prior_pool(cc_ctx* ctx, const cc_layer_desc* desc, const float* scores,
                       const float* prior, float* fused, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if ((!scores && desc->fill_mode != CC_FILL_NEAREST) || !prior || !fused)
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  return run_fuse(ctx, desc, p, scores, prior, fused, stream);
}

int cc_topk_select(cc_ctx* ctx, const cc_layer_desc* desc, const float* fused, const float* prior,
                   int32_t* idx, int32_t* count, void* ws, size_t ws_bytes, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (!fused || !prior || !count || (!idx && p.bt.b_tot > 0))
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if ((rc = check_ws(ctx, p, ws, ws_bytes)) != CC_OK) return rc;
  return run_select(ctx, desc, p, fused, prior, idx, count, (char*)ws, stream);
}

int cc_topk_select_static(cc_ctx* ctx, const cc_layer_desc* desc, const float* fused,
                          const float* prior, int32_t* idx, int32_t* count, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (!fused || !prior || !count || (!idx && p.bt.b_tot > 0))
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  const long long need = (long long)p.g.hkv * (long long)p.bt.m_tot;
  if (need > (long long)select_static_capacity())
    return fail(ctx, CC_ERR_UNSUPPORTED,
                "cc_topk_select_static: %lld flag bytes needed, the static scratch holds %lld",
                need, (long long)select_static_capacity());
  cudaError_t e = launch_select_static(make_launch(ctx, stream), p.bt, p.g, desc->force_threshold,
                                       fused, prior, idx, count, ctx->device);
  if (e == cudaErrorInvalidDevice)
    return fail(ctx, CC_ERR_INVALID_ARG,
                "cc_topk_select_static: the context's device must be the current device");
  if (e != cudaSuccess) return cuda_fail(ctx, e, "static-scratch select launch");
  return CC_OK;
}

int cc_compact_kv(cc_ctx* ctx, const cc_layer_desc* desc, const void* k, const void* v,
                  const int32_t* idx, void* k_out, void* v_out, const int32_t* free_pages,
                  int32_t* out_page_table, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (p.bt.b_tot == 0) return CC_OK;
  if (!k || !v || !idx || !k_out || !v_out) return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if ((uintptr_t)k % 16 || (uintptr_t)v % 16 || (uintptr_t)k_out % 16 || (uintptr_t)v_out % 16)
    return fail(ctx, CC_ERR_INVALID_ARG, "K/V pointers must be 16-byte aligned");
  return run_compact(ctx, desc, p, k, v, idx, k_out, v_out, free_pages, out_page_table, stream);
}

namespace {

// One layer of the fused step with a plan that is already built and checked.
int compress_one(cc_ctx* ctx, const cc_layer_desc* desc, const Plan& p, const void* q_win,
                 const void* k, const void* v, const float* prior, void* k_out, void* v_out,
                 int32_t* idx, int32_t* count, const int32_t* free_pages, int32_t* out_page_table,
                 char* w, void* stream) {
  if (!q_win || !k || !v || !prior || !count || (p.bt.b_tot > 0 && (!k_out || !v_out || !idx)))
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if ((uintptr_t)q_win % 16 || (uintptr_t)k % 16 || (uintptr_t)v % 16 || (uintptr_t)k_out % 16 ||
      (uintptr_t)v_out % 16)
    return fail(ctx, CC_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
  int rc;
  float* scores = (float*)(w + p.off_scores);
  float* fused = (float*)(w + p.off_fused);
  const bool nearest = desc->fill_mode == CC_FILL_NEAREST;   // the scores play no part then
  if (!nearest && (rc = run_score(ctx, desc, p, q_win, k, scores, nullptr, w, stream)) != CC_OK) return rc;
  const int cluster = select_cluster_size(p.bt, p.g.hkv);
  if (cluster > 0 && !nearest) {
    rc = run_fuse_select(ctx, desc, p, cluster, scores, prior, fused, idx, count, stream);
    if (rc != CC_OK) return rc;
  } else {
    if ((rc = run_fuse(ctx, desc, p, scores, prior, fused, stream)) != CC_OK) return rc;
    if ((rc = run_select(ctx, desc, p, fused, prior, idx, count, w, stream)) != CC_OK) return rc;
  }
  if (p.bt.b_tot == 0) return CC_OK;
  return run_compact(ctx, desc, p, k, v, idx, k_out, v_out, free_pages, out_page_table, stream);
}

}  // namespace

int cc_compress_layer(cc_ctx* ctx, const cc_layer_desc* desc, const void* q_win, const void* k,
                      const void* v, const float* prior, void* k_out, void* v_out, int32_t* idx,
                      int32_t* count, const int32_t* free_pages, int32_t* out_page_table,
                      void* ws, size_t ws_bytes, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if ((rc = check_ws(ctx, p, ws, ws_bytes)) != CC_OK) return rc;
  return compress_one(ctx, desc, p, q_win, k, v, prior, k_out, v_out, idx, count, free_pages,
                      out_page_table, (char*)ws, stream);
}

int cc_compress_layers(cc_ctx* ctx, const cc_layer_desc* desc, int32_t n_layers,
                       const void* const* q_win, const void* const* k, const void* const* v,
                       const float* prior, void* const* k_out, void* const* v_out,
                       int32_t* const* idx, int32_t* const* count,
                       const int32_t* const* free_pages, int32_t* const* out_page_table,
                       void* ws, size_t ws_bytes, void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (n_layers < 0) return fail(ctx, CC_ERR_INVALID_ARG, "negative layer count");
  if (n_layers == 0) return CC_OK;
  if (!q_win || !k || !v || !k_out || !v_out || !idx || !count)
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL pointer array");
  if (p.bt.page_size > 0 && (!free_pages || !out_page_table))
    return fail(ctx, CC_ERR_INVALID_ARG, "paged compaction needs free_pages and out_page_table");
  if ((rc = check_ws(ctx, p, ws, ws_bytes)) != CC_OK) return rc;
  for (int l = 0; l < n_layers; ++l) {
    rc = compress_one(ctx, desc, p, q_win[l], k[l], v[l], prior, k_out[l], v_out[l], idx[l], count[l],
                      free_pages ? free_pages[l] : nullptr, out_page_table ? out_page_table[l] : nullptr,
                      (char*)ws, stream);
    if (rc != CC_OK) return rc;
  }
  return CC_OK;
}

int cc_structural_score(cc_ctx* ctx, const cc_layer_desc* desc, const int32_t* idx,
                        const float* prior, float threshold, float* score, int32_t* counts,
                        void* stream) {
  Plan p;
  int rc = build_plan(ctx, desc, &p);
  if (rc != CC_OK) return rc;
  if (!prior || !score || (!idx && p.bt.b_tot > 0))
    return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if (threshold != threshold) return fail(ctx, CC_ERR_INVALID_ARG, "threshold is NaN");
  for (int s = 0; s < p.bt.num_seqs; ++s)
    if (p.bt.seq[s].n >= (1 << 24))
      return fail(ctx, CC_ERR_UNSUPPORTED, "sequence %d is too long for exact f32 counts", s);
  cudaError_t e = launch_str_score(make_launch(ctx, stream), p.bt, p.g, threshold, idx, prior,
                                   score, counts);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "structural score launch");
  return CC_OK;
}

int cc_ppl_chunk_scores(cc_ctx* ctx, const void* logits, int32_t logits_dtype, int32_t num_chunks,
                        int32_t num_tokens, int32_t vocab, int64_t stride_chunk,
                        int64_t stride_token, const int32_t* targets, float* nll, float* score,
                        void* stream) {
  if (!ctx) return CC_ERR_INVALID_ARG;
  if (logits_dtype != CC_BF16 && logits_dtype != CC_F32)
    return fail(ctx, CC_ERR_UNSUPPORTED, "logits must be CC_BF16 or CC_F32");
  if (num_chunks < 0 || num_tokens < 1 || vocab < 1)
    return fail(ctx, CC_ERR_INVALID_ARG, "num_chunks >= 0, num_tokens >= 1 and vocab >= 1 are needed");
  if (num_chunks == 0) return CC_OK;
  if (!logits || !targets || !nll || !score) return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  if ((long long)num_chunks * num_tokens > 0x7fffffffLL)
    return fail(ctx, CC_ERR_UNSUPPORTED, "more than 2^31 rows of logits");
  if (stride_token < vocab || stride_chunk < (int64_t)num_tokens * stride_token)
    return fail(ctx, CC_ERR_INVALID_ARG, "strides smaller than the rows they separate");
  if ((uintptr_t)logits % (logits_dtype == CC_F32 ? 4 : 2))
    return fail(ctx, CC_ERR_INVALID_ARG, "logits pointer is not aligned to its element type");
  cudaError_t e = launch_ppl_scores(make_launch(ctx, stream), logits, logits_dtype == CC_F32,
                                    num_chunks, num_tokens, vocab, stride_chunk, stride_token,
                                    targets, nll, score);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "perplexity score launch");
  return CC_OK;
}

int cc_select_chunks(cc_ctx* ctx, const float* score, int32_t num_chunks, int32_t k,
                     int32_t* chosen, void* stream) {
  if (!ctx) return CC_ERR_INVALID_ARG;
  if (num_chunks < 0 || k < 0) return fail(ctx, CC_ERR_INVALID_ARG, "negative count");
  if (num_chunks > CC_MAX_CHUNKS)
    return fail(ctx, CC_ERR_UNSUPPORTED, "more than %d chunks", CC_MAX_CHUNKS);
  if (k > num_chunks) k = num_chunks;
  if (k == 0) return CC_OK;
  if (!score || !chosen) return fail(ctx, CC_ERR_INVALID_ARG, "NULL tensor pointer");
  cudaError_t e = launch_select_chunks(make_launch(ctx, stream), score, num_chunks, k, chosen);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "chunk selection launch");
  return CC_OK;
}

int cc_exp_rate_probe(cc_ctx* ctx, int32_t from_tmem, int32_t iters, double* per_clock_per_sm,
                      void* stream) {
  if (!ctx || !per_clock_per_sm) return CC_ERR_INVALID_ARG;
  if (iters < 1 || iters > (1 << 24)) return fail(ctx, CC_ERR_INVALID_ARG, "iters must be in [1, 2^24]");
  cudaError_t e = run_exp_probe(make_launch(ctx, stream), from_tmem != 0, iters, ctx->d_probe,
                                per_clock_per_sm);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "exponential-rate probe");
  return CC_OK;
}

int cc_workspace_views(const cc_ctx* ctx, const cc_layer_desc* desc, void* ws, float** scores,
                       float** fused) {
  Plan p;
  int rc = build_plan(const_cast<cc_ctx*>(ctx), desc, &p);
  if (rc != CC_OK) return rc;
  if (!ws) return CC_ERR_WORKSPACE;
  if (scores) *scores = (float*)((char*)ws + p.off_scores);
  if (fused) *fused = (float*)((char*)ws + p.off_fused);
  return CC_OK;
}

}  // extern "C"
