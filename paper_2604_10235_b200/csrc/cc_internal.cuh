// Internal declarations shared by the kernels and the C-ABI layer of libcodecomp.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

#include "codecomp.h"

namespace cc {

constexpr int kHeadDim = 128;
constexpr int kTileKeys = 128;       // keys per score tile (tensor-core path)
constexpr int kMaxRows = 512;        // w * G limit

// Per-sequence geometry, derived on the host from the descriptor.
struct SeqInfo {
  int n;             // tokens
  int budget;        // B_s as given
  int keep;          // min(B_s, n)
  int n_items;       // tokens, or chunks when chunk > 1
  int tok_off;       // offset of the sequence in [N_tot] arrays
  int item_off;      // offset in [M_tot] arrays
  int idx_off;       // offset in [B_tot] arrays
  int tile_off;      // first score tile of the sequence (per KV head)
  int n_tiles;       // ceil(n / kTileKeys)
  int out_page_off;  // first entry of free_pages used by the sequence
  int span_cap;      // B_span, or -1 when protected tokens are not capped
  int pad_;
};

struct BatchTable {
  int num_seqs;
  int page_size;     // 0 = contiguous
  int chunk;         // >= 1
  int n_tot, m_tot, b_tot;
  int tiles_per_head;   // sum of n_tiles
  int max_items;
  SeqInfo seq[CC_MAX_SEQS];
};

struct Geometry {
  int hq, hkv, group, window, rows;       // rows = window * group
  int64_t q_stride_seq, q_stride_row, q_stride_head;
  int64_t kv_stride_tok, kv_stride_head;
  int64_t out_stride_tok, out_stride_head;
  const int32_t* page_table;
  int page_table_stride, out_page_table_stride;
  int causal;      // window rows are the last w tokens of the sequence: row t sees keys <= n - w + t
  int pool_pages;  // pages in the K/V pool (paged layout): page ids must lie in [0, pool_pages)
};

// Device status word: [0] = first error code, [1] = detail (where it happened).
struct DeviceStatus {
  int code;
  int detail;
  int pad[2];
};

__device__ __forceinline__ void report_error(DeviceStatus* st, int code, int detail) {
  if (atomicCAS(&st->code, 0, code) == 0) st->detail = detail;
}

// Pool row of token j of a sequence (paged or contiguous).  Returns -1 for a page id outside
// [0, pool_pages): the caller skips the access and records CC_ERR_DEVICE_FLAG.
__device__ __forceinline__ int64_t token_row(const BatchTable& bt, const Geometry& g, int s, int j) {
  if (bt.page_size == 0) return (int64_t)bt.seq[s].tok_off + j;
  const int page = g.page_table[(int64_t)s * g.page_table_stride + j / bt.page_size];
  if (page < 0 || page >= g.pool_pages) return -1;
  return (int64_t)page * bt.page_size + j % bt.page_size;
}

struct Launch {
  cudaStream_t stream;
  DeviceStatus* status;
  int sm_count;
};

// Programmatic dependent launch: every kernel of the library lets its successor in the stream
// start its prologue early (pdl_launch_dependents at the top) and touches global memory only
// after pdl_wait, which returns once the preceding kernels have completed and flushed.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with the programmatic-serialization attribute (and a cluster width when > 1).
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- kernels' host-side launchers (each returns a cudaError_t from the launch) ----------
size_t score_simt_ws_bytes(const BatchTable& bt, const Geometry& g, int sm_count);
cudaError_t launch_score_simt(const Launch& L, const BatchTable& bt, const Geometry& g,
                              const void* q, const void* k, float* scores, float* lse, void* ws);

size_t score_tc_ws_bytes(const BatchTable& bt, const Geometry& g, int sm_count);
// encode = cuTensorMapEncodeTiled entry point; err receives a CUresult-like code on failure
cudaError_t launch_score_tc(const Launch& L, const BatchTable& bt, const Geometry& g,
                            const void* q, const void* k, float* scores, float* lse, void* ws,
                            void* encode_fn, int64_t pool_rows, int* drv_err);

// fused[h][j] = -(distance of token j to the closest token with prior >= threshold), every head
cudaError_t launch_nearest_fill(const Launch& L, const BatchTable& bt, const Geometry& g,
                                float force_threshold, const float* prior, float* fused);

cudaError_t launch_fuse_pool(const Launch& L, const BatchTable& bt, const Geometry& g,
                             int pool_kind, int pool_size, float alpha, float beta,
                             const float* scores, const float* prior, float* fused);

size_t select_ws_bytes(const BatchTable& bt, const Geometry& g);
cudaError_t launch_select(const Launch& L, const BatchTable& bt, const Geometry& g,
                          float force_threshold, const float* fused, const float* prior,
                          int32_t* idx, int32_t* count, void* ws);

// cluster kernel: items resident in shared memory, optionally starting from the raw scores
// (pooling and prior fusion done in the same launch).  select_cluster_size returns the CTAs per
// (sequence, head) to use, or 0 when a sequence has too many items for it.
int select_cluster_size(const BatchTable& bt, int hkv);
cudaError_t launch_select_cluster(const Launch& L, const BatchTable& bt, const Geometry& g,
                                  float force_threshold, bool fused_input, int pool_kind,
                                  int pool_size, float alpha, float beta, const float* scores,
                                  float* fused, const float* prior, int32_t* idx, int32_t* count,
                                  int cluster);

// variant of launch_select whose scratch is a static device array (no workspace argument)
int64_t select_static_capacity();
cudaError_t launch_select_static(const Launch& L, const BatchTable& bt, const Geometry& g,
                                 float force_threshold, const float* fused, const float* prior,
                                 int32_t* idx, int32_t* count, int device);

cudaError_t launch_compact(const Launch& L, const BatchTable& bt, const Geometry& g,
                           const void* k, const void* v, const int32_t* idx, void* k_out,
                           void* v_out, const int32_t* free_pages, int32_t* out_page_table);

// chunk selection by query-conditioned perplexity (Section 4.1)
cudaError_t launch_ppl_scores(const Launch& L, const void* logits, bool is_f32, int num_chunks,
                              int num_tokens, int vocab, int64_t stride_chunk, int64_t stride_token,
                              const int32_t* targets, float* nll, float* score);
cudaError_t launch_select_chunks(const Launch& L, const float* score, int num_chunks, int k,
                                 int32_t* chosen);

// fraction of the critical tokens (prior >= threshold) that each head's index list retains
cudaError_t launch_str_score(const Launch& L, const BatchTable& bt, const Geometry& g,
                             float threshold, const int32_t* idx, const float* prior,
                             float* score, int32_t* counts);

// throughput probe of the score kernel's inner loop (exp_probe.cu)
cudaError_t run_exp_probe(const Launch& L, bool from_tmem, int iters, long long* scratch,
                          double* rate);

}  // namespace cc
