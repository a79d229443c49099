// A2 + A3: sliding-window pooling of the scores and fusion with the structural prior.
// Token level: one thread per token; the 2*half neighbours come from L1/L2 (the whole score
// array of a layer is about 1 MB).  Chunk level: one thread per chunk.
// Every floating-point operation is an explicitly rounded f32 operation (no contraction into
// FMA), in a fixed order, so that the result is reproducible bit for bit.
#include "cc_internal.cuh"

namespace cc {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float canonical(float x) { return __fadd_rn(x, 0.0f); }  // -0 -> +0

__global__ void __launch_bounds__(kThreads)
fuse_pool_kernel(const __grid_constant__ BatchTable bt, int pool_kind, int pool_size,
                 float alpha, float beta, const float* __restrict__ scores,
                 const float* __restrict__ prior, float* __restrict__ fused) {
  const int s = blockIdx.z;
  const int h = blockIdx.y;
  const SeqInfo& q = bt.seq[s];
  const float* u = scores + (int64_t)h * bt.n_tot + q.tok_off;
  const float* p = prior + q.tok_off;
  float* f = fused + (int64_t)h * bt.m_tot + q.item_off;

  for (int i = blockIdx.x * kThreads + threadIdx.x; i < q.n_items; i += gridDim.x * kThreads) {
    float val, pr;
    if (bt.chunk > 1) {
      const int lo = i * bt.chunk;
      const int hi = min(q.n, lo + bt.chunk);
      val = u[lo];
      pr = p[lo];
      for (int j = lo + 1; j < hi; ++j) {
        val = __fadd_rn(val, u[j]);
        pr = fmaxf(pr, p[j]);
      }
    } else {
      pr = p[i];
      if (pool_kind == CC_POOL_NONE || pool_size <= 1) {
        val = u[i];
      } else {
        const int half = pool_size / 2;
        if (pool_kind == CC_POOL_MAX) {
          val = u[i];
          for (int j = max(0, i - half); j <= min(q.n - 1, i + half); ++j) val = fmaxf(val, u[j]);
        } else {
          val = 0.0f;
          bool first = true;
          for (int j = i - half; j <= i + half; ++j) {
            const float x = (j >= 0 && j < q.n) ? u[j] : 0.0f;
            val = first ? x : __fadd_rn(val, x);
            first = false;
          }
          val = __fdiv_rn(val, (float)pool_size);
        }
      }
    }
    f[i] = canonical(__fadd_rn(__fmul_rn(alpha, val), __fmul_rn(beta, pr)));
  }
}

}  // namespace

cudaError_t launch_fuse_pool(const Launch& L, const BatchTable& bt, const Geometry& g,
                             int pool_kind, int pool_size, float alpha, float beta,
                             const float* scores, const float* prior, float* fused) {
  int blocks = (bt.max_items + kThreads - 1) / kThreads;
  if (blocks < 1) blocks = 1;
  dim3 grid(blocks, g.hkv, bt.num_seqs);
  fuse_pool_kernel<<<grid, kThreads, 0, L.stream>>>(bt, pool_kind, pool_size, alpha, beta, scores,
                                                    prior, fused);
  return cudaGetLastError();
}

}  // namespace cc
