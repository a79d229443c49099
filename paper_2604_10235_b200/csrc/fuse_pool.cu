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

// Nearest-to-protected fill (Section 4.4, last sentence of "Token-level protection"): one CTA per
// sequence.  Every thread owns a contiguous segment of the tokens; the position of the last
// protected token before a segment and of the first one after it come from two block-wide scans,
// then each thread sweeps its segment forwards and backwards.  The value, minus the distance to
// the closest protected token (minus n when there is none), is the same for every head: it is
// computed into head 0's row and copied to the others.
constexpr int kNearThreads = 1024;

__global__ void __launch_bounds__(kNearThreads)
nearest_fill_kernel(const __grid_constant__ BatchTable bt, int hkv, float theta,
                    const float* __restrict__ prior, float* __restrict__ fused) {
  __shared__ int s_last[kNearThreads], s_first[kNearThreads];
  const int s = blockIdx.x;
  const SeqInfo& q = bt.seq[s];
  const int n = q.n;
  if (n == 0) return;
  const float* p = prior + q.tok_off;
  float* f0 = fused + q.item_off;
  const int t = threadIdx.x;
  const int seg = (n + kNearThreads - 1) / kNearThreads;
  const int lo = min(n, t * seg), hi = min(n, lo + seg);
  int last = -1, first = n + n;              // "none": far enough that the distance exceeds n
  for (int j = lo; j < hi; ++j)
    if (p[j] >= theta) { last = j; if (first > n) first = j; }
  s_last[t] = last;
  s_first[t] = first;
  __syncthreads();
  // inclusive scans: maximum of `last` over the threads up to t, minimum of `first` from t on
  for (int d = 1; d < kNearThreads; d <<= 1) {
    const int a = t >= d ? s_last[t - d] : -1;
    const int b = t + d < kNearThreads ? s_first[t + d] : n + n;
    __syncthreads();
    s_last[t] = max(s_last[t], a);
    s_first[t] = min(s_first[t], b);
    __syncthreads();
  }
  int before = t > 0 ? s_last[t - 1] : -1;                       // last protected token before lo
  const int after = t + 1 < kNearThreads ? s_first[t + 1] : n + n;   // first one at or after hi
  for (int j = lo; j < hi; ++j) {
    if (p[j] >= theta) before = j;
    f0[j] = before >= 0 ? (float)(j - before) : (float)n;
  }
  int next = after;
  for (int j = hi - 1; j >= lo; --j) {
    if (p[j] >= theta) next = j;
    const float d = next < n ? (float)(next - j) : (float)n;
    f0[j] = -fminf(f0[j], d);
  }
  __syncthreads();
  for (int h = 1; h < hkv; ++h)
    for (int j = t; j < n; j += kNearThreads) fused[(int64_t)h * bt.m_tot + q.item_off + j] = f0[j];
}

}  // namespace

cudaError_t launch_nearest_fill(const Launch& L, const BatchTable& bt, const Geometry& g,
                                float force_threshold, const float* prior, float* fused) {
  nearest_fill_kernel<<<bt.num_seqs, kNearThreads, 0, L.stream>>>(bt, g.hkv, force_threshold, prior, fused);
  return cudaGetLastError();
}

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
