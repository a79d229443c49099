// Str. Score (Section 5.3, caption of the bug-localization table): the fraction of the
// structurally critical tokens of a sequence (prior >= threshold) that the retained set of a
// KV head contains.  One block per (head, sequence): a pass over the sequence's prior counts the
// critical tokens, a pass over the head's index list counts the retained ones; both are
// coalesced reads of a few hundred KB that stay in L2 across the heads.
#include "cc_internal.cuh"

namespace cc {

namespace {

constexpr int kThreads = 512;

__device__ __forceinline__ int block_sum(int v, int* scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                       // scratch may still be read from the previous call
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  int t = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) t += scratch[w];
  return t;
}

__global__ void __launch_bounds__(kThreads)
str_score_kernel(const __grid_constant__ BatchTable bt, int hkv, float threshold,
                 const int32_t* __restrict__ idx, const float* __restrict__ prior,
                 float* __restrict__ score, int32_t* __restrict__ counts) {
  __shared__ int scratch[kThreads / 32];
  const int h = blockIdx.x, s = blockIdx.y;
  const SeqInfo& q = bt.seq[s];
  const float* p = prior + q.tok_off;
  const int32_t* list = idx + (int64_t)h * bt.b_tot + q.idx_off;
  int critical = 0, kept = 0;
  for (int j = threadIdx.x; j < q.n; j += kThreads) critical += p[j] >= threshold;
  for (int i = threadIdx.x; i < q.keep; i += kThreads) {
    const int tok = list[i];
    if (tok >= 0 && tok < q.n) kept += p[tok] >= threshold;
  }
  critical = block_sum(critical, scratch);
  kept = block_sum(kept, scratch);
  if (threadIdx.x == 0) {
    const int o = s * hkv + h;
    // both counts are below 2^24, so the conversions are exact and the quotient is the
    // correctly rounded fraction
    score[o] = critical > 0 ? __fdiv_rn((float)kept, (float)critical) : 1.0f;
    if (counts != nullptr) {
      counts[2 * o] = kept;
      counts[2 * o + 1] = critical;
    }
  }
}

}  // namespace

cudaError_t launch_str_score(const Launch& L, const BatchTable& bt, const Geometry& g,
                             float threshold, const int32_t* idx, const float* prior,
                             float* score, int32_t* counts) {
  str_score_kernel<<<dim3(g.hkv, bt.num_seqs), kThreads, 0, L.stream>>>(bt, g.hkv, threshold, idx,
                                                                        prior, score, counts);
  return cudaGetLastError();
}

}  // namespace cc
