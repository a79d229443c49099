// Query-conditioned perplexity scores of chunks (Section 4.1): for every (chunk, query position)
// the negative log-likelihood of the query token, logsumexp(row) - row[target], from one
// streaming pass over the row of V logits, then the mean over the query positions, and the
// choice of the k chunks with the lowest score.
//
// The scoring kernel is bound by HBM: every logit is read once (V * 2 or 4 bytes per row, rows
// of several hundred KB), the arithmetic per element is one scale, one exponential and one add.
// One CTA per row; a thread reads 16-byte vectors, four of them in flight, and keeps a running
// (maximum, sum) in base 2 that is rescaled only when a vector raises the maximum; the threads'
// pairs are merged with shuffles.  One exponential pair in three is evaluated on the FMA pipe
// (the special-function unit alone would be as slow as the memory for 2-byte logits).
#include <math.h>

#include "cc_internal.cuh"
#include "exp2_poly.cuh"

namespace cc {

namespace {

constexpr int kThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float max3f(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

struct Running {
  float m, s;       // maximum (base-2 units) and sum of 2^(x log2(e) - m)
  // eight raw logits: the scaling by log2(e) is folded into the subtraction of the maximum
  __device__ __forceinline__ void add8(const float (&x)[8]) {
    const float vm = max3f(max3f(x[0], x[1], x[2]), max3f(x[3], x[4], x[5]), fmaxf(x[6], x[7])) * kLog2e;
    if (vm > m) {
      s *= ex2(m - vm);          // m = -inf at the start: the factor is 0 and s is 0
      m = vm;
    }
    const float nm = -m;
    float a = 0.f, b = 0.f;
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      a += ex2(fmaf(x[i], kLog2e, nm));
      // one value in eight goes to the FMA pipe, which otherwise idles
      b += (i == 2) ? ex2_poly(fmaf(x[i + 1], kLog2e, nm)) : ex2(fmaf(x[i + 1], kLog2e, nm));
    }
    s += a + b;
  }
  __device__ __forceinline__ void merge(float om, float os) {
    const float nm = fmaxf(m, om);
    if (nm == -INFINITY) return;
    s = s * ex2(m - nm) + os * ex2(om - nm);
    m = nm;
  }
};

// A streaming 16-byte load that the compiler keeps where it is written, so that the loads of a
// batch are all issued before the first of them is used.
__device__ __forceinline__ uint4 ld16(const void* p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Eight consecutive logits: their raw 16-byte words and the conversion to f32.
template <typename T> struct Vec;
template <> struct Vec<float> {
  uint4 a, b;
  __device__ __forceinline__ void load(const float* p) { a = ld16(p); b = ld16(p + 4); }
  __device__ __forceinline__ void get(float (&x)[8]) const {
    x[0] = __uint_as_float(a.x); x[1] = __uint_as_float(a.y); x[2] = __uint_as_float(a.z);
    x[3] = __uint_as_float(a.w); x[4] = __uint_as_float(b.x); x[5] = __uint_as_float(b.y);
    x[6] = __uint_as_float(b.z); x[7] = __uint_as_float(b.w);
  }
  __device__ static float one(const float* p) { return *p; }
};
template <> struct Vec<uint16_t> {       // bf16 bit patterns
  uint4 a;
  __device__ __forceinline__ void load(const uint16_t* p) { a = ld16(p); }
  __device__ __forceinline__ void get(float (&x)[8]) const {
    x[0] = __uint_as_float(a.x << 16); x[1] = __uint_as_float(a.x & 0xffff0000u);
    x[2] = __uint_as_float(a.y << 16); x[3] = __uint_as_float(a.y & 0xffff0000u);
    x[4] = __uint_as_float(a.z << 16); x[5] = __uint_as_float(a.z & 0xffff0000u);
    x[6] = __uint_as_float(a.w << 16); x[7] = __uint_as_float(a.w & 0xffff0000u);
  }
  __device__ static float one(const uint16_t* p) { return __uint_as_float((uint32_t)*p << 16); }
};
template <typename T> constexpr int kBatch = sizeof(T) == 2 ? 8 : 4;   // 128 bytes per thread in flight

template <typename T>
__global__ void __launch_bounds__(kThreads)
ppl_nll_kernel(const T* __restrict__ logits, int num_tokens, int vocab, int64_t stride_chunk,
               int64_t stride_token, int vectors, const int32_t* __restrict__ targets,
               float* __restrict__ nll, DeviceStatus* status) {
  __shared__ float sm_m[kThreads / 32], sm_s[kThreads / 32];
  const int row = blockIdx.x, chunk = row / num_tokens, t = row % num_tokens;
  const T* x = logits + (int64_t)chunk * stride_chunk + (int64_t)t * stride_token;
  Running r{-INFINITY, 0.f};
  const int n_vec = vectors ? vocab / 8 : 0;   // rows off the 16-byte grid are read value by value
  int i = threadIdx.x;
  constexpr int kB = kBatch<T>;
  for (; i + (kB - 1) * kThreads < n_vec; i += kB * kThreads) {
    Vec<T> raw[kB];
#pragma unroll
    for (int u = 0; u < kB; ++u) raw[u].load(x + (int64_t)(i + u * kThreads) * 8);
#pragma unroll
    for (int u = 0; u < kB; ++u) {
      float v[8];
      raw[u].get(v);
      r.add8(v);
    }
  }
  for (; i < n_vec; i += kThreads) {
    Vec<T> raw;
    raw.load(x + (int64_t)i * 8);
    float v[8];
    raw.get(v);
    r.add8(v);
  }
  // the up to seven values after the last whole vector
  for (int j = n_vec * 8 + threadIdx.x; j < vocab; j += kThreads) r.merge(Vec<T>::one(x + j) * kLog2e, 1.0f);

#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
    r.merge(__shfl_xor_sync(0xffffffffu, r.m, o), __shfl_xor_sync(0xffffffffu, r.s, o));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sm_m[warp] = r.m; sm_s[warp] = r.s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    Running all{-INFINITY, 0.f};
    for (int w = 0; w < kThreads / 32; ++w) all.merge(sm_m[w], sm_s[w]);
    const int target = targets[t];
    float out = __int_as_float(0x7fc00000);                   // NaN for an invalid token id
    if (target >= 0 && target < vocab)
      out = (all.m + log2f(all.s)) * kLn2 - Vec<T>::one(x + target);
    else
      report_error(status, CC_ERR_DEVICE_FLAG, 600);
    nll[row] = out;
  }
}

// mean over the query positions, summed in order
__global__ void ppl_mean_kernel(const float* __restrict__ nll, int num_chunks, int num_tokens,
                                float* __restrict__ score) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= num_chunks) return;
  float acc = 0.f;
  for (int t = 0; t < num_tokens; ++t) acc = __fadd_rn(acc, nll[(int64_t)c * num_tokens + t]);
  score[c] = __fdiv_rn(acc, (float)num_tokens);
}

// rank of every chunk by (score, index); the k best are written in rank order
__global__ void __launch_bounds__(1024)
select_chunks_kernel(const float* __restrict__ score, int num_chunks, int k, int32_t* __restrict__ chosen) {
  extern __shared__ float key[];
  for (int i = threadIdx.x; i < num_chunks; i += blockDim.x) {
    const float s = score[i];
    key[i] = s != s ? INFINITY : s;                           // NaN ranks last
  }
  __syncthreads();
  for (int i = threadIdx.x; i < num_chunks; i += blockDim.x) {
    const float mine = key[i];
    int rank = 0;
    for (int j = 0; j < num_chunks; ++j) rank += key[j] < mine || (key[j] == mine && j < i);
    if (rank < k) chosen[rank] = i;
  }
}

}  // namespace

cudaError_t launch_ppl_scores(const Launch& L, const void* logits, bool is_f32, int num_chunks,
                              int num_tokens, int vocab, int64_t stride_chunk, int64_t stride_token,
                              const int32_t* targets, float* nll, float* score) {
  const int rows = num_chunks * num_tokens;
  const int64_t per16 = is_f32 ? 4 : 8;
  const int vectors = (uintptr_t)logits % 16 == 0 && stride_token % per16 == 0 && stride_chunk % per16 == 0;
  if (is_f32)
    ppl_nll_kernel<float><<<rows, kThreads, 0, L.stream>>>((const float*)logits, num_tokens, vocab,
                                                           stride_chunk, stride_token, vectors, targets,
                                                           nll, L.status);
  else
    ppl_nll_kernel<uint16_t><<<rows, kThreads, 0, L.stream>>>((const uint16_t*)logits, num_tokens,
                                                              vocab, stride_chunk, stride_token,
                                                              vectors, targets, nll, L.status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ppl_mean_kernel<<<(num_chunks + 127) / 128, 128, 0, L.stream>>>(nll, num_chunks, num_tokens, score);
  return cudaGetLastError();
}

cudaError_t launch_select_chunks(const Launch& L, const float* score, int num_chunks, int k,
                                 int32_t* chosen) {
  select_chunks_kernel<<<1, 1024, (size_t)num_chunks * sizeof(float), L.stream>>>(score, num_chunks, k,
                                                                                 chosen);
  return cudaGetLastError();
}

}  // namespace cc
