// A1, verification mode (CC_MODE_FP32): window attention scores with every product and sum
// in fp32 on the CUDA cores.  Two passes over the keys:
//   pass 1  per query row r: running maximum and sum of exp of the scaled logits over the
//           keys of one split of the sequence (the sum is kept in fp64);
//   pass 2  L_r = log sum exp merged over the splits, then
//           u(j) = sum_r exp(s_rj - L_r), reduced over the rows with warp shuffles and a
//           fixed-order sum of the per-warp partials.
// One thread owns one query row (row r = g * w + t of KV head h is window row t of query
// head h * G + g) and keeps it in registers as 64 packed bf16 pairs; a tile of 64 keys is
// staged in shared memory as fp32.
#include <math.h>

#include "cc_internal.cuh"

namespace cc {

namespace {

constexpr int kTile = 64;
constexpr int kGroup = 8;   // keys per register block

__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

struct SimtArgs {
  const uint16_t* q;
  const uint16_t* k;
  float* scores;
  float* lse;
  float2* part;     // [S][H_kv][splits][rows] (max, sum)
  int splits;
};

template <int PASS>
__global__ void __launch_bounds__(512, 1)
score_simt_kernel(const __grid_constant__ BatchTable bt, const Geometry g, const SimtArgs a,
                  DeviceStatus* status) {
  __shared__ __align__(16) float ktile[kTile * kHeadDim];      // 32 KB
  __shared__ float colpart[16][kTile];                          // per-warp column partials
  const int c = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
  const SeqInfo& sq = bt.seq[s];
  const int rows = g.rows;
  const int r = threadIdx.x;
  const bool active = r < rows;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_warps = blockDim.x >> 5;
  const float scale = 1.0f / sqrtf((float)kHeadDim);

  uint32_t qp[kHeadDim / 2];
  // last key this row attends to: all of them, or (causal window) its own position n - w + t
  const int last_key = (g.causal && active) ? sq.n - g.window + r % g.window : sq.n - 1;
  if (active) {
    const int gi = r / g.window, t = r % g.window;
    const uint4* src = reinterpret_cast<const uint4*>(
        a.q + (int64_t)s * g.q_stride_seq + (int64_t)t * g.q_stride_row +
        (int64_t)(h * g.group + gi) * g.q_stride_head);
#pragma unroll
    for (int i = 0; i < kHeadDim / 8; ++i) {
      const uint4 v = src[i];
      qp[4 * i + 0] = v.x; qp[4 * i + 1] = v.y; qp[4 * i + 2] = v.z; qp[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < kHeadDim / 2; ++i) qp[i] = 0;
  }

  const int64_t part_base = (((int64_t)s * g.hkv + h) * a.splits) * rows;
  float L = 0.0f;
  if (PASS == 2 && active) {
    float m = -INFINITY;
    for (int i = 0; i < a.splits; ++i) m = fmaxf(m, a.part[part_base + (int64_t)i * rows + r].x);
    double sum = 0.0;
    for (int i = 0; i < a.splits; ++i) {
      const float2 p = a.part[part_base + (int64_t)i * rows + r];
      if (p.y > 0.0f) sum += (double)p.y * exp((double)p.x - (double)m);
    }
    L = (float)((double)m + log(sum));
    if (c == 0 && a.lse != nullptr)
      a.lse[((int64_t)s * g.hq + h * g.group) * g.window + r] = L;
  }

  float run_max = -INFINITY;
  double run_sum = 0.0;

  const int n_tiles = (sq.n + kTile - 1) / kTile;
  for (int tile = c; tile < n_tiles; tile += a.splits) {
    const int base = tile * kTile;
    const int valid = min(kTile, sq.n - base);
    __syncthreads();
    // stage the tile as fp32; rows past the sequence end are zero
    for (int e = threadIdx.x; e < kTile * (kHeadDim / 8); e += blockDim.x) {
      const int j = e / (kHeadDim / 8), part = e % (kHeadDim / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (j < valid) {
        const int64_t row = token_row(bt, g, s, base + j);
        if (row < 0) {
          report_error(status, CC_ERR_DEVICE_FLAG, 100);
        } else {
          v = reinterpret_cast<const uint4*>(a.k + row * g.kv_stride_tok +
                                             (int64_t)h * g.kv_stride_head)[part];
        }
      }
      float* dst = ktile + j * kHeadDim + part * 8;
      dst[0] = bf16_lo(v.x); dst[1] = bf16_hi(v.x); dst[2] = bf16_lo(v.y); dst[3] = bf16_hi(v.y);
      dst[4] = bf16_lo(v.z); dst[5] = bf16_hi(v.z); dst[6] = bf16_lo(v.w); dst[7] = bf16_hi(v.w);
    }
    __syncthreads();

    for (int j0 = 0; j0 < valid; j0 += kGroup) {
      float acc[kGroup];
#pragma unroll
      for (int j = 0; j < kGroup; ++j) acc[j] = 0.0f;
#pragma unroll
      for (int cb = 0; cb < kHeadDim / 4; ++cb) {
        const float q0 = bf16_lo(qp[2 * cb]), q1 = bf16_hi(qp[2 * cb]);
        const float q2 = bf16_lo(qp[2 * cb + 1]), q3 = bf16_hi(qp[2 * cb + 1]);
#pragma unroll
        for (int j = 0; j < kGroup; ++j) {
          const float4 kv = *reinterpret_cast<const float4*>(ktile + (j0 + j) * kHeadDim + cb * 4);
          acc[j] = fmaf(q0, kv.x, acc[j]);
          acc[j] = fmaf(q1, kv.y, acc[j]);
          acc[j] = fmaf(q2, kv.z, acc[j]);
          acc[j] = fmaf(q3, kv.w, acc[j]);
        }
      }
      if (PASS == 1) {
        float gmax = -INFINITY;
#pragma unroll
        for (int j = 0; j < kGroup; ++j) {
          acc[j] = (j0 + j < valid && base + j0 + j <= last_key) ? acc[j] * scale : -INFINITY;
          gmax = fmaxf(gmax, acc[j]);
        }
        if (gmax > -INFINITY) {          // a causal row may see none of the eight keys
          const float new_max = fmaxf(run_max, gmax);
          float add = 0.0f;
#pragma unroll
          for (int j = 0; j < kGroup; ++j) add += expf(acc[j] - new_max);
          run_sum = run_sum * (double)expf(run_max - new_max) + (double)add;
          run_max = new_max;
        }
      } else {
#pragma unroll
        for (int j = 0; j < kGroup; ++j) {
          float v = (active && j0 + j < valid && base + j0 + j <= last_key)
                        ? expf(acc[j] * scale - L) : 0.0f;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0) colpart[warp][j0 + j] = v;
        }
      }
    }
    if (PASS == 2) {
      __syncthreads();
      for (int j = threadIdx.x; j < valid; j += blockDim.x) {
        float sum = 0.0f;
        for (int wi = 0; wi < n_warps; ++wi) sum += colpart[wi][j];
        a.scores[(int64_t)h * bt.n_tot + sq.tok_off + base + j] = sum;
      }
    }
  }
  if (PASS == 1 && active)
    a.part[part_base + (int64_t)c * rows + r] = make_float2(run_max, (float)run_sum);
}

int pick_splits(const BatchTable& bt, const Geometry& g, int sm_count) {
  int max_tiles = 1;
  for (int s = 0; s < bt.num_seqs; ++s)
    max_tiles = max(max_tiles, (bt.seq[s].n + kTile - 1) / kTile);
  int want = (2 * sm_count + g.hkv * bt.num_seqs - 1) / (g.hkv * bt.num_seqs);
  if (want < 1) want = 1;
  if (want > max_tiles) want = max_tiles;
  if (want > 64) want = 64;
  return want;
}

}  // namespace

size_t score_simt_ws_bytes(const BatchTable& bt, const Geometry& g, int sm_count) {
  const size_t n = (size_t)bt.num_seqs * g.hkv * pick_splits(bt, g, sm_count) * g.rows;
  return (n * sizeof(float2) + 255) / 256 * 256;
}

cudaError_t launch_score_simt(const Launch& L, const BatchTable& bt, const Geometry& g,
                              const void* q, const void* k, float* scores, float* lse, void* ws) {
  SimtArgs a;
  a.q = (const uint16_t*)q;
  a.k = (const uint16_t*)k;
  a.scores = scores;
  a.lse = lse;
  a.part = (float2*)ws;
  a.splits = pick_splits(bt, g, L.sm_count);
  const int threads = (g.rows + 31) / 32 * 32;
  dim3 grid(a.splits, g.hkv, bt.num_seqs);
  score_simt_kernel<1><<<grid, threads, 0, L.stream>>>(bt, g, a, L.status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  score_simt_kernel<2><<<grid, threads, 0, L.stream>>>(bt, g, a, L.status);
  return cudaGetLastError();
}

}  // namespace cc
