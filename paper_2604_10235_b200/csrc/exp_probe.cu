// Throughput probe of the score kernel's inner loop (no counterpart in the paper): how many
// exponentials per clock one SM sustains when sixteen warps do nothing but the loop
// acc += 2^(v * c + off) of score_tc.cu (same code: exp2_poly.cuh), on values held in registers
// or on values read from tensor memory with tcgen05.ld as the kernel reads its accumulators.
// The figure is the ceiling that binds the score stage, reported by the benchmark next to the
// HBM and tensor-core rooflines.
#include "cc_internal.cuh"
#include "exp2_poly.cuh"

namespace cc {

namespace {

constexpr int kProbeThreads = 512;                 // sixteen warps, as the score kernel's epilogue
constexpr size_t kProbeSmem = 160 * 1024;          // one CTA per SM, so a CTA may take all of TMEM

__device__ __forceinline__ void probe_tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}

// out[2 * block] = cycles of the timed loop, out[2 * block + 1] = a value that depends on every
// exponential (so that none of them is optimised away).
template <bool FROM_TMEM>
__global__ void __launch_bounds__(kProbeThreads, 1)
exp_probe_kernel(long long* out, int iters, float c, float off) {
  extern __shared__ uint8_t probe_smem[];
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(probe_smem);
  const int warp = threadIdx.x >> 5;
  uint32_t tmem_base = 0;
  if (FROM_TMEM) {
    if (warp == 0) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"((uint32_t)__cvta_generic_to_shared(tmem_slot)), "r"(512u) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    tmem_base = *tmem_slot;
  }
  // lanes of the warp's quadrant, one of the four 128-column blocks
  const uint32_t addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
  uint32_t v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i)
    v[i] = __float_as_uint(-30.0f + (float)((threadIdx.x * 37 + i * 11) % 64) * 0.5f);
  uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
  const uint64_t c2 = pack2(c, c);
  uint64_t off2 = pack2(off, off);
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
    if (FROM_TMEM) {
      probe_tmem_ld32(addr + (uint32_t)((it & 3) * 32), v);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    } else {
      off2 = add2(off2, pack2(-1.0e-4f, -1.0e-4f));     // new arguments every round
    }
    exp_accumulate<false, 32>(v, c2, off2, 0u, acc);
  }
  const long long t1 = clock64();
  const float total = acc_total(acc);
  if (threadIdx.x == 0) out[2 * blockIdx.x] = t1 - t0;
  if (total == 123.456f) out[2 * blockIdx.x + 1] = 1;    // keeps the sums alive
  if (FROM_TMEM) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u)
                   : "memory");
    }
  }
}

}  // namespace

// Runs the probe on every SM and returns the mean rate (values per clock per SM) in *rate.
// Synchronises the stream.  scratch: device memory for 2 * sm_count 64-bit words.
cudaError_t run_exp_probe(const Launch& L, bool from_tmem, int iters, long long* scratch,
                          double* rate) {
  auto kern = from_tmem ? exp_probe_kernel<true> : exp_probe_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProbeSmem);
  if (e != cudaSuccess) return e;
  const float c = 0.12751743f;     // log2(e) / sqrt(128)
  kern<<<L.sm_count, kProbeThreads, kProbeSmem, L.stream>>>(scratch, iters, c, -1.0f);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  long long host[2 * 256];
  const int n = L.sm_count < 256 ? L.sm_count : 256;
  e = cudaMemcpyAsync(host, scratch, sizeof(long long) * 2 * n, cudaMemcpyDeviceToHost, L.stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(L.stream);
  if (e != cudaSuccess) return e;
  double sum = 0.0;
  for (int i = 0; i < n; ++i)
    sum += (double)(kProbeThreads * 32) * (double)iters / (double)(host[2 * i] > 0 ? host[2 * i] : 1);
  *rate = sum / n;
  return cudaSuccess;
}

}  // namespace cc
