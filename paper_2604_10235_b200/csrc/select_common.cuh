// Helpers shared by the two selection kernels (select.cu: one CTA per (sequence, head);
// select_cluster.cu: a thread-block cluster per (sequence, head)).
#pragma once

namespace cc {

// Order-preserving map from f32 to u32 (larger float <=> larger key); -0.0 ranks equal to +0.0.
__device__ __forceinline__ unsigned mono_key(float x) {
  unsigned b = __float_as_uint(__fadd_rn(x, 0.0f));
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ unsigned warp_sum(unsigned v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace cc
