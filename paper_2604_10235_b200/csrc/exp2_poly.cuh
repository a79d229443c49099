// 2^x helpers shared by the score kernel, the chunk-scoring kernel and the throughput probe:
// the special-function instruction, the FMA-pipe polynomial, and the packed f32x2 arithmetic
// that the inner loops are written in.
#pragma once

#include <stdint.h>

namespace cc {

constexpr float kEx2Magic = 12582912.0f;         // 1.5 * 2^23: adding it rounds to the nearest integer
// degree-3 minimax polynomial of 2^f on [-0.5, 0.5], relative error 7.8e-5
constexpr float kEx2C3 = 0.05516434833407402f;
constexpr float kEx2C2 = 0.24259322881698608f;
constexpr float kEx2C1 = 0.693260669708252f;
constexpr float kEx2C0 = 0.9999293088912964f;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x on the FMA pipe: x = n + f with n = round(x) taken from the low mantissa bits of
// x + 1.5 * 2^23, 2^f by the polynomial, n added into the exponent field.  Arguments are
// clamped at -125 so that the exponent never wraps (2^-125 is far below anything a score or a
// likelihood can resolve); the caller keeps x below 127.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -125.0f);
  const float t = x + kEx2Magic;
  const float f = x - (t - kEx2Magic);
  float p = fmaf(f, kEx2C3, kEx2C2);
  p = fmaf(p, f, kEx2C1);
  p = fmaf(p, f, kEx2C0);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// packed f32x2 arithmetic (two values in a 64-bit register pair per instruction)
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for a pair on the special-function unit
__device__ __forceinline__ uint64_t ex2_pair_sfu(uint64_t x) {
  float a, b;
  unpack2(x, a, b);
  return pack2(ex2(a), ex2(b));
}
// 2^x for a pair on the FMA pipe (packed form of ex2_poly, same clamp)
__device__ __forceinline__ uint64_t ex2_pair_fma(uint64_t x) {
  float a, b;
  unpack2(x, a, b);
  x = pack2(fmaxf(a, -125.0f), fmaxf(b, -125.0f));
  const uint64_t magic = pack2(kEx2Magic, kEx2Magic);
  const uint64_t t = add2(x, magic);
  const uint64_t f = sub2(x, sub2(t, magic));
  uint64_t p = fma2(f, pack2(kEx2C3, kEx2C3), pack2(kEx2C2, kEx2C2));
  p = fma2(p, f, pack2(kEx2C1, kEx2C1));
  p = fma2(p, f, pack2(kEx2C0, kEx2C0));
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(t, t0, t1);
  // p * 2^n: n (low mantissa bits of t) shifted into the exponent field by one multiply-add
  int r0, r1;
  asm("mad.lo.s32 %0, %1, 8388608, %2;" : "=r"(r0) : "r"(__float_as_int(t0)), "r"(__float_as_int(p0)));
  asm("mad.lo.s32 %0, %1, 8388608, %2;" : "=r"(r1) : "r"(__float_as_int(t1)), "r"(__float_as_int(p1)));
  return pack2(__int_as_float(r0), __int_as_float(r1));
}

#ifndef CC_POLY_EVERY
#define CC_POLY_EVERY 3
#endif
constexpr int kPolyEvery = CC_POLY_EVERY;        // one pair in this many takes the polynomial path

// acc += 2^(v * c + off) over the first kWidth of 32 values; off is one pair for all of them or
// read per value from shared memory (off_col: shared-space address of the first value's offset).
// Of every kPolyEvery pairs one goes to the FMA pipe, the
// others to the special-function unit.
template <bool kPerColumn, int kWidth>
__device__ __forceinline__ void exp_accumulate(const uint32_t (&v)[32], uint64_t c2, uint64_t off2,
                                               uint32_t off_col, uint64_t (&acc)[4]) {
#pragma unroll
  for (int i = 0; i < kWidth; i += 4) {
    uint64_t o[2] = {off2, off2};
    if (kPerColumn) {
      // off_col is the shared-space address of the offsets: a shared-space load at a constant
      // distance from it needs no address arithmetic per load
      float4 L;
      asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                   : "=f"(L.x), "=f"(L.y), "=f"(L.z), "=f"(L.w)
                   : "r"(off_col + (uint32_t)(i * 4)));
      o[0] = pack2(L.x, L.y);
      o[1] = pack2(L.z, L.w);
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int pair = (i >> 1) + k;
      const uint64_t x = fma2(pack2(__uint_as_float(v[i + 2 * k]), __uint_as_float(v[i + 2 * k + 1])), c2, o[k]);
      if (pair % kPolyEvery == kPolyEvery - 1) acc[3] = add2(acc[3], ex2_pair_fma(x));
      else acc[pair % 3] = add2(acc[pair % 3], ex2_pair_sfu(x));
    }
  }
}
__device__ __forceinline__ float acc_total(const uint64_t (&acc)[4]) {
  float a, b, c, d;
  unpack2(add2(acc[0], acc[1]), a, b);
  unpack2(add2(acc[2], acc[3]), c, d);
  return (a + b) + (c + d);
}

}  // namespace cc
