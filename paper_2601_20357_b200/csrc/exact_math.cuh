// Order-independent decision arithmetic for the vocabulary-wide kernels.
//
// Token ids, accept counts and the weight argmax are integers decided by floating point
// (Algorithm 1 steps 6-7; Sec. 3 item 3; Sec. 4.1).  To make them independent of grid shape and
// scheduling every floating-point step below is ONE correctly rounded binary32 operation
// (the *_rn intrinsics are never contracted into fused multiply-adds), exp and log are built
// from such steps, and every sum over the vocabulary is a sum of integers: a probability q
// becomes the mass trunc(q * 2^40) before it is added.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tabed {

constexpr int   kMassBits  = 40;
constexpr float kMassScale = 1099511627776.0f;            // 2^40
constexpr float kMassInv   = 9.094947017729282e-13f;      // 2^-40
constexpr float kFltMin    = 1.17549435e-38f;

__device__ __forceinline__ float f32(uint32_t bits) { return __uint_as_float(bits); }

// exp(x) for x <= 0, exactly 0 below -80.
// n = rint(x*log2(e)); r = (x - n*LN2_HI) - n*LN2_LO; Horner of sum r^i/i!, i<=7; scale by 2^n.
__device__ __forceinline__ float xexp(float x) {
  if (x < -80.0f) return 0.0f;
  const float n = rintf(__fmul_rn(x, f32(0x3FB8AA3Bu)));            // log2(e)
  float r = __fsub_rn(x, __fmul_rn(n, f32(0x3F318000u)));            // 355/512
  r = __fsub_rn(r, __fmul_rn(n, f32(0xB95E8083u)));                  // ln2 - 355/512
  float p = f32(0x39500D01u);                                        // 1/5040
  p = __fadd_rn(__fmul_rn(p, r), f32(0x3AB60B61u));                  // 1/720
  p = __fadd_rn(__fmul_rn(p, r), f32(0x3C088889u));                  // 1/120
  p = __fadd_rn(__fmul_rn(p, r), f32(0x3D2AAAABu));                  // 1/24
  p = __fadd_rn(__fmul_rn(p, r), f32(0x3E2AAAABu));                  // 1/6
  p = __fadd_rn(__fmul_rn(p, r), 0.5f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  const int ni = (int)n;
  return __fmul_rn(p, __int_as_float((ni + 127) << 23));
}

// ln(x) for normal positive x.  x = m*2^e, m in (sqrt2/2, sqrt2]; s = (m-1)/(m+1);
// ln m = 2s(1 + s^2/3 + s^4/5 + s^6/7 + s^8/9); ln x = e*LN2_HI + (ln m + e*LN2_LO).
__device__ __forceinline__ float xlog(float x) {
  const uint32_t b = __float_as_uint(x);
  int e = (int)(b >> 23) - 127;
  float m = __uint_as_float((b & 0x007FFFFFu) | 0x3F800000u);
  if (m > f32(0x3FB504F3u)) { m = __fmul_rn(m, 0.5f); e += 1; }
  const float s = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
  const float z = __fmul_rn(s, s);
  float poly = f32(0x3DE38E39u);                                     // 1/9
  poly = __fadd_rn(__fmul_rn(poly, z), f32(0x3E124925u));            // 1/7
  poly = __fadd_rn(__fmul_rn(poly, z), f32(0x3E4CCCCDu));            // 1/5
  poly = __fadd_rn(__fmul_rn(poly, z), f32(0x3EAAAAABu));            // 1/3
  poly = __fadd_rn(__fmul_rn(poly, z), 1.0f);
  const float lnm = __fmul_rn(__fadd_rn(s, s), poly);
  const float ef = (float)e;
  return __fadd_rn(__fmul_rn(ef, f32(0x3F318000u)),
                   __fadd_rn(lnm, __fmul_rn(ef, f32(0xB95E8083u))));
}

// integer mass of a non-negative probability
__device__ __forceinline__ unsigned long long mass_of(float q) {
  return __float2ull_rz(__fmul_rn(q, kMassScale));
}
// normaliser S = float(sum of masses) * 2^-40
__device__ __forceinline__ float norm_of(unsigned long long total) {
  return __fmul_rn(__ull2float_rn(total), kMassInv);
}

// order-preserving map float -> uint32 so that a maximum can be taken with an integer atomic
__device__ __forceinline__ uint32_t ord_encode(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_decode(uint32_t u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// threshold of the inverse-CDF draw: ((2k+1) * T) >> 24 with k = floor(u * 2^23)
__device__ __forceinline__ unsigned long long draw_threshold(float u, unsigned long long T) {
  const unsigned long long k2 = 2ull * (unsigned long long)__float2uint_rd(__fmul_rn(u, 8388608.0f)) + 1ull;
  const unsigned long long lo = k2 * T;
  const unsigned long long hi = __umul64hi(k2, T);
  return (hi << 40) | (lo >> 24);
}

// ---- warp / block reductions -------------------------------------------------------------
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ long long warp_sum_i64(long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

}  // namespace tabed
