// Shared device/host helpers of the RCP W2A4 library (sm_100a).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rcp {

constexpr int kMaxTokens = 16;   // skinny regime of the GEMV
constexpr int kMaxK = 65536;

__device__ __forceinline__ int sext4(uint32_t nib) { return (int)((nib ^ 8u) & 0xFu) - 8; }

// y = s * (L0*S0 + L1*S1 + L2*S2 + L3*S3), fp32 arithmetic, integers converted exactly (|S| < 2^24).
__device__ __forceinline__ __half lut_finish(float s, uint2 lut4, int S0, int S1, int S2, int S3) {
  const __half2 l01 = *reinterpret_cast<const __half2*>(&lut4.x);
  const __half2 l23 = *reinterpret_cast<const __half2*>(&lut4.y);
  float acc = __half2float(__low2half(l01)) * (float)S0;
  acc = fmaf(__half2float(__high2half(l01)), (float)S1, acc);
  acc = fmaf(__half2float(__low2half(l23)), (float)S2, acc);
  acc = fmaf(__half2float(__high2half(l23)), (float)S3, acc);
  return __float2half_rn(s * acc);
}

// L0*S0 + L1*S1 + L2*S2 + L3*S3 alone, in the same order and arithmetic.
__device__ __forceinline__ float lut_sum(uint2 lut4, int S0, int S1, int S2, int S3) {
  const __half2 l01 = *reinterpret_cast<const __half2*>(&lut4.x);
  const __half2 l23 = *reinterpret_cast<const __half2*>(&lut4.y);
  float acc = __half2float(__low2half(l01)) * (float)S0;
  acc = fmaf(__half2float(__high2half(l01)), (float)S1, acc);
  acc = fmaf(__half2float(__low2half(l23)), (float)S2, acc);
  acc = fmaf(__half2float(__high2half(l23)), (float)S3, acc);
  return acc;
}

// q[e] = clamp(round-half-even(v[e] / s), -8, 7) for NV values, the quotient being the IEEE fp32
// division the definition asks for, without dividing in the common case. With rinv = 1 / s (correctly
// rounded), t = v * rinv lies within 2^-23 |v / s| of the exact quotient and the IEEE quotient within half
// an ulp of it; clamped to [-8, 7] (rounding and clamping commute: the bounds are integers) the two differ
// by less than 1.7e-6, so they round to the same integer unless t lies that close to a half-integer.
// Only then (and on exact ties) does the warp redo its values with the division itself; the vote keeps
// the warp together. Rounding: adding 1.5 * 2^23 leaves the rounded integer in the low mantissa bits.
// s > 0 and finite. Every lane of the warp must call.
template <int NV>
__device__ __forceinline__ void quantize_int4(const float (&v)[NV], float s, int (&q)[NV]) {
  const float rinv = __frcp_rn(s);
  bool doubt = false;
#pragma unroll
  for (int e = 0; e < NV; e++) {
    const float t = fminf(fmaxf(__fmul_rn(v[e], rinv), -8.f), 7.f);
    const float biased = __fadd_rn(t, 12582912.f);
    q[e] = __float_as_int(biased) - 0x4B400000;
    doubt |= fabsf(__fsub_rn(t, __fsub_rn(biased, 12582912.f))) > 0.499996f;
  }
  if (__any_sync(0xffffffffu, doubt)) {
#pragma unroll
    for (int e = 0; e < NV; e++) q[e] = max(-8, min(7, __float2int_rn(__fdiv_rn(v[e], s))));
  }
}

// One group's term of the group-wise form: L0*S0 + L1*S1 + L2*S2 + L3*S3 in fp32.
__device__ __forceinline__ float lut_dot(uint2 lut4, int S0, int S1, int S2, int S3) {
  const float2 l01 = __half22float2(*reinterpret_cast<const __half2*>(&lut4.x));
  const float2 l23 = __half22float2(*reinterpret_cast<const __half2*>(&lut4.y));
  float acc = l01.x * (float)S0;
  acc = fmaf(l01.y, (float)S1, acc);
  acc = fmaf(l23.x, (float)S2, acc);
  acc = fmaf(l23.y, (float)S3, acc);
  return acc;
}

}  // namespace rcp
