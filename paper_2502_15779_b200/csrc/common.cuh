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
