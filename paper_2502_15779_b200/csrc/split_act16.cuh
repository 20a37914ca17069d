// Weight-only form of the GEMV (Section 5, W2-only setting): fp16 activations as block fixed point.
// Per token, E = floor(log2(max |x|)); X = round-half-even(x * 2^(21 - E)) is an integer below 2^22 in
// magnitude (exactly x for every element within 2^-11 of the maximum, half a unit off at most otherwise);
// X = q0 + 64 q1 + 64^2 q2 + 64^3 q3 with q0..q2 in [-32, 31]. The four digit planes are four int8
// "tokens" of the integer GEMV, with units 2^(E - 21) * 64^d.
#pragma once
#include <cuda_fp16.h>
#include <cstdint>

namespace rcp {

constexpr int kSplitThreads = 512;

// floor(log2) of the largest magnitude of a token from its fp16 bit pattern (0 for an all-zero token)
__device__ __forceinline__ int split_exponent(unsigned amax_bits) {
  if (amax_bits >= 0x0400u) return (int)(amax_bits >> 10) - 15;        // normal
  if (amax_bits > 0u) return (31 - __clz((int)amax_bits)) - 24;        // subnormal: mantissa * 2^-24
  return 0;
}
// largest magnitude bit pattern among the eight fp16 values of v
__device__ __forceinline__ unsigned split_amax8(uint4 v, unsigned amax) {
  const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; j++) {
    amax = max(amax, w[j] & 0x7FFFu);
    amax = max(amax, (w[j] >> 16) & 0x7FFFu);
  }
  return amax;
}
// the four digit planes of eight consecutive fp16 values: out[d] = eight signed bytes of digit d
__device__ __forceinline__ void split_digits8(uint4 v, float mult, uint32_t (&out)[4][2]) {
  const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int d = 0; d < 4; d++) { out[d][0] = 0; out[d][1] = 0; }
#pragma unroll
  for (int j = 0; j < 8; j++) {
    const __half h = __ushort_as_half((unsigned short)(j & 1 ? w[j >> 1] >> 16 : w[j >> 1] & 0xFFFFu));
    int X = __float2int_rn(__fmul_rn(__half2float(h), mult));   // exact product, half-to-even
#pragma unroll
    for (int d = 0; d < 4; d++) {
      int q = X;
      if (d < 3) {
        q = ((X + 32) & 63) - 32;   // residue in [-32, 31]
        X = (X - q) >> 6;           // divisible: the shift is exact
      }
      out[d][j >> 2] |= (uint32_t)(q & 0xFF) << (8 * (j & 3));
    }
  }
}

// grid: one CTA per token. digits [M][4][K] int8, unit [M][4] fp32. K % 8 == 0, x 16-byte aligned.
__global__ void __launch_bounds__(kSplitThreads) split_act16_kernel(const __half* __restrict__ x, int K,
                                                                     int8_t* __restrict__ digits,
                                                                     float* __restrict__ unit) {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __shared__ unsigned s_max[kSplitThreads / 32];
  const int m = blockIdx.x, tid = threadIdx.x;
  const uint4* const xv = reinterpret_cast<const uint4*>(x + (size_t)m * K);
  const int nvec = K / 8;
  // largest magnitude: the bit patterns of finite fp16 magnitudes order like the values
  unsigned amax = 0;
  for (int i = tid; i < nvec; i += kSplitThreads) amax = split_amax8(__ldg(xv + i), amax);
  amax = __reduce_max_sync(0xffffffffu, amax);
  if ((tid & 31) == 0) s_max[tid >> 5] = amax;
  __syncthreads();
  amax = 0;
#pragma unroll
  for (int i = 0; i < kSplitThreads / 32; i++) amax = max(amax, s_max[i]);
  const int E = split_exponent(amax);
  const float mult = __int_as_float((21 - E + 127) << 23);  // 2^(21 - E), between 2^6 and 2^45
  if (tid < 4) unit[m * 4 + tid] = __int_as_float((E - 21 + 6 * tid + 127) << 23);
  int8_t* const dg = digits + (size_t)m * 4 * K;
  for (int i = tid; i < nvec; i += kSplitThreads) {
    uint32_t out[4][2];
    split_digits8(__ldg(xv + i), mult, out);
#pragma unroll
    for (int d = 0; d < 4; d++)
      *reinterpret_cast<uint2*>(dg + (size_t)d * K + (size_t)i * 8) = make_uint2(out[d][0], out[d][1]);
  }
}

}  // namespace rcp
