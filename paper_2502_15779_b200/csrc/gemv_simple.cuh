// Reference-shaped GEMV kernel: one warp per (row, token), scalar decode of every code.
// Used for S_dbg (it materialises the exact per-code sums S_c) and for shapes the tuned
// variants do not take. Section 4.4: O = S * X_q * LUT[W_q].
#pragma once
#include "common.cuh"

namespace rcp {

__global__ void __launch_bounds__(256) gemv_simple_kernel(const uint32_t* __restrict__ words,
                                                          const uint2* __restrict__ lut,
                                                          const uint8_t* __restrict__ xq,
                                                          const __half* __restrict__ scale, int M, int N,
                                                          int K, __half* __restrict__ y,
                                                          int32_t* __restrict__ S_dbg) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= N) return;
  const int n = warp;
  const int W = K / 16;
  const uint32_t* wrow = words + (size_t)n * W;
  for (int m = 0; m < M; m++) {
    const uint2* xrow = reinterpret_cast<const uint2*>(xq + (size_t)m * (K / 2));
    int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    for (int w = lane; w < W; w += 32) {
      const uint32_t cw = __ldg(wrow + w);
      const uint2 xa = __ldg(xrow + w);  // 16 nibbles
#pragma unroll
      for (int j = 0; j < 16; j++) {
        const uint32_t nib = ((j < 8 ? xa.x : xa.y) >> (4 * (j & 7))) & 0xFu;
        const int q = sext4(nib);
        const uint32_t c = (cw >> (2 * j)) & 3u;
        s0 += (c == 0) ? q : 0;
        s1 += (c == 1) ? q : 0;
        s2 += (c == 2) ? q : 0;
        s3 += (c == 3) ? q : 0;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      s0 += __shfl_xor_sync(0xffffffffu, s0, d);
      s1 += __shfl_xor_sync(0xffffffffu, s1, d);
      s2 += __shfl_xor_sync(0xffffffffu, s2, d);
      s3 += __shfl_xor_sync(0xffffffffu, s3, d);
    }
    if (lane == 0) {
      y[(size_t)m * N + n] = lut_finish(__half2float(scale[m]), __ldg(lut + n), s0, s1, s2, s3);
      if (S_dbg) {
        int4 out = make_int4(s0, s1, s2, s3);
        *reinterpret_cast<int4*>(S_dbg + ((size_t)m * N + n) * 4) = out;
      }
    }
  }
}

// Group-wise grid (Section 4.4: the grid has one four-entry row per group of G weights of an
// output row): lut is [N][K/G][4]. One warp per row, a lane takes whole groups, so the exact
// per-group per-code sums S_c[m][n][j] exist in registers and can be exported.
__global__ void __launch_bounds__(256) gemv_simple_grouped_kernel(const uint32_t* __restrict__ words,
                                                                  const uint2* __restrict__ lut,
                                                                  const uint8_t* __restrict__ xq,
                                                                  const __half* __restrict__ scale, int M, int N,
                                                                  int K, int G, __half* __restrict__ y,
                                                                  int32_t* __restrict__ S_dbg) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= N) return;
  const int n = warp;
  const int W = K / 16, NG = K / G, WG = G / 16;
  const uint32_t* wrow = words + (size_t)n * W;
  for (int m = 0; m < M; m++) {
    const uint2* xrow = reinterpret_cast<const uint2*>(xq + (size_t)m * (K / 2));
    float acc = 0.f;
    for (int j = lane; j < NG; j += 32) {
      int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
      for (int w = j * WG; w < (j + 1) * WG; w++) {
        const uint32_t cw = __ldg(wrow + w);
        const uint2 xa = __ldg(xrow + w);  // 16 nibbles
#pragma unroll
        for (int i = 0; i < 16; i++) {
          const uint32_t nib = ((i < 8 ? xa.x : xa.y) >> (4 * (i & 7))) & 0xFu;
          const int q = sext4(nib);
          const uint32_t c = (cw >> (2 * i)) & 3u;
          s0 += (c == 0) ? q : 0;
          s1 += (c == 1) ? q : 0;
          s2 += (c == 2) ? q : 0;
          s3 += (c == 3) ? q : 0;
        }
      }
      acc += lut_dot(__ldg(lut + (size_t)n * NG + j), s0, s1, s2, s3);
      if (S_dbg) *reinterpret_cast<int4*>(S_dbg + (((size_t)m * N + n) * NG + j) * 4) = make_int4(s0, s1, s2, s3);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) y[(size_t)m * N + n] = __float2half_rn(__half2float(scale[m]) * acc);
  }
}

}  // namespace rcp
