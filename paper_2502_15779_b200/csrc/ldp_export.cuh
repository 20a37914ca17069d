// Export of a layer trained with learnable direct partitioning to the GEMV's inputs (Section 4.3:
// Eq. "partition", the grid t_i, Eq. "quant", Eq. "dequantgrid"; Section 4.4 Eq. "deqgrid"; the
// clipping range of Section 4.2). An offline, one-pass kernel: 2 bytes read and a quarter byte
// written per weight. One warp per quantization unit (G consecutive weights of a row): the range by
// shuffles, the three thresholds and four levels in fp32 with one rounding per operation (so the
// 2-bit decision is reproducible bit for bit), codes packed 16 to a word straight away.
#pragma once
#include "common.cuh"

namespace rcp {

struct LdpParams {
  const __half* w;     // [N][K] rotated weights
  const float* sb;     // [N][K/G] sigmoid(beta): lower clipping fraction
  const float* sg;     // sigmoid(gamma)
  const float* s1;     // sigmoid(s_1)
  const float* s2;     // sigmoid(s_2)
  uint32_t* words;     // [N][K/16]
  uint2* lut;          // [N][K/G] four fp16 levels
  int N, K, G;
  long long units;     // N * K / G
};

__global__ void __launch_bounds__(256) ldp_export_kernel(const LdpParams p) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int NG = p.K / p.G;
  for (long long u = warp0; u < p.units; u += nwarps) {
    const long long n = u / NG;
    const int j = (int)(u - n * NG);
    const __half* wu = p.w + n * p.K + (long long)j * p.G;
    // range of the unit: a lane takes 4 consecutive weights per round of 128
    float wmin = INFINITY, wmax = -INFINITY;
    for (int k0 = lane * 4; k0 < p.G; k0 += 128) {
      const uint2 raw = __ldg(reinterpret_cast<const uint2*>(wu + k0));
      const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
      const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
      wmin = fminf(fminf(wmin, fminf(a.x, a.y)), fminf(b.x, b.y));
      wmax = fmaxf(fmaxf(wmax, fmaxf(a.x, a.y)), fmaxf(b.x, b.y));
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      wmin = fminf(wmin, __shfl_xor_sync(0xffffffffu, wmin, d));
      wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, d));
    }
    const float lo = __fmul_rn(__ldg(p.sb + u), wmin);
    const float hi = __fmul_rn(__ldg(p.sg + u), wmax);
    const float h = __fsub_rn(hi, lo);
    const float p1 = __ldg(p.s1 + u), r2 = __ldg(p.s2 + u);
    const float rest = __fsub_rn(1.0f, p1);
    const float p2 = __fmul_rn(rest, r2);
    const float p3 = __fmul_rn(rest, __fsub_rn(1.0f, r2));
    const float t1 = __fdiv_rn(p1, 2.0f);
    const float t2 = __fadd_rn(t1, __fdiv_rn(__fadd_rn(p1, p2), 2.0f));
    const float t3 = __fadd_rn(t2, __fdiv_rn(__fadd_rn(p2, p3), 2.0f));
    const bool ok = h > 0.0f;
    if (lane == 0) {
      const float w1 = __fdiv_rn(__fadd_rn(t1, t2), 2.0f), w2 = __fdiv_rn(__fadd_rn(t2, t3), 2.0f);
      float lv[4] = {__fadd_rn(lo, __fmul_rn(h, 0.0f)), __fadd_rn(lo, __fmul_rn(h, w1)), __fadd_rn(lo, __fmul_rn(h, w2)), __fadd_rn(lo, __fmul_rn(h, 1.0f))};
      if (!ok) lv[0] = lv[1] = lv[2] = lv[3] = lo;
      const __half2 l01 = __halves2half2(__float2half_rn(lv[0]), __float2half_rn(lv[1]));
      const __half2 l23 = __halves2half2(__float2half_rn(lv[2]), __float2half_rn(lv[3]));
      uint2 out;
      out.x = *reinterpret_cast<const uint32_t*>(&l01);
      out.y = *reinterpret_cast<const uint32_t*>(&l23);
      p.lut[u] = out;
    }
    // codes: 4 per lane, 16 per group of four lanes = one packed word
    uint32_t* wordrow = p.words + n * (p.K / 16) + (long long)j * (p.G / 16);
    for (int k0 = lane * 4; k0 - lane * 4 < p.G; k0 += 128) {   // all lanes stay in the loop for the shuffles
      uint32_t byte = 0;
      if (k0 < p.G && ok) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(wu + k0));
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        const float v[4] = {a.x, a.y, b.x, b.y};
#pragma unroll
        for (int e = 0; e < 4; e++) {
          const float c = fminf(fmaxf(v[e], lo), hi);
          const float x = __fdiv_rn(__fsub_rn(c, lo), h);
          const uint32_t code = (uint32_t)(x >= t1) + (uint32_t)(x >= t2) + (uint32_t)(x >= t3);
          byte |= code << (2 * e);
        }
      }
      uint32_t word = byte << (8 * (lane & 3));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      if ((lane & 3) == 0 && k0 < p.G) wordrow[k0 >> 4] = word;
    }
  }
}

}  // namespace rcp
