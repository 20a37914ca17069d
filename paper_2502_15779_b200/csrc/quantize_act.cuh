// Fused activation path: block-Hadamard rotation (Appendix A.2, normalized Sylvester matrix) ->
// per-token absmax symmetric int4 quantization -> nibble packing (Section 4.4 tensor formats).
//
// One CTA per token. Every thread owns groups of 8 consecutive elements, so the butterfly
// strides run in ascending order: 1,2,4 inside the thread's registers, 8..128 by warp
// shuffles, 256 and above through shared memory in radix-8 passes. Each butterfly is one fp32
// add and one fp32 subtract (lower index first), then one fp32 multiply by 1/sqrt(B): the
// rounding order is fixed, so the int4 decision is reproducible bit for bit.
#pragma once
#include "common.cuh"

namespace rcp {

template <int G>
__global__ void __launch_bounds__(1024) quantize_act_kernel(const __half* __restrict__ x, int K, int B, int lgB,
                                                            float inv_sqrt_b, float clip_ratio,
                                                            uint8_t* __restrict__ xq,
                                                            __half* __restrict__ scale) {
  extern __shared__ float sbuf[];  // 8 * blockDim.x floats when B > 256
  __shared__ float s_red[32];
  const int m = blockIdx.x;
  const int T = blockDim.x;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const __half* xm = x + (size_t)m * K;
  // Launched with programmatic stream serialization: let the next kernel get started, then wait
  // for the kernel before this one, whose output x may be and whose input xq and scale may be.
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  float v[G][8];
#pragma unroll
  for (int g = 0; g < G; g++) {
    const int base = (g * T + tid) * 8;
    if (base < K) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xm + base));
      const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const float2 f = __half22float2(h2[e]);
        v[g][2 * e] = f.x;
        v[g][2 * e + 1] = f.y;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; e++) v[g][e] = 0.f;
    }
  }

  if (B > 1) {
#pragma unroll
    for (int g = 0; g < G; g++) {
      // strides 1, 2, 4: inside the registers
#pragma unroll
      for (int h = 1; h < 8; h *= 2) {
        if (h < B) {
#pragma unroll
          for (int e = 0; e < 8; e++) {
            if ((e & h) == 0) {
              const float u = v[g][e], w = v[g][e + h];
              v[g][e] = __fadd_rn(u, w);
              v[g][e + h] = __fsub_rn(u, w);
            }
          }
        }
      }
      // strides 8 .. 128: lane exchanges (element stride 8*d <-> lane distance d)
#pragma unroll
      for (int d = 1; d < 32; d *= 2) {
        if (8 * d < B) {
          const bool upper = (lane & d) != 0;
#pragma unroll
          for (int e = 0; e < 8; e++) {
            const float other = __shfl_xor_sync(0xffffffffu, v[g][e], d);
            v[g][e] = upper ? __fsub_rn(other, v[g][e]) : __fadd_rn(v[g][e], other);
          }
        }
      }
    }
    // strides 256 and above: passes of up to three strides (radix 8) through shared memory.
    // A pass over strides s, 2s, .. (r = 2, 4 or 8 of them combined) works on tuples of r elements
    // s apart; B is a multiple of r s, so the tuple index maps to an element index with shifts only:
    // element = ((tuple >> log2 s) << log2(r s)) | (tuple & (s - 1)), plus j s for the j-th member.
    if (B > 256) {
#pragma unroll
      for (int g = 0; g < G; g++) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 8; e++) sbuf[tid * 8 + e] = v[g][e];
        __syncthreads();
        for (int ls = 8; ls < lgB;) {
          const int lr = min(3, lgB - ls);   // log2 of the radix of this pass
          float w[8];
          int idx[8];
#pragma unroll
          for (int e = 0; e < 8; e++) {
            const int tau = (tid << (3 - lr)) + (e >> lr);   // tuple index over the whole buffer
            const int j = e & ((1 << lr) - 1);
            idx[e] = ((tau >> ls) << (ls + lr)) + (tau & ((1 << ls) - 1)) + (j << ls);
            w[e] = sbuf[idx[e]];
          }
#pragma unroll
          for (int t = 0; t < 3; t++) {
            const int hh = 1 << t;  // tuple-local stride
            if (t < lr) {
#pragma unroll
              for (int e = 0; e < 8; e++) {
                if ((e & hh) == 0) {
                  const float u = w[e], z = w[e + hh];
                  w[e] = __fadd_rn(u, z);
                  w[e + hh] = __fsub_rn(u, z);
                }
              }
            }
          }
#pragma unroll
          for (int e = 0; e < 8; e++) sbuf[idx[e]] = w[e];
          __syncthreads();
          ls += lr;
        }
#pragma unroll
        for (int e = 0; e < 8; e++) v[g][e] = sbuf[tid * 8 + e];
      }
    }
#pragma unroll
    for (int g = 0; g < G; g++)
#pragma unroll
      for (int e = 0; e < 8; e++) v[g][e] = __fmul_rn(v[g][e], inv_sqrt_b);
  }

  // token-wide absmax
  float amax = 0.f;
#pragma unroll
  for (int g = 0; g < G; g++)
#pragma unroll
    for (int e = 0; e < 8; e++) amax = fmaxf(amax, fabsf(v[g][e]));
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  __syncthreads();
  if (lane == 0) s_red[tid >> 5] = amax;
  __syncthreads();
  amax = 0.f;
  for (int w = 0; w < (T + 31) / 32; w++) amax = fmaxf(amax, s_red[w]);

  const float s32 = __fdiv_rn(__fmul_rn(amax, clip_ratio), 7.0f);
  const __half s16 = __float2half_rn(s32);
  const float s = __half2float(s16);
  if (tid == 0) scale[m] = s16;

  uint8_t* xqm = xq + (size_t)m * (K / 2);
#pragma unroll
  for (int g = 0; g < G; g++) {
    const int base = (g * T + tid) * 8;
    if (base < K) {
      uint32_t packed = 0;
#pragma unroll
      for (int e = 0; e < 8; e++) {
        int q = 0;
        if (s != 0.f) {
          q = __float2int_rn(__fdiv_rn(v[g][e], s));
          q = max(-8, min(7, q));
        }
        packed |= (uint32_t)(q & 0xF) << (4 * e);
      }
      *reinterpret_cast<uint32_t*>(xqm + base / 2) = packed;
    }
  }
}

}  // namespace rcp
