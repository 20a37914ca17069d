// Fused activation path: block-Hadamard rotation (Appendix A.2, normalized Sylvester matrix) ->
// per-token absmax symmetric int4 quantization -> nibble packing (Section 4.4 tensor formats).
//
// A token is one vector of K elements and the whole job is latency: a thread-block cluster of C
// CTAs (1, 2, 4 or 8) shares it, each CTA a contiguous slice, every thread 8 consecutive
// elements. The butterfly strides run in ascending order: 1,2,4 inside the thread's registers,
// 8..128 by warp shuffles, 256 up to the slice through the CTA's shared memory in radix-8 passes,
// and the strides that span slices (a rotation block larger than a slice) across the cluster:
// every CTA reads the partner slices through distributed shared memory and redoes the small
// butterfly network over the ranks, keeping its own output. Each butterfly is one fp32 add and
// one fp32 subtract (lower index first), then one fp32 multiply by 1/sqrt(B): the rounding order
// is fixed, so the int4 decision is reproducible bit for bit. The token's absmax meets in
// distributed shared memory as well.
#pragma once
#include "common.cuh"

namespace rcp {

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// reads a float at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ float ld_cluster_f32(const float* local, uint32_t rank) {
  const uint32_t laddr = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(rank));
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(raddr) : "memory");
  return v;
}
// the same for four consecutive floats (16-byte aligned)
__device__ __forceinline__ float4 ld_cluster_f32x4(const float* local, uint32_t rank) {
  const uint32_t laddr = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(rank));
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(raddr)
               : "memory");
  return v;
}

struct QuantParams {
  const __half* x;
  uint8_t* xq;
  __half* scale;
  int K, B, lgB;
  int unit, nunits;     // cross == 1: the token is shared out in units of `unit` elements (a multiple of B and 64)
  int slice;            // cross > 1: elements per CTA (a power of two, 256 .. 8192), K == B == cross * slice
  int lg_local;         // B > 256: log2 of min(B, slice): strides below it stay inside the CTA
  int cross;            // CTAs one rotation block is split over (1, 2, 4 or 8)
  float inv_sqrt_b, clip_ratio;
};

// C = CTAs per token (the cluster size; grid = tokens * C)
template <int C>
__global__ void __launch_bounds__(1024) quantize_act_kernel(const QuantParams p) {
  extern __shared__ float sbuf[];   // 8 floats per thread when B > 256
  __shared__ float s_red[32];
  __shared__ float s_amax;
  const int m = blockIdx.x / C;
  const uint32_t rank = blockIdx.x % C;   // == %cluster_ctarank for a cluster of C along x
  const int tid = threadIdx.x, lane = tid & 31;
  const int B = p.B;
  // Launched with programmatic stream serialization: let the next kernel get started, then wait
  // for the kernel before this one, whose output x may be and whose input xq and scale may be.
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // this CTA's slice of the token
  int start, len;
  if (p.cross == 1) {
    const int u0 = (int)((long long)p.nunits * rank / C), u1 = (int)((long long)p.nunits * (rank + 1) / C);
    start = u0 * p.unit;
    len = (u1 - u0) * p.unit;
  } else {
    start = (int)rank * p.slice;
    len = p.slice;
  }
  const int base = start + tid * 8;
  const bool mine = tid * 8 < len;
  const __half* xm = p.x + (size_t)m * p.K;

  float v[8];
  if (mine) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xm + base));
    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float2 f = __half22float2(h2[e]);
      v[2 * e] = f.x;
      v[2 * e + 1] = f.y;
    }
  } else {
#pragma unroll
    for (int e = 0; e < 8; e++) v[e] = 0.f;
  }

  if (B > 1) {
    // strides 1, 2, 4: inside the registers
#pragma unroll
    for (int h = 1; h < 8; h *= 2) {
      if (h < B) {
#pragma unroll
        for (int e = 0; e < 8; e++) {
          if ((e & h) == 0) {
            const float u = v[e], w = v[e + h];
            v[e] = __fadd_rn(u, w);
            v[e + h] = __fsub_rn(u, w);
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
          const float other = __shfl_xor_sync(0xffffffffu, v[e], d);
          v[e] = upper ? __fsub_rn(other, v[e]) : __fadd_rn(v[e], other);
        }
      }
    }
    if (B > 256) {
      // strides 256 .. below min(B, slice): passes of up to three strides (radix 8) through shared
      // memory. A pass over strides s, 2s, .. (r = 2, 4 or 8 of them combined) works on tuples of r
      // elements s apart; the tuple index maps to an element index with shifts only:
      // element = ((tuple >> log2 s) << log2(r s)) | (tuple & (s - 1)), plus j s for the j-th member.
#pragma unroll
      for (int e = 0; e < 8; e++) sbuf[tid * 8 + e] = v[e];
      __syncthreads();
      for (int ls = 8; ls < p.lg_local;) {
        const int lr = min(3, p.lg_local - ls);   // log2 of the radix of this pass
        float w[8];
        int idx[8];
#pragma unroll
        for (int e = 0; e < 8; e++) {
          const int tau = (tid << (3 - lr)) + (e >> lr);   // tuple index over the slice
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
      if constexpr (C > 1) {
        if (p.cross > 1) {
          // strides slice .. B/2: the partner elements sit at the same offset in the other CTAs of
          // an aligned group of `cross` ranks; run the butterflies over the ranks, keep this rank's
          cluster_sync_all();
          const uint32_t g0 = rank & ~(uint32_t)(p.cross - 1), me = rank - g0;
          float w[C][8];
#pragma unroll
          for (int r = 0; r < C; r++) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            if (r < p.cross) {
              a = ld_cluster_f32x4(&sbuf[tid * 8], g0 + r);
              b = ld_cluster_f32x4(&sbuf[tid * 8 + 4], g0 + r);
            }
            w[r][0] = a.x; w[r][1] = a.y; w[r][2] = a.z; w[r][3] = a.w;
            w[r][4] = b.x; w[r][5] = b.y; w[r][6] = b.z; w[r][7] = b.w;
          }
#pragma unroll
          for (int e = 0; e < 8; e++) {
#pragma unroll
            for (int h = 1; h < C; h *= 2) {
              if (h < p.cross) {
#pragma unroll
                for (int r = 0; r < C; r++) {
                  if ((r & h) == 0) {
                    const float u = w[r][e], z = w[r + h][e];
                    w[r][e] = __fadd_rn(u, z);
                    w[r + h][e] = __fsub_rn(u, z);
                  }
                }
              }
            }
            float out = w[0][e];
#pragma unroll
            for (int r = 1; r < C; r++) out = (me == (uint32_t)r) ? w[r][e] : out;
            v[e] = out;
          }
        } else {
#pragma unroll
          for (int e = 0; e < 8; e++) v[e] = sbuf[tid * 8 + e];
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; e++) v[e] = sbuf[tid * 8 + e];
      }
    }
#pragma unroll
    for (int e = 0; e < 8; e++) v[e] = __fmul_rn(v[e], p.inv_sqrt_b);
  }

  // token-wide absmax: warp, CTA, cluster
  float amax = 0.f;
#pragma unroll
  for (int e = 0; e < 8; e++) amax = fmaxf(amax, fabsf(v[e]));
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  if (lane == 0) s_red[tid >> 5] = amax;
  __syncthreads();
  if (tid < 32) {
    float a = (tid < (int)((blockDim.x + 31) >> 5)) ? s_red[tid] : 0.f;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, d));
    if (tid == 0) s_amax = a;
  }
  if constexpr (C > 1) {
    cluster_sync_all();   // every CTA's s_amax is written (and every partner read of sbuf is done)
    amax = 0.f;
#pragma unroll
    for (int r = 0; r < C; r++) amax = fmaxf(amax, ld_cluster_f32(&s_amax, r));
    cluster_sync_all();   // nobody leaves while a partner may still read its shared memory
  } else {
    __syncthreads();
    amax = s_amax;
  }

  const float s32 = __fdiv_rn(__fmul_rn(amax, p.clip_ratio), 7.0f);
  const __half s16 = __float2half_rn(s32);
  const float s = __half2float(s16);
  if (rank == 0 && tid == 0) p.scale[m] = s16;

  if (mine) {
    uint32_t packed = 0;
    if (s != 0.f) {
#pragma unroll
      for (int e = 0; e < 8; e++) {
        int q = __float2int_rn(__fdiv_rn(v[e], s));
        q = max(-8, min(7, q));
        packed |= (uint32_t)(q & 0xF) << (4 * e);
      }
    }
    *reinterpret_cast<uint32_t*>(p.xq + (size_t)m * (p.K / 2) + base / 2) = packed;
  }
}

}  // namespace rcp
