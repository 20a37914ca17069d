// Fused activation path: block-Hadamard rotation (Appendix A.2, normalized Sylvester matrix) ->
// per-token absmax symmetric int4 quantization -> nibble packing (Section 4.4 tensor formats).
//
// A token is one vector of K elements and the whole job is latency: a thread-block cluster of C
// CTAs (1, 2, 4 or 8) shares it, each CTA whole rotation blocks, every thread 8 consecutive
// elements. The butterfly strides run in ascending order: 1,2,4 inside the thread's registers,
// 8..128 by warp shuffles, 256 and up through the CTA's shared memory in radix-8 passes. (A rotation
// block never spans CTAs: one block over a token of 4096 or 8192 elements takes the one-CTA kernel
// further down, shorter tokens fit one CTA.) Each butterfly is one fp32 add and one fp32 subtract
// (lower index first), then one fp32 multiply by 1/sqrt(B): the rounding order is fixed, so the int4
// decision is reproducible bit for bit. The token's absmax meets in distributed shared memory.
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

struct QuantParams {
  const __half* x;
  uint8_t* xq;
  __half* scale;
  int K, B, lgB;
  int unit, nunits;     // the token is shared out over the cluster in units of `unit` elements (a multiple of B and 64)
  int lg_local;         // B > 256: log2 B, the strides that go through shared memory end below it
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
  const int u0 = (int)((long long)p.nunits * rank / C), u1 = (int)((long long)p.nunits * (rank + 1) / C);
  const int start = u0 * p.unit, len = (u1 - u0) * p.unit;
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
      // strides 256 .. B/2: passes of up to three strides (radix 8) through shared
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
#pragma unroll
      for (int e = 0; e < 8; e++) v[e] = sbuf[tid * 8 + e];
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

  int q[8];
  if (s != 0.f) {   // the same for the whole cluster; threads beyond the slice hold zeros
    quantize_int4<8>(v, s, q);
  } else {
#pragma unroll
    for (int e = 0; e < 8; e++) q[e] = 0;
  }
  if (mine) {
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 8; e++) packed |= (uint32_t)(q[e] & 0xF) << (4 * e);
    *reinterpret_cast<uint32_t*>(p.xq + (size_t)m * (p.K / 2) + base / 2) = packed;
  }
}

// ---------------------------------------------------------------------------------------------
// One token of W = K / 16 words (256 or 512) under a single rotation block, by NT = 512 threads of one
// CTA: thread tid holds word tid (16 consecutive activations). Every butterfly stage runs in registers, the
// data changing hands through shared memory in between, in ascending order of the strides (the order of
// quantize_act_kernel: same operations on the same operands, bit-identical results):
//   strides 1..8      inside the word;
//   strides 16..128   after a transposition inside the warp (thread (h, e) of a warp, h = lane >> 4,
//                     e = lane & 15, takes element e of the warp's words 16 h .. 16 h + 15);
//   stride 256        one lane exchange (lane ^ 16);
//   strides 512 ..    after a transposition across the warps (thread (warp = element, lane) takes the
//                     R = W / 32 values of its column, 32 words apart);
// then the scale by 1/sqrt(K) and the token's absmax. Leaves the rotated, scaled activations of the thread's
// word in v and returns the quantization scale (as rounded to fp16). Uses named barrier 1 with NT threads;
// qbuf: rotate_scratch_bytes(K) bytes, 16-byte aligned; s_amax: NT / 32 floats.
__host__ __device__ constexpr size_t rotate_scratch_bytes(int K) { return (size_t)17 * (K / 16) * 4; }

template <int NT>
__device__ __forceinline__ float rotate_token_words(const __half* x, int W, float inv_sqrt_b, float clip_ratio,
                                                    float* qbuf, float* s_amax, float (&v)[16]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kPitch = 17;   // rows of the in-warp transposition: 16 floats and one of padding (no bank conflicts)
  const int QP = W + 4;        // pitch of the cross-warp buffer [16 elements][W words]: the 16-byte stores of eight
                               // lanes with different elements then fall into different banks
  if (tid < W) {
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)tid * 16);
    const uint4 r0 = __ldg(src), r1 = __ldg(src + 1);
    const __half2* h0 = reinterpret_cast<const __half2*>(&r0);
    const __half2* h1 = reinterpret_cast<const __half2*>(&r1);
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float2 f0 = __half22float2(h0[e]), f1 = __half22float2(h1[e]);
      v[2 * e] = f0.x; v[2 * e + 1] = f0.y; v[8 + 2 * e] = f1.x; v[8 + 2 * e + 1] = f1.y;
    }
  } else {
#pragma unroll
    for (int e = 0; e < 16; e++) v[e] = 0.f;
  }
  // sixteen values in registers: the four stages that pair them
  auto butterflies16 = [](float (&a)[16]) {
#pragma unroll
    for (int h = 1; h < 16; h *= 2) {
#pragma unroll
      for (int e = 0; e < 16; e++) {
        if ((e & h) == 0) {
          const float u = a[e], w = a[e + h];
          a[e] = __fadd_rn(u, w);
          a[e + h] = __fsub_rn(u, w);
        }
      }
    }
  };
  butterflies16(v);   // strides 1..8
  const bool data_warp = warp * 32 < W;   // (W is a multiple of 256: a warp holds 32 words or none)
  const int e1 = lane & 15, hi = lane & 16;
  float u[16];
#pragma unroll
  for (int j = 0; j < 16; j++) u[j] = 0.f;
  if (data_warp) {
    float* const wbuf = qbuf + warp * (32 * kPitch);
#pragma unroll
    for (int e = 0; e < 16; e++) wbuf[lane * kPitch + e] = v[e];
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 16; j++) u[j] = wbuf[(hi | j) * kPitch + e1];   // element e1 of the words hi + j
    butterflies16(u);   // strides 16..128
#pragma unroll
    for (int j = 0; j < 16; j++) {   // stride 256
      const float other = __shfl_xor_sync(0xffffffffu, u[j], 16);
      u[j] = hi ? __fsub_rn(other, u[j]) : __fadd_rn(u[j], other);
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");   // every warp is done with its transposition area
  if (data_warp) {   // u[j]: element e1 of word warp * 32 + hi + j
    float4* const dst = reinterpret_cast<float4*>(qbuf + e1 * QP + warp * 32 + hi);
#pragma unroll
    for (int j = 0; j < 4; j++) dst[j] = make_float4(u[4 * j], u[4 * j + 1], u[4 * j + 2], u[4 * j + 3]);
  }
  asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
  {
    const int R = W >> 5;   // 8 or 16 warps hold data
    float* const colp = qbuf + warp * QP + lane;
    float tv[16];
#pragma unroll
    for (int w = 0; w < 16; w++) tv[w] = (w < R) ? colp[w * 32] : 0.f;
#pragma unroll
    for (int h = 1; h < 16; h *= 2) {
      if (h < R) {
#pragma unroll
        for (int w = 0; w < 16; w++) {
          if ((w & h) == 0) {
            const float a = tv[w], z = tv[w + h];
            tv[w] = __fadd_rn(a, z);
            tv[w + h] = __fsub_rn(a, z);
          }
        }
      }
    }
#pragma unroll
    for (int w = 0; w < 16; w++) if (w < R) colp[w * 32] = tv[w];
  }
  asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
  if (tid < W) {
#pragma unroll
    for (int e = 0; e < 16; e++) v[e] = qbuf[e * QP + tid];
  }
  float amax = 0.f;
#pragma unroll
  for (int e = 0; e < 16; e++) {
    v[e] = __fmul_rn(v[e], inv_sqrt_b);
    amax = fmaxf(amax, fabsf(v[e]));
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
  if (lane == 0) s_amax[warp] = amax;
  asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
#pragma unroll
  for (int w = 0; w < NT / 32; w++) amax = fmaxf(amax, s_amax[w]);
  const float s32 = __fdiv_rn(__fmul_rn(amax, clip_ratio), 7.0f);
  return __half2float(__float2half_rn(s32));
}

// One CTA of 512 threads per token, for a token of 4096 or 8192 elements under one rotation block:
// faster than the cluster form above for these shapes (no cluster launch, no passes through
// distributed shared memory).
__global__ void __launch_bounds__(512) quantize_act_wide_kernel(const QuantParams p) {
  extern __shared__ __align__(16) float sbuf[];   // rotate_scratch_bytes(K)
  __shared__ float s_amax[16];
  const int m = blockIdx.x, tid = threadIdx.x;
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int W = p.K / 16;
  float v[16];
  const float s = rotate_token_words<512>(p.x + (size_t)m * p.K, W, p.inv_sqrt_b, p.clip_ratio, sbuf, s_amax, v);
  if (tid == 0) p.scale[m] = __float2half_rn(s);
  int q[16];
  if (s != 0.f) {   // the same for the whole CTA; threads beyond the token hold zeros
    quantize_int4<16>(v, s, q);
  } else {
#pragma unroll
    for (int e = 0; e < 16; e++) q[e] = 0;
  }
  if (tid < W) {
    uint32_t lo32 = 0, hi32 = 0;
#pragma unroll
    for (int e = 0; e < 8; e++) {
      lo32 |= (uint32_t)(q[e] & 0xF) << (4 * e);
      hi32 |= (uint32_t)(q[8 + e] & 0xF) << (4 * e);
    }
    *reinterpret_cast<uint2*>(p.xq + (size_t)m * (p.K / 2) + (size_t)tid * 8) = make_uint2(lo32, hi32);
  }
}

}  // namespace rcp
