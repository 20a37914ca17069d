// 3-bit weights (Section 4.3, paragraph "Application of LDP on NF3 format"; Table "memory", W3 column):
// packing and the W3A4 look-up-table GEMV with eight levels per quantization unit.
//
// Storage. The low two bits of a code are stored exactly like a 2-bit code (words2 [N][K/16]); the top bit goes
// to a plane of its own (words1 [N][K/32]): word v covers the codes 32v .. 32v+31 and holds the top bit of code
// 32v + i in bit 2i and of code 32v + 16 + i in bit 2i + 1. Masked with 0x55555555 (shifted down by one for the
// second half) a plane word therefore lines up with the b0 bits of the matching words2 word.
//
// Exact integer formulation. With b0, b1, b2 the bits of a code, the sums of q over the seven products
//   b0, b1, b0 b1, b2, b0 b2, b1 b2, b0 b1 b2      (T_S for the non-empty subsets S of {0,1,2})
// and T_0 = sum of q give every per-code sum by inclusion and exclusion:
//   S_c = sum over S containing the set bits of c of (-1)^(|S| - popcount(c)) T_S.
// Each product is a bit plane of 16 single bits (one logic operation per plane and word); masked at in-byte
// position p it is the A operand of an 8-bit dot product (dp4a) against the int8 activations, even positions
// meeting activations pre-multiplied by 4 so that positions {0,1} and {2,3} share an accumulator.
// 2.3 times the mask and dot-product work of the 2-bit kernel per weight. One warp per output row, lanes along
// K in units of 64 codes (a 16-byte and an 8-byte load), two units = one group of 128 per lane step.
#pragma once
#include "common.cuh"

namespace rcp {

__global__ void pack_weights3_kernel(const uint4* __restrict__ codes, size_t nplane, uint32_t* __restrict__ words2,
                                     uint32_t* __restrict__ words1, int* __restrict__ bad) {
  for (size_t v = blockIdx.x * (size_t)blockDim.x + threadIdx.x; v < nplane; v += (size_t)gridDim.x * blockDim.x) {
    const uint4 a = __ldg(codes + 2 * v), b = __ldg(codes + 2 * v + 1);   // codes 32v .. 32v+15, 32v+16 .. 32v+31
    const uint32_t c[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t lo[2] = {0, 0}, top = 0, over = 0;
#pragma unroll
    for (int i = 0; i < 8; i++) {
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const uint32_t code = (c[i] >> (8 * j)) & 0xFFu;
        const int k = 4 * i + j;                       // 0..31 inside the plane word
        over |= code & ~7u;
        lo[k >> 4] |= (code & 3u) << (2 * (k & 15));
        top |= ((code >> 2) & 1u) << (k < 16 ? 2 * k : 2 * (k - 16) + 1);
      }
    }
    words2[2 * v] = lo[0];
    words2[2 * v + 1] = lo[1];
    words1[v] = top;
    if (over) atomicExch(bad, 1);
  }
}

constexpr int kW3Threads = 256;

struct W3Params {
  const uint32_t* words2;
  const uint32_t* words1;
  const uint4* lut;        // [N][8] fp16 (GRP: [N][K/128][8])
  const uint8_t* xq;       // [K/2] of the token
  const __half* scale;     // of the token
  __half* y;               // [N] of the token
  int32_t* S_out;          // SDBG: [N][8] (GRP: [N][K/128][8]) of the token
  int N, K;
};

// S_c from the eight subset sums (index = bit set of the subset; t[0] = sum of q)
__device__ __forceinline__ void w3_percode(const int (&t)[8], int (&S)[8]) {
  S[7] = t[7];
  S[6] = t[6] - t[7];
  S[5] = t[5] - t[7];
  S[3] = t[3] - t[7];
  S[4] = t[4] - t[5] - t[6] + t[7];
  S[2] = t[2] - t[3] - t[6] + t[7];
  S[1] = t[1] - t[3] - t[5] + t[7];
  S[0] = t[0] - t[1] - t[2] - t[4] + t[3] + t[5] + t[6] - t[7];
}

__device__ __forceinline__ float w3_lut_dot(uint4 l, const int (&S)[8]) {
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&l.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&l.y));
  const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&l.z));
  const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&l.w));
  float acc = a.x * (float)S[0];
  acc = fmaf(a.y, (float)S[1], acc);
  acc = fmaf(b.x, (float)S[2], acc);
  acc = fmaf(b.y, (float)S[3], acc);
  acc = fmaf(c.x, (float)S[4], acc);
  acc = fmaf(c.y, (float)S[5], acc);
  acc = fmaf(d.x, (float)S[6], acc);
  acc = fmaf(d.y, (float)S[7], acc);
  return acc;
}

// One token per launch. Shared memory: the token's activations expanded to one byte per code, 16 bytes per
// word of 16 codes: { position 0 (times 4), position 1, position 2 (times 4), position 3 }, byte j of a position =
// activation of code 16 w + 4 j + p. Word i of unit u (64 codes) sits at index ((u & 1) * 4 + i) * npair + (u >> 1):
// the lanes of a warp, which take consecutive pairs of units, then read consecutive 16-byte slots (no bank
// conflicts).
template <bool GRP, bool SDBG>
__global__ void __launch_bounds__(kW3Threads) gemv_w3a4_kernel(const W3Params p) {
  extern __shared__ uint4 s_act[];           // [K / 16]
  __shared__ int s_t0[kW3Threads / 32];
  __shared__ int s_t0g[GRP ? 512 : 1];       // sum of q per group of 128 (K <= 65536)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = p.K / 16;
  const int nunit = p.K / 64, npair = (nunit + 1) / 2;
  // ---- expand the activations
  int tsum = 0;
  for (int w0 = 0; w0 < W; w0 += kW3Threads) {   // the same trip count for every thread: the shuffles below need whole warps
    const int w = w0 + tid;
    const bool in = w < W;
    uint2 x = make_uint2(0, 0);
    if (in) x = __ldg(reinterpret_cast<const uint2*>(p.xq) + w);   // 16 nibbles
    uint32_t pos[4] = {0, 0, 0, 0};
    int wsum = 0;
#pragma unroll
    for (int j = 0; j < 4; j++)
#pragma unroll
      for (int pp = 0; pp < 4; pp++) {
        const int k = 4 * j + pp;
        const int q = sext4(((k < 8 ? x.x : x.y) >> (4 * (k & 7))) & 0xFu);
        wsum += q;
        pos[pp] |= (uint32_t)(((pp & 1) ? q : 4 * q) & 0xFF) << (8 * j);
      }
    if (in) s_act[(((w >> 2) & 1) * 4 + (w & 3)) * npair + (w >> 3)] = make_uint4(pos[0], pos[1], pos[2], pos[3]);
    if constexpr (GRP) {
      // eight consecutive words are one group; they belong to eight consecutive lanes
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 1);
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 2);
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 4);
      if (in && (w & 7) == 0) s_t0g[w >> 3] = wsum;
    } else {
      tsum += wsum;
    }
  }
  if constexpr (!GRP) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, d);
    if (lane == 0) s_t0[warp] = tsum;
  }
  __syncthreads();
  int T0 = 0;
  if constexpr (!GRP) {
#pragma unroll
    for (int i = 0; i < kW3Threads / 32; i++) T0 += s_t0[i];
  }
  const float s = __half2float(p.scale[0]);
  const int ngrp = p.K / 128;
  const int warps = gridDim.x * (kW3Threads / 32);
  // The weights of a lane step (two units: a 16-byte and an 8-byte load each) are fetched one step ahead, across
  // the end of a row as well, so that the loads of the next step are in flight while this one is computed.
  const int nit = (nunit + 63) / 64;                         // lane steps per row
  const int row_first = blockIdx.x * (kW3Threads / 32) + warp;
  auto fetch = [&](int row, int it, uint4 (&a)[2], uint2 (&z)[2]) {
#pragma unroll
    for (int h = 0; h < 2; h++) {
      const int u = 2 * lane + 64 * it + h;
      a[h] = make_uint4(0, 0, 0, 0);
      z[h] = make_uint2(0, 0);
      if (row < p.N && u < nunit) {
        a[h] = __ldg(reinterpret_cast<const uint4*>(p.words2 + (size_t)row * W) + u);
        z[h] = __ldg(reinterpret_cast<const uint2*>(p.words1 + (size_t)row * (W / 2)) + u);
      }
    }
  };
  uint4 an[2];
  uint2 zn[2];
  fetch(row_first, 0, an, zn);
  for (int row = row_first; row < p.N; row += warps) {
    int acc[7][2];
#pragma unroll
    for (int f = 0; f < 7; f++) { acc[f][0] = 0; acc[f][1] = 0; }
    float yacc = 0.f;
    // a lane takes units u = 2 (lane + 32 i), +1: 128 consecutive codes, one group of the group-wise grid
    for (int it = 0; it < nit; it++) {
      const int u0 = 2 * lane + 64 * it;
      uint4 ac[2] = {an[0], an[1]};
      uint2 zc[2] = {zn[0], zn[1]};
      if (it + 1 < nit) fetch(row, it + 1, an, zn); else fetch(row + warps, 0, an, zn);
      if (u0 >= nunit) continue;   // (only in the last step of a row; the prefetch above has been issued)
#pragma unroll
      for (int h = 0; h < 2; h++) {
        const int u = u0 + h;
        if (u < nunit) {
          const uint32_t ww[4] = {ac[h].x, ac[h].y, ac[h].z, ac[h].w};
#pragma unroll
          for (int i = 0; i < 4; i++) {
            const uint32_t w = ww[i], hb = w >> 1, whb = w & hb;
            const uint32_t zsel = (i < 2) ? zc[h].x : zc[h].y;
            const uint32_t zz = (i & 1) ? (zsel >> 1) : zsel;   // top bits lined up with the b0 bits (odd bits: the other half's)
            const uint4 q = s_act[(h * 4 + i) * npair + (u0 >> 1)];
            const uint32_t qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int pp = 0; pp < 4; pp++) {
              // the seven products of code bits at in-byte position pp: one logic operation each (the mask keeps
              // the even bit of the position, so stray odd bits of hb and zz drop out)
              const uint32_t m = 0x01010101u << (2 * pp);
              uint32_t P[7];
              P[0] = w & m;                   // b0
              P[1] = hb & m;                  // b1
              P[2] = whb & m;                 // b0 b1
              P[3] = zz & m;                  // b2
              asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(P[4]) : "r"(w), "r"(zz), "r"(m));     // b0 b2
              asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(P[5]) : "r"(hb), "r"(zz), "r"(m));    // b1 b2
              asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(P[6]) : "r"(whb), "r"(zz), "r"(m));   // b0 b1 b2
#pragma unroll
              for (int f = 0; f < 7; f++) acc[f][pp >> 1] = __dp4a((int)P[f], (int)qq[pp], acc[f][pp >> 1]);
            }
          }
        }
      }
      if constexpr (GRP) {
        // this lane's 128 codes are group u0 / 2: finish it here
        const int gi = u0 >> 1;
        int t[8], S[8];
        t[0] = s_t0g[gi];
        t[1] = (acc[0][0] >> 2) + (acc[0][1] >> 6);
        t[2] = (acc[1][0] >> 2) + (acc[1][1] >> 6);
        t[3] = (acc[2][0] >> 2) + (acc[2][1] >> 6);
        t[4] = (acc[3][0] >> 2) + (acc[3][1] >> 6);
        t[5] = (acc[4][0] >> 2) + (acc[4][1] >> 6);
        t[6] = (acc[5][0] >> 2) + (acc[5][1] >> 6);
        t[7] = (acc[6][0] >> 2) + (acc[6][1] >> 6);
        w3_percode(t, S);
        yacc += w3_lut_dot(__ldg(p.lut + (size_t)row * ngrp + gi), S);
        if constexpr (SDBG) {
          int4* o = reinterpret_cast<int4*>(p.S_out + ((size_t)row * ngrp + gi) * 8);
          o[0] = make_int4(S[0], S[1], S[2], S[3]);
          o[1] = make_int4(S[4], S[5], S[6], S[7]);
        }
#pragma unroll
        for (int f = 0; f < 7; f++) { acc[f][0] = 0; acc[f][1] = 0; }
      }
    }
    if constexpr (GRP) {
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) yacc += __shfl_xor_sync(0xffffffffu, yacc, d);
      if (lane == 0) p.y[row] = __float2half_rn(s * yacc);
    } else {
      int t[8], S[8];
      t[0] = T0;
#pragma unroll
      for (int f = 0; f < 7; f++) {
        int v = (acc[f][0] >> 2) + (acc[f][1] >> 6);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        t[f + 1] = v;
      }
      if (lane == 0) {
        w3_percode(t, S);
        p.y[row] = __float2half_rn(s * w3_lut_dot(__ldg(p.lut + row), S));
        if constexpr (SDBG) {
          int4* o = reinterpret_cast<int4*>(p.S_out + (size_t)row * 8);
          o[0] = make_int4(S[0], S[1], S[2], S[3]);
          o[1] = make_int4(S[4], S[5], S[6], S[7]);
        }
      }
    }
  }
}

}  // namespace rcp
