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
// 2.4 times the mask and dot-product work of the 2-bit kernel per weight. One warp per output row, lanes along
// K in units of 64 codes (a 16-byte and an 8-byte load), two units = one group of 128 per lane step; one resident
// wave of CTAs, rows dealt round-robin to its warps.
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

// Export of a 3-bit layer trained with a learnable centre (Section 4.3, paragraph "Application of LDP on NF3
// format", Eq. "nf3scales", Eq. "nf3") to the inputs of the kernel below: packed codes and the eight levels of
// every quantization unit. Offline, one pass: 2 bytes read and 3/8 byte written per weight. One warp per unit
// (G consecutive weights of a row, G a multiple of 32): the range by shuffles; centre, the two scales and the
// levels in fp32 with one rounding per operation, so that the 3-bit decision is reproducible bit for bit; a
// lane takes four consecutive weights per round of 128, four lanes make a word of low bits, eight lanes a word
// of the top-bit plane. `table`: the eight ascending normalized levels of the format, table[zero] == 0.
struct Nf3Params {
  const __half* w;     // [N][K] rotated weights
  const float* sb;     // [N][K/G] sigmoid(beta): lower clipping fraction
  const float* sg;     // sigmoid(gamma)
  const float* s1;     // sigmoid(s_1): the centre as a fraction of the clipped range
  uint32_t* words2;    // [N][K/16]
  uint32_t* words1;    // [N][K/32]
  uint4* lut;          // [N][K/G] eight fp16 levels
  float table[8];
  int zero;
  int N, K, G;
  long long units;     // N * K / G
};

__global__ void __launch_bounds__(256) nf3_export_kernel(const Nf3Params p) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int NG = p.K / p.G;
  for (long long u = warp0; u < p.units; u += nwarps) {
    const long long n = u / NG;
    const int j = (int)(u - n * NG);
    const __half* wu = p.w + n * p.K + (long long)j * p.G;
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
    const float c = __fadd_rn(lo, __fmul_rn(h, __ldg(p.s1 + u)));
    const float s_neg = fabsf(__fsub_rn(c, lo)), s_pos = fabsf(__fsub_rn(hi, c));
    const bool ok = h > 0.0f;
    if (lane < 8) {   // lane i makes level i; the eight halves are gathered into one 16-byte store
      const float level = __fadd_rn(c, __fmul_rn(p.table[lane], lane > p.zero ? s_pos : s_neg));
      const uint32_t bits = __half_as_ushort(__float2half_rn(ok ? level : lo));
      const uint32_t other = __shfl_down_sync(0x000000ffu, bits, 1, 8);
      const uint32_t pair = bits | (other << 16);                    // valid in even lanes
      uint4 out;
      out.x = __shfl_sync(0x000000ffu, pair, 0);
      out.y = __shfl_sync(0x000000ffu, pair, 2);
      out.z = __shfl_sync(0x000000ffu, pair, 4);
      out.w = __shfl_sync(0x000000ffu, pair, 6);
      if (lane == 0) p.lut[u] = out;
    }
    __syncwarp();
    uint32_t* row2 = p.words2 + n * (p.K / 16) + (long long)j * (p.G / 16);
    uint32_t* row1 = p.words1 + n * (p.K / 32) + (long long)j * (p.G / 32);
    for (int k0 = lane * 4; k0 - lane * 4 < p.G; k0 += 128) {   // all lanes stay in the loop for the shuffles
      uint32_t low = 0, top = 0;
      if (k0 < p.G) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(wu + k0));
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        const float v[4] = {a.x, a.y, b.x, b.y};
#pragma unroll
        for (int e = 0; e < 4; e++) {
          int code = p.zero;
          if (ok) {
            const float cl = fminf(fmaxf(v[e], lo), hi);
            const bool pos = cl > c;            // a weight equal to the centre belongs to the negative side
            const float sc = pos ? s_pos : s_neg;
            if (sc > 0.0f) {
              const float x = __fdiv_rn(__fsub_rn(cl, c), sc);
              const int first = pos ? p.zero : 0, last = pos ? 7 : p.zero;
              code = first;
              float best = fabsf(__fsub_rn(x, p.table[first]));
              for (int i = first + 1; i <= last; i++) {
                const float dist = fabsf(__fsub_rn(x, p.table[i]));
                if (dist < best) { best = dist; code = i; }   // strict: a tie keeps the lower level
              }
            }
          }
          low |= (uint32_t)(code & 3) << (2 * e);
          const int kk = (k0 + e) & 31;       // place in the plane word: codes 0..15 even bits, 16..31 odd bits
          top |= (uint32_t)(code >> 2) << (kk < 16 ? 2 * kk : 2 * (kk - 16) + 1);
        }
      }
      uint32_t word = low << (8 * (lane & 3));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      top |= __shfl_xor_sync(0xffffffffu, top, 1);
      top |= __shfl_xor_sync(0xffffffffu, top, 2);
      top |= __shfl_xor_sync(0xffffffffu, top, 4);
      if ((lane & 3) == 0 && k0 < p.G) row2[k0 >> 4] = word;
      if ((lane & 7) == 0 && k0 < p.G) row1[k0 >> 5] = top;
    }
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

// Four 4-bit two's-complement values, one in the low nibble of each byte (high nibbles zero), sign-extended to
// bytes: with t = v ^ 8 per byte the result is t - 8; the bytes are lifted to 0x80 + t first so that no borrow
// crosses a byte, and the lift is taken out again.
__device__ __forceinline__ uint32_t w3_sext4x4(uint32_t v) {
  return (((v ^ 0x08080808u) | 0x80808080u) - 0x08080808u) ^ 0x80808080u;
}
// a & b & MASK as one logic operation with the mask as an immediate
template <uint32_t MASK>
__device__ __forceinline__ uint32_t w3_and_mask(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(d) : "r"(a), "r"(b), "n"(MASK));
  return d;
}
// In-byte position PP of a word: the seven products of code bits, one logic operation each (the mask keeps the
// even bit of the position, so stray odd bits of hb and zz drop out), and their seven dot products.
template <int PP>
__device__ __forceinline__ void w3_position(uint32_t w, uint32_t hb, uint32_t whb, uint32_t zz, uint32_t q,
                                            int (&acc)[7][2]) {
  constexpr uint32_t m = 0x01010101u << (2 * PP);
  uint32_t P[7];
  P[0] = w & m;                          // b0
  P[1] = hb & m;                         // b1
  P[2] = whb & m;                        // b0 b1
  P[3] = zz & m;                         // b2
  P[4] = w3_and_mask<m>(w, zz);          // b0 b2
  P[5] = w3_and_mask<m>(hb, zz);         // b1 b2
  P[6] = w3_and_mask<m>(whb, zz);        // b0 b1 b2
#pragma unroll
  for (int f = 0; f < 7; f++) acc[f][PP >> 1] = __dp4a((int)P[f], (int)q, acc[f][PP >> 1]);
}

// One token per launch. Shared memory: the token's activations expanded to one byte per code, 16 bytes per
// word of 16 codes: { position 0 (times 4), position 1, position 2 (times 4), position 3 }, byte j of a position =
// activation of code 16 w + 4 j + p. A lane step covers 64 units of 64 codes; lane l takes units 2l and 2l + 1 of
// it (128 consecutive codes, one group of the group-wise grid), i.e. eight words c = 0..7. Word c of lane l in
// step `it` sits at 16-byte slot (it * 8 + c) * 32 + l: the lanes of a warp read consecutive slots (no bank
// conflicts) at offsets from one address that are known at compile time. K is padded to whole lane steps with
// zeros (weights beyond K are loaded as zeros as well, so the padding contributes nothing).
// Four CTAs per SM (64 registers, no spills): 32 warps hide the weight loads better than the 24 that the
// compiler's own choice of 80 registers leaves (57344x8192: 74.5 against 76.8 us).
template <bool GRP, bool SDBG>
__global__ void __launch_bounds__(kW3Threads, 4) gemv_w3a4_kernel(const W3Params p) {
  extern __shared__ uint4 s_act[];           // [lane steps][8][32]
  __shared__ int s_t0[kW3Threads / 32];
  __shared__ int s_t0g[GRP ? 512 : 1];       // sum of q per group of 128 (K <= 65536)
  constexpr int kWarps = kW3Threads / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = p.K / 16;
  const int nunit = p.K / 64;
  const int nit = (nunit + 63) / 64;         // lane steps per row
  const int warps = gridDim.x * kWarps;
  const uint4* const w2 = reinterpret_cast<const uint4*>(p.words2) + 2 * lane;   // a unit: one uint4 of words2,
  const uint2* const w1 = reinterpret_cast<const uint2*>(p.words1) + 2 * lane;   // one uint2 of words1
  struct Step { uint4 a[2]; uint2 z[2]; };   // the weights of a lane step: two units
  auto fetch = [&](int row, int it, Step& d) {
    const size_t e = (size_t)row * nunit + 64 * it;
    const int u = 2 * lane + 64 * it;
#pragma unroll
    for (int h = 0; h < 2; h++) {
      const bool ok = row < p.N && u + h < nunit;
      d.a[h] = ok ? __ldg(w2 + e + h) : make_uint4(0, 0, 0, 0);
      d.z[h] = ok ? __ldg(w1 + e + h) : make_uint2(0, 0);
    }
  };
  // Rows are dealt round-robin to all warps of the grid (one resident wave of CTAs). The first weights are
  // requested before anything else, so that their way from memory overlaps the expansion.
  const int gw = blockIdx.x * kWarps + warp;
  Step A, B;
  fetch(gw, 0, A);
  // ---- expand the activations (256 words per lane step: the same trip count for every thread)
  int tsum = 0;
  for (int w = tid; w < nit * 256; w += kW3Threads) {
    uint2 x = make_uint2(0, 0);
    if (w < W) x = __ldg(reinterpret_cast<const uint2*>(p.xq) + w);   // 16 nibbles
    // four nibbles at a time: nibble k of a register goes to byte k / 2 of e (k even) or o (k odd), is sign-extended
    // inside its byte, then the bytes are gathered by position (byte j of position pp = code 4 j + pp)
    const uint32_t e0 = w3_sext4x4(x.x & 0x0F0F0F0Fu), o0 = w3_sext4x4((x.x >> 4) & 0x0F0F0F0Fu);   // codes 0,2,4,6 / 1,3,5,7
    const uint32_t e1 = w3_sext4x4(x.y & 0x0F0F0F0Fu), o1 = w3_sext4x4((x.y >> 4) & 0x0F0F0F0Fu);   // codes 8,.. / 9,..
    uint4 pos;
    pos.x = (__byte_perm(e0, e1, 0x6420) << 2) & 0xFCFCFCFCu;   // codes 0,4,8,12, times 4 inside each byte
    pos.y = __byte_perm(o0, o1, 0x6420);                        // codes 1,5,9,13
    pos.z = (__byte_perm(e0, e1, 0x7531) << 2) & 0xFCFCFCFCu;   // codes 2,6,10,14, times 4
    pos.w = __byte_perm(o0, o1, 0x7531);                        // codes 3,7,11,15
    int wsum = __dp4a((int)e0, 0x01010101, __dp4a((int)o0, 0x01010101, __dp4a((int)e1, 0x01010101, __dp4a((int)o1, 0x01010101, 0))));
    // word w = 8 (32 it + l) + c
    s_act[((w >> 8) * 8 + (w & 7)) * 32 + ((w >> 3) & 31)] = pos;
    if constexpr (GRP) {
      // eight consecutive words are one group; they belong to eight consecutive lanes
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 1);
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 2);
      wsum += __shfl_xor_sync(0xffffffffu, wsum, 4);
      if (w < W && (w & 7) == 0) s_t0g[w >> 3] = wsum;
    } else {
      tsum += wsum;
    }
  }
  if constexpr (!GRP) {
    tsum = __reduce_add_sync(0xffffffffu, tsum);
    if (lane == 0) s_t0[warp] = tsum;
  }
  __syncthreads();
  int T0 = 0;
  if constexpr (!GRP) {
#pragma unroll
    for (int i = 0; i < kWarps; i++) T0 += s_t0[i];
  }
  const float s = __half2float(p.scale[0]);
  const int ngrp = p.K / 128;
  // The arithmetic of a lane step into the fourteen accumulators (weights beyond K are zeros: no guard needed).
  int acc[7][2];
#pragma unroll
  for (int f = 0; f < 7; f++) { acc[f][0] = 0; acc[f][1] = 0; }
  const uint4* const act_lane = s_act + lane;
  auto lane_step = [&](const Step& c, int it) {
    const uint4* const act = act_lane + it * 256;
#pragma unroll
    for (int h = 0; h < 2; h++) {
      const uint32_t ww[4] = {c.a[h].x, c.a[h].y, c.a[h].z, c.a[h].w};
#pragma unroll
      for (int i = 0; i < 4; i++) {
        const uint32_t w = ww[i], hb = w >> 1, whb = w & hb;
        const uint32_t zsel = (i < 2) ? c.z[h].x : c.z[h].y;
        const uint32_t zz = (i & 1) ? (zsel >> 1) : zsel;   // top bits lined up with the b0 bits (odd bits: the other half's)
        const uint4 q = act[(h * 4 + i) * 32];
        w3_position<0>(w, hb, whb, zz, q.x, acc);
        w3_position<1>(w, hb, whb, zz, q.y, acc);
        w3_position<2>(w, hb, whb, zz, q.z, acc);
        w3_position<3>(w, hb, whb, zz, q.w, acc);
      }
    }
  };
  // Group-wise grid: this lane's 128 codes of step `it` are group lane + 32 it of the row; its term of y.
  auto finish_group = [&](int row, int it) -> float {
    const int gi = lane + 32 * it;
    int t[8], S[8];
#pragma unroll
    for (int f = 0; f < 7; f++) {
      t[f + 1] = (acc[f][0] >> 2) + (acc[f][1] >> 6);
      acc[f][0] = 0;
      acc[f][1] = 0;
    }
    if (gi >= ngrp) return 0.f;
    t[0] = s_t0g[GRP ? gi : 0];
    w3_percode(t, S);
    if constexpr (SDBG) {
      int4* o = reinterpret_cast<int4*>(p.S_out + ((size_t)row * ngrp + gi) * 8);
      o[0] = make_int4(S[0], S[1], S[2], S[3]);
      o[1] = make_int4(S[4], S[5], S[6], S[7]);
    }
    return w3_lut_dot(__ldg(p.lut + (size_t)row * ngrp + gi), S);
  };
  // Per-row grid: the row's result from its eight sums (one thread).
  auto finish_row = [&](int row, const int (&t)[8]) {
    int S[8];
    w3_percode(t, S);
    p.y[row] = __float2half_rn(s * w3_lut_dot(__ldg(p.lut + row), S));
    if constexpr (SDBG) {
      int4* o = reinterpret_cast<int4*>(p.S_out + (size_t)row * 8);
      o[0] = make_int4(S[0], S[1], S[2], S[3]);
      o[1] = make_int4(S[4], S[5], S[6], S[7]);
    }
  };
  // A row: the weights are fetched one lane step ahead into two buffers used in turn; on entry A holds step 0
  // of the row, on exit step 0 of row nrow (the warp's next one; nothing beyond the last row).
  float yacc = 0.f;
  auto step = [&](const Step& c, int row, int it) {
    lane_step(c, it);
    if constexpr (GRP) yacc += finish_group(row, it);
  };
  auto run_row = [&](int row, int nrow) {
    int it = 0;
    for (; it + 1 < nit; it += 2) {
      fetch(row, it + 1, B);
      step(A, row, it);
      if (it + 2 < nit) fetch(row, it + 2, A); else fetch(nrow, 0, A);
      step(B, row, it + 1);
    }
    if (it < nit) {   // an odd count: one step left, in A
      fetch(nrow, 0, B);
      step(A, row, it);
      A = B;
    }
  };
  for (int row = gw; row < p.N; row += warps) {
    run_row(row, row + warps);
    if constexpr (GRP) {
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) yacc += __shfl_xor_sync(0xffffffffu, yacc, d);
      if (lane == 0) p.y[row] = __float2half_rn(s * yacc);
      yacc = 0.f;
    } else {
      int t[8];
      t[0] = T0;
#pragma unroll
      for (int f = 0; f < 7; f++) {
        t[f + 1] = __reduce_add_sync(0xffffffffu, (acc[f][0] >> 2) + (acc[f][1] >> 6));   // one instruction per sum
        acc[f][0] = 0;
        acc[f][1] = 0;
      }
      if (lane == 0) finish_row(row, t);
    }
  }
}

}  // namespace rcp
