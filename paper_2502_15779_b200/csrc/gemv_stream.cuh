// Streaming LUT GEMV for sm_100a (Section 4.4 of the paper: O = S * X_q * LUT[W_q]).
//
// Exact integer formulation. With b0 = code & 1, b1 = code >> 1 and, per output row,
//   T1 = sum_k b0 q,  T2 = sum_k b1 q,  T3 = sum_k b0 b1 q,  T0 = sum_k q   (T0 is row independent)
// the per-code sums are S3 = T3, S1 = T1 - T3, S2 = T2 - T3, S0 = T0 - T1 - T2 + T3.
// A 32-bit weight word holds 16 codes; byte j holds codes 4j..4j+3 at in-byte positions p = 0..3.
// Masking the word with 0x01010101 << 2p leaves one b0 bit per byte, scaled by 4^p: four such bytes
// are the A operand of an 8-bit integer dot product whose B operand is the four matching int8
// activations. Twelve masked words (three functions x four positions) cover a word; each costs
// one LOP3, the scarce resource (the logic pipe issues 64 lanes/clk/SM on B200). The products go
// to the int8 mma.sync path (16 rows x 32 bytes per instruction, tokens in the n dimension)
// and/or to dp4a on the FMA pipe.
//
// Data movement: the packed weights are the only large stream. One persistent CTA per SM takes an
// equal, contiguous share of the (row tile, K chunk) work items; a producer warp streams
// 128-row x 128-byte boxes into a shared-memory ring with TMA (cp.async.bulk.tensor, 128B swizzle,
// mbarrier completion), eight consumer warps (16 rows each) read them bank-conflict free. The
// int4 activations are expanded once per CTA into the B-operand byte layout in shared memory.
// Tiles split between CTAs are combined with integer atomics in a caller-provided scratch buffer
// (order independent, hence deterministic); the last contributor finishes the tile and re-zeroes it.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace rcp {

constexpr int kTileRows = 128;       // rows per work item (8 consumer warps x 16)
constexpr int kChunkWords = 32;      // 32-bit words per row per work item (128 bytes, 512 codes)
constexpr int kStageBytes = kTileRows * kChunkWords * 4;
constexpr int kConsumerWarps = 8;
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 8;
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded waits: give up, flag the error, drain and exit

enum StreamMode { kModeMma = 0, kModeHybrid = 1, kModeDp4a = 2 };

struct StreamParams {
  const uint2* lut;
  const uint8_t* xq;
  const __half* scale;
  __half* y;
  int32_t* ws_status;   // [4]
  uint32_t* ws_count;   // [ntiles][8]
  int32_t* ws_sum;      // [ntiles*128][M][3]
  int M, N, K;
  int ntiles;
  int nchunks;          // K chunks in total
  int ch_per_super;     // K chunks per super-chunk (blockIdx.y)
  int stages;
  int ncol;             // token columns stored in the expanded activation buffer (power of two >= M)
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false after kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; i++) {
    if (mbar_try(bar, parity)) return true;
    if (i > 64) __nanosleep(32);
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void dp4a_u8s8(int& d, uint32_t a, uint32_t b) {
  asm volatile("dp4a.u32.s32 %0, %1, %2, %0;" : "+r"(d) : "r"(a), "r"(b));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// Physical 16-byte unit of (word index inside the super-chunk, token column) in the expanded
// activation buffer. The permutation spreads the four k-slices a quad reads at once over banks.
__device__ __forceinline__ uint32_t bs_unit(uint32_t widx_rel, uint32_t col, uint32_t ncol) {
  const uint32_t t = (widx_rel >> 3) & 3u;
  if (ncol >= 8) return widx_rel * ncol + (col & ~7u) + ((col + 2u * t) & 7u);
  const uint32_t x = ncol == 1 ? 2u * t : (ncol == 2 ? t : (t & 1u));
  return (widx_rel ^ x) * ncol + col;
}

// ----------------------------------------------------------------------------- the kernel
template <int MT, int MODE>
__global__ void __launch_bounds__(kStreamThreads, 1)
gemv_stream_kernel(const __grid_constant__ CUtensorMap tmap, const StreamParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;           // TMA 128B swizzle wants 1024-byte alignment
  uint8_t* const gen = smem_raw + (base - raw);
  const int stages = p.stages;
  const uint32_t a_base = base;
  const uint32_t misc_off = (uint32_t)stages * kStageBytes;
  uint64_t* const bars = reinterpret_cast<uint64_t*>(gen + misc_off);          // full[8], empty[8]
  int* const s_T0 = reinterpret_cast<int*>(gen + misc_off + 128);               // [16]
  float* const s_scale = reinterpret_cast<float*>(gen + misc_off + 192);        // [16]
  volatile int* const s_abort = reinterpret_cast<volatile int*>(gen + misc_off + 256);
  const uint32_t bs_off = misc_off + 512;
  const uint32_t bs_base = base + bs_off;
  const uint32_t full0 = base + misc_off, empty0 = full0 + 64;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;

  // work range of this CTA inside its super-chunk
  const int ch0 = blockIdx.y * p.ch_per_super;
  const int nch = min(p.ch_per_super, p.nchunks - ch0);
  const long long total = (long long)p.ntiles * nch;
  const int it_begin = (int)(total * blockIdx.x / gridDim.x);
  const int it_end = (int)(total * (blockIdx.x + 1) / gridDim.x);
  if (it_begin >= it_end) return;

  if (tid == 0) {
    for (int s = 0; s < stages; s++) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kConsumerWarps);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int armed = 0;
      for (int it = it_begin; it < it_end; it++) {
        const int n = it - it_begin;
        const int s = n % stages;
        if (n >= stages) {
          if (!mbar_wait(empty0 + 8 * s, ((n / stages) - 1) & 1)) {
            atomicExch(p.ws_status, 1);
            *s_abort = 1;
            break;
          }
        }
        if (*s_abort) break;
        const int tile = it / nch, ch = ch0 + it % nch;
        mbar_expect_tx(full0 + 8 * s, kStageBytes);
        tma_load_2d(a_base + s * kStageBytes, &tmap, ch * kChunkWords, tile * kTileRows, full0 + 8 * s);
        armed = n + 1;
      }
      if (*s_abort) {
        // drain: every armed box must have landed before the CTA may exit
        for (int n = max(0, armed - stages); n < armed; n++) mbar_wait(full0 + 8 * (n % stages), (n / stages) & 1);
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers: prologue
  const int ctid = tid;  // 0..255
  const int W = p.K / 16;
  const int w0 = ch0 * kChunkWords;
  const int nwords_super = nch * kChunkWords;
  // (a) T0[m] = sum_k q[m][k] over the whole K, and the scales
  for (int m = warp; m < p.M; m += kConsumerWarps) {
    const uint32_t* xr = reinterpret_cast<const uint32_t*>(p.xq + (size_t)m * (p.K / 2));
    int acc = 0;
    for (int i = lane; i < p.K / 8; i += 32) {
      const uint32_t x = __ldg(xr + i);
      int d = 0;
      dp4a_u8s8(d, x & 0x0F0F0F0Fu, 0x01010101u);
      dp4a_u8s8(d, (x >> 4) & 0x0F0F0F0Fu, 0x01010101u);
      acc += d - 16 * __popc(x & 0x88888888u);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) {
      s_T0[m] = acc;
      s_scale[m] = __half2float(p.scale[m]);
    }
  }
  // (b) expanded activations: unit (word, token) = 4 x u32, one per in-byte position p,
  //     byte j of word p = q[token][16*word + 4j + p]
  {
    const uint32_t ncol = p.ncol;
    const int nunits = nwords_super * (int)ncol;
    for (int u = ctid; u < nunits; u += kConsumerWarps * 32) {
      const uint32_t wr = u / ncol, col = u % ncol;
      const int widx = w0 + (int)wr;
      uint4 out = make_uint4(0, 0, 0, 0);
      if ((int)col < p.M && widx < W) {
        const uint2 x = __ldg(reinterpret_cast<const uint2*>(p.xq + (size_t)col * (p.K / 2)) + widx);
        uint32_t r[4];
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
          const uint32_t lo = (x.x >> (4 * pp)) & 0x000F000Fu;
          const uint32_t hi = (x.y >> (4 * pp)) & 0x000F000Fu;
          const uint32_t v = __byte_perm(lo, hi, 0x6420);
          r[pp] = v | ((v & 0x08080808u) * 0x1Eu);  // sign-extend each nibble to a byte
        }
        out = make_uint4(r[0], r[1], r[2], r[3]);
      }
      *reinterpret_cast<uint4*>(gen + bs_off + (size_t)bs_unit(wr, col, ncol) * 16) = out;
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");

  // -------------------------------------------------------------------- consumers: main loop
  constexpr int NTOK_DP = (MODE == kModeMma) ? 0 : 2;  // dp4a modes serve at most two tokens
  int accM[MODE == kModeDp4a ? 1 : MT][MODE == kModeDp4a ? 1 : (MODE == kModeHybrid ? 2 : 3)][4][4];
  int accD[NTOK_DP == 0 ? 1 : NTOK_DP][2][MODE == kModeDp4a ? 3 : 1][4];
#pragma unroll
  for (int a = 0; a < (MODE == kModeDp4a ? 1 : MT); a++)
#pragma unroll
    for (int f = 0; f < (MODE == kModeDp4a ? 1 : (MODE == kModeHybrid ? 2 : 3)); f++)
#pragma unroll
      for (int pp = 0; pp < 4; pp++)
#pragma unroll
        for (int r = 0; r < 4; r++) accM[a][f][pp][r] = 0;
#pragma unroll
  for (int a = 0; a < (NTOK_DP == 0 ? 1 : NTOK_DP); a++)
#pragma unroll
    for (int r = 0; r < 2; r++)
#pragma unroll
      for (int f = 0; f < (MODE == kModeDp4a ? 3 : 1); f++)
#pragma unroll
        for (int pp = 0; pp < 4; pp++) accD[a][r][f][pp] = 0;

  const uint32_t ncol = p.ncol;
  const int M = p.M;
  // token column this lane feeds to the MMA B operand (columns beyond the stored ones repeat)
  uint32_t bcol[MT];
#pragma unroll
  for (int mt = 0; mt < MT; mt++) bcol[mt] = (uint32_t)(8 * mt + g) % ncol;

  const uint32_t a_lane = (uint32_t)(warp * 16 + g) * 128u;
  int cur_tile = it_begin / nch;
  int done_in_tile = 0;
  bool aborted = false;

  auto flush = [&](int tile, int ndone) {
    // ---- gather this lane's (row, token) results as T1,T2,T3
    // MODE kModeMma: lane (g,t) owns tokens 8mt+2t, 8mt+2t+1 for rows g and g+8.
    // dp4a modes:    columns repeat the tokens; partial dp4a sums are reduced over the quad and
    //                lane t==0 owns tokens 0..M-1 for rows g and g+8.
    constexpr int NE = (MODE == kModeMma) ? 4 * MT : 4;
    int T1[NE], T2[NE], T3[NE], etok[NE], erow[NE];
    if constexpr (MODE == kModeMma) {
#pragma unroll
      for (int mt = 0; mt < MT; mt++)
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const int e = mt * 4 + r;
          etok[e] = 8 * mt + 2 * t + (r & 1);
          erow[e] = g + 8 * (r >> 1);
          int a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
          for (int pp = 0; pp < 4; pp++) {
            a1 += accM[mt][0][pp][r] >> (2 * pp);
            a2 += accM[mt][1][pp][r] >> (2 * pp + 1);
            a3 += accM[mt][2][pp][r] >> (2 * pp + 1);
          }
          T1[e] = a1; T2[e] = a2; T3[e] = a3;
        }
    } else {
#pragma unroll
      for (int tok = 0; tok < 2; tok++)
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const int e = tok * 2 + rr;
          etok[e] = (t == 0) ? tok : kMaxTokens;  // only lane t==0 of a quad emits
          erow[e] = g + 8 * rr;
          int a1 = 0, a2 = 0, a3 = 0;
          if constexpr (MODE == kModeHybrid) {
            // MMA column c carries token c % M; lane t==0 holds columns 0 and 1
            const int r = (M == 1 ? 0 : tok) + 2 * rr;
#pragma unroll
            for (int pp = 0; pp < 4; pp++) {
              a1 += accM[0][0][pp][r] >> (2 * pp);
              a2 += accM[0][1][pp][r] >> (2 * pp + 1);
              a3 += accD[tok][rr][0][pp] >> (2 * pp + 1);
            }
          } else {
#pragma unroll
            for (int pp = 0; pp < 4; pp++) {
              a1 += accD[tok][rr][0][pp] >> (2 * pp);
              a2 += accD[tok][rr][1][pp] >> (2 * pp + 1);
              a3 += accD[tok][rr][2][pp] >> (2 * pp + 1);
            }
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            a2 += __shfl_xor_sync(0xffffffffu, a2, 1); a2 += __shfl_xor_sync(0xffffffffu, a2, 2);
          }
          a3 += __shfl_xor_sync(0xffffffffu, a3, 1); a3 += __shfl_xor_sync(0xffffffffu, a3, 2);
          T1[e] = a1; T2[e] = a2; T3[e] = a3;
        }
    }
    const int row0 = tile * kTileRows + warp * 16;
    bool finish = true;
    if (ndone != p.nchunks) {
      // ---- partial tile: add into the scratch sums, the last contributor finishes
#pragma unroll
      for (int e = 0; e < NE; e++) {
        if (etok[e] < M && row0 + erow[e] < p.N) {
          int32_t* dst = p.ws_sum + ((size_t)(row0 + erow[e]) * M + etok[e]) * 3;
          atomicAdd(dst + 0, T1[e]);
          atomicAdd(dst + 1, T2[e]);
          atomicAdd(dst + 2, T3[e]);
        }
      }
      __threadfence();
      __syncwarp();
      uint32_t old = 0;
      if (lane == 0) old = atomicAdd(p.ws_count + tile * kConsumerWarps + warp, (uint32_t)ndone);
      old = __shfl_sync(0xffffffffu, old, 0);
      finish = (old + (uint32_t)ndone == (uint32_t)p.nchunks);
      if (finish) {
        __threadfence();
#pragma unroll
        for (int e = 0; e < NE; e++) {
          if (etok[e] < M && row0 + erow[e] < p.N) {
            int32_t* src = p.ws_sum + ((size_t)(row0 + erow[e]) * M + etok[e]) * 3;
            T1[e] = atomicExch(src + 0, 0);
            T2[e] = atomicExch(src + 1, 0);
            T3[e] = atomicExch(src + 2, 0);
          }
        }
        if (lane == 0) atomicExch(p.ws_count + tile * kConsumerWarps + warp, 0u);
      }
    }
    if (finish) {
#pragma unroll
      for (int e = 0; e < NE; e++) {
        const int row = row0 + erow[e];
        if (etok[e] < M && row < p.N) {
          const int S3 = T3[e], S1 = T1[e] - T3[e], S2 = T2[e] - T3[e];
          const int S0 = s_T0[etok[e]] - S1 - S2 - S3;
          p.y[(size_t)etok[e] * p.N + row] = lut_finish(s_scale[etok[e]], __ldg(p.lut + row), S0, S1, S2, S3);
        }
      }
    }
    // reset accumulators
#pragma unroll
    for (int a = 0; a < (MODE == kModeDp4a ? 1 : MT); a++)
#pragma unroll
      for (int f = 0; f < (MODE == kModeDp4a ? 1 : (MODE == kModeHybrid ? 2 : 3)); f++)
#pragma unroll
        for (int pp = 0; pp < 4; pp++)
#pragma unroll
          for (int r = 0; r < 4; r++) accM[a][f][pp][r] = 0;
#pragma unroll
    for (int a = 0; a < (NTOK_DP == 0 ? 1 : NTOK_DP); a++)
#pragma unroll
      for (int r = 0; r < 2; r++)
#pragma unroll
        for (int f = 0; f < (MODE == kModeDp4a ? 3 : 1); f++)
#pragma unroll
          for (int pp = 0; pp < 4; pp++) accD[a][r][f][pp] = 0;
  };

  for (int it = it_begin; it < it_end; it++) {
    const int n = it - it_begin;
    const int s = n % stages;
    const int tile = it / nch, chrel = it % nch;
    if (tile != cur_tile) {
      flush(cur_tile, done_in_tile);
      cur_tile = tile;
      done_in_tile = 0;
    }
    if (!mbar_wait(full0 + 8 * s, (n / stages) & 1)) {
      if (lane == 0) atomicExch(p.ws_status, 2);
      *s_abort = 1;
      aborted = true;
      break;
    }
    const uint32_t a_stage = a_base + s * kStageBytes + a_lane;
#pragma unroll
    for (int i = 0; i < 2; i++) {
      const uint32_t chunk16 = (uint32_t)((2 * t + i) ^ (g & 7)) << 4;
      const uint4 U = lds128(a_stage + chunk16);
      const uint4 V = lds128(a_stage + 8 * 128 + chunk16);
      const uint32_t uw[4] = {U.x, U.y, U.z, U.w};
      const uint32_t vw[4] = {V.x, V.y, V.z, V.w};
      const uint32_t wrel = (uint32_t)chrel * kChunkWords + 8u * t + 4u * i;  // + e
#pragma unroll
      for (int pr = 0; pr < 2; pr++) {
        const int e0 = 2 * pr, e1 = 2 * pr + 1;
        // activation operands for the two k-words, per MMA column group / dp4a token
        uint4 bm0[MT], bm1[MT];
        if constexpr (MODE != kModeDp4a) {
#pragma unroll
          for (int mt = 0; mt < MT; mt++) {
            bm0[mt] = lds128(bs_base + bs_unit(wrel + e0, bcol[mt], ncol) * 16);
            bm1[mt] = lds128(bs_base + bs_unit(wrel + e1, bcol[mt], ncol) * 16);
          }
        }
        uint4 bd0[2], bd1[2];
        if constexpr (MODE != kModeMma) {
#pragma unroll
          for (int tok = 0; tok < 2; tok++) {
            if (tok < M) {
              if (MODE == kModeHybrid && M == 1) {
                bd0[tok] = bm0[0];
                bd1[tok] = bm1[0];
              } else {
                bd0[tok] = lds128(bs_base + bs_unit(wrel + e0, tok, ncol) * 16);
                bd1[tok] = lds128(bs_base + bs_unit(wrel + e1, tok, ncol) * 16);
              }
            } else {
              bd0[tok] = make_uint4(0, 0, 0, 0);
              bd1[tok] = make_uint4(0, 0, 0, 0);
            }
          }
        }
        const uint32_t u0 = uw[e0], u1 = uw[e1], v0 = vw[e0], v1 = vw[e1];
        const uint32_t u0s = u0 + u0, u1s = u1 + u1, v0s = v0 + v0, v1s = v1 + v1;  // b0 moved onto b1's bit
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
          const uint32_t m0 = 0x01010101u << (2 * pp), m1 = m0 << 1;
          if constexpr (MODE != kModeDp4a) {
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
              const uint32_t b0 = (&bm0[mt].x)[pp], b1 = (&bm1[mt].x)[pp];
              mma_u8s8(accM[mt][0][pp], u0 & m0, v0 & m0, u1 & m0, v1 & m0, b0, b1);
              mma_u8s8(accM[mt][1][pp], u0 & m1, v0 & m1, u1 & m1, v1 & m1, b0, b1);
              if constexpr (MODE == kModeMma)
                mma_u8s8(accM[mt][2][pp], u0 & u0s & m1, v0 & v0s & m1, u1 & u1s & m1, v1 & v1s & m1, b0, b1);
            }
          }
          if constexpr (MODE == kModeHybrid) {
            const uint32_t pu0 = u0 & u0s & m1, pv0 = v0 & v0s & m1, pu1 = u1 & u1s & m1, pv1 = v1 & v1s & m1;
#pragma unroll
            for (int tok = 0; tok < 2; tok++) {
              if (tok < M) {
                const uint32_t b0 = (&bd0[tok].x)[pp], b1 = (&bd1[tok].x)[pp];
                dp4a_u8s8(accD[tok][0][0][pp], pu0, b0);
                dp4a_u8s8(accD[tok][0][0][pp], pu1, b1);
                dp4a_u8s8(accD[tok][1][0][pp], pv0, b0);
                dp4a_u8s8(accD[tok][1][0][pp], pv1, b1);
              }
            }
          }
          if constexpr (MODE == kModeDp4a) {
            const uint32_t au0[3] = {u0 & m0, u0 & m1, u0 & u0s & m1};
            const uint32_t au1[3] = {u1 & m0, u1 & m1, u1 & u1s & m1};
            const uint32_t av0[3] = {v0 & m0, v0 & m1, v0 & v0s & m1};
            const uint32_t av1[3] = {v1 & m0, v1 & m1, v1 & v1s & m1};
#pragma unroll
            for (int tok = 0; tok < 2; tok++) {
              if (tok < M) {
                const uint32_t b0 = (&bd0[tok].x)[pp], b1 = (&bd1[tok].x)[pp];
#pragma unroll
                for (int f = 0; f < 3; f++) {
                  dp4a_u8s8(accD[tok][0][f][pp], au0[f], b0);
                  dp4a_u8s8(accD[tok][0][f][pp], au1[f], b1);
                  dp4a_u8s8(accD[tok][1][f][pp], av0[f], b0);
                  dp4a_u8s8(accD[tok][1][f][pp], av1[f], b1);
                }
              }
            }
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + 8 * s);
    done_in_tile++;
  }
  if (!aborted) flush(cur_tile, done_in_tile);
}

}  // namespace rcp
