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
// Data movement: the packed weights are the only large stream. Persistent CTAs (two per SM) take
// equal, contiguous shares of the (128-row tile, 512-code K chunk) work items. Each of the eight
// warps of a CTA owns 16 rows of the tile and runs its own pipeline: lane 0 streams 16-row x
// 128-byte boxes into the warp's shared-memory ring with TMA (cp.async.bulk.tensor, 128B swizzle,
// mbarrier completion) and the warp reads them bank-conflict free; warps never wait on each other
// after the prologue. The int4 activations are expanded once per CTA into the B-operand byte
// layout in shared memory.
// Tiles split between CTAs are combined with integer atomics in a caller-provided scratch buffer
// (order independent, hence deterministic); the last contributor finishes the tile and re-zeroes it.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace rcp {

constexpr int kTileRows = 128;       // rows per work item (8 consumer warps x 16)
constexpr int kChunkWords = 32;      // 32-bit words per row per work item (128 bytes, 512 codes)
constexpr int kWarps = 8;
constexpr int kWarpRows = kTileRows / kWarps;                  // 16 = the m of mma.m16n8k32
constexpr int kBoxBytes = kWarpRows * kChunkWords * 4;         // 2 KB per warp per work item
constexpr int kStageBytes = kWarps * kBoxBytes;                // 16 KB per CTA per ring slot
constexpr int kStreamThreads = kWarps * 32;
constexpr int kMaxStages = 8;
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded waits: give up, flag the error, drain and exit

enum StreamMode { kModeMma = 0, kModeHybrid = 1, kModeDp4a = 2 };
#ifdef RCP_EXPERIMENTS
// measurement-only switches (wrong results): 1 = stream the boxes but skip the math, 2 = do the math
// on whatever the ring holds without streaming
__device__ int g_experiment = 0;
#endif

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
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void dp4a_u8s8(int& d, uint32_t a, uint32_t b) {
  asm("dp4a.u32.s32 %0, %1, %2, %0;" : "+r"(d) : "r"(a), "r"(b));
}

// Byte offset of the 32-byte unit of (word pair inside the super-chunk, token column) in the
// expanded activation buffer. A unit holds, for the two words of the pair and the four in-byte
// positions p, the u32 of four int8 activations: index p*2 + (word & 1), so that the two B
// registers of one MMA are adjacent. The low two bits of the pair index are XORed with the k-slice
// (t = bits 2..3) so that the four slices a quad reads at once fall into different banks.
__device__ __forceinline__ uint32_t bs_pair_off(uint32_t pair_rel, uint32_t col, uint32_t ncol) {
  const uint32_t sw = (pair_rel & ~3u) | ((pair_rel ^ (pair_rel >> 2)) & 3u);
  return (sw * ncol + col) * 32u;
}

// ----------------------------------------------------------------------------- the kernel
// MT    column groups of 8 tokens fed to the MMA (1 or 2)
// MODE  kModeMma: all three planes on the tensor cores; kModeHybrid: b0 and b1 planes on the tensor
//       cores, the b0*b1 plane on dp4a; kModeDp4a: everything on dp4a (CUDA cores only)
// MTOK  tokens, fixed at compile time for the dp4a modes (1 or 2); 0 = run-time (kModeMma)
// MINB  CTAs per SM the register budget is sized for
template <int MT, int MODE, int MTOK, int MINB>
__global__ void __launch_bounds__(kStreamThreads, MINB)
gemv_stream_kernel(const __grid_constant__ CUtensorMap tmap, const StreamParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;           // TMA 128B swizzle wants 1024-byte alignment
  uint8_t* const gen = smem_raw + (base - raw);
  const int stages = p.stages;
  const uint32_t misc_off = (uint32_t)stages * kStageBytes;
  // misc: full barriers [warp][stage] (512 B), T0 [16], scales [16]
  int* const s_T0 = reinterpret_cast<int*>(gen + misc_off + 512);
  float* const s_scale = reinterpret_cast<float*>(gen + misc_off + 576);
  const uint32_t bs_off = misc_off + 640;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const uint32_t full0 = base + misc_off + (uint32_t)warp * (kMaxStages * 8);   // this warp's barriers
  const uint32_t ring0 = base + (uint32_t)warp * kBoxBytes;                     // slot s at + s*kStageBytes

  // work range of this CTA inside its super-chunk
  const int ch0 = blockIdx.y * p.ch_per_super;
  const int nch = min(p.ch_per_super, p.nchunks - ch0);
  const long long total = (long long)p.ntiles * nch;
  const int it_begin = (int)(total * blockIdx.x / gridDim.x);
  const int it_end = (int)(total * (blockIdx.x + 1) / gridDim.x);
  if (it_begin >= it_end) return;
  const int nitems = it_end - it_begin;

  if (lane == 0) {
    for (int s = 0; s < stages; s++) mbar_init(full0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kMaxTokens) s_T0[tid] = 0;
  __syncwarp();

  // The weights do not depend on the preceding kernel: start streaming at once.
  auto issue = [&](int s, int tile, int chrel) {  // lane 0 only
    mbar_expect_tx(full0 + 8 * s, kBoxBytes);
    tma_load_2d(ring0 + s * kStageBytes, &tmap, (ch0 + chrel) * kChunkWords, tile * kTileRows + warp * kWarpRows,
                full0 + 8 * s);
  };
  // (tile, chunk) of the next item to request; advanced without divisions in the main loop
  int ld_tile = it_begin / nch, ld_ch = it_begin % nch;
  const int pre = min(stages, nitems);
#ifdef RCP_EXPERIMENTS
  const int experiment = g_experiment;
#else
  constexpr int experiment = 0;
#endif
  for (int n = 0; n < pre; n++) {
    if (lane == 0 && experiment != 2) issue(n, ld_tile, ld_ch);
    if (++ld_ch == nch) { ld_ch = 0; ld_tile++; }
  }
  __syncthreads();

  // -------------------------------------------------------------------- prologue
  const int M = (MTOK > 0) ? MTOK : p.M;
  const uint32_t ncol = (MTOK > 0) ? (uint32_t)MTOK : (uint32_t)p.ncol;
  const int W = p.K / 16;
  const int w0 = ch0 * kChunkWords;
  // (a) T0[m] = sum_k q[m][k] over the whole K (all threads share the pass), and the scales
  {
    const int per_tok = p.K / 8;
    for (int idx = tid; idx < M * per_tok; idx += kStreamThreads) {
      const int m = idx / per_tok;
      const uint32_t x = __ldg(reinterpret_cast<const uint32_t*>(p.xq) + idx);
      int d = 0;
      dp4a_u8s8(d, x & 0x0F0F0F0Fu, 0x01010101u);
      dp4a_u8s8(d, (x >> 4) & 0x0F0F0F0Fu, 0x01010101u);
      atomicAdd(&s_T0[m], d - 16 * __popc(x & 0x88888888u));
    }
    if (tid < M) s_scale[tid] = __half2float(p.scale[tid]);
  }
  // (b) expanded activations, see bs_pair_off: byte j of the u32 (word, p) = q[token][16*word + 4j + p]
  {
    const int nwords_super = nch * kChunkWords;
    const int nunits = nwords_super * (int)ncol;
    for (int u = tid; u < nunits; u += kStreamThreads) {
      const uint32_t wr = (uint32_t)u / ncol, col = (uint32_t)u % ncol;
      const int widx = w0 + (int)wr;
      uint32_t r[4] = {0, 0, 0, 0};
      if ((int)col < M && widx < W) {
        const uint2 x = __ldg(reinterpret_cast<const uint2*>(p.xq + (size_t)col * (p.K / 2)) + widx);
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
          const uint32_t lo = (x.x >> (4 * pp)) & 0x000F000Fu;
          const uint32_t hi = (x.y >> (4 * pp)) & 0x000F000Fu;
          const uint32_t v = __byte_perm(lo, hi, 0x6420);
          r[pp] = v | ((v & 0x08080808u) * 0x1Eu);  // sign-extend each nibble to a byte
        }
      }
      uint32_t* dst = reinterpret_cast<uint32_t*>(gen + bs_off + bs_pair_off(wr >> 1, col, ncol)) + (wr & 1u);
#pragma unroll
      for (int pp = 0; pp < 4; pp++) dst[2 * pp] = r[pp];
    }
  }
  __syncthreads();

  // -------------------------------------------------------------------- main loop (per warp)
  constexpr int NF_M = (MODE == kModeDp4a) ? 0 : (MODE == kModeHybrid ? 2 : 3);  // planes on the MMA
  constexpr int NF_D = (MODE == kModeDp4a) ? 3 : (MODE == kModeHybrid ? 1 : 0);  // planes on dp4a
  constexpr int NTD = (NF_D == 0) ? 1 : MTOK;
  int accM[MT][NF_M == 0 ? 1 : NF_M][4][4];
  int accD[NTD][2][NF_D == 0 ? 1 : NF_D][4];
  auto zero_acc = [&]() {
#pragma unroll
    for (int a = 0; a < MT; a++)
#pragma unroll
      for (int f = 0; f < (NF_M == 0 ? 1 : NF_M); f++)
#pragma unroll
        for (int pp = 0; pp < 4; pp++)
#pragma unroll
          for (int r = 0; r < 4; r++) accM[a][f][pp][r] = 0;
#pragma unroll
    for (int a = 0; a < NTD; a++)
#pragma unroll
      for (int r = 0; r < 2; r++)
#pragma unroll
        for (int f = 0; f < (NF_D == 0 ? 1 : NF_D); f++)
#pragma unroll
          for (int pp = 0; pp < 4; pp++) accD[a][r][f][pp] = 0;
  };
  zero_acc();

  // per-lane constant parts of the shared-memory addresses
  //   weights: row g (and g+8) of the warp's box, 16-byte chunk (2t+i) ^ (row & 7) under the 128B swizzle
  const uint8_t* const a_lane = gen + (size_t)warp * kBoxBytes + (size_t)g * 128;
  uint32_t a_chunk[2];
#pragma unroll
  for (int i = 0; i < 2; i++) a_chunk[i] = (uint32_t)((2 * t + i) ^ (g & 7)) << 4;
  //   activations: the four word pairs (2i+pr) this lane's k-slice covers inside a chunk
  const uint8_t* const bs_gen = gen + bs_off;
  uint32_t bM_off[MT][4];
  uint32_t bD_off[NTD][4];
#pragma unroll
  for (int c = 0; c < 4; c++) {
#pragma unroll
    for (int mt = 0; mt < MT; mt++) bM_off[mt][c] = bs_pair_off(4u * t + c, (uint32_t)(8 * mt + g) % ncol, ncol);
#pragma unroll
    for (int tok = 0; tok < NTD; tok++) bD_off[tok][c] = bs_pair_off(4u * t + c, (uint32_t)tok % ncol, ncol);
  }
  const uint32_t b_chunk_stride = (kChunkWords / 2) * ncol * 32;  // bytes of expanded activations per K chunk

  int cur_tile = it_begin / nch;
  int done_in_tile = 0;
  uint2 lut_g[2];  // LUT rows g and g+8 of the current tile, fetched ahead of the epilogue
  auto fetch_lut = [&](int tile) {
#pragma unroll
    for (int rr = 0; rr < 2; rr++) {
      const int row = tile * kTileRows + warp * kWarpRows + g + 8 * rr;
      lut_g[rr] = row < p.N ? __ldg(p.lut + row) : make_uint2(0, 0);
    }
  };
  fetch_lut(cur_tile);

  auto flush = [&](int tile, int ndone) {
    // ---- this lane's (row, token) results as T1,T2,T3
    // kModeMma:   lane (g,t) owns tokens 8mt+2t, 8mt+2t+1 for rows g and g+8.
    // dp4a modes: MMA columns repeat the tokens; dp4a partial sums are reduced over the quad and
    //             lane t==0 owns tokens 0..MTOK-1 for rows g and g+8.
    constexpr int NE = (MODE == kModeMma) ? 4 * MT : 2 * NTD;
    int T1[NE], T2[NE], T3[NE], etok[NE], err[NE];
    if constexpr (MODE == kModeMma) {
#pragma unroll
      for (int mt = 0; mt < MT; mt++)
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const int e = mt * 4 + r;
          etok[e] = 8 * mt + 2 * t + (r & 1);
          err[e] = r >> 1;
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
      for (int tok = 0; tok < NTD; tok++)
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const int e = tok * 2 + rr;
          etok[e] = (t == 0) ? tok : kMaxTokens;  // only lane t==0 of a quad emits
          err[e] = rr;
          int a1 = 0, a2 = 0, a3 = 0;
          if constexpr (MODE == kModeHybrid) {
            // MMA column c carries token c % MTOK; lane t==0 holds columns 0 and 1
            const int r = tok + 2 * rr;
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
    const int row0 = tile * kTileRows + warp * kWarpRows + g;
    bool finish = true;
    if (ndone != p.nchunks) {
      // ---- partial tile: add into the scratch sums, the last contributor finishes
#pragma unroll
      for (int e = 0; e < NE; e++) {
        const int row = row0 + 8 * err[e];
        if (etok[e] < M && row < p.N) {
          int32_t* dst = p.ws_sum + ((size_t)row * M + etok[e]) * 3;
          atomicAdd(dst + 0, T1[e]);
          atomicAdd(dst + 1, T2[e]);
          atomicAdd(dst + 2, T3[e]);
        }
      }
      __threadfence();
      __syncwarp();
      uint32_t old = 0;
      if (lane == 0) old = atomicAdd(p.ws_count + tile * kWarps + warp, (uint32_t)ndone);
      old = __shfl_sync(0xffffffffu, old, 0);
      finish = (old + (uint32_t)ndone == (uint32_t)p.nchunks);
      if (finish) {
        __threadfence();
#pragma unroll
        for (int e = 0; e < NE; e++) {
          const int row = row0 + 8 * err[e];
          if (etok[e] < M && row < p.N) {
            int32_t* src = p.ws_sum + ((size_t)row * M + etok[e]) * 3;
            T1[e] = atomicExch(src + 0, 0);
            T2[e] = atomicExch(src + 1, 0);
            T3[e] = atomicExch(src + 2, 0);
          }
        }
        if (lane == 0) atomicExch(p.ws_count + tile * kWarps + warp, 0u);
      }
    }
    if (finish) {
#pragma unroll
      for (int e = 0; e < NE; e++) {
        const int row = row0 + 8 * err[e];
        if (etok[e] < M && row < p.N) {
          const int S3 = T3[e], S1 = T1[e] - T3[e], S2 = T2[e] - T3[e];
          const int S0 = s_T0[etok[e]] - S1 - S2 - S3;
          p.y[(size_t)etok[e] * p.N + row] = lut_finish(s_scale[etok[e]], lut_g[err[e]], S0, S1, S2, S3);
        }
      }
    }
    zero_acc();
  };

  int tile = cur_tile, chrel = it_begin % nch;  // item being consumed
  int s = 0;                                    // its ring slot
  uint32_t parity = 0;                          // phase of the slot's barrier
  for (int n = 0; n < nitems; n++) {
    if (tile != cur_tile) {
      flush(cur_tile, done_in_tile);
      cur_tile = tile;
      done_in_tile = 0;
      fetch_lut(tile);
    }
    if (experiment != 2 && !mbar_wait(full0 + 8 * s, parity)) {
      // give up: flag the error, wait (bounded) for the boxes still in flight, leave
      if (lane == 0) atomicExch(p.ws_status, 2);
      for (int k = n + 1; k < min(nitems, n + stages); k++) mbar_wait(full0 + 8 * (k % stages), (k / stages) & 1);
      return;
    }
    const uint8_t* const a_stage = a_lane + (size_t)s * kStageBytes;
    const uint8_t* const b_chunk = bs_gen + (size_t)chrel * b_chunk_stride;
#pragma unroll
    for (int i = 0; i < (experiment == 1 ? 0 : 2); i++) {
      const uint4 U = *reinterpret_cast<const uint4*>(a_stage + a_chunk[i]);
      const uint4 V = *reinterpret_cast<const uint4*>(a_stage + 8 * 128 + a_chunk[i]);
      const uint32_t uw[4] = {U.x, U.y, U.z, U.w};
      const uint32_t vw[4] = {V.x, V.y, V.z, V.w};
#pragma unroll
      for (int pr = 0; pr < 2; pr++) {
        const int e0 = 2 * pr, e1 = 2 * pr + 1, c = 2 * i + pr;
        // activation operands of the word pair: [position p][word]
        uint32_t bM[MT][4][2];
        uint32_t bD[NTD][4][2];
        if constexpr (NF_D > 0) {
#pragma unroll
          for (int tok = 0; tok < NTD; tok++) {
            const uint4 x = *reinterpret_cast<const uint4*>(b_chunk + bD_off[tok][c]);
            const uint4 y = *reinterpret_cast<const uint4*>(b_chunk + bD_off[tok][c] + 16);
            bD[tok][0][0] = x.x; bD[tok][0][1] = x.y; bD[tok][1][0] = x.z; bD[tok][1][1] = x.w;
            bD[tok][2][0] = y.x; bD[tok][2][1] = y.y; bD[tok][3][0] = y.z; bD[tok][3][1] = y.w;
          }
        }
        if constexpr (NF_M > 0) {
          if constexpr (MODE == kModeHybrid && MTOK == 1) {
#pragma unroll
            for (int pp = 0; pp < 4; pp++) { bM[0][pp][0] = bD[0][pp][0]; bM[0][pp][1] = bD[0][pp][1]; }
          } else {
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
              const uint4 x = *reinterpret_cast<const uint4*>(b_chunk + bM_off[mt][c]);
              const uint4 y = *reinterpret_cast<const uint4*>(b_chunk + bM_off[mt][c] + 16);
              bM[mt][0][0] = x.x; bM[mt][0][1] = x.y; bM[mt][1][0] = x.z; bM[mt][1][1] = x.w;
              bM[mt][2][0] = y.x; bM[mt][2][1] = y.y; bM[mt][3][0] = y.z; bM[mt][3][1] = y.w;
            }
          }
        }
        const uint32_t u0 = uw[e0], u1 = uw[e1], v0 = vw[e0], v1 = vw[e1];
        const uint32_t u0s = u0 + u0, u1s = u1 + u1, v0s = v0 + v0, v1s = v1 + v1;  // b0 moved onto b1's bit
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
          const uint32_t m0 = 0x01010101u << (2 * pp), m1 = m0 << 1;
          // the three planes of the four words: b0, b1, b0*b1 (the last two scaled by 2)
          const uint32_t au0[3] = {u0 & m0, u0 & m1, u0 & u0s & m1};
          const uint32_t au1[3] = {u1 & m0, u1 & m1, u1 & u1s & m1};
          const uint32_t av0[3] = {v0 & m0, v0 & m1, v0 & v0s & m1};
          const uint32_t av1[3] = {v1 & m0, v1 & m1, v1 & v1s & m1};
#pragma unroll
          for (int f = 0; f < NF_M; f++)
#pragma unroll
            for (int mt = 0; mt < MT; mt++)
              mma_u8s8(accM[mt][f][pp], au0[f], av0[f], au1[f], av1[f], bM[mt][pp][0], bM[mt][pp][1]);
#pragma unroll
          for (int f = 0; f < NF_D; f++) {
            const int fa = 3 - NF_D + f;  // hybrid: plane 2 only; dp4a: planes 0..2
#pragma unroll
            for (int tok = 0; tok < NTD; tok++) {
              dp4a_u8s8(accD[tok][0][f][pp], au0[fa], bD[tok][pp][0]);
              dp4a_u8s8(accD[tok][1][f][pp], av0[fa], bD[tok][pp][0]);
              dp4a_u8s8(accD[tok][0][f][pp], au1[fa], bD[tok][pp][1]);
              dp4a_u8s8(accD[tok][1][f][pp], av1[fa], bD[tok][pp][1]);
            }
          }
        }
      }
    }
    __syncwarp();
    // the slot is free again: refill it with the item `stages` ahead
    if (n + stages < nitems) {
      if (lane == 0 && experiment != 2) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(s, ld_tile, ld_ch);
      }
      if (++ld_ch == nch) { ld_ch = 0; ld_tile++; }
    }
    done_in_tile++;
    if (++chrel == nch) { chrel = 0; tile++; }
    if (++s == stages) { s = 0; parity ^= 1u; }
  }
  flush(cur_tile, done_in_tile);
}

}  // namespace rcp
