// Streaming LUT GEMV for sm_100a (Section 4.4 of the paper: O = S * X_q * LUT[W_q]).
//
// Exact integer formulation. With b0 = code & 1, b1 = code >> 1 and, per output row,
//   T1 = sum_k b0 q,  T2 = sum_k b1 q,  T3 = sum_k b0 b1 q,  T0 = sum_k q   (T0 is row independent)
// the per-code sums are S3 = T3, S1 = T1 - T3, S2 = T2 - T3, S0 = T0 - T1 - T2 + T3.
// A 32-bit weight word holds 16 codes; byte j holds codes 4j..4j+3 at in-byte positions p = 0..3.
// Masking the word with 0x01010101 << 2p leaves one b0 bit per byte, scaled by 4^p: four such bytes
// are the A operand of an 8-bit integer dot product whose B operand is the four matching int8
// activations. Twelve masked words (three planes x four positions) cover a word; each costs one
// LOP3 on the 64-lane/clk logic pipe, the scarce resource. The products go to int8 mma.sync
// (16 rows x 32 bytes per instruction, tokens in the n dimension) and/or to dp4a on the FMA pipe.
// Even positions meet activations pre-multiplied by 4, so positions {0,1} and {2,3} share an
// accumulator (scaled by 4 and 64, twice that for the planes masked at the b1 bit).
//
// Data movement. The packed weights are the only large stream. One persistent CTA per SM: a
// producer thread streams 256-row x 128-byte boxes (32 KB) into a shared-memory ring with TMA
// (cp.async.bulk.tensor, 128B swizzle, mbarrier completion); sixteen consumer warps each own 16
// rows of the box over the whole K range, read their MMA fragments bank-conflict free, keep the
// partial sums in registers and finish their rows themselves, so the consumers never wait on one
// another. Tiles (256 rows x K) are dealt round-robin over the CTAs; the tiles left over are split
// along K between CTAs and come first. Their partial sums meet in a caller-provided scratch buffer
// (integer atomics, order independent, hence deterministic); the memory fence, the count of
// contributions and the finishing of a completed tile are the job of a separate warp, so that
// their latency stays off the consumers' path; the last contributor re-zeroes the scratch. The
// int4 activations are expanded once per CTA into the B-operand byte layout in shared memory.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace rcp {

constexpr int kCWarps = 16;                       // consumer warps
constexpr int kGThreads = (kCWarps + 2) * 32;     // + one producer warp + one finishing warp
constexpr int kPartRing = 8;                      // partial segments in flight between consumers and finisher
constexpr int kTileRows = 16 * kCWarps;           // rows of a TMA box
constexpr int kStageWords = 32;                   // 128 bytes of K per row per stage (512 codes)
constexpr int kStageBytes = kTileRows * kStageWords * 4;
constexpr int kMaxStages = 8;
constexpr int kMaxSps = 64;                       // stages per tile one CTA may handle
constexpr uint32_t kSpinLimit = 1u << 22;         // bounded waits: give up, flag the error and exit

enum GemvMode { kModeMma = 0, kModeHybrid = 1, kModeDp4a = 2 };

struct GemvParams {
  const uint2* lut;
  const uint8_t* xq;
  const __half* scale;
  __half* y;
  int32_t* ws_status;   // [4]
  uint32_t* ws_count;   // [ntiles]
  int32_t* ws_T0;       // [ntiles][M]
  int32_t* ws_sum;      // [ntiles * 256][M][3]
  int M, N, K;
  int ntiles;           // 256-row tiles
  int spt_all;          // stages per tile over the whole K
  int sps;              // stages per tile handled by one blockIdx.y
  int stages;           // ring depth
  int off_bar, off_T0st, off_T0, off_scale, off_bs;   // shared-memory byte offsets from the aligned base
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
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
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

// One segment of a CTA's work: stages [sb, se) of a tile (stage indices relative to blockIdx.y's range).
struct Segment { int tile, sb, se; };

// The work of CTA b of G: first an equal share of the stages of the tiles left over when the tiles
// are dealt round-robin (at most two segments), then the rounds of whole tiles.
struct WorkList {
  int G, b, R, spt, tail_tile, tail_sb, tail_n, ntail, nseg;
  __device__ __forceinline__ WorkList(int ntiles, int spt_, int G_, int b_) : G(G_), b(b_), spt(spt_) {
    R = ntiles / G;
    const long long rem = (long long)(ntiles - R * G) * spt;
    const int lo = (int)(rem * b / G), hi = (int)(rem * (b + 1) / G);
    tail_n = hi - lo;
    tail_sb = tail_n > 0 ? lo % spt : 0;
    tail_tile = R * G + (tail_n > 0 ? lo / spt : 0);
    ntail = (tail_n > 0 ? 1 : 0) + (tail_sb + tail_n > spt ? 1 : 0);
    nseg = R + ntail;
  }
  __device__ __forceinline__ Segment get(int i) const {
    Segment s;
    if (i >= ntail) { s.tile = (i - ntail) * G + b; s.sb = 0; s.se = spt; }
    else if (i == 0) { s.tile = tail_tile; s.sb = tail_sb; s.se = min(spt, tail_sb + tail_n); }
    else { s.tile = tail_tile + 1; s.sb = 0; s.se = tail_sb + tail_n - spt; }
    return s;
  }
};

// Expanded activations. A stage is 32 words of a row; consumer lane t reads 16-byte chunk 2t+i of
// the row in sub-step i, i.e. words 8t+4i .. 8t+4i+3, as two word pairs pr. For every
// (stage, i, pr) and token column there are two 16-byte halves per lane slice t; half h holds
// positions 2h and 2h+1:
//   { q[p=2h][word x], q[2h][word y], q[2h+1][word x], q[2h+1][word y] },  byte j of q[p][w] =
//   activation of code 16 w + 4 j + p, times 4 when p is even.
// Byte address of (stage, i, pr, half, col, t): ((((stage*2 + i)*2 + pr)*2 + half)*ncol + col)*64 + t*16.

// MT    column groups of 8 tokens fed to the MMA (1 or 2)
// MODE  kModeMma: all three planes on the tensor cores; kModeHybrid: b0 and b1 planes on the tensor
//       cores, the b0*b1 plane on dp4a; kModeDp4a: everything on dp4a (CUDA cores only)
// MTOK  tokens, fixed at compile time for the dp4a modes (1 or 2); 0 = run-time (kModeMma)
template <int MT, int MODE, int MTOK>
__global__ void __launch_bounds__(kGThreads, 1)
gemv_stream_kernel(const __grid_constant__ CUtensorMap tmap, const GemvParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;           // TMA 128B swizzle wants 1024-byte alignment
  uint8_t* const gen = smem_raw + (base - raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int M = (MTOK > 0) ? MTOK : p.M;
  const int ncol = M;
  const int stages = p.stages;
  const uint32_t full0 = base + p.off_bar, empty0 = full0 + 8 * kMaxStages;
  const uint32_t part0 = empty0 + 8 * kMaxStages, done0 = part0 + 8 * kPartRing;
  int* const s_T0st = reinterpret_cast<int*>(gen + p.off_T0st);         // [M][kMaxSps]
  float* const s_scale = reinterpret_cast<float*>(gen + p.off_scale);   // [16]
  uint8_t* const bs = gen + p.off_bs;

  const int st0 = blockIdx.y * p.sps;                  // first stage (of a tile) handled here
  const int spt = min(p.sps, p.spt_all - st0);         // stages per tile handled here
  const WorkList work(p.ntiles, spt, gridDim.x, blockIdx.x);
  if (work.nseg == 0) return;
  const bool one_range = (gridDim.y == 1);
  auto is_whole = [&](const Segment& sg) { return one_range && sg.sb == 0 && sg.se == p.spt_all; };

  // ------------------------------------------------------------------ producer prologue
  // The weights do not depend on the preceding kernel: start streaming at once.
  int pr_seg = 0, pr_slot = 0;
  uint32_t pr_phase = 0;
  Segment pr_cur = work.get(0);
  int pr_st = pr_cur.sb;
  auto produce = [&]() {  // one stage; the producer thread only
    mbar_expect_tx(full0 + 8 * pr_slot, kStageBytes);
    tma_load_2d(base + pr_slot * kStageBytes, &tmap, (st0 + pr_st) * kStageWords, pr_cur.tile * kTileRows,
                full0 + 8 * pr_slot);
    if (++pr_st == pr_cur.se) {
      if (++pr_seg < work.nseg) { pr_cur = work.get(pr_seg); pr_st = pr_cur.sb; }
    }
    if (++pr_slot == stages) { pr_slot = 0; pr_phase ^= 1u; }
  };
  if (tid == kCWarps * 32) {
    // the producer thread sets up every barrier itself and starts the stream before the CTA meets
    for (int s = 0; s < stages; s++) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, kCWarps); }
    for (int s = 0; s < kPartRing; s++) { mbar_init(part0 + 8 * s, kCWarps); mbar_init(done0 + 8 * s, 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < stages && pr_seg < work.nseg; i++) produce();
  }

  // ------------------------------------------------------------------ activations (all threads)
  // Expands the activations of this K range; one unit = (column, stage, i, pr, t) = two words.
  // The 16 units of a (column, stage) are 16 consecutive lanes: their sum of q is T0 of the stage.
  {
    const int W = p.K / 16;
    const int total = ncol * spt * 16;
    for (int u0 = warp * 32; u0 < total; u0 += kGThreads) {
      const int u = u0 + lane;
      int tsum = 0;
      const int pair = u >> 4;
      const int col = pair / spt, st = pair - col * spt;
      if (u < total) {
        const int tt = u & 3, pr = (u >> 2) & 1, i = (u >> 3) & 1;
        const int wx = (st0 + st) * kStageWords + 8 * tt + 4 * i + 2 * pr;   // word index in the row
        uint4 x = make_uint4(0, 0, 0, 0);
        if (wx < W) x = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2)) + (wx >> 1));
        uint32_t q[4][2];
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
#pragma unroll
          for (int w = 0; w < 2; w++) {
            const uint32_t lo32 = w ? x.z : x.x, hi32 = w ? x.w : x.y;   // codes 0..7 and 8..15 of the word
            const uint32_t a = (lo32 >> (4 * pp)) & 0x000F000Fu;
            const uint32_t c = (hi32 >> (4 * pp)) & 0x000F000Fu;
            uint32_t v = __byte_perm(a, c, 0x6420);        // nibbles of codes p, 4+p, 8+p, 12+p
            v |= (v & 0x08080808u) * 0x1Eu;                 // sign-extend each nibble to a byte
            tsum = __dp4a((int)v, 0x01010101, tsum);
            if ((pp & 1) == 0) v = (v << 2) & 0xFCFCFCFCu;  // even positions carry 4 q
            q[pp][w] = v;
          }
        }
        uint8_t* dst = bs + ((size_t)((((st * 2 + i) * 2 + pr) * 2) * ncol + col)) * 64 + tt * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(q[0][0], q[0][1], q[1][0], q[1][1]);
        *reinterpret_cast<uint4*>(dst + (size_t)ncol * 64) = make_uint4(q[2][0], q[2][1], q[3][0], q[3][1]);
      }
#pragma unroll
      for (int d = 8; d > 0; d >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, d);
      if ((lane & 15) == 0 && u < total) s_T0st[col * kMaxSps + st] = tsum;
    }
    if (tid < M) s_scale[tid] = __half2float(p.scale[tid]);
  }
  __syncthreads();

  // ------------------------------------------------------------------ producer main loop
  if (warp == kCWarps) {
    if (lane == 0) {
      while (pr_seg < work.nseg) {
        // the slot was filled one ring turn ago: wait until every consumer warp has released it
        if (!mbar_wait(empty0 + 8 * pr_slot, pr_phase ^ 1u)) { atomicExch(p.ws_status, 2); break; }
        produce();
      }
    }
    return;
  }

  // ------------------------------------------------------------------ finishing warp
  // For every partial segment, once all consumer warps have added their sums to the scratch:
  // fence, count the contribution, and if it completes the tile, finish its 256 rows.
  if (warp == kCWarps + 1) {
    int pk = 0;
    for (int si = 0; si < work.nseg; si++) {
      const Segment sg = work.get(si);
      if (is_whole(sg)) continue;
      const int ps = pk & (kPartRing - 1);
      if (!mbar_wait(part0 + 8 * ps, (uint32_t)(pk / kPartRing) & 1u)) {
        if (lane == 0) atomicExch(p.ws_status, 4);
        return;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(done0 + 8 * ps);   // the ring slot may be used again
      pk++;
      if (!one_range && lane < M) {
        int a = 0;
        for (int st = sg.sb; st < sg.se; st++) a += s_T0st[lane * kMaxSps + st];
        atomicAdd(p.ws_T0 + (size_t)sg.tile * M + lane, a);
      }
      __threadfence();
      __syncwarp();
      uint32_t old = 0;
      if (lane == 0) old = atomicAdd(p.ws_count + sg.tile, (uint32_t)(sg.se - sg.sb));
      old = __shfl_sync(0xffffffffu, old, 0);
      if (old + (uint32_t)(sg.se - sg.sb) != (uint32_t)p.spt_all) continue;
      __threadfence();
      const int nout = kTileRows * M;
      for (int idx = lane; idx < nout; idx += 32) {
        const int r = idx / M, m = idx - r * M;
        const int row = sg.tile * kTileRows + r;
        if (row < p.N) {
          int32_t* src = p.ws_sum + ((size_t)row * M + m) * 3;
          const int T1 = __ldcg(src + 0), T2 = __ldcg(src + 1), T3 = __ldcg(src + 2);
          src[0] = 0; src[1] = 0; src[2] = 0;
          int T0;
          if (one_range) {
            T0 = 0;
            for (int st = 0; st < spt; st++) T0 += s_T0st[m * kMaxSps + st];
          } else {
            T0 = __ldcg(p.ws_T0 + (size_t)sg.tile * M + m);
          }
          const int S3 = T3, S1 = T1 - T3, S2 = T2 - T3;
          const int S0 = T0 - S1 - S2 - S3;
          p.y[(size_t)m * p.N + row] = lut_finish(s_scale[m], __ldg(p.lut + row), S0, S1, S2, S3);
        }
      }
      __syncwarp();
      if (!one_range && lane < M) p.ws_T0[(size_t)sg.tile * M + lane] = 0;
      if (lane == 0) p.ws_count[sg.tile] = 0u;
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  constexpr int NF_M = (MODE == kModeDp4a) ? 0 : (MODE == kModeHybrid ? 2 : 3);  // planes on the MMA
  constexpr int NF_D = (MODE == kModeDp4a) ? 3 : (MODE == kModeHybrid ? 1 : 0);  // planes on dp4a
  constexpr int NTD = (NF_D == 0) ? 1 : MTOK;
  int accM[MT][NF_M == 0 ? 1 : NF_M][2][4];
  int accD[NTD][2][NF_D == 0 ? 1 : NF_D][2];
  auto zero_acc = [&]() {
#pragma unroll
    for (int a = 0; a < MT; a++)
#pragma unroll
      for (int f = 0; f < (NF_M == 0 ? 1 : NF_M); f++)
#pragma unroll
        for (int h = 0; h < 2; h++)
#pragma unroll
          for (int r = 0; r < 4; r++) accM[a][f][h][r] = 0;
#pragma unroll
    for (int a = 0; a < NTD; a++)
#pragma unroll
      for (int r = 0; r < 2; r++)
#pragma unroll
        for (int f = 0; f < (NF_D == 0 ? 1 : NF_D); f++)
#pragma unroll
          for (int h = 0; h < 2; h++) accD[a][r][f][h] = 0;
  };
  zero_acc();

  // per-lane constant parts of the shared-memory addresses
  //   weights: rows g and g+8 of the warp's 16 rows; 16-byte chunk (2t+i) ^ (row & 7) under the 128B swizzle
  const uint32_t a_row = base + (uint32_t)((warp * 16 + g) * 128);
  uint32_t a_chunk[2];
#pragma unroll
  for (int i = 0; i < 2; i++) a_chunk[i] = (uint32_t)(((2 * t + i) ^ g) << 4);
  const uint32_t bs_u32 = smem_u32(bs);
  const uint32_t half_stride = (uint32_t)ncol * 64;
  const uint32_t stage_stride = 8 * half_stride;   // 2 (i) x 2 (pr) x 2 (half) per stage
  uint32_t bM_lane[MT], bD_lane[NTD];
#pragma unroll
  for (int mt = 0; mt < MT; mt++) {
    int col = 8 * mt + g;
    if constexpr (MTOK > 0) col = g % MTOK;
    else if (col >= M) col = M - 1;
    bM_lane[mt] = bs_u32 + (uint32_t)(col * 64 + t * 16);
  }
#pragma unroll
  for (int tok = 0; tok < NTD; tok++) bD_lane[tok] = bs_u32 + (uint32_t)(tok * 64 + t * 16);

  int part_k = 0;  // partial segments handed over so far
  uint2 lut_g[2];  // LUT rows g and g+8 of the current tile, fetched ahead of the epilogue
  auto fetch_lut = [&](int tile) {
#pragma unroll
    for (int rr = 0; rr < 2; rr++) {
      const int row = tile * kTileRows + warp * 16 + g + 8 * rr;
      lut_g[rr] = row < p.N ? __ldg(p.lut + row) : make_uint2(0, 0);
    }
  };

  // finishes this warp's 16 rows of a segment
  auto flush = [&](const Segment& sg) {
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
          T1[e] = (accM[mt][0][0][r] >> 2) + (accM[mt][0][1][r] >> 6);
          T2[e] = (accM[mt][1][0][r] >> 3) + (accM[mt][1][1][r] >> 7);
          T3[e] = (accM[mt][2][0][r] >> 3) + (accM[mt][2][1][r] >> 7);
        }
    } else {
#pragma unroll
      for (int tok = 0; tok < NTD; tok++)
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const int e = tok * 2 + rr;
          etok[e] = (t == 0) ? tok : kMaxTokens;  // only lane t==0 of a quad emits
          err[e] = rr;
          int a1, a2, a3;
          if constexpr (MODE == kModeHybrid) {
            const int r = tok + 2 * rr;  // MMA column c carries token c % MTOK; lane t==0 holds columns 0, 1
            a1 = (accM[0][0][0][r] >> 2) + (accM[0][0][1][r] >> 6);
            a2 = (accM[0][1][0][r] >> 3) + (accM[0][1][1][r] >> 7);
            a3 = (accD[tok][rr][0][0] >> 3) + (accD[tok][rr][0][1] >> 7);
          } else {
            a1 = (accD[tok][rr][0][0] >> 2) + (accD[tok][rr][0][1] >> 6);
            a2 = (accD[tok][rr][1][0] >> 3) + (accD[tok][rr][1][1] >> 7);
            a3 = (accD[tok][rr][2][0] >> 3) + (accD[tok][rr][2][1] >> 7);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            a2 += __shfl_xor_sync(0xffffffffu, a2, 1); a2 += __shfl_xor_sync(0xffffffffu, a2, 2);
          }
          a3 += __shfl_xor_sync(0xffffffffu, a3, 1); a3 += __shfl_xor_sync(0xffffffffu, a3, 2);
          T1[e] = a1; T2[e] = a2; T3[e] = a3;
        }
    }
    const int row0 = sg.tile * kTileRows + warp * 16 + g;
    if (is_whole(sg)) {
#pragma unroll
      for (int e = 0; e < NE; e++) {
        const int row = row0 + 8 * err[e];
        if (etok[e] < M && row < p.N) {
          int T0 = 0;
          for (int st = 0; st < spt; st++) T0 += s_T0st[etok[e] * kMaxSps + st];
          const int S3 = T3[e], S1 = T1[e] - T3[e], S2 = T2[e] - T3[e];
          const int S0 = T0 - S1 - S2 - S3;
          p.y[(size_t)etok[e] * p.N + row] = lut_finish(s_scale[etok[e]], lut_g[err[e]], S0, S1, S2, S3);
        }
      }
    } else {
      // partial rows: add into the scratch sums and hand the segment to the finishing warp
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
      const int ps = part_k & (kPartRing - 1);
      bool ok = true;
      if (part_k >= kPartRing) ok = mbar_wait(done0 + 8 * ps, (uint32_t)(part_k / kPartRing - 1) & 1u);
      __syncwarp();
      if (lane == 0) {
        if (ok) mbar_arrive(part0 + 8 * ps);
        else atomicExch(p.ws_status, 5);
      }
      part_k++;
    }
    zero_acc();
  };

  int slot = 0;
  uint32_t phase = 0;
  for (int si = 0; si < work.nseg; si++) {
    const Segment sg = work.get(si);
    if (is_whole(sg)) fetch_lut(sg.tile);
    uint32_t b_stage = (uint32_t)sg.sb * stage_stride;
    for (int st = sg.sb; st < sg.se; st++, b_stage += stage_stride) {
      if (!mbar_wait(full0 + 8 * slot, phase)) {
        if (lane == 0) atomicExch(p.ws_status, 3);
        return;
      }
      const uint32_t a_stage = a_row + (uint32_t)slot * kStageBytes;
#pragma unroll
      for (int i = 0; i < 2; i++) {
        const uint4 U = lds128(a_stage + a_chunk[i]);
        const uint4 V = lds128(a_stage + 8 * 128 + a_chunk[i]);
        const uint32_t uw[4] = {U.x, U.y, U.z, U.w};
        const uint32_t vw[4] = {V.x, V.y, V.z, V.w};
#pragma unroll
        for (int pr = 0; pr < 2; pr++) {
          const uint32_t b_off = b_stage + (uint32_t)((i * 2 + pr) * 2) * half_stride;
          // activation operands of the word pair: [position p][word]
          uint32_t bM[MT][4][2];
          uint32_t bD[NTD][4][2];
          if constexpr (NF_D > 0) {
#pragma unroll
            for (int tok = 0; tok < NTD; tok++) {
              const uint4 x = lds128(bD_lane[tok] + b_off);
              const uint4 y = lds128(bD_lane[tok] + b_off + half_stride);
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
                const uint4 x = lds128(bM_lane[mt] + b_off);
                const uint4 y = lds128(bM_lane[mt] + b_off + half_stride);
                bM[mt][0][0] = x.x; bM[mt][0][1] = x.y; bM[mt][1][0] = x.z; bM[mt][1][1] = x.w;
                bM[mt][2][0] = y.x; bM[mt][2][1] = y.y; bM[mt][3][0] = y.z; bM[mt][3][1] = y.w;
              }
            }
          }
          const uint32_t u0 = uw[2 * pr], u1 = uw[2 * pr + 1], v0 = vw[2 * pr], v1 = vw[2 * pr + 1];
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
                mma_u8s8(accM[mt][f][pp >> 1], au0[f], av0[f], au1[f], av1[f], bM[mt][pp][0], bM[mt][pp][1]);
#pragma unroll
            for (int f = 0; f < NF_D; f++) {
              const int fa = 3 - NF_D + f;  // hybrid: plane 2 only; dp4a: planes 0..2
#pragma unroll
              for (int tok = 0; tok < NTD; tok++) {
                dp4a_u8s8(accD[tok][0][f][pp >> 1], au0[fa], bD[tok][pp][0]);
                dp4a_u8s8(accD[tok][1][f][pp >> 1], av0[fa], bD[tok][pp][0]);
                dp4a_u8s8(accD[tok][0][f][pp >> 1], au1[fa], bD[tok][pp][1]);
                dp4a_u8s8(accD[tok][1][f][pp >> 1], av1[fa], bD[tok][pp][1]);
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * slot);   // this warp is done with the slot
      if (++slot == stages) { slot = 0; phase ^= 1u; }
    }
    flush(sg);
  }
}

}  // namespace rcp
