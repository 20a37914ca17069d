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
// producer thread streams boxes of rows x 128 bytes into a shared-memory ring with TMA
// (cp.async.bulk.tensor, 128B swizzle, mbarrier completion); sixteen consumer warps read their MMA
// fragments bank-conflict free and keep the partial sums in registers.
//   Groups of 16 rows are the unit of work, and the work is cut into phases. In a phase every
//   CTA takes gpc consecutive groups (gpc = 16, 8, 4, 2 or 1) and KS = 16 / gpc warps share a
//   group, each taking every KS-th 128-byte chunk of K; a stage of the ring is KS boxes of
//   16 gpc rows x 128 bytes (32 KB). With gpc = 16 (as many rounds as the row count allows, tiles
//   dealt round-robin so that the GPU sweeps memory in order) a warp owns its group over the whole
//   K and finishes its rows from its registers. The groups left over go in phases of 8, 4, 2, 1
//   groups per CTA, so that all sixteen warps stay busy; there the sums of the KS warps of a group
//   meet in shared memory (integer atomics) and one of them finishes the rows.
// Group-wise grid (GRP; the grid of Section 4.4 has one four-entry row per group of 128 weights):
//   the integer sums live for one group only. A 128-byte chunk of a row is four groups. On the
//   CUDA-core path lane t of a quad already holds exactly group t of the chunk, so after every
//   chunk each lane turns its own sums into one fp32 term with its group's grid. On the tensor
//   cores an MMA adds up the k of all four lanes of a quad, so there the quad reads one group at a
//   time (8 bytes per lane instead of 16, rows dealt to the lanes so that the reads stay free of
//   bank conflicts) and finishes it after twelve MMAs. The fp32 terms add up in a fixed order.
// Nothing is exchanged between CTAs, no scratch memory is needed, and the result does not depend
// on timing. The int4 activations are expanded once per CTA into the B-operand byte layout in
// shared memory.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "quantize_act.cuh"
#include "split_act16.cuh"

// Guarded build (-DRCP_CHECKED): compute-sanitizer's stand-in. Every shared-memory address the streaming kernel
// forms for the weight ring, the expanded activations, the reduction buffers and the parked sums, and every TMA
// request, is checked against the area the host laid out; a violation skips the access and leaves 16 + the
// number of the site in the status word (the largest such code wins) instead of faulting. The production build
// compiles none of it.
#ifdef RCP_CHECKED
#define RCP_CK(cond, site) ((cond) ? true : (ck_fail(site), false))
#define RCP_LDS128(addr, lo, hi, site) \
  ([&]() -> uint4 { const uint32_t a__ = (addr); \
     if (!RCP_CK(a__ >= (lo) && a__ + 16u <= (hi) && (a__ & 15u) == 0, site)) return make_uint4(0, 0, 0, 0); \
     return lds128(a__); }())
#define RCP_LDS64(addr, lo, hi, site) \
  ([&]() -> uint2 { const uint32_t a__ = (addr); \
     if (!RCP_CK(a__ >= (lo) && a__ + 8u <= (hi) && (a__ & 7u) == 0, site)) return make_uint2(0, 0); \
     return lds64(a__); }())
#else
#define RCP_CK(cond, site) (true)
#define RCP_LDS128(addr, lo, hi, site) lds128(addr)
#define RCP_LDS64(addr, lo, hi, site) lds64(addr)
#endif

namespace rcp {

constexpr int kCWarps = 16;                       // consumer warps
constexpr int kGThreads = (kCWarps + 1) * 32;     // + one producer warp
constexpr int kTileRows = 16 * kCWarps;           // rows of a round's TMA box
constexpr int kChunkWords = 32;                   // 128 bytes of K per row per box (512 codes)
constexpr int kGroupBytes = 16 * kChunkWords * 4; // one group's rows in a box: 2 KB
constexpr int kStageBytes = kTileRows * kChunkWords * 4;
constexpr int kMaxStages = 8;
constexpr int kExpWarps = 4;                      // SB: warps that expand the activations of the stages (one per scheduler)
constexpr uint32_t kSpinLimit = 1u << 22;         // bounded waits: give up, flag the error and exit

enum GemvMode { kModeMma = 0, kModeHybrid = 1, kModeDp4a = 2 };

constexpr int kMaxPhases = 6;
// One phase, repeated reps times: `total` groups starting at group first + rep * total are shared out
// evenly over the CTAs b < ncta: with q = total / ncta and r = total % ncta the first r CTAs take q + 1
// consecutive groups, the others q (at most gpc). KS = 16 / gpc warps share a group; the TMA box has
// 16 gpc rows. The host works out everything that would need a division in the kernel.
struct GemvPhase {
  int gpc, first, total, ncta, reps;
  int q, r;        // total / ncta, total % ncta
  int ks, inv_ks;  // KS, and ceil(256 / KS): warp / KS == (warp * inv_ks) >> 8 for warp < 16
  int sa;          // stages per repetition: ceil(nchunk / KS)
};
struct GemvMaps { CUtensorMap m[kMaxPhases]; };   // box of 16 gpc rows x 128 bytes for phase i

struct GemvParams {
  const uint2* lut;
  const uint8_t* xq;
  const __half* scale;
  const float* unit;     // A16: fp32 unit of each digit column (scale unused)
  float* unit_out;       // A16 with x set (one token): every CTA makes the digit planes itself (kept in shared
                         // memory at off_qbuf); CTA 0 also stores them to xq_out ([4][K] bytes) and the units here
  __half* y;
  int32_t* status;      // optional: receives a code when a bounded wait gives up
  int32_t* S_out;       // SDBG instantiations only: the exact per-code sums, [M][N][4] (group-wise: [M][N][ngrp][4];
                        // digit columns: one "token" per column)
  int M, N, K;
  int ngrp;             // group-wise grid: groups of 128 weights per row (K / 128), lut is [N][ngrp]; else 0
  int nchunk;           // 128-byte chunks per row, ceil(K / 512); with nsplit > 1: per part of K
  int nchunk_total;     // chunks per row over the whole K
  int nsplit;           // parts of K gone through one after the other (tensor-core kernels of the per-row grid; else 1)
  int off_part;         // nsplit > 1: partial sums of this CTA's rows between the parts
  int inv_nchunk;       // ceil(2^20 / nchunk): x / nchunk == (x * inv_nchunk) >> 20 for x < 2^20 / nchunk
  int nphase;
  GemvPhase phase[kMaxPhases];
  // fused activation quantizer (FQ): x fp16 [M][K] replaces xq and scale as input
  const __half* x;
  uint8_t* xq_out;      // optional [M][K/2]: the int4 activations, written by CTA 0
  __half* scale_out;    // optional [M]
  float inv_sqrt_b, clip_ratio;   // the rotation block is the whole token, K = 4096 or 8192
  int off_qbuf;         // the quantizer's scratch (rotate_scratch_bytes(K)) in shared memory
  int stages;           // ring depth
  int ramp_clk;         // clocks between the first `stages` requests of a CTA
  int off_bar, off_T0c, off_scale, off_red, off_bs;   // shared-memory byte offsets from the aligned base
  int bs_bytes, red_bytes, part_bytes;                // sizes of the areas at off_bs, off_red, off_part (guarded build)
  int stage_stride;     // bytes from one ring stage to the next: kStageBytes, plus the stage's activation area (SB)
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
// Bounded wait. Returns false after `limit` polls.
__device__ __forceinline__ bool mbar_wait_n(uint32_t bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; i++) {
    if (mbar_try(bar, parity)) return true;
    __nanosleep(64);   // leave the issue slots to the warps that have work
  }
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) { return mbar_wait_n(bar, parity, kSpinLimit); }
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
// the same with the A operand read as signed bytes
__device__ __forceinline__ void mma_s8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same with a zero accumulator coming in
__device__ __forceinline__ void mma_u8s8_zero(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
// int -> float for |x| < 2^22 with one integer add and one float add (no conversion unit)
__device__ __forceinline__ float small_int_to_float(int x) {
  return __int_as_float(x + 0x4B400000) - 12582912.0f;   // 1.5 * 2^23 + x, exactly
}
// a & b & c as one three-input logic operation (written out: the compiler would otherwise keep a & b as a
// common subexpression of the four positions and spend a fifth operation per word)
__device__ __forceinline__ uint32_t and3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ void dp4a_u8s8(int& d, uint32_t a, uint32_t b) {
  asm("dp4a.u32.s32 %0, %1, %2, %0;" : "+r"(d) : "r"(a), "r"(b));
}
__device__ __forceinline__ void dp4a_s8s8(int& d, uint32_t a, uint32_t b) {
  asm("dp4a.s32.s32 %0, %1, %2, %0;" : "+r"(d) : "r"(a), "r"(b));
}

// Self-test of the bounded wait and its report (a test aid, not part of the data path): one thread waits, with
// the routine the GEMV kernels wait with and a limit of the caller's choice, on a barrier that nobody ever
// arrives at. The wait gives up, the status word receives the consumer-side code, the kernel returns.
__global__ void wait_timeout_kernel(int32_t* status, uint32_t polls) {
  __shared__ __align__(8) unsigned long long bar_mem;
  if (threadIdx.x == 0) {
    const uint32_t bar = smem_u32(&bar_mem);
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_n(bar, 0, polls)) atomicExch(status, 3);
  }
}

// Expanded activations. A chunk is 32 words of a row; consumer lane t reads 16-byte chunk 2t+i of
// the row in sub-step i, i.e. words 8t+4i .. 8t+4i+3, as two word pairs pr. For every
// (chunk, i, pr) and token column there are two 16-byte halves per lane slice t; half h holds
// positions 2h and 2h+1:
//   { q[p=2h][word x], q[2h][word y], q[2h+1][word x], q[2h+1][word y] },  byte j of q[p][w] =
//   activation of code 16 w + 4 j + p, times 4 when p is even.
// Byte address of (chunk, i, pr, half, col, t): ((((chunk*2 + i)*2 + pr)*2 + half)*ncol + col)*64 + t*16.

// MODE  kModeMma: all three planes on the tensor cores; kModeHybrid: b0 and b1 planes on the tensor
//       cores, the b0*b1 plane on dp4a; kModeDp4a: everything on dp4a (CUDA cores only)
// MTOK  tokens, fixed at compile time for the dp4a modes (1 or 2); kModeMma: 0 = run-time, up to 8; 8 = exactly eight
//       (one MMA column tile), 16 = run-time, 9 to 16 (two column tiles fed from the same masks)
// GRP   one grid per group of 128 weights instead of one per row (kModeHybrid has no such form)
// FQ    one token of 4096 or 8192 activations under one rotation block: the activations arrive as
//       fp16 and every CTA rotates and quantizes them itself (Appendix A.2, Section 4.4), in the
//       arithmetic order of the stand-alone quantizer: bit-identical int4 values. For these shapes
//       (where the stand-alone kernel needs a cluster and passes through distributed shared memory)
//       it costs less than a kernel of its own. A thread takes one word (16 consecutive activations):
//       strides 1..8 in registers, 16..256 by lane exchanges, 512 and up through shared memory, one
//       thread per (lane, element) column over the warps.
// A16   weight-only form: the "tokens" are the four base-64 fixed-point digits of up to two (MTOK 16: four)
//       fp16 tokens, one signed byte per element (p.xq is [4 tokens][K] bytes, p.unit their fp32 units, p.M
//       the number of digit columns); the digits of a token are combined in fp32 when its rows are finished.
// SPLIT K in parts (see below): the eight-column tensor-core kernels of the per-row grid, when asked to.
// SDBG  checked instantiation: the same kernel also stores the integer sums S_0..S_3 it finishes its rows
//       from (p.S_out), so that a test can compare them with a reference bit for bit. The production
//       instantiations (SDBG false) contain none of this.
// SB    activations streamed with the weights (tensor-core kernels of the per-row grid): nothing is expanded up
//       front. Every ring stage carries, behind its boxes of weights, the expanded activations of the chunks
//       those boxes cover (tokens x 512 bytes per chunk), written by one more warp that runs ahead of the
//       consumers like the producer does. The token count and K then no longer meet in shared memory: no K in
//       parts, up to sixteen tokens for any K, and the expansion (2 us at eight tokens of 8192) leaves the
//       critical path. The host keeps (warps sharing a group) x tokens at 32 or less per stage.
template <int MODE, int MTOK, bool GRP, bool FQ = false, bool A16 = false, bool SPLIT = false, bool SDBG = false,
          bool SB = false>
__global__ void __launch_bounds__(SB ? kGThreads + 32 * kExpWarps : kGThreads, 1)
gemv_stream_kernel(const __grid_constant__ GemvMaps maps, const GemvParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;           // TMA 128B swizzle wants 1024-byte alignment
  uint8_t* const gen = smem_raw + (base - raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int M = (MTOK > 0 && MTOK != 16) ? MTOK : p.M;   // (kModeMma with MTOK 8: exactly eight tokens, known at compile time)
  constexpr bool kTwoTiles = (MODE == kModeMma && MTOK == 16);   // tokens 8..15 in a second set of accumulators
  static_assert(!(kTwoTiles && (GRP || FQ)), "two column tiles: per-row grid, quantized activations only");
  static_assert(!A16 || (MODE == kModeMma && !GRP && !FQ), "digit columns: tensor-core mode, per-row grid");
  // Long K with several tokens: the expanded activations of the whole K do not fit in shared memory. The kernel
  // then goes through K in nsplit parts: activations of the part expanded, every phase run over the part's
  // chunks, the integer sums of this CTA's rows parked in shared memory until the last part finishes them. The
  // plan is the same for every part, so the same lane meets the same sums again: nothing crosses warps.
  // A form of its own, so that the kernels that never need it keep their code.
  constexpr bool kSplit = SPLIT;
  static_assert(!SPLIT || (MODE == kModeMma && MTOK == 0 && !GRP && !FQ), "K in parts: eight-column tensor-core kernels, per-row grid");
  static_assert(!SB || (MODE == kModeMma && !FQ && !A16 && !SPLIT), "streamed activations: tensor-core kernels");
  constexpr int kThreads = SB ? kGThreads + 32 * kExpWarps : kGThreads;   // consumers, producer warp, and the expander warps (SB)
  const uint32_t stage_stride = SB ? (uint32_t)p.stage_stride : (uint32_t)kStageBytes;
  const int nsplit = kSplit ? p.nsplit : 1;
  const int ncol = M;
  const int stages = p.stages;
  const uint32_t full0 = base + p.off_bar, empty0 = full0 + 8 * kMaxStages;
  static_assert(!(GRP && MODE == kModeHybrid), "no group-wise hybrid mode");
  constexpr bool kRelabel = GRP && MODE == kModeMma;   // a quad shares a group: lane t takes words 8j+2t, 8j+2t+1
  int* const s_T0c = reinterpret_cast<int*>(gen + p.off_T0c);           // [M][nchunk]: sum of q per chunk; GRP: [M][4 nchunk] per group
  float* const s_scale = reinterpret_cast<float*>(gen + p.off_scale);   // [16]
  int* const s_red = reinterpret_cast<int*>(gen + p.off_red);           // [2][8 groups][16 rows][M][3]
  float* const s_redf = reinterpret_cast<float*>(gen + p.off_red);      // GRP: [2][16 warps][16 rows][M]
  // tensor-core GRP: the same area as floats [4 nchunk][Mp], 8 x the sum of q of a group, tokens padded to even
  float* const s_T0f = reinterpret_cast<float*>(gen + p.off_T0c);
  const int ng4 = 4 * p.nchunk;
  const int Mp = (M + 1) & ~1;
  uint8_t* const bs = gen + p.off_bs;
#ifdef RCP_CHECKED
  auto ck_fail = [&](int site) { if (p.status) atomicMax(p.status, 16 + site); };
#endif
  // areas of the layout (used by the guarded build's checks only)
  const uint32_t ring_lo = base, ring_hi = base + (uint32_t)stages * stage_stride;
  const uint32_t bs_lo = SB ? ring_lo : base + (uint32_t)p.off_bs, bs_hi = SB ? ring_hi : bs_lo + (uint32_t)p.bs_bytes;
  (void)ring_lo; (void)ring_hi; (void)bs_lo; (void)bs_hi;

  const int b = blockIdx.x;
  // Launched with programmatic stream serialization: the next kernel may start as CTAs retire.
  asm volatile("griddepcontrol.launch_dependents;");
  int* const s_T0tot = reinterpret_cast<int*>(s_scale + 32);   // [16]: sum of q per token, behind scales and maxima
  // The producer warp sets up the ring's barriers and only announces that (bar.arrive): its first
  // requests go out without waiting for anybody. The consumer warps wait for the announcement.
  if (warp != kCWarps) {
    if (tid < kMaxTokens) s_T0tot[tid] = 0;
    asm volatile("bar.sync 3, %0;" ::"n"(kThreads) : "memory");
  }

  // ------------------------------------------------------------------ producer
  // One thread requests every stage of this CTA in order. The weights do not depend on the
  // preceding kernel, so it starts at once (before griddepcontrol.wait), and it never meets the
  // other warps again.
  if (warp == kCWarps) {
    if (lane == 0) {
      // a stage is full when its weights have landed (one arrival with the byte count) and, SB, the expander has arrived
      for (int s = 0; s < stages; s++) { mbar_init(full0 + 8 * s, SB ? 1 + kExpWarps : 1); mbar_init(empty0 + 8 * s, kCWarps); }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("bar.arrive 3, %0;" ::"n"(kThreads) : "memory");
    if (lane != 0) return;
    int slot = 0;
    uint32_t phase = 0;
    int issued = 0;
    // The first ring-full of requests is spaced out by the time HBM needs to serve one stage for the
    // whole grid: issued all at once, the stages of all CTAs share the bandwidth and even the first
    // one lands only when nearly all of them have.
    const long long t_start = clock64();
    for (int kp = 0; kp < nsplit; kp++) {
    const int chunk0 = kSplit ? kp * p.nchunk : 0;                                    // this part of K
    const int nch = kSplit ? min(p.nchunk, p.nchunk_total - chunk0) : p.nchunk;
    for (int pi = 0; pi < p.nphase; pi++) {
      const GemvPhase ph = p.phase[pi];
      if (b >= ph.ncta) continue;
      if (kp == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.m[pi]) : "memory");
      const int KS = ph.ks;
      const uint32_t box = (uint32_t)ph.gpc * kGroupBytes;
      const int lo = ph.q * b + min(b, ph.r);
      const int SA = ph.sa;
      for (int rp = 0; rp < ph.reps; rp++) {
        const int row0 = (ph.first + rp * ph.total + lo) * 16;
        for (int s = 0; s < SA; s++) {
          // a slot filled one ring turn ago must have been released by every consumer warp
          if (issued >= stages) {
            if (!mbar_wait(empty0 + 8 * slot, phase ^ 1u)) {
              if (p.status) atomicExch(p.status, 2);
              return;
            }
          } else {
            const long long due = t_start + (long long)issued * p.ramp_clk;
            while (clock64() < due) { }
          }
          const uint32_t bar = full0 + 8 * slot, dst = base + (uint32_t)slot * stage_stride;
          const int nbox = kSplit ? max(0, min(KS, nch - s * KS)) : min(KS, nch - s * KS);   // a short last part can leave a stage empty
          mbar_expect_tx(bar, (uint32_t)nbox * box);
          for (int j = 0; j < nbox; j++) {
            const int xw = (chunk0 + s * KS + j) * kChunkWords;   // first word of the box: a multiple of 32, so 16-byte aligned
            if (RCP_CK(dst + (uint32_t)(j + 1) * box <= ring_hi && ((dst + (uint32_t)j * box) & 1023u) == 0 && xw >= 0 &&
                       xw < p.K / 16 && (xw & 3) == 0 && row0 >= 0 && row0 < p.N && pi < kMaxPhases, 1))
              tma_load_2d(dst + (uint32_t)j * box, &maps.m[pi], xw, row0, bar);
          }
          issued++;
          if (++slot == stages) { slot = 0; phase ^= 1u; }
        }
      }
    }
    }
    return;
  }

  // ------------------------------------------------------------------ expander (SB)
  // One warp walks the same sequence of stages as the producer and fills each stage's activation area:
  // for every box of the stage (a chunk of K) and every token, the chunk's 512 int4 activations as int8 in the
  // B-fragment order the consumers read. It waits for a slot to be released like the producer does.
  if constexpr (SB) {
    if (warp > kCWarps) {
      const int ew = warp - (kCWarps + 1);   // which of the expander warps
      asm volatile("griddepcontrol.wait;" ::: "memory");   // xq may belong to the kernel before this one
      int slot = 0;
      uint32_t phase = 0;
      int issued = 0;
      const int W = p.K / 16;
      for (int pi = 0; pi < p.nphase; pi++) {
        const GemvPhase ph = p.phase[pi];
        if (b >= ph.ncta) continue;
        const int KS = ph.ks, SA = ph.sa;
        for (int rp = 0; rp < ph.reps; rp++) {
          for (int s = 0; s < SA; s++) {
            // The stage's work is (boxes x tokens x 16) units of two words, dealt to the lanes four at a time.
            // The packed activations of a batch are fetched (global memory, L2) before the wait for the slot and
            // before the previous batch is stored: the latency stays off the path.
            const int nbox = min(KS, p.nchunk - s * KS);
            const int per_box = M * 16, total = nbox * per_box;
            const uint32_t inv_box = ((1u << 20) + per_box - 1) / per_box;   // v / per_box == (v * inv_box) >> 20 for v < 512
            constexpr int kLaneStep = 32 * kExpWarps;
            auto fetch = [&](int v0, uint4 (&x)[4]) {
#pragma unroll
              for (int r = 0; r < 4; r++) {
                const int v = v0 + kLaneStep * r;
                x[r] = make_uint4(0, 0, 0, 0);
                if (v < total) {
                  const int j = (int)(((uint32_t)v * inv_box) >> 20), w = v - j * per_box;
                  const int col = w >> 4, lo = w & 3, hi = (w >> 2) & 3;
                  const int wx = (s * KS + j) * kChunkWords + (kRelabel ? 8 * hi + 2 * lo : 8 * lo + 2 * hi);   // first of the unit's two words
                  if (wx < W) x[r] = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2)) + (wx >> 1));
                }
              }
            };
            uint4 xa[4];
            fetch(ew * 32 + lane, xa);
            if (issued >= stages) {
              if (!mbar_wait(empty0 + 8 * slot, phase ^ 1u)) {
                if (lane == 0 && p.status) atomicExch(p.status, 4);
                return;
              }
            }
            uint8_t* const sb = gen + (size_t)slot * stage_stride + kStageBytes;
            for (int v0 = ew * 32 + lane; v0 < total; v0 += 4 * kLaneStep) {
              uint4 xn[4];
              if (v0 + 4 * kLaneStep < total) fetch(v0 + 4 * kLaneStep, xn);
#pragma unroll
              for (int r = 0; r < 4; r++) {
                const int v = v0 + kLaneStep * r;
                if (v < total) {
                  const int j = (int)(((uint32_t)v * inv_box) >> 20), w = v - j * per_box;
                  const int col = w >> 4, lo = w & 3, hi = (w >> 2) & 3;
                  const uint4 x = xa[r];
                  uint32_t q[4][2];
#pragma unroll
                  for (int ww = 0; ww < 2; ww++) {
                    const uint32_t lo32 = ww ? x.z : x.x, hi32 = ww ? x.w : x.y;
                    uint32_t n4[4] = {lo32 & 0x0F0F0F0Fu, (lo32 >> 4) & 0x0F0F0F0Fu, hi32 & 0x0F0F0F0Fu, (hi32 >> 4) & 0x0F0F0F0Fu};
#pragma unroll
                    for (int h = 0; h < 4; h++) n4[h] |= (n4[h] & 0x08080808u) * 0x1Eu;   // sign-extend the nibbles
                    const uint32_t e0 = __byte_perm(n4[0], n4[2], 0x6420), e2 = __byte_perm(n4[0], n4[2], 0x7531);
                    q[0][ww] = (e0 << 2) & 0xFCFCFCFCu;
                    q[1][ww] = __byte_perm(n4[1], n4[3], 0x6420);
                    q[2][ww] = (e2 << 2) & 0xFCFCFCFCu;
                    q[3][ww] = __byte_perm(n4[1], n4[3], 0x7531);
                  }
                  uint8_t* dst = sb + ((size_t)(((j * 4 + hi) * 2) * ncol + col)) * 64 + lo * 16;
                  if (RCP_CK(dst >= gen && dst + (size_t)ncol * 64 + 16 <= gen + (size_t)(slot + 1) * stage_stride, 13)) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(q[0][0], q[0][1], q[1][0], q[1][1]);
                    *reinterpret_cast<uint4*>(dst + (size_t)ncol * 64) = make_uint4(q[2][0], q[2][1], q[3][0], q[3][1]);
                  }
                }
              }
#pragma unroll
              for (int r = 0; r < 4; r++) xa[r] = xn[r];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(full0 + 8 * slot);   // release: the stores above are visible to whoever sees the phase complete
            issued++;
            if (++slot == stages) { slot = 0; phase ^= 1u; }
          }
        }
      }
      return;
    }
  }

  // The packed weights and the LUT are constants of the layer; everything else (xq, scale, y) may
  // belong to the kernel before this one: wait for it.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ring position, barrier parity and reduction-buffer parity carried from one part of K to the next
  int slot_keep = 0, nred_keep = 0;
  uint32_t phase_keep = 0;
  int* const s_part = reinterpret_cast<int*>(gen + p.off_part);   // [group of this CTA][16 rows][M][3]
  for (int kp = 0; kp < nsplit; kp++) {
  const int chunk0 = kSplit ? kp * p.nchunk : 0;                                    // this part of K
  const int nch = kSplit ? min(p.nchunk, p.nchunk_total - chunk0) : p.nchunk;
  if (kp > 0) asm volatile("bar.sync 1, %0;" ::"n"(kCWarps * 32) : "memory");        // every warp is done with the last part's activations
  // ------------------------------------------------------------------ fused quantizer (consumer warps)
  if constexpr (FQ) {
    static_assert(!FQ || (MODE == kModeDp4a && MTOK == 1), "the fused quantizer serves the one-token kernels");
    constexpr int NT = kCWarps * 32;
    const int W = p.K / 16;                                           // 256 or 512 words: one per thread
    float* const qbuf = reinterpret_cast<float*>(gen + p.off_qbuf);   // rotate_scratch_bytes(K)
    float* const s_amax = s_scale + 16;                               // [16 warps] behind the scales
    float v[16];
    const float sc = rotate_token_words<NT>(p.x, W, p.inv_sqrt_b, p.clip_ratio, qbuf, s_amax, v);
    if (tid == 0) {
      s_scale[0] = sc;
      if (b == 0 && p.scale_out) p.scale_out[0] = __float2half_rn(sc);
    }
    int q[16];
    int tsum = 0;
    if (sc != 0.f) {   // the same for the whole CTA; threads beyond the token hold zeros
      quantize_int4<16>(v, sc, q);
    } else {
#pragma unroll
      for (int e = 0; e < 16; e++) q[e] = 0;
    }
#pragma unroll
    for (int e = 0; e < 16; e++) tsum += q[e];
    const int ch = tid >> 5, wi = tid & 31;
    if (tid < p.nchunk * kChunkWords) {
      uint32_t Q[4];
#pragma unroll
      for (int pp = 0; pp < 4; pp++) {
        const int m = (pp & 1) ? 1 : 4;   // even positions carry 4 q
        Q[pp] = (uint32_t)((q[pp] * m) & 0xFF) | ((uint32_t)((q[4 + pp] * m) & 0xFF) << 8) |
                ((uint32_t)((q[8 + pp] * m) & 0xFF) << 16) | ((uint32_t)((q[12 + pp] * m) & 0xFF) << 24);
      }
      uint8_t* dst = bs + (size_t)((ch * 4 + ((wi >> 1) & 3)) * 2) * 64 + (wi >> 3) * 16 + (wi & 1) * 4;
      if (RCP_CK(dst >= bs && dst + 64 + 12 <= bs + p.bs_bytes, 2)) {
        *reinterpret_cast<uint32_t*>(dst) = Q[0];
        *reinterpret_cast<uint32_t*>(dst + 8) = Q[1];
        *reinterpret_cast<uint32_t*>(dst + 64) = Q[2];
        *reinterpret_cast<uint32_t*>(dst + 64 + 8) = Q[3];
      }
    }
    if (b == 0 && p.xq_out && tid < W) {
      uint32_t lo32 = 0, hi32 = 0;
#pragma unroll
      for (int e = 0; e < 8; e++) {
        lo32 |= (uint32_t)(q[e] & 0xF) << (4 * e);
        hi32 |= (uint32_t)(q[8 + e] & 0xF) << (4 * e);
      }
      *reinterpret_cast<uint2*>(p.xq_out + (size_t)tid * 8) = make_uint2(lo32, hi32);
    }
    // sums of q: a warp holds exactly one chunk (32 consecutive words), eight lanes one group of 128
    tsum += __shfl_xor_sync(0xffffffffu, tsum, 1);
    tsum += __shfl_xor_sync(0xffffffffu, tsum, 2);
    tsum += __shfl_xor_sync(0xffffffffu, tsum, 4);
    if constexpr (GRP) {
      if ((lane & 7) == 0 && ch < p.nchunk) s_T0c[tid >> 3] = tsum;
    } else {
      tsum += __shfl_xor_sync(0xffffffffu, tsum, 8);
      tsum += __shfl_xor_sync(0xffffffffu, tsum, 16);
      if (lane == 0 && ch < p.nchunk) atomicAdd(&s_T0tot[0], tsum);
    }
    if constexpr (!GRP)
      for (int i = tid; i < 2 * 8 * 16 * M * 3; i += kCWarps * 32) s_red[i] = 0;
  } else if constexpr (SB && GRP) {
    // Streamed activations, group-wise grid: the sum of q of every (token, group of 128) is needed up front, as
    // 8 x the sum in fp32 (what the finish works with). A group is 64 bytes of packed activations.
    // (the last chunk may reach beyond K: its missing groups get a sum of zero, they meet a grid of zeros)
    const int ngroups = p.K / 128;
    for (int i = tid; i < M * ng4; i += kCWarps * 32) {
      const int col = i / ng4, gi = i - col * ng4;
      const uint4* src = reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2) + (size_t)gi * 64);
      int tsum = 0;
#pragma unroll
      for (int v4 = 0; v4 < 4; v4++) {
        const uint4 x = gi < ngroups ? __ldg(src + v4) : make_uint4(0, 0, 0, 0);
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int h = 0; h < 4; h++) {
          uint32_t e = xs[h] & 0x0F0F0F0Fu, o = (xs[h] >> 4) & 0x0F0F0F0Fu;
          e |= (e & 0x08080808u) * 0x1Eu;
          o |= (o & 0x08080808u) * 0x1Eu;
          tsum = __dp4a((int)e, 0x01010101, tsum);
          tsum = __dp4a((int)o, 0x01010101, tsum);
        }
      }
      s_T0f[gi * Mp + col] = (float)(8 * tsum);
    }
    if (tid < M) s_scale[tid] = __half2float(p.scale[tid]);
  } else if constexpr (SB) {
    // Streamed activations: only the sum of q per token is needed up front (S_0 = T0 - S_1 - S_2 - S_3).
    const int nvec = p.K / 32;   // 16-byte vectors of packed activations per token
    for (int col = 0; col < M; col++) {
      int tsum = 0;
      for (int i = tid; i < nvec; i += kCWarps * 32) {
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2)) + i);
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int h = 0; h < 4; h++) {
          uint32_t e = xs[h] & 0x0F0F0F0Fu, o = (xs[h] >> 4) & 0x0F0F0F0Fu;
          e |= (e & 0x08080808u) * 0x1Eu;
          o |= (o & 0x08080808u) * 0x1Eu;
          tsum = __dp4a((int)e, 0x01010101, tsum);
          tsum = __dp4a((int)o, 0x01010101, tsum);
        }
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, d);
      if (lane == 0) atomicAdd(&s_T0tot[col], tsum);
    }
    if (tid < M) s_scale[tid] = __half2float(p.scale[tid]);
    for (int i = tid; i < 2 * 8 * 16 * M * 3; i += kCWarps * 32) s_red[i] = 0;
  } else
  // ------------------------------------------------------------------ activations (consumer warps)
  // One unit = (column, chunk, i, pr, t) = two words. The 16 units of a (column, chunk) are 16
  // consecutive lanes: their sum of q is added to the token's total s_T0tot (per-row grid) or kept per group
  // of 128 in s_T0c (group-wise grid).
  {
    // Weight-only form with the activations still in fp16: the digit planes of this CTA's copy are made
    // here (the arithmetic of split_act16_kernel) and kept in shared memory.
    uint8_t* const stg = gen + p.off_qbuf;   // [column][K] signed bytes
    if constexpr (A16) {
      if (p.x) {
        // One token (the host asks for this form only then: with two, the stand-alone kernel in front was
        // measured faster), its values held in registers between the two passes (up to four vectors of eight
        // per thread: K <= 16384, which the host checks).
        unsigned* const s_am = reinterpret_cast<unsigned*>(s_red);   // [16 warps]; s_red is cleared further down
        const int nvec = p.K / 8;
        uint4 xr[4];
        unsigned amax = 0u;
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const int i = tid + r * (kCWarps * 32);
          xr[r] = make_uint4(0, 0, 0, 0);
          if (i < nvec) xr[r] = __ldg(reinterpret_cast<const uint4*>(p.x) + i);
          amax = split_amax8(xr[r], amax);
        }
        amax = __reduce_max_sync(0xffffffffu, amax);
        if (lane == 0) s_am[warp] = amax;
        asm volatile("bar.sync 1, %0;" ::"n"(kCWarps * 32) : "memory");
        amax = 0;
#pragma unroll
        for (int i = 0; i < kCWarps; i++) amax = max(amax, s_am[i]);
        const int E = split_exponent(amax);
        const float mult = __int_as_float((21 - E + 127) << 23);
        if (tid < 4) {
          const float un = __int_as_float((E - 21 + 6 * tid + 127) << 23);
          s_scale[tid] = un;
          if (b == 0 && p.unit_out) p.unit_out[tid] = un;
        }
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const int i = tid + r * (kCWarps * 32);
          if (i < nvec) {
            uint32_t out[4][2];
            split_digits8(xr[r], mult, out);
#pragma unroll
            for (int d = 0; d < 4; d++) {
              const size_t at = (size_t)d * p.K + (size_t)i * 8;
              *reinterpret_cast<uint2*>(stg + at) = make_uint2(out[d][0], out[d][1]);
              if (b == 0 && p.xq_out) *reinterpret_cast<uint2*>(p.xq_out + at) = make_uint2(out[d][0], out[d][1]);
            }
          }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kCWarps * 32) : "memory");   // planes complete; s_red free to be cleared
      }
    }
    const int W = p.K / 16;
    const int total = ncol * p.nchunk * 16;
    // the two words of unit u (zeros past the end of the row or of the units)
    auto load_unit = [&](int u) {
      const int pair = u >> 4;
      const int col = (int)(((uint32_t)pair * (uint32_t)p.inv_nchunk) >> 20), ch = pair - col * p.nchunk;   // pair / nchunk
      const int lo = u & 3, hi = (u >> 2) & 3;
      const int wx = (chunk0 + ch) * kChunkWords + (kRelabel ? 8 * hi + 2 * lo : 8 * lo + 2 * hi);   // word index in the row
      uint4 x = make_uint4(0, 0, 0, 0);
      if (u < total && wx < W) x = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2)) + (wx >> 1));
      return x;
    };
    // digit columns: the 16 bytes of word wx + w of unit u
    auto load_unit_bytes = [&](int u, int w) {
      const int pair = u >> 4;
      const int col = (int)(((uint32_t)pair * (uint32_t)p.inv_nchunk) >> 20), ch = pair - col * p.nchunk;
      const int lo = u & 3, hi = (u >> 2) & 3;
      const int wx = (chunk0 + ch) * kChunkWords + 8 * lo + 2 * hi + w;
      uint4 x = make_uint4(0, 0, 0, 0);
      if (u < total && wx < W) {
        if (p.x) x = *(reinterpret_cast<const uint4*>(stg + (size_t)col * p.K) + wx);   // planes made above
        else x = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * p.K) + wx);
      }
      return x;
    };
    // tensor-core kernels of the per-row grid (several tokens, so several units per thread): the next unit's
    // words are fetched while this one is expanded. Measured: the one- and two-token kernels lose 1 % with
    // it, the group-wise kernels have no registers to spare for it.
    constexpr bool kPrefetch = !GRP && !A16 && MODE == kModeMma;
    uint4 x_next = make_uint4(0, 0, 0, 0);
    if constexpr (kPrefetch) x_next = load_unit(warp * 32 + lane);
    for (int u0 = warp * 32; u0 < total; u0 += kCWarps * 32) {
      const int u = u0 + lane;
      int tsum = 0;
      const int pair = u >> 4;
      const int col = (int)(((uint32_t)pair * (uint32_t)p.inv_nchunk) >> 20), ch = pair - col * p.nchunk;   // pair / nchunk
      uint4 x = x_next;
      if constexpr (kPrefetch) x_next = load_unit(u + kCWarps * 32);
      if (u < total) {
        const int lo = u & 3, hi = (u >> 2) & 3;   // lo: 16-byte slot t of the column block; hi: 2 i + pr, or the group
        if constexpr (!kPrefetch && !A16) {
          const int wx = (chunk0 + ch) * kChunkWords + (kRelabel ? 8 * hi + 2 * lo : 8 * lo + 2 * hi);   // word index in the row
          if (wx < W) x = __ldg(reinterpret_cast<const uint4*>(p.xq + (size_t)col * (p.K / 2)) + (wx >> 1));
        }
        uint32_t q[4][2];
        if constexpr (A16) {
#pragma unroll
          for (int w = 0; w < 2; w++) {
            const uint4 d = load_unit_bytes(u, w);   // bytes 4b..4b+3 of d: the digits that meet byte b of the weight word
            tsum = __dp4a((int)d.x, 0x01010101, tsum); tsum = __dp4a((int)d.y, 0x01010101, tsum);
            tsum = __dp4a((int)d.z, 0x01010101, tsum); tsum = __dp4a((int)d.w, 0x01010101, tsum);
            // 4 x 4 byte transpose: position p gathers byte p of each of the four
            const uint32_t t01 = __byte_perm(d.x, d.y, 0x5140), t23 = __byte_perm(d.z, d.w, 0x5140);
            const uint32_t s01 = __byte_perm(d.x, d.y, 0x7362), s23 = __byte_perm(d.z, d.w, 0x7362);
            q[0][w] = (__byte_perm(t01, t23, 0x5410) << 2) & 0xFCFCFCFCu;   // even positions carry 4 q (|q| <= 32)
            q[1][w] = __byte_perm(t01, t23, 0x7632);
            q[2][w] = (__byte_perm(s01, s23, 0x5410) << 2) & 0xFCFCFCFCu;
            q[3][w] = __byte_perm(s01, s23, 0x7632);
          }
        } else
#pragma unroll
        for (int w = 0; w < 2; w++) {
          const uint32_t lo32 = w ? x.z : x.x, hi32 = w ? x.w : x.y;   // codes 0..7 and 8..15 of the word
          // even and odd codes of each half as bytes, each nibble sign-extended to a byte
          uint32_t n4[4] = {lo32 & 0x0F0F0F0Fu, (lo32 >> 4) & 0x0F0F0F0Fu, hi32 & 0x0F0F0F0Fu, (hi32 >> 4) & 0x0F0F0F0Fu};
#pragma unroll
          for (int h = 0; h < 4; h++) {
            n4[h] |= (n4[h] & 0x08080808u) * 0x1Eu;
            tsum = __dp4a((int)n4[h], 0x01010101, tsum);
          }
          // position p of a byte of codes: codes p, 4+p, 8+p, 12+p; even positions carry 4 q
          const uint32_t v0 = __byte_perm(n4[0], n4[2], 0x6420), v2 = __byte_perm(n4[0], n4[2], 0x7531);
          q[0][w] = (v0 << 2) & 0xFCFCFCFCu;
          q[1][w] = __byte_perm(n4[1], n4[3], 0x6420);
          q[2][w] = (v2 << 2) & 0xFCFCFCFCu;
          q[3][w] = __byte_perm(n4[1], n4[3], 0x7531);
        }
        uint8_t* dst = bs + ((size_t)(((ch * 4 + hi) * 2) * ncol + col)) * 64 + lo * 16;
        if (RCP_CK(dst >= bs && dst + (size_t)ncol * 64 + 16 <= bs + p.bs_bytes, 3)) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(q[0][0], q[0][1], q[1][0], q[1][1]);
          *reinterpret_cast<uint4*>(dst + (size_t)ncol * 64) = make_uint4(q[2][0], q[2][1], q[3][0], q[3][1]);
        }
      }
      if constexpr (!GRP) {
#pragma unroll
        for (int d = 8; d > 0; d >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, d);
        if ((lane & 15) == 0 && u < total) atomicAdd(&s_T0tot[col], tsum);   // integer: any order gives the same sum
      } else if constexpr (kRelabel) {   // the group is bits 2,3 of the unit: add up over bits 0,1
        tsum += __shfl_xor_sync(0xffffffffu, tsum, 1);
        tsum += __shfl_xor_sync(0xffffffffu, tsum, 2);
        if ((u & 3) == 0 && u < total) s_T0f[(ch * 4 + ((u >> 2) & 3)) * Mp + col] = (float)(8 * tsum);
      } else {                           // the group is bits 0,1 of the unit: add up over bits 2,3
        tsum += __shfl_xor_sync(0xffffffffu, tsum, 4);
        tsum += __shfl_xor_sync(0xffffffffu, tsum, 8);
        if ((u & 12) == 0 && u < total) s_T0c[col * ng4 + ch * 4 + (u & 3)] = tsum;
      }
    }
    if (tid < M && !(A16 && p.x)) s_scale[tid] = A16 ? p.unit[tid] : __half2float(p.scale[tid]);
    if constexpr (!GRP)
      for (int i = tid; i < 2 * 8 * 16 * M * 3; i += kCWarps * 32) s_red[i] = 0;
  }
  asm volatile("bar.sync 1, %0;" ::"n"(kCWarps * 32) : "memory");   // consumer warps only

  // ------------------------------------------------------------------ consumers
  constexpr int NF_M = (MODE == kModeDp4a) ? 0 : (MODE == kModeHybrid ? 2 : 3);  // planes on the MMA
  constexpr int NF_D = (MODE == kModeDp4a) ? 3 : (MODE == kModeHybrid ? 1 : 0);  // planes on dp4a
  constexpr int NTD = (NF_D == 0) ? 1 : MTOK;
  int accM[NF_M == 0 ? 1 : NF_M][2][4];
  int accN[kTwoTiles ? 3 : 1][1][4];   // second column tile
  int accD[NTD][2][NF_D == 0 ? 1 : NF_D][2];
  // kModeDp4a: position 3 sits in bits 6 and 7 of a byte. One mask keeps both; read as unsigned
  // bytes they weigh 64 b0 + 128 b1, read as signed bytes 64 b0 - 128 b1, so two dp4a on the same
  // operand separate the b0 and b1 planes and a mask is saved.
  constexpr bool kSign3 = (MODE == kModeDp4a);
  int accP[NTD][2][2];   // [token][row][unsigned, signed]
  // The same on the tensor cores (per-row grid): the operand masked at bits 6,7 goes through one MMA that
  // reads it as unsigned and one that reads it as signed bytes.
  constexpr bool kSign3M = (MODE == kModeMma && !GRP && !kTwoTiles);   // two tiles: no registers for its accumulators
  int accPu[4], accPs[4];
  auto zero_acc = [&]() {
#pragma unroll
    for (int f = 0; f < (NF_M == 0 ? 1 : NF_M); f++)
#pragma unroll
      for (int h = 0; h < 2; h++)
#pragma unroll
        for (int r = 0; r < 4; r++) accM[f][h][r] = 0;
#pragma unroll
    for (int a = 0; a < NTD; a++)
#pragma unroll
      for (int r = 0; r < 2; r++)
#pragma unroll
        for (int f = 0; f < (NF_D == 0 ? 1 : NF_D); f++)
#pragma unroll
          for (int h = 0; h < 2; h++) accD[a][r][f][h] = 0;
#pragma unroll
    for (int a = 0; a < NTD; a++)
#pragma unroll
      for (int r = 0; r < 2; r++) { accP[a][r][0] = 0; accP[a][r][1] = 0; }
#pragma unroll
    for (int r = 0; r < 4; r++) { accPu[r] = 0; accPs[r] = 0; }
#pragma unroll
    for (int f = 0; f < (kTwoTiles ? 3 : 1); f++)
#pragma unroll
      for (int r = 0; r < 4; r++) accN[f][0][r] = 0;
  };
  zero_acc();

  // (row, token) entries this lane emits.
  // kModeMma:   lane (g,t) owns tokens 2t, 2t+1 (and 8+2t, 9+2t with two column tiles) for rows g and g+8.
  // dp4a modes: MMA columns repeat the tokens (column c carries token c % MTOK); dp4a partial sums
  //             are reduced over the quad and lane t==0 owns tokens 0..MTOK-1 for rows g and g+8.
  constexpr int NE = (MODE == kModeMma) ? (kTwoTiles ? 8 : 4) : 2 * NTD;
  int etok[NE], err[NE], T0v[NE];
#pragma unroll
  for (int e = 0; e < NE; e++) {
    if constexpr (MODE == kModeMma) { etok[e] = 8 * (e >> 2) + 2 * t + (e & 1); err[e] = (e >> 1) & 1; }
    else { etok[e] = (t == 0) ? (e >> 1) : kMaxTokens; err[e] = e & 1; }
    T0v[e] = 0;
  }
  // T0 of the tokens this lane emits (added up while the activations were expanded)
  if constexpr (!GRP && !kTwoTiles) {   // two tiles: read when needed, the registers are taken
#pragma unroll
    for (int e = 0; e < NE; e++) if (etok[e] < M) T0v[e] = s_T0tot[etok[e]];
  }

  // per-lane constant parts of the shared-memory addresses
  //   weights: 16-byte chunk (2t+i) ^ (row & 7) of rows g and g+8 under the 128B swizzle
  uint32_t a_chunk[2];
#pragma unroll
  for (int i = 0; i < 2; i++) a_chunk[i] = (uint32_t)(g * 128 + (((2 * t + i) ^ g) << 4));
  const uint32_t half_stride = (uint32_t)ncol * 64;
  const uint32_t chunk_stride = 8 * half_stride;   // 2 (i) x 2 (pr) x 2 (half) per chunk
  uint32_t bM_lane, bD_lane[NTD];
  {
    int col = g;
    if constexpr (MTOK > 0) col = g % MTOK;
    else if (col >= M) col = M - 1;
    bM_lane = (uint32_t)(col * 64 + t * 16);
  }
  const uint32_t bN_lane = (uint32_t)(min(8 + g, M - 1) * 64 + t * 16);   // column of the second tile
#pragma unroll
  for (int tok = 0; tok < NTD; tok++) bD_lane[tok] = (uint32_t)(tok * 64 + t * 16);

  // 16 rows x 128 bytes of weights at shared address a_grp against the activations of one chunk
  auto compute_chunk = [&](uint32_t a_grp, uint32_t b_ptr) {   // b_ptr: the chunk's expanded activations
    const uint32_t a_ptr = a_grp;                          // 32-bit shared-memory addresses throughout
#pragma unroll
    for (int i = 0; i < 2; i++) {
      const uint4 U = RCP_LDS128(a_ptr + a_chunk[i], ring_lo, ring_hi, 4);
      const uint4 V = RCP_LDS128(a_ptr + 8 * 128 + a_chunk[i], ring_lo, ring_hi, 4);
      const uint32_t uw[4] = {U.x, U.y, U.z, U.w};
      const uint32_t vw[4] = {V.x, V.y, V.z, V.w};
#pragma unroll
      for (int pr = 0; pr < 2; pr++) {
        const uint32_t b_off = (uint32_t)((i * 2 + pr) * 2) * half_stride;
        // activation operands of the word pair: [position p][word]
        uint32_t bM[4][2];
        uint32_t bD[NTD][4][2];
        if constexpr (NF_D > 0) {
#pragma unroll
          for (int tok = 0; tok < NTD; tok++) {
            const uint4 x = RCP_LDS128(b_ptr + bD_lane[tok] + b_off, bs_lo, bs_hi, 5);
            const uint4 y = RCP_LDS128(b_ptr + bD_lane[tok] + b_off + half_stride, bs_lo, bs_hi, 5);
            bD[tok][0][0] = x.x; bD[tok][0][1] = x.y; bD[tok][1][0] = x.z; bD[tok][1][1] = x.w;
            bD[tok][2][0] = y.x; bD[tok][2][1] = y.y; bD[tok][3][0] = y.z; bD[tok][3][1] = y.w;
          }
        }
        if constexpr (NF_M > 0) {
          if constexpr (MODE == kModeHybrid && MTOK == 1) {
#pragma unroll
            for (int pp = 0; pp < 4; pp++) { bM[pp][0] = bD[0][pp][0]; bM[pp][1] = bD[0][pp][1]; }
          } else {
            const uint4 x = RCP_LDS128(b_ptr + bM_lane + b_off, bs_lo, bs_hi, 6);
            const uint4 y = RCP_LDS128(b_ptr + bM_lane + b_off + half_stride, bs_lo, bs_hi, 6);
            bM[0][0] = x.x; bM[0][1] = x.y; bM[1][0] = x.z; bM[1][1] = x.w;
            bM[2][0] = y.x; bM[2][1] = y.y; bM[3][0] = y.z; bM[3][1] = y.w;
          }
        }
        uint32_t bN[4][2];
        if constexpr (kTwoTiles) {
          const uint4 x = RCP_LDS128(b_ptr + bN_lane + b_off, bs_lo, bs_hi, 7);
          const uint4 y = RCP_LDS128(b_ptr + bN_lane + b_off + half_stride, bs_lo, bs_hi, 7);
          bN[0][0] = x.x; bN[0][1] = x.y; bN[1][0] = x.z; bN[1][1] = x.w;
          bN[2][0] = y.x; bN[2][1] = y.y; bN[3][0] = y.z; bN[3][1] = y.w;
        }
        const uint32_t u0 = uw[2 * pr], u1 = uw[2 * pr + 1], v0 = vw[2 * pr], v1 = vw[2 * pr + 1];
        const uint32_t u0s = u0 + u0, u1s = u1 + u1, v0s = v0 + v0, v1s = v1 + v1;  // b0 moved onto b1's bit
#pragma unroll
        for (int po = 0; po < 4; po++) {
          // positions in the order 0, 2, 1, 3: consecutive iterations feed different accumulators
          const int pp = ((po & 1) << 1) | (po >> 1);
          // Two column tiles: positions 2 and 3 are moved down onto the bits of 0 and 1 first, so that all
          // four positions add into one set of accumulators (there are no registers for two sets per tile).
          const bool down = kTwoTiles && pp >= 2;
          const uint32_t m0 = 0x01010101u << (2 * (down ? pp - 2 : pp)), m1 = m0 << 1;
          const uint32_t w_u0 = down ? u0 >> 4 : u0, w_u1 = down ? u1 >> 4 : u1;
          const uint32_t w_v0 = down ? v0 >> 4 : v0, w_v1 = down ? v1 >> 4 : v1;
          const uint32_t s_u0 = down ? w_u0 + w_u0 : u0s, s_u1 = down ? w_u1 + w_u1 : u1s;
          const uint32_t s_v0 = down ? w_v0 + w_v0 : v0s, s_v1 = down ? w_v1 + w_v1 : v1s;
          // the three planes of the four words: b0, b1, b0*b1 (the last two scaled by 2)
          const uint32_t au0[3] = {w_u0 & m0, w_u0 & m1, and3(w_u0, s_u0, m1)};
          const uint32_t au1[3] = {w_u1 & m0, w_u1 & m1, and3(w_u1, s_u1, m1)};
          const uint32_t av0[3] = {w_v0 & m0, w_v0 & m1, and3(w_v0, s_v0, m1)};
          const uint32_t av1[3] = {w_v1 & m0, w_v1 & m1, and3(w_v1, s_v1, m1)};
#pragma unroll
          for (int f = 0; f < NF_M; f++) {
            if (kSign3M && pp == 3 && f < 2) continue;
            const int half = kTwoTiles ? 0 : pp >> 1;
            mma_u8s8(accM[f][half], au0[f], av0[f], au1[f], av1[f], bM[pp][0], bM[pp][1]);
            if constexpr (kTwoTiles) mma_u8s8(accN[f][0], au0[f], av0[f], au1[f], av1[f], bN[pp][0], bN[pp][1]);
          }
          if (kSign3M && pp == 3) {
            const uint32_t k3 = 0xC0C0C0C0u;
            const uint32_t ku0 = u0 & k3, kv0 = v0 & k3, ku1 = u1 & k3, kv1 = v1 & k3;
            mma_u8s8(accPu, ku0, kv0, ku1, kv1, bM[3][0], bM[3][1]);
            mma_s8s8(accPs, ku0, kv0, ku1, kv1, bM[3][0], bM[3][1]);
          }
          if (kSign3 && pp == 3) {
            const uint32_t k3 = 0xC0C0C0C0u;
#pragma unroll
            for (int tok = 0; tok < NTD; tok++) {
              dp4a_u8s8(accP[tok][0][0], u0 & k3, bD[tok][3][0]);
              dp4a_s8s8(accP[tok][0][1], u0 & k3, bD[tok][3][0]);
              dp4a_u8s8(accP[tok][1][0], v0 & k3, bD[tok][3][0]);
              dp4a_s8s8(accP[tok][1][1], v0 & k3, bD[tok][3][0]);
              dp4a_u8s8(accP[tok][0][0], u1 & k3, bD[tok][3][1]);
              dp4a_s8s8(accP[tok][0][1], u1 & k3, bD[tok][3][1]);
              dp4a_u8s8(accP[tok][1][0], v1 & k3, bD[tok][3][1]);
              dp4a_s8s8(accP[tok][1][1], v1 & k3, bD[tok][3][1]);
            }
          }
#pragma unroll
          for (int f = 0; f < NF_D; f++) {
            const int fa = 3 - NF_D + f;  // hybrid: plane 2 only; dp4a: planes 0..2
            if (kSign3 && pp == 3 && fa < 2) continue;
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
  };

  // ---- group-wise grid
  // Tensor-core mode: MMA row g of the fragment is row grow of the 16 (rows 0,2,4,6 in the first
  // half-warp, 1,3,5,7 in the second: the 8-byte reads of a half-warp then hit all 32 banks once).
  const int grow = kRelabel ? (2 * (g & 3) + (g >> 2)) : g;
  float yacc[NE];
#pragma unroll
  for (int e = 0; e < NE; e++) yacc[e] = 0.f;
  const int tok2 = min(2 * t, Mp - 2);   // tensor-core mode: this lane's pair of token columns, kept inside the table
  // grids of the groups of chunk ch for this lane's rows: [group of the chunk][row]; the CUDA-core
  // path needs group t only
  constexpr int NLG = 1;
  auto fetch_lut_grp = [&](int row_first, int ch, uint2 (&dst)[NLG][2]) {
    const int gi = ch * 4 + t;   // lane t of a quad fetches group t; the tensor-core path passes it round the quad
#pragma unroll
    for (int rr = 0; rr < 2; rr++) {
      const int row = row_first + grow + 8 * rr;
      dst[0][rr] = (row < p.N && gi < p.ngrp) ? __ldg(p.lut + (size_t)row * p.ngrp + gi) : make_uint2(0, 0);
    }
  };
  // CUDA-core mode, after a chunk: this lane's sums are those of group t of the chunk
  auto flush_grp_dp4a = [&](int ch, const uint2 (&lg)[NLG][2], int row_first) {
    if constexpr (GRP && MODE == kModeDp4a) {
      const int gi = ch * 4 + t;
#pragma unroll
      for (int tok = 0; tok < NTD; tok++)
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const int a1 = (accD[tok][rr][0][0] >> 2) + (accD[tok][rr][0][1] >> 6) + ((accP[tok][rr][0] + accP[tok][rr][1]) >> 7);
          const int a2 = (accD[tok][rr][1][0] >> 3) + (accD[tok][rr][1][1] >> 7) + ((accP[tok][rr][0] - accP[tok][rr][1]) >> 8);
          const int a3 = (accD[tok][rr][2][0] >> 3) + (accD[tok][rr][2][1] >> 7);
          const int T0 = s_T0c[tok * ng4 + gi];
          const int S1 = a1 - a3, S2 = a2 - a3;
          yacc[tok * 2 + rr] += lut_dot(lg[0][rr], T0 - S1 - S2 - a3, S1, S2, a3);
          if constexpr (SDBG) {
            const int row = row_first + g + 8 * rr;
            if (row < p.N && gi < p.ngrp)
              *reinterpret_cast<int4*>(p.S_out + (((size_t)tok * p.N + row) * p.ngrp + gi) * 4) =
                  make_int4(T0 - S1 - S2 - a3, S1, S2, a3);
          }
        }
      zero_acc();
    }
  };
  // Tensor-core mode: one chunk = four groups, each read by the whole quad, finished after its
  // twelve MMAs.
  auto compute_chunk_grp_mma = [&](uint32_t a_grp, uint32_t b_abs, int ch, const uint2 (&lg)[NLG][2], int row_first) {   // b_abs: the chunk's expanded activations
    if constexpr (kRelabel) {
      const uint32_t a_row = a_grp + (uint32_t)(grow * 128 + ((t & 1) << 3));
      const uint32_t b_grp = b_abs + bM_lane;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const uint32_t a_sw = (uint32_t)(((2 * j + (t >> 1)) ^ (grow & 7)) << 4);
        const uint2 U = RCP_LDS64(a_row + a_sw, ring_lo, ring_hi, 8);
        const uint2 V = RCP_LDS64(a_row + 8 * 128 + a_sw, ring_lo, ring_hi, 8);
        const uint32_t b_ptr = b_grp + (uint32_t)(j * 2) * half_stride;
        const uint4 x = RCP_LDS128(b_ptr, bs_lo, bs_hi, 9);
        const uint4 y = RCP_LDS128(b_ptr + half_stride, bs_lo, bs_hi, 9);
        const uint32_t bM[4][2] = {{x.x, x.y}, {x.z, x.w}, {y.x, y.y}, {y.z, y.w}};
        // Positions 2 and 3 are moved down onto the bits of 0 and 1 first, so that all four positions add into one
        // set of accumulators: the finish below then converts three sums per entry, not six halves.
        const uint32_t wu[2][2] = {{U.x, U.y}, {U.x >> 4, U.y >> 4}}, wv[2][2] = {{V.x, V.y}, {V.x >> 4, V.y >> 4}};
        uint32_t su[2][2], sv[2][2];   // b0 moved onto b1's bit
#pragma unroll
        for (int d = 0; d < 2; d++)
#pragma unroll
          for (int w = 0; w < 2; w++) { su[d][w] = wu[d][w] + wu[d][w]; sv[d][w] = wv[d][w] + wv[d][w]; }
#pragma unroll
        for (int po = 0; po < 4; po++) {
          const int pp = ((po & 1) << 1) | (po >> 1);   // positions in the order 0, 2, 1, 3
          const int d = pp >> 1;
          const uint32_t m0 = 0x01010101u << (2 * (pp & 1)), m1 = m0 << 1;
          const uint32_t au0[3] = {wu[d][0] & m0, wu[d][0] & m1, and3(wu[d][0], su[d][0], m1)};
          const uint32_t au1[3] = {wu[d][1] & m0, wu[d][1] & m1, and3(wu[d][1], su[d][1], m1)};
          const uint32_t av0[3] = {wv[d][0] & m0, wv[d][0] & m1, and3(wv[d][0], sv[d][0], m1)};
          const uint32_t av1[3] = {wv[d][1] & m0, wv[d][1] & m1, and3(wv[d][1], sv[d][1], m1)};
#pragma unroll
          for (int f = 0; f < 3; f++) {
            if (po == 0) mma_u8s8_zero(accM[f][0], au0[f], av0[f], au1[f], av1[f], bM[pp][0], bM[pp][1]);
            else mma_u8s8(accM[f][0], au0[f], av0[f], au1[f], av1[f], bM[pp][0], bM[pp][1]);
          }
        }
        // The accumulators hold 4 T1, 8 T2 and 8 T3. Everything below works on 8 x the sums, in fp32 (small
        // integers: exact); the 1/8 goes into the final scale. With the levels L0..L3 of the (row, group),
        //   8 y = L0 (8 T0) + 2 (L1 - L0) (4 T1) + (L2 - L0) (8 T2) + ((L3 - L1) - (L2 - L0)) (8 T3):
        // the coefficients are made once per row and serve all its tokens.
        const int gi = ch * 4 + j;
        const float2 t0 = *reinterpret_cast<const float2*>(s_T0f + gi * Mp + tok2);
        float cf[2][4];
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const uint32_t lx = __shfl_sync(0xffffffffu, lg[0][rr].x, (lane & ~3) | j);
          const uint32_t ly = __shfl_sync(0xffffffffu, lg[0][rr].y, (lane & ~3) | j);
          const float2 l01 = __half22float2(*reinterpret_cast<const __half2*>(&lx));
          const float2 l23 = __half22float2(*reinterpret_cast<const __half2*>(&ly));
          const float d1 = l01.y - l01.x, d2 = l23.x - l01.x;
          cf[rr][0] = l01.x;
          cf[rr][1] = d1 + d1;
          cf[rr][2] = d2;
          cf[rr][3] = (l23.y - l01.y) - d2;
        }
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const float F1 = small_int_to_float(accM[0][0][r]);   // 4 T1
          const float F2 = small_int_to_float(accM[1][0][r]);   // 8 T2
          const float F3 = small_int_to_float(accM[2][0][r]);   // 8 T3
          const float (&c)[4] = cf[r >> 1];
          yacc[r] = fmaf(c[0], (r & 1) ? t0.y : t0.x, fmaf(c[1], F1, fmaf(c[2], F2, fmaf(c[3], F3, yacc[r]))));
          if constexpr (SDBG) {
            // the same sums as integers
            const int I1 = accM[0][0][r] >> 2, I2 = accM[1][0][r] >> 3, I3 = accM[2][0][r] >> 3;
            const int tok = 2 * t + (r & 1), row = row_first + grow + 8 * (r >> 1);
            if (tok < M && row < p.N && gi < p.ngrp) {
              const int I0 = __float2int_rn(0.125f * ((r & 1) ? t0.y : t0.x)) - (I1 - I3) - (I2 - I3) - I3;
              *reinterpret_cast<int4*>(p.S_out + (((size_t)tok * p.N + row) * p.ngrp + gi) * 4) =
                  make_int4(I0, I1 - I3, I2 - I3, I3);
            }
          }
        }
      }
    }
  };
  // end of a row group: the fp32 sums of this warp's chunks, for the entries this lane emits
  auto emit_grp = [&](int row_first, bool active, int KS, int grp, int ks, int& nred) {
    if constexpr (GRP) {
      if constexpr (MODE == kModeDp4a) {   // the four lanes of a quad hold four groups each: add them up
#pragma unroll
        for (int e = 0; e < NE; e++) {
          yacc[e] += __shfl_xor_sync(0xffffffffu, yacc[e], 1);
          yacc[e] += __shfl_xor_sync(0xffffffffu, yacc[e], 2);
        }
      }
      if (KS > 1) {
        // every warp of the group leaves its sums in its own slot; the first adds them up in order
        float* const red = s_redf + (nred & 1) * (kCWarps * 16 * M);
        nred++;
#pragma unroll
        for (int e = 0; e < NE; e++)
          if (active && etok[e] < M &&
              RCP_CK(((nred - 1) & 1) * (kCWarps * 16 * M) + (warp * 16 + g + 8 * err[e]) * M + etok[e] < p.red_bytes / 4, 10))
            red[(warp * 16 + g + 8 * err[e]) * M + etok[e]] = yacc[e];
        asm volatile("bar.sync 2, %0;" ::"n"(kCWarps * 32) : "memory");   // consumer warps only
        if (active && ks == 0) {
#pragma unroll
          for (int e = 0; e < NE; e++) {
            if (etok[e] < M) {
              float a = 0.f;
              for (int k = 0; k < KS; k++) a += red[((grp * KS + k) * 16 + g + 8 * err[e]) * M + etok[e]];
              yacc[e] = a;
            }
          }
        }
      }
      if (active && ks == 0) {
#pragma unroll
        for (int e = 0; e < NE; e++) {
          const int row = row_first + grow + 8 * err[e];
          if (etok[e] < M && row < p.N)
            p.y[(size_t)etok[e] * p.N + row] = __float2half_rn(s_scale[etok[e]] * (kRelabel ? 0.125f * yacc[e] : yacc[e]));
        }
      }
#pragma unroll
      for (int e = 0; e < NE; e++) yacc[e] = 0.f;
    }
  };

  // this lane's entries as T1, T2, T3 from the accumulators (and clears them)
  auto collect = [&](int (&T1)[NE], int (&T2)[NE], int (&T3)[NE]) {
    if constexpr (MODE == kModeMma) {
#pragma unroll
      for (int r = 0; r < 4; r++) {
        T1[r] = (accM[0][0][r] >> 2) + (accM[0][1][r] >> 6);
        T2[r] = (accM[1][0][r] >> 3) + (accM[1][1][r] >> 7);
        T3[r] = (accM[2][0][r] >> 3) + (accM[2][1][r] >> 7);
        if constexpr (kSign3M) {
          T1[r] += (accPu[r] + accPs[r]) >> 7;
          T2[r] += (accPu[r] - accPs[r]) >> 8;
        }
      }
      if constexpr (kTwoTiles) {
#pragma unroll
        for (int r = 0; r < 4; r++) {
          T1[4 + r] = accN[0][0][r] >> 2;   // one set of accumulators: accM[.][1] stayed zero above
          T2[4 + r] = accN[1][0][r] >> 3;
          T3[4 + r] = accN[2][0][r] >> 3;
        }
      }
    } else {
#pragma unroll
      for (int tok = 0; tok < NTD; tok++)
#pragma unroll
        for (int rr = 0; rr < 2; rr++) {
          const int e = tok * 2 + rr;
          int a1, a2, a3;
          if constexpr (MODE == kModeHybrid) {
            const int r = tok + 2 * rr;  // lane t==0 holds columns 0, 1
            a1 = (accM[0][0][r] >> 2) + (accM[0][1][r] >> 6);
            a2 = (accM[1][0][r] >> 3) + (accM[1][1][r] >> 7);
            a3 = (accD[tok][rr][0][0] >> 3) + (accD[tok][rr][0][1] >> 7);
          } else {
            a1 = (accD[tok][rr][0][0] >> 2) + (accD[tok][rr][0][1] >> 6) + ((accP[tok][rr][0] + accP[tok][rr][1]) >> 7);
            a2 = (accD[tok][rr][1][0] >> 3) + (accD[tok][rr][1][1] >> 7) + ((accP[tok][rr][0] - accP[tok][rr][1]) >> 8);
            a3 = (accD[tok][rr][2][0] >> 3) + (accD[tok][rr][2][1] >> 7);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            a2 += __shfl_xor_sync(0xffffffffu, a2, 1); a2 += __shfl_xor_sync(0xffffffffu, a2, 2);
          }
          a3 += __shfl_xor_sync(0xffffffffu, a3, 1); a3 += __shfl_xor_sync(0xffffffffu, a3, 2);
          T1[e] = a1; T2[e] = a2; T3[e] = a3;
        }
    }
    zero_acc();
  };
  uint2 lut_g[2];  // LUT rows g and g+8 of the current group, fetched ahead of the epilogue
  auto fetch_lut = [&](int row_first) {
#pragma unroll
    for (int rr = 0; rr < 2; rr++) {
      const int row = row_first + g + 8 * rr;
      lut_g[rr] = row < p.N ? __ldg(p.lut + row) : make_uint2(0, 0);
    }
  };
  auto emit = [&](int row_first, const int (&T1)[NE], const int (&T2)[NE], const int (&T3)[NE]) {
    if constexpr (A16) {
      // Columns 4j..4j+3 are the digits of token j: lane t holds two of them, lane t ^ 1 the other two.
      // y = (u_a D_a + u_b D_b) + (u_c D_c + u_d D_d) in fp32, D the grid-weighted sum of a digit column.
#pragma unroll
      for (int e = 0; e < NE; e += 2) {
        float v = 0.f;
#pragma unroll
        for (int h = 0; h < 2; h++) {
          const int c = etok[e + h];
          if (c < M) {
            const int S3 = T3[e + h], S1 = T1[e + h] - T3[e + h], S2 = T2[e + h] - T3[e + h];
            const int S0 = (kTwoTiles ? s_T0tot[c] : T0v[e + h]) - S1 - S2 - S3;
            const float d = lut_sum(lut_g[err[e]], S0, S1, S2, S3);
            if constexpr (SDBG) {
              const int row_s = row_first + g + 8 * err[e];
              if (row_s < p.N) *reinterpret_cast<int4*>(p.S_out + ((size_t)c * p.N + row_s) * 4) = make_int4(S0, S1, S2, S3);
            }
            v = h ? __fmaf_rn(s_scale[c], d, v) : __fmul_rn(s_scale[c], d);
          }
        }
        v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, 1));   // both lanes add the same two numbers
        const int row = row_first + g + 8 * err[e], tok = etok[e] >> 2;
        if ((t & 1) == 0 && etok[e] < M && row < p.N) p.y[(size_t)tok * p.N + row] = __float2half_rn(v);
      }
    } else {
#pragma unroll
      for (int e = 0; e < NE; e++) {
        const int row = row_first + g + 8 * err[e];
        if (etok[e] < M && row < p.N) {
          const int S3 = T3[e], S1 = T1[e] - T3[e], S2 = T2[e] - T3[e];
          const int S0 = (kTwoTiles ? s_T0tot[etok[e]] : T0v[e]) - S1 - S2 - S3;
          p.y[(size_t)etok[e] * p.N + row] = lut_finish(s_scale[etok[e]], lut_g[err[e]], S0, S1, S2, S3);
          if constexpr (SDBG)
            *reinterpret_cast<int4*>(p.S_out + ((size_t)etok[e] * p.N + row) * 4) = make_int4(S0, S1, S2, S3);
        }
      }
    }
  };

  int T1[NE], T2[NE], T3[NE];
  // finishes the rows of a group, or (K in parts) parks their sums until the last part has added its share
  auto finish = [&](int row_first, int gslot) {
    if (kSplit && nsplit > 1) {
#pragma unroll
      for (int e = 0; e < NE; e++) {
        if (etok[e] < M) {
          int* d = s_part + ((gslot * 16 + g + 8 * err[e]) * M + etok[e]) * 3;
          if (!RCP_CK(gslot >= 0 && (((gslot * 16 + g + 8 * err[e]) * M + etok[e]) * 3 + 3) * 4 <= p.part_bytes, 11)) continue;
          if (kp > 0) { T1[e] += d[0]; T2[e] += d[1]; T3[e] += d[2]; }
          if (kp + 1 < nsplit) { d[0] = T1[e]; d[1] = T2[e]; d[2] = T3[e]; }
        }
      }
      if (kp + 1 < nsplit) return;
    }
    emit(row_first, T1, T2, T3);
  };

  int slot = slot_keep;
  uint32_t phase = phase_keep;
  int nred = nred_keep;   // phases with a shared-memory reduction so far (its two buffers alternate)
  int gbase = 0;   // groups of this CTA before the current repetition, the same count in every part
  for (int pi = 0; pi < p.nphase; pi++) {
    const GemvPhase ph = p.phase[pi];
    if (b >= ph.ncta) continue;
    const int KS = ph.ks;
    const int grp = (warp * ph.inv_ks) >> 8, ks = warp - grp * KS;
    const int SA = ph.sa;
    const int lo = ph.q * b + min(b, ph.r), hi = lo + ph.q + (b < ph.r ? 1 : 0);
    const bool active = grp < hi - lo;   // fewer groups than gpc here, or warps beyond gpc KS
    const uint32_t a_off = (uint32_t)ks * ((uint32_t)ph.gpc * kGroupBytes) + (uint32_t)grp * kGroupBytes;
    for (int rp = 0; rp < ph.reps; rp++) {
      const int row_first = (ph.first + rp * ph.total + lo + grp) * 16;
      const int gslot = gbase + grp;
      gbase += hi - lo;
      uint32_t b_chunk = (uint32_t)ks * chunk_stride;
      int ch = ks;
      if constexpr (GRP) {
        // the grids of a chunk are fetched one chunk ahead
        uint2 lg_cur[NLG][2], lg_nxt[NLG][2];
        fetch_lut_grp(active ? row_first : p.N, ch, lg_nxt);
        for (int s = 0; s < SA; s++, ch += KS, b_chunk += (uint32_t)KS * chunk_stride) {
#pragma unroll
          for (int j = 0; j < NLG; j++) { lg_cur[j][0] = lg_nxt[j][0]; lg_cur[j][1] = lg_nxt[j][1]; }
          if (s + 1 < SA) fetch_lut_grp(active ? row_first : p.N, ch + KS, lg_nxt);
          if (!mbar_wait(full0 + 8 * slot, phase)) {
            if (lane == 0 && p.status) atomicExch(p.status, 3);
            return;
          }
          if (active && ch < p.nchunk) {
            const uint32_t st = base + (uint32_t)slot * stage_stride;   // (stage_stride == kStageBytes unless SB)
            const uint32_t a_grp = st + a_off;
            if constexpr (kRelabel) {
              compute_chunk_grp_mma(a_grp, SB ? st + kStageBytes + (uint32_t)ks * chunk_stride : base + (uint32_t)p.off_bs + b_chunk,
                                    ch, lg_cur, row_first);
            } else {
              compute_chunk(a_grp, base + (uint32_t)p.off_bs + b_chunk);
              flush_grp_dp4a(ch, lg_cur, row_first);
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty0 + 8 * slot);   // this warp is done with the slot
          if (++slot == stages) { slot = 0; phase ^= 1u; }
        }
        emit_grp(row_first, active, KS, grp, ks, nred);
        continue;
      }
      if (active) fetch_lut(row_first);
      for (int s = 0; s < SA; s++, ch += KS, b_chunk += (uint32_t)KS * chunk_stride) {
        if (!mbar_wait(full0 + 8 * slot, phase)) {
          if (lane == 0 && p.status) atomicExch(p.status, 3);
          return;
        }
        if (active && ch < nch) {
          if constexpr (SB) {
            const uint32_t st = base + (uint32_t)slot * stage_stride;
            compute_chunk(st + a_off, st + kStageBytes + (uint32_t)ks * chunk_stride);
          } else {
            compute_chunk(base + (uint32_t)slot * kStageBytes + a_off, base + (uint32_t)p.off_bs + b_chunk);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * slot);   // this warp is done with the slot
        if (++slot == stages) { slot = 0; phase ^= 1u; }
      }
      collect(T1, T2, T3);
      if (KS == 1) {
        if (active) finish(row_first, gslot);
      } else {
        // the KS warps of a group add up in shared memory; the first of them finishes the rows
        int* const red = s_red + (nred & 1) * (8 * 16 * M * 3);
        nred++;
#pragma unroll
        for (int e = 0; e < NE; e++) {
          if (active && etok[e] < M &&
              RCP_CK(grp < 8 && (((nred - 1) & 1) * (8 * 16 * M * 3) + ((grp * 16 + g + 8 * err[e]) * M + etok[e]) * 3 + 3) * 4 <= p.red_bytes, 12)) {
            int* d = red + ((grp * 16 + g + 8 * err[e]) * M + etok[e]) * 3;
            atomicAdd(d + 0, T1[e]);
            atomicAdd(d + 1, T2[e]);
            atomicAdd(d + 2, T3[e]);
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kCWarps * 32) : "memory");   // consumer warps only
        if (active && ks == 0) {
#pragma unroll
          for (int e = 0; e < NE; e++) {
            if (etok[e] < M) {
              int* d = red + ((grp * 16 + g + 8 * err[e]) * M + etok[e]) * 3;
              T1[e] = d[0]; T2[e] = d[1]; T3[e] = d[2];
              d[0] = 0; d[1] = 0; d[2] = 0;   // ready for the reduction after next
            }
          }
          finish(row_first, gslot);
        }
      }
    }
  }
  slot_keep = slot; phase_keep = phase; nred_keep = nred;
  }   // parts of K
}

}  // namespace rcp
