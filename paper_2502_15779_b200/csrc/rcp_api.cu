// C ABI of the RCP W2A4 library: argument validation, launch configuration, status codes.
#include "../../include/rcp.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <utility>

#include "common.cuh"
#include "gemv_simple.cuh"
#include "gemv_stream.cuh"
#include "gemv_w3.cuh"
#include "ldp_export.cuh"
#include "split_act16.cuh"
#include "pack.cuh"
#include "quantize_act.cuh"

namespace {

thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return RCP_ERR_CUDA;
}

#define RCP_CUDA(call)                            \
  do {                                            \
    cudaError_t e__ = (call);                     \
    if (e__ != cudaSuccess) return cuda_fail(e__); \
  } while (0)

// Launches with programmatic stream serialization: the kernel may start while the preceding
// kernel on the stream is still running and must execute griddepcontrol.wait before it touches
// anything that kernel may read or write.
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool k_ok(int K) { return K >= 64 && K <= rcp::kMaxK && K % 64 == 0; }

// Set by pack_weights_kernel when it meets a code above 3. One slot per call in flight (calls from several host
// threads or on several streams take different slots, so that none clears or reads another's flag).
constexpr unsigned kPackSlots = 64;
__device__ int g_pack_bad[kPackSlots];
std::atomic<unsigned> g_pack_next{0};

// ---------------------------------------------------------------------------------------------
// Streaming GEMV: launch plan.
struct StreamPlan {
  int nchunk, nchunk_total, nsplit, nphase, stages, grid;   // nchunk: chunks per row in one part of K
  rcp::GemvPhase phase[rcp::kMaxPhases];
  int off_bar, off_T0c, off_scale, off_red, off_bs, off_qbuf, off_part;
  int bs_bytes, red_bytes, part_bytes;
  int stage_stride;   // ring stage: boxes of weights, plus the stage's expanded activations when they are streamed
  size_t smem;
};

constexpr size_t kSmemMax = 232448;            // 227 KB of dynamic shared memory per CTA on sm_100
constexpr size_t kExpandBudget = 128 * 1024;   // expanded activations (one byte per code and token) per CTA
constexpr size_t kExpandBudgetTwoTiles = 80 * 1024;   // the same with 9 to 16 tokens (their reduction buffers are larger)

// Tokens one launch can take: their expanded activations must fit beside a ring of three stages.
// cap 16: the tensor-core kernel with two column tiles takes 9 to 16 tokens at once where they fit.
int tokens_per_pass(int M, int K, int cap) {
  if (cap > 8) {
    if (M > 8 && (size_t)M * K <= kExpandBudgetTwoTiles) return M;
    cap = 8;
  }
  int m = std::min(M, cap);
  while (m > 1 && (size_t)m * K > kExpandBudget) m--;
  return m;
}

// The tensor-core kernels of the per-row grid rather keep their (up to eight) tokens and go through K in
// parts when the expanded activations of the whole K would not fit: the weights are then streamed once, not
// once per launch. Falls back to fewer tokens when the sums parked between the parts leave no room for a
// ring of three stages (very many rows per CTA). Returns the tokens per launch, *nsplit the parts of K.
StreamPlan make_plan(int M, int N, int K, int sms, bool grouped = false, size_t qbuf = 0, int nsplit = 1,
                     bool stream_act = false);
int tokens_and_parts(int M, int N, int K, int cap, int sms, int* nsplit) {
  *nsplit = 1;
  const int m = tokens_per_pass(M, K, cap);
  if (cap < 8 || m > 8) return m;
  const int want = std::min(M, 8);
  if (m == want) return m;   // everything fits at once (measured: parts cost more than a ring of two stages does)
  for (int parts = (int)(((size_t)want * K + kExpandBudget - 1) / kExpandBudget); parts <= 8; parts++) {
    const StreamPlan pl = make_plan(want, N, K, sms, false, 0, parts);
    if (pl.stages >= 3 && pl.smem <= kSmemMax) {
      *nsplit = pl.nsplit;
      return want;
    }
  }
  return m;
}

// Cost model of a phase in clocks: stages x (warps sharing a scheduler) x clocks per warp and
// chunk on one of the four schedulers, plus a fixed cost per phase (LUT fetch, reduction, barrier).
long long phase_cost(int gpc, int nchunk) {
  const int KS = rcp::kCWarps / gpc;
  const int stages = (nchunk + KS - 1) / KS;
  const int per_sched = (gpc * KS + 3) / 4;
  return (long long)stages * per_sched * 504 + 2000;
}

// A phase with the quotients the kernel would otherwise divide for.
rcp::GemvPhase make_phase(int gpc, int first, int total, int ncta, int reps, int nchunk, int ks_cap = rcp::kCWarps) {
  rcp::GemvPhase ph;
  ph.gpc = gpc; ph.first = first; ph.total = total; ph.ncta = ncta; ph.reps = reps;
  ph.q = total / ncta;
  ph.r = total % ncta;
  ph.ks = std::min(rcp::kCWarps / gpc, ks_cap);
  ph.inv_ks = (256 + ph.ks - 1) / ph.ks;
  ph.sa = (nchunk + ph.ks - 1) / ph.ks;
  return ph;
}

// Splits `rem` leftover groups (fewer than 16 per CTA) into phases: shares of 8, 4, 2 or 1 groups
// per CTA keep all warps busy but cost a phase each; one last phase takes whatever is left,
// ceil(left / CTAs) groups per CTA. Picks the cheapest combination. Returns the number of phases.
// ks_cap: most warps that may share a group along K (streamed activations: a stage holds the activations of
// that many chunks); phases that would need more are left out, the last phase uses fewer warps per group.
int plan_leftover(int rem, int sms, int nchunk, rcp::GemvPhase* out, int ks_cap = rcp::kCWarps) {
  int best_mask = 0;
  long long best = -1;
  for (int mask = 0; mask < 16; mask++) {   // bit i: a phase of 8 >> i groups per CTA
    int left = rem;
    long long cost = 0;
    bool ok = true;
    for (int i = 0; i < 4; i++) {
      if (!(mask >> i & 1)) continue;
      const int gpc = 8 >> i;
      if (rcp::kCWarps / gpc > ks_cap) { ok = false; break; }
      if (left < gpc * sms) { ok = false; break; }
      left -= gpc * sms;
      cost += phase_cost(gpc, nchunk);
    }
    if (!ok) continue;
    if (left >= 16 * sms) continue;
    if (left > 0) cost += phase_cost((left + sms - 1) / sms, nchunk);
    if (best < 0 || cost < best) { best = cost; best_mask = mask; }
  }
  int n = 0, first = 0, left = rem;
  for (int i = 0; i < 4; i++) {
    if (!(best_mask >> i & 1)) continue;
    const int gpc = 8 >> i;
    out[n++] = make_phase(gpc, first, gpc * sms, sms, 1, nchunk, ks_cap);
    first += gpc * sms;
    left -= gpc * sms;
  }
  if (left > 0) {
    const int ncta = std::min(left, sms);
    out[n++] = make_phase((left + ncta - 1) / ncta, first, left, ncta, 1, nchunk, ks_cap);
  }
  return n;
}

// qbuf: bytes of staging for the fused quantizer's cross-warp rotation strides (0 if unused)
// nsplit: parts of K the kernel goes through one after the other (tensor-core kernels of the per-row grid)
// stream_act: the expanded activations travel with the ring stages (tensor-core kernels of the per-row grid)
// instead of being expanded for the whole K up front.
StreamPlan make_plan(int M, int N, int K, int sms, bool grouped, size_t qbuf, int nsplit, bool stream_act) {
  StreamPlan pl;
  pl.grid = sms;
  pl.nchunk_total = (K / 16 + rcp::kChunkWords - 1) / rcp::kChunkWords;
  pl.nsplit = std::max(1, std::min(nsplit, pl.nchunk_total));
  pl.nchunk = (pl.nchunk_total + pl.nsplit - 1) / pl.nsplit;
  pl.nsplit = (pl.nchunk_total + pl.nchunk - 1) / pl.nchunk;   // no empty part
  // Phases: first the groups left over when every CTA takes 16 per round, then the rounds.
  const int groups = (N + 15) / 16;
  const int per_round = sms * rcp::kCWarps;
  const int R = groups / per_round;
  const int ks_cap = stream_act ? std::max(1, 32 / M) : rcp::kCWarps;
  pl.nphase = plan_leftover(groups - R * per_round, sms, pl.nchunk, pl.phase, ks_cap);
  int first = groups - R * per_round;
  if (R > 0) pl.phase[pl.nphase++] = make_phase(rcp::kCWarps, first, per_round, sms, R, pl.nchunk);
  int ks_max = 1;
  for (int i = 0; i < pl.nphase; i++) ks_max = std::max(ks_max, pl.phase[i].ks);
  // streamed: per stage, 512 bytes per token and chunk of the stage, rounded so that the stages stay 1024-byte aligned
  const size_t bstage = stream_act ? ((size_t)ks_max * M * 512 + 1023) / 1024 * 1024 : 0;
  pl.stage_stride = (int)(rcp::kStageBytes + bstage);
  const size_t bs_bytes = stream_act ? 0 : (size_t)pl.nchunk * rcp::kChunkWords * 16 * M;
  // sums of q per chunk (per group of 128: four per chunk); reduction buffers: integer sums of 8
  // row groups x 3 planes, or (group-wise grid) one fp32 term per warp
  const size_t t0c_bytes = grouped ? (size_t)(M + 1) * pl.nchunk * 16 : (((size_t)M * pl.nchunk * 4) + 15) / 16 * 16;
  const size_t red_bytes = grouped ? (size_t)2 * rcp::kCWarps * 16 * M * 4 : (size_t)2 * 8 * 16 * M * 3 * 4;
  // K in parts: the integer sums of every group this CTA owns wait in shared memory between the parts
  int own_groups = 0;
  for (int i = 0; i < pl.nphase; i++) own_groups += pl.phase[i].reps * (pl.phase[i].q + (pl.phase[i].r ? 1 : 0));
  const size_t part_bytes = pl.nsplit > 1 ? (size_t)own_groups * 16 * M * 3 * 4 : 0;
  const size_t misc = 128 + t0c_bytes + 256 + red_bytes + qbuf + part_bytes;
  const size_t fixed = 1024 + misc + bs_bytes;
  pl.stages = fixed >= kSmemMax ? 0 : (int)std::min<size_t>(rcp::kMaxStages, (kSmemMax - fixed) / pl.stage_stride);
  size_t off = (size_t)pl.stages * pl.stage_stride;
  pl.off_bar = (int)off; off += 128;
  pl.off_T0c = (int)off; off += t0c_bytes;
  pl.off_scale = (int)off; off += 256;   // 16 scales, 16 per-warp maxima of the fused quantizer, 16 token totals
  pl.off_red = (int)off; off += red_bytes;
  pl.off_bs = (int)off; off += bs_bytes;
  pl.off_qbuf = (int)off; off += qbuf;
  pl.off_part = (int)off; off += part_bytes;
  pl.bs_bytes = (int)bs_bytes; pl.red_bytes = (int)red_bytes; pl.part_bytes = (int)part_bytes;
  pl.smem = off + 1024;
  return pl;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

constexpr int kMaxDevices = 64;

// SMs of the current device (remembered per device; 148 if the query fails)
int sm_count() {
  static std::mutex mu;
  static int n[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  std::lock_guard<std::mutex> lock(mu);
  if (!n[dev] && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 148;
  return n[dev];
}

template <int MODE, int MTOK, bool GRP, bool FQ, bool A16, bool SPLIT, bool SDBG, bool SB = false>
int launch_stream_s(const rcp::GemvMaps& maps, const rcp::GemvParams& gp, const StreamPlan& pl, cudaStream_t st) {
  // cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the (kernel, device) pair: set once per device
  static std::mutex mu;
  static bool attr_set[kMaxDevices] = {};
  auto kern = rcp::gemv_stream_kernel<MODE, MTOK, GRP, FQ, A16, SPLIT, SDBG, SB>;
  int dev = 0;
  RCP_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return RCP_ERR_LIMIT;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
      RCP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax));
      attr_set[dev] = true;
    }
  }
  RCP_CUDA(launch_overlapped(kern, dim3(pl.grid), dim3(SB ? rcp::kGThreads + 32 * rcp::kExpWarps : rcp::kGThreads), pl.smem, st, maps, gp));
  return RCP_OK;
}

// streamed activations (tensor-core kernels of the per-row grid; MTOK 0: up to eight tokens, 16: nine to sixteen)
template <int MTOK>
int launch_stream_sb(const rcp::GemvMaps& maps, const rcp::GemvParams& gp, const StreamPlan& pl, cudaStream_t st) {
  if (gp.S_out) return launch_stream_s<rcp::kModeMma, MTOK, false, false, false, false, true, true>(maps, gp, pl, st);
  return launch_stream_s<rcp::kModeMma, MTOK, false, false, false, false, false, true>(maps, gp, pl, st);
}

// gp.S_out set: the checked instantiation of the same kernel, which also stores its integer sums.
template <int MODE, int MTOK, bool GRP = false, bool FQ = false, bool A16 = false, bool SPLIT = false>
int launch_stream_t(const rcp::GemvMaps& maps, const rcp::GemvParams& gp, const StreamPlan& pl, cudaStream_t st) {
  if (gp.S_out) return launch_stream_s<MODE, MTOK, GRP, FQ, A16, SPLIT, true>(maps, gp, pl, st);
  return launch_stream_s<MODE, MTOK, GRP, FQ, A16, SPLIT, false>(maps, gp, pl, st);
}

// One launch: M tokens (their expanded activations fit in shared memory). grouped: lut_f16 is
// [N][K/128][4], one grid per group of 128 weights.
// Activations still to be rotated and quantized, for the kernels that do it themselves.
struct FusedAct {
  const void* x_f16;     // [M][K]
  int B;                 // rotation block, 1 = none
  float clip_ratio;
  uint8_t* xq_out;       // optional
  void* scale_out;       // optional
};

// Shapes the in-kernel quantizer takes: one token of 4096 or 8192 elements under one rotation block.
// Measured on B200: there the fused kernel beats the two kernels by 0.7 to 1.9 us a call; for shorter
// tokens, block-wise rotation or two tokens the stand-alone quantizer (several CTAs per token) wins.
// Weight-only form, activations still in fp16: the GEMV kernel makes the digit planes itself.
struct SplitAct {
  const void* x_f16;    // [tokens][K]
  int8_t* digits_out;   // [tokens][4][K], written by CTA 0
  float* unit_out;      // [tokens][4], written by CTA 0
};

bool fused_ok(int M, int K, int B) { return M == 1 && B == K && (K == 4096 || K == 8192); }

int launch_stream(int mode, const uint32_t* words, const void* lut_f16, const uint8_t* xq, const void* scale_f16,
                  int M, int N, int K, void* y_f16, void* workspace, cudaStream_t st, bool grouped = false,
                  const FusedAct* fa = nullptr, const float* unit = nullptr, int nsplit = 1,
                  const SplitAct* sa = nullptr, int32_t* S_out = nullptr, bool stream_act = false) {
  if (stream_act && (mode != rcp::kModeMma || fa || unit || sa || nsplit > 1 || M > (grouped ? 8 : rcp::kMaxTokens))) return RCP_ERR_VARIANT;
  if (nsplit > 1 && (mode != rcp::kModeMma || grouped || fa || M > 8)) return RCP_ERR_VARIANT;
  if (sa && (mode != rcp::kModeMma || grouped || fa || unit || nsplit > 1 || M != 4 || K > 16384)) return RCP_ERR_VARIANT;
  // unit: weight-only form; xq then holds M digit columns of K signed bytes (four per token), scale_f16 is unused
  if (unit && (mode != rcp::kModeMma || grouped || fa || M % 4)) return RCP_ERR_VARIANT;
  if (mode != rcp::kModeMma && M > 2) return RCP_ERR_VARIANT;
  if (M > 8 && (grouped || fa || M > rcp::kMaxTokens)) return RCP_ERR_VARIANT;
  if (grouped && (mode == rcp::kModeHybrid || K % 128)) return RCP_ERR_VARIANT;
  if (fa && (mode != rcp::kModeDp4a || !fused_ok(M, K, fa->B))) return RCP_ERR_VARIANT;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return cuda_fail(cudaErrorNotSupported);
  const StreamPlan pl = make_plan(M, N, K, sm_count(), grouped, fa ? rcp::rotate_scratch_bytes(K) : (sa ? (size_t)M * K : 0), nsplit,
                                  stream_act);
  if (pl.stages < 2 || pl.smem > kSmemMax) return RCP_ERR_SHAPE;
  // Tensor maps of the phases in use (the others repeat the first). Encoding one costs the host about a
  // microsecond, so the maps of the last few (weights, shape, boxes) combinations are remembered per thread.
  struct MapKey { const void* words; int N, K, nphase, gpc[rcp::kMaxPhases]; };
  struct MapSlot { MapKey key; rcp::GemvMaps maps; bool used; };
  constexpr int kMapSlots = 16;
  thread_local MapSlot map_cache[kMapSlots] = {};
  thread_local int map_next = 0;
  MapKey key = {};
  key.words = words; key.N = N; key.K = K; key.nphase = pl.nphase;
  for (int i = 0; i < pl.nphase; i++) key.gpc[i] = pl.phase[i].gpc;
  const rcp::GemvMaps* cached = nullptr;
  for (int i = 0; i < kMapSlots; i++)
    if (map_cache[i].used && std::memcmp(&map_cache[i].key, &key, sizeof(MapKey)) == 0) { cached = &map_cache[i].maps; break; }
  if (!cached) {
    MapSlot& slot = map_cache[map_next];
    map_next = (map_next + 1) % kMapSlots;
    slot.used = false;
    const cuuint64_t gdim[2] = {(cuuint64_t)(K / 16), (cuuint64_t)N};
    const cuuint64_t gstride[1] = {(cuuint64_t)(K / 4)};
    const cuuint32_t estr[2] = {1, 1};
    for (int i = 0; i < rcp::kMaxPhases; i++) {
      if (i >= pl.nphase && i > 0) { slot.maps.m[i] = slot.maps.m[0]; continue; }
      const int gpc = i < pl.nphase ? pl.phase[i].gpc : 1;
      const cuuint32_t box[2] = {(cuuint32_t)rcp::kChunkWords, (cuuint32_t)(16 * gpc)};
      const CUresult r = enc(&slot.maps.m[i], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(words), gdim,
                             gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);
    }
    slot.key = key;
    slot.used = true;
    cached = &slot.maps;
  }
  const rcp::GemvMaps& maps = *cached;
  rcp::GemvParams gp;
  gp.lut = static_cast<const uint2*>(lut_f16);
  gp.xq = xq;
  gp.scale = static_cast<const __half*>(scale_f16);
  gp.unit = unit;
  gp.y = static_cast<__half*>(y_f16);
  gp.status = static_cast<int32_t*>(workspace);
  gp.S_out = S_out;
  gp.M = M; gp.N = N; gp.K = K;
  gp.ngrp = grouped ? K / 128 : 0;
  gp.nchunk = pl.nchunk;
  gp.nchunk_total = pl.nchunk_total;
  gp.nsplit = pl.nsplit;
  gp.off_part = pl.off_part;
  gp.inv_nchunk = ((1 << 20) + pl.nchunk - 1) / pl.nchunk;
  gp.nphase = pl.nphase;
  for (int i = 0; i < rcp::kMaxPhases; i++) gp.phase[i] = i < pl.nphase ? pl.phase[i] : make_phase(1, 0, 0, 1, 0, pl.nchunk);
  gp.stages = pl.stages;
  // one 32 KB stage per CTA at about 6 TB/s for the whole grid, in SM clocks (about 2 GHz)
  gp.ramp_clk = (int)((double)rcp::kStageBytes * pl.grid / 6.0e12 * 1.9e9);
  gp.off_bar = pl.off_bar; gp.off_T0c = pl.off_T0c; gp.off_scale = pl.off_scale; gp.off_red = pl.off_red;
  gp.off_bs = pl.off_bs;
  gp.bs_bytes = pl.bs_bytes; gp.red_bytes = pl.red_bytes; gp.part_bytes = pl.part_bytes;
  gp.stage_stride = pl.stage_stride;
  gp.off_qbuf = pl.off_qbuf;
  gp.x = nullptr; gp.xq_out = nullptr; gp.scale_out = nullptr; gp.unit_out = nullptr;
  gp.inv_sqrt_b = 1.f; gp.clip_ratio = 1.f;
  if (fa) {
    gp.x = static_cast<const __half*>(fa->x_f16);
    gp.xq_out = fa->xq_out;
    gp.scale_out = static_cast<__half*>(fa->scale_out);
    gp.inv_sqrt_b = (float)(1.0 / std::sqrt((double)fa->B));
    gp.clip_ratio = fa->clip_ratio;
    return grouped ? launch_stream_t<rcp::kModeDp4a, 1, true, true>(maps, gp, pl, st)
                   : launch_stream_t<rcp::kModeDp4a, 1, false, true>(maps, gp, pl, st);
  }
  if (sa) {
    gp.x = static_cast<const __half*>(sa->x_f16);
    gp.xq_out = reinterpret_cast<uint8_t*>(sa->digits_out);
    gp.unit_out = sa->unit_out;
    return launch_stream_t<rcp::kModeMma, 0, false, false, true>(maps, gp, pl, st);
  }
  if (unit) {
    if (pl.nsplit > 1) return launch_stream_t<rcp::kModeMma, 0, false, false, true, true>(maps, gp, pl, st);
    return M > 8 ? launch_stream_t<rcp::kModeMma, 16, false, false, true>(maps, gp, pl, st)
                 : launch_stream_t<rcp::kModeMma, 0, false, false, true>(maps, gp, pl, st);
  }
  if (grouped) {
    if (mode == rcp::kModeDp4a)
      return M == 1 ? launch_stream_t<rcp::kModeDp4a, 1, true>(maps, gp, pl, st)
                    : launch_stream_t<rcp::kModeDp4a, 2, true>(maps, gp, pl, st);
    if (stream_act)
      return gp.S_out ? launch_stream_s<rcp::kModeMma, 0, true, false, false, false, true, true>(maps, gp, pl, st)
                      : launch_stream_s<rcp::kModeMma, 0, true, false, false, false, false, true>(maps, gp, pl, st);
    if (M == 8 && !gp.S_out) return launch_stream_s<rcp::kModeMma, 8, true, false, false, false, false>(maps, gp, pl, st);
    return launch_stream_t<rcp::kModeMma, 0, true>(maps, gp, pl, st);
  }
  if (mode == rcp::kModeHybrid)
    return M == 1 ? launch_stream_t<rcp::kModeHybrid, 1>(maps, gp, pl, st)
                  : launch_stream_t<rcp::kModeHybrid, 2>(maps, gp, pl, st);
  if (mode == rcp::kModeDp4a)
    return M == 1 ? launch_stream_t<rcp::kModeDp4a, 1>(maps, gp, pl, st)
                  : launch_stream_t<rcp::kModeDp4a, 2>(maps, gp, pl, st);
  if (stream_act) {
    if (M == 8 && !gp.S_out) return launch_stream_sb<8>(maps, gp, pl, st);
    return M > 8 ? launch_stream_sb<16>(maps, gp, pl, st) : launch_stream_sb<0>(maps, gp, pl, st);
  }
  if (pl.nsplit > 1) return launch_stream_t<rcp::kModeMma, 0, false, false, false, true>(maps, gp, pl, st);
  if (M == 8 && !gp.S_out) return launch_stream_s<rcp::kModeMma, 8, false, false, false, false, false>(maps, gp, pl, st);   // token count known at compile time
  return M > 8 ? launch_stream_t<rcp::kModeMma, 16>(maps, gp, pl, st) : launch_stream_t<rcp::kModeMma, 0>(maps, gp, pl, st);
}

// All M tokens: as many launches as it takes for the expanded activations to fit (`cap` tokens at most each).
int launch_stream_passes(int mode, int cap, const uint32_t* words, const void* lut_f16, const uint8_t* xq,
                         const void* scale_f16, int M, int N, int K, void* y_f16, void* workspace, cudaStream_t st,
                         bool grouped = false, int32_t* S_out = nullptr) {
  int nsplit = 1;
  const int mp = (grouped || cap < 8) ? tokens_per_pass(M, K, cap) : tokens_and_parts(M, N, K, cap, sm_count(), &nsplit);
  // Where the launch would have to go through K in parts (several tokens, a long K), the form that streams the
  // activations beside the weights is faster (measured: 8192 x 28672 at eight tokens 29.4 against 32.9 us); elsewhere
  // expanding once up front wins, because the expansion competes with the mask arithmetic for the logic pipe.
  if (mode == rcp::kModeMma && !grouped && nsplit > 1 && mp == std::min(M, 8)) {
    const StreamPlan sp = make_plan(mp, N, K, sm_count(), false, 0, 1, true);
    if (sp.stages >= 3 && sp.smem <= kSmemMax) {
      for (int m0 = 0; m0 < M; m0 += mp) {
        const int mm = std::min(mp, M - m0);
        const int rc = launch_stream(mode, words, lut_f16, xq + (size_t)m0 * (K / 2),
                                     static_cast<const __half*>(scale_f16) + m0, mm, N, K,
                                     static_cast<__half*>(y_f16) + (size_t)m0 * N, workspace, st, false, nullptr, nullptr, 1,
                                     nullptr, S_out ? S_out + (size_t)m0 * N * 4 : nullptr, true);
        if (rc != RCP_OK) return rc;
      }
      return RCP_OK;
    }
  }
  // Group-wise grid on the tensor cores, a K so long that not even eight tokens' expanded activations fit: the form
  // with the activations streamed beside the weights takes up to eight tokens in one pass over the weights
  // (8192 x 28672 at eight tokens: one launch instead of two of four tokens).
  if (mode == rcp::kModeMma && grouped && mp < std::min(M, 8)) {
    const int m8 = std::min(M, 8);
    const StreamPlan sp = make_plan(m8, N, K, sm_count(), true, 0, 1, true);
    if (sp.stages >= 3 && sp.smem <= kSmemMax) {
      for (int m0 = 0; m0 < M; m0 += m8) {
        const int mm = std::min(m8, M - m0);
        const int rc = launch_stream(mode, words, lut_f16, xq + (size_t)m0 * (K / 2),
                                     static_cast<const __half*>(scale_f16) + m0, mm, N, K,
                                     static_cast<__half*>(y_f16) + (size_t)m0 * N, workspace, st, true, nullptr, nullptr, 1,
                                     nullptr, S_out ? S_out + (size_t)m0 * N * 4 * (K / 128) : nullptr, true);
        if (rc != RCP_OK) return rc;
      }
      return RCP_OK;
    }
  }
  for (int m0 = 0; m0 < M; m0 += mp) {
    const int mm = std::min(mp, M - m0);
    int md = mode;
    if (md == rcp::kModeHybrid && mm > 2) md = rcp::kModeMma;
    const int rc = launch_stream(md, words, lut_f16, xq + (size_t)m0 * (K / 2),
                                 static_cast<const __half*>(scale_f16) + m0, mm, N, K,
                                 static_cast<__half*>(y_f16) + (size_t)m0 * N, workspace, st, grouped, nullptr, nullptr,
                                 md == rcp::kModeMma ? nsplit : 1, nullptr,
                                 S_out ? S_out + (size_t)m0 * N * 4 * (grouped ? K / 128 : 1) : nullptr);
    if (rc != RCP_OK) return rc;
  }
  return RCP_OK;
}

// ---------------------------------------------------------------------------------------------
// Scratch of rcp_gemv_w2a4_static: part of the device image, one copy per GPU that loads the library.
static __device__ __align__(256) unsigned char g_static_scratch[RCP_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device. In host code the array's name only
// stands for the symbol; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device with that device current and remembered afterwards.
int static_scratch_address(void** out) {
  static std::mutex mu;
  static void* addr[kMaxDevices] = {};
  int dev = 0;
  RCP_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return RCP_ERR_LIMIT;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    RCP_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    addr[dev] = p;
  }
  *out = addr[dev];
  return RCP_OK;
}

template <bool GRP, bool SDBG>
int launch_w3(const rcp::W3Params& wp, size_t smem, cudaStream_t st) {
  static std::mutex mu;
  static bool attr_set[kMaxDevices] = {};
  auto kern = rcp::gemv_w3a4_kernel<GRP, SDBG>;
  int dev = 0;
  RCP_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return RCP_ERR_LIMIT;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
      RCP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, rcp::kMaxK + 128));
      attr_set[dev] = true;
    }
  }
  // One wave of resident CTAs, rows dealt round-robin to their warps (measured: CTAs beyond the resident wave,
  // and warps sharing a row along K, both cost more than the evener load returns).
  int per_sm = 0;
  RCP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, rcp::kW3Threads, smem));
  const int warps_per_cta = rcp::kW3Threads / 32;
  const int grid = std::min(sm_count() * std::max(per_sm, 1), (wp.N + warps_per_cta - 1) / warps_per_cta);
  kern<<<grid, rcp::kW3Threads, smem, st>>>(wp);
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

}  // namespace

extern "C" {

const char* rcp_status_str(int status) {
  switch (status) {
    case RCP_OK: return "ok";
    case RCP_ERR_NULL: return "null pointer";
    case RCP_ERR_SHAPE: return "unsupported shape";
    case RCP_ERR_ALIGN: return "pointer not 16-byte aligned";
    case RCP_ERR_CODE: return "weight code above 3";
    case RCP_ERR_WORKSPACE: return "workspace missing";
    case RCP_ERR_CUDA: return "CUDA error";
    case RCP_ERR_VARIANT: return "kernel variant unknown or not applicable to this shape";
    case RCP_ERR_LIMIT: return "size beyond the entry point's fixed capacity";
    default: return "unknown status";
  }
}

int rcp_last_cuda_error(void) { return g_last_cuda_error; }

int rcp_pack_weights(const uint8_t* codes, int N, int K, uint32_t* words, void* stream) {
  if (!codes || !words) return RCP_ERR_NULL;
  if (N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (!aligned16(codes) || !aligned16(words)) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* bad = nullptr;
  RCP_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&bad), g_pack_bad));
  bad += g_pack_next.fetch_add(1) % kPackSlots;
  RCP_CUDA(cudaMemsetAsync(bad, 0, sizeof(int), st));
  const size_t nwords = (size_t)N * (K / 16);
  const int block = 256;
  const int grid = (int)std::min<size_t>((nwords + block - 1) / block, (size_t)148 * 32);
  rcp::pack_weights_kernel<<<grid, block, 0, st>>>(reinterpret_cast<const uint4*>(codes), nwords, words, bad);
  RCP_CUDA(cudaGetLastError());
  int h_bad = 0;
  RCP_CUDA(cudaMemcpyAsync(&h_bad, bad, sizeof(int), cudaMemcpyDeviceToHost, st));
  RCP_CUDA(cudaStreamSynchronize(st));
  return h_bad ? RCP_ERR_CODE : RCP_OK;
}

int rcp_pack_weights3(const uint8_t* codes, int N, int K, uint32_t* words2, uint32_t* words1, void* stream) {
  if (!codes || !words2 || !words1) return RCP_ERR_NULL;
  if (N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (!aligned16(codes) || !aligned16(words2) || !aligned16(words1)) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* bad = nullptr;
  RCP_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&bad), g_pack_bad));
  bad += g_pack_next.fetch_add(1) % kPackSlots;
  RCP_CUDA(cudaMemsetAsync(bad, 0, sizeof(int), st));
  const size_t nplane = (size_t)N * (K / 32);
  const int block = 256;
  const int grid = (int)std::min<size_t>((nplane + block - 1) / block, (size_t)sm_count() * 32);
  rcp::pack_weights3_kernel<<<grid, block, 0, st>>>(reinterpret_cast<const uint4*>(codes), nplane, words2, words1, bad);
  RCP_CUDA(cudaGetLastError());
  int h_bad = 0;
  RCP_CUDA(cudaMemcpyAsync(&h_bad, bad, sizeof(int), cudaMemcpyDeviceToHost, st));
  RCP_CUDA(cudaStreamSynchronize(st));
  return h_bad ? RCP_ERR_CODE : RCP_OK;
}

int rcp_gemv_w3a4(const uint32_t* words2, const uint32_t* words1, const void* lut_f16, int group, const uint8_t* xq,
                  const void* scale_f16, int M, int N, int K, void* y_f16, int32_t* S_dbg, void* stream) {
  if (!words2 || !words1 || !lut_f16 || !xq || !scale_f16 || !y_f16) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (group != 0 && (group != 128 || K % 128)) return RCP_ERR_SHAPE;
  if (!aligned16(words2) || !aligned16(words1) || !aligned16(lut_f16) || !aligned16(xq) || !aligned16(S_dbg) ||
      (reinterpret_cast<uintptr_t>(y_f16) & 1u) || (reinterpret_cast<uintptr_t>(scale_f16) & 1u))
    return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int ngrp = group ? K / 128 : 1;
  const size_t smem = (size_t)((K / 64 + 63) / 64) * 4096;   // expanded activations, K padded to whole lane steps of 4096 codes
  for (int m = 0; m < M; m++) {   // one token per launch: the variant is tuned for decoding one token
    rcp::W3Params wp;
    wp.words2 = words2; wp.words1 = words1;
    wp.lut = static_cast<const uint4*>(lut_f16);
    wp.xq = xq + (size_t)m * (K / 2);
    wp.scale = static_cast<const __half*>(scale_f16) + m;
    wp.y = static_cast<__half*>(y_f16) + (size_t)m * N;
    wp.S_out = S_dbg ? S_dbg + (size_t)m * N * ngrp * 8 : nullptr;
    wp.N = N; wp.K = K;
    int rc;
    if (group) rc = S_dbg ? launch_w3<true, true>(wp, smem, st) : launch_w3<true, false>(wp, smem, st);
    else rc = S_dbg ? launch_w3<false, true>(wp, smem, st) : launch_w3<false, false>(wp, smem, st);
    if (rc != RCP_OK) return rc;
  }
  return RCP_OK;
}

int rcp_nf3_export(const void* w_f16, const float* sig_beta, const float* sig_gamma, const float* sig_s1,
                   const float* table8_host, int zero_index, int N, int K, int group, uint32_t* words2,
                   uint32_t* words1, void* lut_f16, void* stream) {
  if (!w_f16 || !sig_beta || !sig_gamma || !sig_s1 || !table8_host || !words2 || !words1 || !lut_f16) return RCP_ERR_NULL;
  if (N < 1 || !k_ok(K) || group < 32 || group % 32 || K % group) return RCP_ERR_SHAPE;
  if (zero_index < 0 || zero_index > 7 || table8_host[zero_index] != 0.0f) return RCP_ERR_SHAPE;
  for (int i = 1; i < 8; i++)
    if (!(table8_host[i] > table8_host[i - 1])) return RCP_ERR_SHAPE;   // ascending (and no NaN)
  if (!aligned16(w_f16) || !aligned16(words2) || !aligned16(words1) || !aligned16(lut_f16) ||
      (reinterpret_cast<uintptr_t>(sig_beta) & 3u) || (reinterpret_cast<uintptr_t>(sig_gamma) & 3u) ||
      (reinterpret_cast<uintptr_t>(sig_s1) & 3u))
    return RCP_ERR_ALIGN;
  rcp::Nf3Params np;
  np.w = static_cast<const __half*>(w_f16);
  np.sb = sig_beta; np.sg = sig_gamma; np.s1 = sig_s1;
  np.words2 = words2; np.words1 = words1;
  np.lut = static_cast<uint4*>(lut_f16);
  for (int i = 0; i < 8; i++) np.table[i] = table8_host[i];
  np.zero = zero_index;
  np.N = N; np.K = K; np.G = group;
  np.units = (long long)N * (K / group);
  const int block = 256;
  const long long want = (np.units + (block / 32) - 1) / (block / 32);
  const int grid = (int)std::min<long long>(want, (long long)sm_count() * 16);
  rcp::nf3_export_kernel<<<grid, block, 0, static_cast<cudaStream_t>(stream)>>>(np);
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int rcp_ldp_export(const void* w_f16, const float* sig_beta, const float* sig_gamma, const float* sig_s1,
                   const float* sig_s2, int N, int K, int group, uint32_t* words, void* lut_f16, void* stream) {
  if (!w_f16 || !sig_beta || !sig_gamma || !sig_s1 || !sig_s2 || !words || !lut_f16) return RCP_ERR_NULL;
  if (N < 1 || !k_ok(K) || group < 16 || group % 16 || K % group) return RCP_ERR_SHAPE;
  if (!aligned16(w_f16) || !aligned16(words) || (reinterpret_cast<uintptr_t>(lut_f16) & 7u) ||
      (reinterpret_cast<uintptr_t>(sig_beta) & 3u) || (reinterpret_cast<uintptr_t>(sig_gamma) & 3u) ||
      (reinterpret_cast<uintptr_t>(sig_s1) & 3u) || (reinterpret_cast<uintptr_t>(sig_s2) & 3u))
    return RCP_ERR_ALIGN;
  rcp::LdpParams lp;
  lp.w = static_cast<const __half*>(w_f16);
  lp.sb = sig_beta; lp.sg = sig_gamma; lp.s1 = sig_s1; lp.s2 = sig_s2;
  lp.words = words;
  lp.lut = static_cast<uint2*>(lut_f16);
  lp.N = N; lp.K = K; lp.G = group;
  lp.units = (long long)N * (K / group);
  const int block = 256;
  const long long want = (lp.units + (block / 32) - 1) / (block / 32);
  const int grid = (int)std::min<long long>(want, (long long)sm_count() * 16);
  rcp::ldp_export_kernel<<<grid, block, 0, static_cast<cudaStream_t>(stream)>>>(lp);
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int rcp_quantize_act(const void* x_f16, int M, int K, int had_block, float clip_ratio, uint8_t* xq,
                     void* scale_f16, void* stream) {
  if (!x_f16 || !xq || !scale_f16) return RCP_ERR_NULL;
  if (M < 1 || M > 65535 || !k_ok(K)) return RCP_ERR_SHAPE;
  int B = had_block <= 1 ? 1 : had_block;
  if (B > 8192 || (B & (B - 1)) || K % B) return RCP_ERR_SHAPE;
  if (!(clip_ratio > 0.f) || !std::isfinite(clip_ratio)) return RCP_ERR_SHAPE;
  if (!aligned16(x_f16) || !aligned16(xq) || (reinterpret_cast<uintptr_t>(scale_f16) & 1u)) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // A cluster of C CTAs per token, 8 elements per thread, about 2048 elements per CTA (8192 at most).
  rcp::QuantParams qp;
  qp.x = static_cast<const __half*>(x_f16);
  qp.xq = xq;
  qp.scale = static_cast<__half*>(scale_f16);
  qp.K = K; qp.B = B;
  qp.lgB = 0;
  while ((1 << qp.lgB) < B) qp.lgB++;
  qp.inv_sqrt_b = (float)(1.0 / std::sqrt((double)B));
  qp.clip_ratio = clip_ratio;
  if (B == K && (K == 4096 || K == 8192)) {
    // one rotation block over a long token: one CTA of 512 threads per token (measured faster than a cluster)
    qp.unit = K; qp.nunits = 1; qp.lg_local = qp.lgB;
    RCP_CUDA(launch_overlapped(rcp::quantize_act_wide_kernel, dim3((unsigned)M), dim3(512), rcp::rotate_scratch_bytes(K), st, qp));
    return RCP_OK;
  }
  // whole rotation blocks per CTA (a block is at most 2048 elements here: longer single blocks went above,
  // and B <= 8192 < K otherwise means at least two blocks)
  int C = 1;
  while (C < 8 && K / (2 * C) >= 2048) C *= 2;
  qp.unit = std::max(B, 64);
  qp.nunits = K / qp.unit;
  qp.lg_local = qp.lgB;
  C = std::min(C, qp.nunits);
  while (C > 1 && (C & (C - 1))) C--;   // power of two
  int per = (qp.nunits + C - 1) / C;
  while ((long long)per * qp.unit > 8192 && C < 8) { C *= 2; per = (qp.nunits + C - 1) / C; }
  if ((long long)per * qp.unit > 8192) return RCP_ERR_SHAPE;
  const int T = (per * qp.unit / 8 + 31) / 32 * 32;
  const size_t smem = B > 256 ? (size_t)T * 8 * sizeof(float) : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)M * C);
  cfg.blockDim = dim3(T);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = C;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = C > 1 ? 2 : 1;
  switch (C) {
    case 1: RCP_CUDA(cudaLaunchKernelEx(&cfg, rcp::quantize_act_kernel<1>, qp)); break;
    case 2: RCP_CUDA(cudaLaunchKernelEx(&cfg, rcp::quantize_act_kernel<2>, qp)); break;
    case 4: RCP_CUDA(cudaLaunchKernelEx(&cfg, rcp::quantize_act_kernel<4>, qp)); break;
    default: RCP_CUDA(cudaLaunchKernelEx(&cfg, rcp::quantize_act_kernel<8>, qp)); break;
  }
  return RCP_OK;
}

int rcp_gemv_plan(int M, int N, int K, int sms, int* out, int cap) {
  if (!out && cap > 0) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (sms <= 0) sms = 148;
  int nsplit = 1;
  const int mp = tokens_and_parts(M, N, K, 16, sms, &nsplit);
  const StreamPlan pl = make_plan(mp, N, K, sms, false, 0, nsplit);
  int v[7 + 5 * rcp::kMaxPhases];
  int n = 0;
  v[n++] = mp;
  v[n++] = (M + mp - 1) / mp;
  v[n++] = pl.stages;
  v[n++] = (int)pl.smem;
  v[n++] = pl.nchunk;
  v[n++] = pl.nphase;
  for (int i = 0; i < pl.nphase; i++) {
    v[n++] = pl.phase[i].gpc; v[n++] = pl.phase[i].first; v[n++] = pl.phase[i].total;
    v[n++] = pl.phase[i].ncta; v[n++] = pl.phase[i].reps;
  }
  v[n++] = pl.nsplit;
  for (int i = 0; i < n && i < cap; i++) out[i] = v[i];
  return n;
}

size_t rcp_gemv_workspace_bytes(int M, int N, int K) {
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return 0;
  return 16;   // a status word for the kernels' bounded waits; no sums pass through global memory
}

int rcp_gemv_w2a4_variant(int variant, const uint32_t* words, const void* lut_f16, const uint8_t* xq,
                          const void* scale_f16, int M, int N, int K, void* y_f16, void* workspace,
                          int32_t* S_dbg, void* stream) {
  if (!words || !lut_f16 || !xq || !scale_f16 || !y_f16) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (!aligned16(words) || !aligned16(xq) || !aligned16(S_dbg) ||
      (reinterpret_cast<uintptr_t>(lut_f16) & 7u) || (reinterpret_cast<uintptr_t>(y_f16) & 1u) ||
      (reinterpret_cast<uintptr_t>(scale_f16) & 1u))
    return RCP_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(workspace) & 3u) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // S_dbg without a variant of the caller's choice: the plain kernel. With one: the checked instantiation of
  // that streaming kernel, which stores the sums it finishes its rows from.
  if (S_dbg && variant == RCP_GEMV_AUTO) variant = RCP_GEMV_SIMPLE;
  // measured on B200: one token runs fastest on the CUDA cores alone, more tokens on the tensor cores
  if (variant == RCP_GEMV_AUTO) variant = (M == 1) ? RCP_GEMV_DP4A : RCP_GEMV_MMA_ONLY;
  // the streaming kernels wait on barriers with a bound and report a wait that gave up through the workspace
  if (variant != RCP_GEMV_SIMPLE && !workspace) return RCP_ERR_WORKSPACE;
  switch (variant) {
    case RCP_GEMV_SIMPLE: {
      const int block = 256;
      const int grid = (N + (block / 32) - 1) / (block / 32);
      rcp::gemv_simple_kernel<<<grid, block, 0, st>>>(words, static_cast<const uint2*>(lut_f16), xq,
                                                      static_cast<const __half*>(scale_f16), M, N, K,
                                                      static_cast<__half*>(y_f16), S_dbg);
      break;
    }
    case RCP_GEMV_MMA:
      // tensor-core path; for one or two tokens the b0*b1 plane goes to dp4a (FMA pipe) instead
      return launch_stream_passes(M <= 2 ? rcp::kModeHybrid : rcp::kModeMma, 16, words, lut_f16, xq, scale_f16, M, N, K,
                                  y_f16, workspace, st, false, S_dbg);
    case RCP_GEMV_MMA_ONLY:
      return launch_stream_passes(rcp::kModeMma, 16, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st, false,
                                  S_dbg);
    case RCP_GEMV_DP4A:
      // CUDA-core path: two tokens per launch
      return launch_stream_passes(rcp::kModeDp4a, 2, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st, false,
                                  S_dbg);
    case RCP_GEMV_MMA_STREAM: {
      // tensor-core path with the activations streamed beside the weights: all tokens in one launch, any K
      const StreamPlan pl = make_plan(M, N, K, sm_count(), false, 0, 1, true);
      if (pl.stages < 2 || pl.smem > kSmemMax) return RCP_ERR_VARIANT;
      return launch_stream(rcp::kModeMma, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st, false, nullptr,
                           nullptr, 1, nullptr, S_dbg, true);
    }
    default:
      return RCP_ERR_VARIANT;
  }
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int rcp_gemv_w2a4(const uint32_t* words, const void* lut_f16, const uint8_t* xq, const void* scale_f16,
                  int M, int N, int K, void* y_f16, void* workspace, int32_t* S_dbg, void* stream) {
  return rcp_gemv_w2a4_variant(RCP_GEMV_AUTO, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace,
                               S_dbg, stream);
}

int rcp_gemv_w2a16_checked(const uint32_t* words, const void* lut_f16, const void* x_f16, int M, int N, int K,
                           void* y_f16, int8_t* digits, float* unit, void* workspace, int32_t* S_dbg, void* stream) {
  if (!words || !lut_f16 || !x_f16 || !y_f16 || !digits || !unit) return RCP_ERR_NULL;
  if (!workspace) return RCP_ERR_WORKSPACE;
  if (!aligned16(S_dbg)) return RCP_ERR_ALIGN;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (!aligned16(words) || !aligned16(x_f16) || !aligned16(digits) || (reinterpret_cast<uintptr_t>(lut_f16) & 7u) ||
      (reinterpret_cast<uintptr_t>(y_f16) & 1u) || (reinterpret_cast<uintptr_t>(unit) & 3u) ||
      (reinterpret_cast<uintptr_t>(workspace) & 3u))
    return RCP_ERR_ALIGN;
  // digit columns per launch: sixteen (four tokens) or eight (two) where their expanded bytes fit, else four
  const int cols = 4 * M;
  int nsplit = 1;
  const int cp = tokens_and_parts(std::min(cols, 16), N, K, 16, sm_count(), &nsplit) & ~3;
  if (cp < 4) return RCP_ERR_SHAPE;   // not even the four digit planes of one token fit (very many rows and a long K)
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // One token of up to 16384 elements: one kernel does both steps (every CTA splits its own copy of the
  // activations, held in registers between the search for the largest magnitude and the digits, which costs
  // less than a launch in front of it: measured 0.4 to 1.2 us a call; with two tokens the launch in front won).
  if (M == 1 && nsplit == 1 && cp == cols && K <= 16384 &&
      make_plan(cols, N, K, sm_count(), false, (size_t)cols * K, 1).stages >= 3) {
    const SplitAct sa{x_f16, digits, unit};
    return launch_stream(rcp::kModeMma, words, lut_f16, nullptr, nullptr, cols, N, K, y_f16, workspace, st, false,
                         nullptr, nullptr, 1, &sa, S_dbg);
  }
  RCP_CUDA(launch_overlapped(rcp::split_act16_kernel, dim3(M), dim3(rcp::kSplitThreads), 0, st,
                             static_cast<const __half*>(x_f16), K, digits, unit));
  for (int c0 = 0; c0 < cols; c0 += cp) {
    const int cc = std::min(cp, cols - c0);
    const int rc = launch_stream(rcp::kModeMma, words, lut_f16, reinterpret_cast<const uint8_t*>(digits) + (size_t)c0 * K,
                                 nullptr, cc, N, K, static_cast<__half*>(y_f16) + (size_t)(c0 / 4) * N, workspace, st,
                                 false, nullptr, unit + c0, nsplit, nullptr, S_dbg ? S_dbg + (size_t)c0 * N * 4 : nullptr);
    if (rc != RCP_OK) return rc;
  }
  return RCP_OK;
}

int rcp_gemv_w2a16(const uint32_t* words, const void* lut_f16, const void* x_f16, int M, int N, int K, void* y_f16,
                   int8_t* digits, float* unit, void* workspace, void* stream) {
  return rcp_gemv_w2a16_checked(words, lut_f16, x_f16, M, N, K, y_f16, digits, unit, workspace, nullptr, stream);
}

int rcp_gemv_w2a4_grouped_variant(int variant, const uint32_t* words, const void* lut_f16, int group,
                                  const uint8_t* xq, const void* scale_f16, int M, int N, int K, void* y_f16,
                                  void* workspace, int32_t* S_dbg, void* stream) {
  if (!words || !lut_f16 || !xq || !scale_f16 || !y_f16) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (group < 16 || group % 16 || K % group) return RCP_ERR_SHAPE;
  if (!aligned16(words) || !aligned16(xq) || !aligned16(S_dbg) ||
      (reinterpret_cast<uintptr_t>(lut_f16) & 7u) || (reinterpret_cast<uintptr_t>(y_f16) & 1u) ||
      (reinterpret_cast<uintptr_t>(scale_f16) & 1u))
    return RCP_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(workspace) & 3u) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the streaming kernels are built for the paper's group size; other sizes take the plain kernel
  if (variant == RCP_GEMV_AUTO && (S_dbg || group != 128)) variant = RCP_GEMV_SIMPLE;
  if (variant == RCP_GEMV_AUTO) variant = (M <= 2) ? RCP_GEMV_DP4A : RCP_GEMV_MMA_ONLY;
  if (variant != RCP_GEMV_SIMPLE && !workspace) return RCP_ERR_WORKSPACE;
  switch (variant) {
    case RCP_GEMV_SIMPLE: {
      const int block = 256;
      const int grid = (N + (block / 32) - 1) / (block / 32);
      rcp::gemv_simple_grouped_kernel<<<grid, block, 0, st>>>(words, static_cast<const uint2*>(lut_f16), xq,
                                                              static_cast<const __half*>(scale_f16), M, N, K, group,
                                                              static_cast<__half*>(y_f16), S_dbg);
      break;
    }
    case RCP_GEMV_MMA_ONLY:
      if (group != 128) return RCP_ERR_VARIANT;
      return launch_stream_passes(rcp::kModeMma, 8, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st, true,
                                  S_dbg);
    case RCP_GEMV_DP4A:
      if (group != 128) return RCP_ERR_VARIANT;
      return launch_stream_passes(rcp::kModeDp4a, 2, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st, true,
                                  S_dbg);
    default:
      return RCP_ERR_VARIANT;
  }
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int rcp_gemv_w2a4_grouped(const uint32_t* words, const void* lut_f16, int group, const uint8_t* xq,
                          const void* scale_f16, int M, int N, int K, void* y_f16, void* workspace, int32_t* S_dbg,
                          void* stream) {
  return rcp_gemv_w2a4_grouped_variant(RCP_GEMV_AUTO, words, lut_f16, group, xq, scale_f16, M, N, K, y_f16, workspace,
                                       S_dbg, stream);
}

int rcp_gemv_w2a4_static(const uint32_t* words, const void* lut_f16, const uint8_t* xq, const void* scale_f16,
                         int M, int N, int K, void* y_f16, void* stream) {
  // the same checks as rcp_gemv_w2a4, before anything is put on the stream
  if (!words || !lut_f16 || !xq || !scale_f16 || !y_f16) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  if (!aligned16(words) || !aligned16(xq) || (reinterpret_cast<uintptr_t>(lut_f16) & 7u) ||
      (reinterpret_cast<uintptr_t>(y_f16) & 1u) || (reinterpret_cast<uintptr_t>(scale_f16) & 1u))
    return RCP_ERR_ALIGN;
  const size_t need = rcp_gemv_workspace_bytes(M, N, K);
  if (need > RCP_STATIC_SCRATCH_BYTES) return RCP_ERR_LIMIT;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != RCP_OK) return rc;
  // the array keeps the previous call's contents: clear what this call's kernel expects to be zero
  if (need > 0) RCP_CUDA(cudaMemsetAsync(scratch, 0, need, static_cast<cudaStream_t>(stream)));
  return rcp_gemv_w2a4_variant(RCP_GEMV_AUTO, words, lut_f16, xq, scale_f16, M, N, K, y_f16, scratch, nullptr,
                               stream);
}

int rcp_gemv_w2a4_static_status(int32_t* status_host, void* stream) {
  if (!status_host) return RCP_ERR_NULL;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != RCP_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  RCP_CUDA(cudaMemcpyAsync(status_host, scratch, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  RCP_CUDA(cudaStreamSynchronize(st));
  return RCP_OK;
}

int rcp_selftest_wait_timeout(void* workspace, int polls, void* stream) {
  if (polls < 1 || polls > (1 << 20)) return RCP_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(workspace) & 3u) return RCP_ERR_ALIGN;
  void* status = workspace;
  if (!status) {
    const int rc = static_scratch_address(&status);
    if (rc != RCP_OK) return rc;
  }
  rcp::wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int32_t*>(status), (uint32_t)polls);
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int rcp_linear_w2a4_launches(int M, int N, int K, int had_block, int group) {
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  const int B = had_block <= 1 ? 1 : had_block;
  if (fused_ok(M, K, B) && (group == 0 || group == 128)) return 1;
  if (group != 0 && group != 128) return 2;
  const int cap = group == 0 ? (M == 1 ? 2 : 16) : (M <= 2 ? 2 : 8);   // tokens per launch of the variant AUTO picks
  int nsplit = 1;
  const int mp = (group != 0 || cap < 8) ? tokens_per_pass(M, K, cap) : tokens_and_parts(M, N, K, cap, sm_count(), &nsplit);
  return 1 + (M + mp - 1) / mp;
}

int rcp_linear_w2a4_checked(const void* x_f16, int M, int K, int had_block, float clip_ratio, const uint32_t* words,
                            const void* lut_f16, int group, int N, void* y_f16, uint8_t* xq, void* scale_f16,
                            void* workspace, int32_t* S_dbg, void* stream) {
  if (!x_f16 || !words || !lut_f16 || !y_f16) return RCP_ERR_NULL;
  if (!aligned16(S_dbg)) return RCP_ERR_ALIGN;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  const int B = had_block <= 1 ? 1 : had_block;
  if (B > 8192 || (B & (B - 1)) || K % B) return RCP_ERR_SHAPE;
  if (!(clip_ratio > 0.f) || !std::isfinite(clip_ratio)) return RCP_ERR_SHAPE;
  if (group != 0 && (group < 16 || group % 16 || K % group)) return RCP_ERR_SHAPE;
  if (!aligned16(x_f16) || !aligned16(words) || !aligned16(xq) || (reinterpret_cast<uintptr_t>(lut_f16) & 7u) ||
      (reinterpret_cast<uintptr_t>(y_f16) & 1u) || (reinterpret_cast<uintptr_t>(scale_f16) & 1u) ||
      (reinterpret_cast<uintptr_t>(workspace) & 3u))
    return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!workspace) return RCP_ERR_WORKSPACE;
  if (fused_ok(M, K, B) && (group == 0 || group == 128)) {
    const FusedAct fa{x_f16, B, clip_ratio, xq, scale_f16};
    return launch_stream(rcp::kModeDp4a, words, lut_f16, nullptr, nullptr, M, N, K, y_f16, workspace, st, group == 128,
                         &fa, nullptr, 1, nullptr, S_dbg);
  }
  // otherwise the two kernels one after the other; they need the staging buffers
  if (!xq || !scale_f16) return RCP_ERR_NULL;
  int rc = rcp_quantize_act(x_f16, M, K, had_block, clip_ratio, xq, scale_f16, stream);
  if (rc != RCP_OK) return rc;
  // with S_dbg: the streaming kernel AUTO would pick, in its checked instantiation
  if (group == 0)
    return rcp_gemv_w2a4_variant(S_dbg ? (M == 1 ? RCP_GEMV_DP4A : RCP_GEMV_MMA_ONLY) : RCP_GEMV_AUTO, words, lut_f16, xq,
                                 scale_f16, M, N, K, y_f16, workspace, S_dbg, stream);
  return rcp_gemv_w2a4_grouped_variant(S_dbg && group == 128 ? (M <= 2 ? RCP_GEMV_DP4A : RCP_GEMV_MMA_ONLY) : RCP_GEMV_AUTO,
                                       words, lut_f16, group, xq, scale_f16, M, N, K, y_f16, workspace, S_dbg, stream);
}

int rcp_linear_w2a4(const void* x_f16, int M, int K, int had_block, float clip_ratio, const uint32_t* words,
                    const void* lut_f16, int group, int N, void* y_f16, uint8_t* xq, void* scale_f16, void* workspace,
                    void* stream) {
  return rcp_linear_w2a4_checked(x_f16, M, K, had_block, clip_ratio, words, lut_f16, group, N, y_f16, xq, scale_f16,
                                 workspace, nullptr, stream);
}

int rcp_linear_w2a4_host(const void* x_host_f16, int M, int K, int had_block, float clip_ratio,
                         const uint32_t* words, const void* lut_f16, int N, void* y_host_f16, void* x_dev,
                         uint8_t* xq_dev, void* scale_dev, void* y_dev, void* workspace, void* stream) {
  if (!x_host_f16 || !y_host_f16 || !x_dev || !y_dev) return RCP_ERR_NULL;   // staging is needed for pageable memory
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Page-locked host memory is visible to the GPU: the quantizer (a handful of CTAs) then reads the
  // few kilobytes of activations straight from it, which saves a trip through the copy engine. The
  // single-kernel form would have every CTA fetch them across the bus, so it is not used here.
  cudaPointerAttributes attr;
  const void* x_mapped = nullptr;
  if (xq_dev && scale_dev && cudaPointerGetAttributes(&attr, x_host_f16) == cudaSuccess &&
      attr.type == cudaMemoryTypeHost && attr.devicePointer && aligned16(attr.devicePointer))
    x_mapped = attr.devicePointer;
  else
    (void)cudaGetLastError();   // an unregistered pointer is not an error here
  // Likewise the GEMV can store its few kilobytes of results straight into page-locked host memory.
  void* y_mapped = nullptr;
  if (cudaPointerGetAttributes(&attr, y_host_f16) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
      attr.devicePointer)
    y_mapped = attr.devicePointer;
  else
    (void)cudaGetLastError();
  void* const y_out = y_mapped ? y_mapped : y_dev;
  int rc;
  if (x_mapped) {
    rc = rcp_quantize_act(x_mapped, M, K, had_block, clip_ratio, xq_dev, scale_dev, stream);
    if (rc == RCP_OK)
      rc = rcp_gemv_w2a4(words, lut_f16, xq_dev, scale_dev, M, N, K, y_out, workspace, nullptr, stream);
  } else {
    RCP_CUDA(cudaMemcpyAsync(x_dev, x_host_f16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st));
    rc = rcp_linear_w2a4(x_dev, M, K, had_block, clip_ratio, words, lut_f16, 0, N, y_out, xq_dev, scale_dev, workspace,
                         stream);
  }
  if (rc != RCP_OK) return rc;
  if (!y_mapped) RCP_CUDA(cudaMemcpyAsync(y_host_f16, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st));
  return RCP_OK;
}

}  // extern "C"
