// C ABI of the RCP W2A4 library: argument validation, launch configuration, status codes.
#include "../../include/rcp.h"

#include <algorithm>
#include <cmath>
#include <mutex>

#include "common.cuh"
#include "gemv_simple.cuh"
#include "gemv_stream.cuh"
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

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool k_ok(int K) { return K >= 64 && K <= rcp::kMaxK && K % 64 == 0; }

__device__ int g_pack_bad;  // set by pack_weights_kernel when it meets a code above 3

// ---------------------------------------------------------------------------------------------
// Streaming GEMV: launch plan shared by rcp_gemv_workspace_bytes and the launcher.
struct StreamPlan {
  int ntiles, spt_all, sps, supers, stages;
  int off_bar, off_T0st, off_T0, off_scale, off_bs;
  size_t smem, ws_count_off, ws_T0_off, ws_sum_off, ws_bytes;
};

constexpr size_t kSmemMax = 232448;           // 227 KB of dynamic shared memory per CTA on sm_100
constexpr size_t kExpandBudget = 96 * 1024;   // expanded activations kept resident per CTA

StreamPlan make_plan(int M, int N, int K) {
  StreamPlan pl;
  pl.ntiles = (N + rcp::kTileRows - 1) / rcp::kTileRows;
  pl.spt_all = (K / 16 + rcp::kStageWords - 1) / rcp::kStageWords;
  // expanded activations: one byte per code and token, 512 M bytes per stage; K ranges whose
  // activations fit in shared memory go to different blockIdx.y
  const size_t bs_per_stage = (size_t)rcp::kStageWords * 16 * M;
  int sps = (int)std::min<size_t>(rcp::kMaxSps, std::max<size_t>(1, kExpandBudget / bs_per_stage));
  sps = std::min(sps, pl.spt_all);
  pl.supers = (pl.spt_all + sps - 1) / sps;
  pl.sps = (pl.spt_all + pl.supers - 1) / pl.supers;
  const size_t bs_bytes = (size_t)pl.sps * bs_per_stage;
  const size_t misc = 256 + (size_t)M * rcp::kMaxSps * 4 + 64 + 64;
  pl.stages = (int)std::min<size_t>(rcp::kMaxStages, (kSmemMax - 1024 - misc - bs_bytes) / rcp::kStageBytes);
  size_t off = (size_t)pl.stages * rcp::kStageBytes;
  pl.off_bar = (int)off; off += 256;
  pl.off_T0st = (int)off; off += (size_t)M * rcp::kMaxSps * 4;
  pl.off_T0 = (int)off; off += 64;
  pl.off_scale = (int)off; off += 64;
  pl.off_bs = (int)off; off += bs_bytes;
  pl.smem = off + 1024;
  pl.ws_count_off = 16;
  pl.ws_T0_off = pl.ws_count_off + (((size_t)pl.ntiles * 4 + 15) / 16) * 16;
  pl.ws_sum_off = pl.ws_T0_off + (((size_t)pl.ntiles * M * 4 + 15) / 16) * 16;
  pl.ws_bytes = pl.ws_sum_off + (size_t)pl.ntiles * rcp::kTileRows * M * 3 * 4;
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

int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      n = 148;
  }
  return n;
}

template <int MT, int MODE, int MTOK>
int launch_stream_t(const CUtensorMap& map, const rcp::GemvParams& gp, const StreamPlan& pl, cudaStream_t st) {
  static bool attr_set = false;
  auto kern = rcp::gemv_stream_kernel<MT, MODE, MTOK>;
  if (!attr_set) {
    RCP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax));
    attr_set = true;
  }
  const int gx = std::max(1, sm_count() / pl.supers);
  kern<<<dim3(gx, pl.supers), rcp::kGThreads, pl.smem, st>>>(map, gp);
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

int launch_stream(int mode, const uint32_t* words, const void* lut_f16, const uint8_t* xq, const void* scale_f16,
                  int M, int N, int K, void* y_f16, void* workspace, cudaStream_t st) {
  if (!workspace) return RCP_ERR_WORKSPACE;
  if (!aligned16(workspace)) return RCP_ERR_ALIGN;
  if (mode != rcp::kModeMma && M > 2) return RCP_ERR_VARIANT;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return cuda_fail(cudaErrorNotSupported);
  const StreamPlan pl = make_plan(M, N, K);
  if (pl.stages < 2 || pl.smem > kSmemMax) return RCP_ERR_SHAPE;
  CUtensorMap map;
  const cuuint64_t gdim[2] = {(cuuint64_t)(K / 16), (cuuint64_t)N};
  const cuuint64_t gstride[1] = {(cuuint64_t)(K / 4)};
  const cuuint32_t box[2] = {(cuuint32_t)rcp::kStageWords, (cuuint32_t)rcp::kTileRows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(words), gdim, gstride, box,
                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);
  rcp::GemvParams gp;
  gp.lut = static_cast<const uint2*>(lut_f16);
  gp.xq = xq;
  gp.scale = static_cast<const __half*>(scale_f16);
  gp.y = static_cast<__half*>(y_f16);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  gp.ws_status = reinterpret_cast<int32_t*>(ws);
  gp.ws_count = reinterpret_cast<uint32_t*>(ws + pl.ws_count_off);
  gp.ws_T0 = reinterpret_cast<int32_t*>(ws + pl.ws_T0_off);
  gp.ws_sum = reinterpret_cast<int32_t*>(ws + pl.ws_sum_off);
  gp.M = M; gp.N = N; gp.K = K;
  gp.ntiles = pl.ntiles; gp.spt_all = pl.spt_all; gp.sps = pl.sps; gp.stages = pl.stages;
  gp.off_bar = pl.off_bar; gp.off_T0st = pl.off_T0st; gp.off_T0 = pl.off_T0; gp.off_scale = pl.off_scale;
  gp.off_bs = pl.off_bs;
  if (mode == rcp::kModeHybrid)
    return M == 1 ? launch_stream_t<1, rcp::kModeHybrid, 1>(map, gp, pl, st)
                  : launch_stream_t<1, rcp::kModeHybrid, 2>(map, gp, pl, st);
  if (mode == rcp::kModeDp4a)
    return M == 1 ? launch_stream_t<1, rcp::kModeDp4a, 1>(map, gp, pl, st)
                  : launch_stream_t<1, rcp::kModeDp4a, 2>(map, gp, pl, st);
  if (M <= 8) return launch_stream_t<1, rcp::kModeMma, 0>(map, gp, pl, st);
  return launch_stream_t<2, rcp::kModeMma, 0>(map, gp, pl, st);
}

// ---------------------------------------------------------------------------------------------
// Scratch of rcp_gemv_w2a4_static: part of the device image, one copy per GPU that loads the library.
static __device__ __align__(256) unsigned char g_static_scratch[RCP_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device. In host code the array's name only
// stands for the symbol; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device with that device current and remembered afterwards.
int static_scratch_address(void** out) {
  constexpr int kMaxDevices = 64;
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

int rcp_quantize_act(const void* x_f16, int M, int K, int had_block, float clip_ratio, uint8_t* xq,
                     void* scale_f16, void* stream) {
  if (!x_f16 || !xq || !scale_f16) return RCP_ERR_NULL;
  if (M < 1 || M > 65535 || !k_ok(K)) return RCP_ERR_SHAPE;
  int B = had_block <= 1 ? 1 : had_block;
  if (B > 8192 || (B & (B - 1)) || K % B) return RCP_ERR_SHAPE;
  if (!(clip_ratio > 0.f) || !std::isfinite(clip_ratio)) return RCP_ERR_SHAPE;
  if (!aligned16(x_f16) || !aligned16(xq) || (reinterpret_cast<uintptr_t>(scale_f16) & 1u)) return RCP_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // Threads: 8 elements each. The thread count is a multiple of one warp (blocks up to 256 stay
  // inside a warp) and of B/8 (larger blocks exchange through shared memory inside the CTA).
  const int unit = B > 256 ? B / 8 : 32;
  int T = ((K / 8 + unit - 1) / unit) * unit;
  if (T > 1024) T = (1024 / unit) * unit;
  const int G = (K / 8 + T - 1) / T;
  const size_t smem = B > 256 ? (size_t)T * 8 * sizeof(float) : 0;
  const float inv_sqrt_b = (float)(1.0 / std::sqrt((double)B));
  const __half* x = static_cast<const __half*>(x_f16);
  __half* sc = static_cast<__half*>(scale_f16);
#define RCP_LAUNCH_Q(GG) \
  rcp::quantize_act_kernel<GG><<<M, T, smem, st>>>(x, K, B, inv_sqrt_b, clip_ratio, xq, sc)
  if (G <= 1) RCP_LAUNCH_Q(1);
  else if (G <= 2) RCP_LAUNCH_Q(2);
  else if (G <= 4) RCP_LAUNCH_Q(4);
  else if (G <= 8) RCP_LAUNCH_Q(8);
  else return RCP_ERR_SHAPE;
#undef RCP_LAUNCH_Q
  RCP_CUDA(cudaGetLastError());
  return RCP_OK;
}

size_t rcp_gemv_workspace_bytes(int M, int N, int K) {
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return 0;
  // the layout grows with M, and the CUDA-core variant runs the tokens in pairs on the same scratch
  return make_plan(M, N, K).ws_bytes;
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
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (S_dbg) variant = RCP_GEMV_SIMPLE;
  if (variant == RCP_GEMV_AUTO) variant = RCP_GEMV_MMA;
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
      return launch_stream(M <= 2 ? rcp::kModeHybrid : rcp::kModeMma, words, lut_f16, xq, scale_f16, M, N, K, y_f16,
                           workspace, st);
    case RCP_GEMV_MMA_ONLY:
      return launch_stream(rcp::kModeMma, words, lut_f16, xq, scale_f16, M, N, K, y_f16, workspace, st);
    case RCP_GEMV_DP4A: {
      // CUDA-core path: two tokens per launch
      for (int m0 = 0; m0 < M; m0 += 2) {
        const int mm = std::min(2, M - m0);
        // later token pairs reuse the same scratch: it is left zeroed by the previous launch
        const int rc = launch_stream(rcp::kModeDp4a, words, lut_f16, xq + (size_t)m0 * (K / 2),
                                     static_cast<const __half*>(scale_f16) + m0, mm, N, K,
                                     static_cast<__half*>(y_f16) + (size_t)m0 * N, workspace, st);
        if (rc != RCP_OK) return rc;
      }
      return RCP_OK;
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

int rcp_gemv_w2a4_static(const uint32_t* words, const void* lut_f16, const uint8_t* xq, const void* scale_f16,
                         int M, int N, int K, void* y_f16, void* stream) {
  const size_t need = rcp_gemv_workspace_bytes(M, N, K);   // 0 on a bad shape: reported by the call below
  if (need > RCP_STATIC_SCRATCH_BYTES) return RCP_ERR_LIMIT;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != RCP_OK) return rc;
  // the array keeps the previous call's contents: clear what this call's kernel expects to be zero
  if (need > 0) RCP_CUDA(cudaMemsetAsync(scratch, 0, need, static_cast<cudaStream_t>(stream)));
  return rcp_gemv_w2a4_variant(RCP_GEMV_AUTO, words, lut_f16, xq, scale_f16, M, N, K, y_f16, scratch, nullptr,
                               stream);
}

int rcp_linear_w2a4_host(const void* x_host_f16, int M, int K, int had_block, float clip_ratio,
                         const uint32_t* words, const void* lut_f16, int N, void* y_host_f16, void* x_dev,
                         uint8_t* xq_dev, void* scale_dev, void* y_dev, void* workspace, void* stream) {
  if (!x_host_f16 || !y_host_f16 || !x_dev || !y_dev) return RCP_ERR_NULL;
  if (M < 1 || M > rcp::kMaxTokens || N < 1 || !k_ok(K)) return RCP_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  RCP_CUDA(cudaMemcpyAsync(x_dev, x_host_f16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st));
  int rc = rcp_quantize_act(x_dev, M, K, had_block, clip_ratio, xq_dev, scale_dev, stream);
  if (rc != RCP_OK) return rc;
  rc = rcp_gemv_w2a4(words, lut_f16, xq_dev, scale_dev, M, N, K, y_dev, workspace, nullptr, stream);
  if (rc != RCP_OK) return rc;
  RCP_CUDA(cudaMemcpyAsync(y_host_f16, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st));
  return RCP_OK;
}

}  // extern "C"
