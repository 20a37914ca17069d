// C ABI of the RCP W2A4 library: argument validation, launch configuration, status codes.
#include "../../include/rcp.h"

#include <cmath>

#include "common.cuh"
#include "gemv_simple.cuh"
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
  return 0;
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
  (void)workspace;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (S_dbg) variant = RCP_GEMV_SIMPLE;
  if (variant == RCP_GEMV_AUTO) variant = RCP_GEMV_SIMPLE;
  switch (variant) {
    case RCP_GEMV_SIMPLE: {
      const int block = 256;
      const int grid = (N + (block / 32) - 1) / (block / 32);
      rcp::gemv_simple_kernel<<<grid, block, 0, st>>>(words, static_cast<const uint2*>(lut_f16), xq,
                                                      static_cast<const __half*>(scale_f16), M, N, K,
                                                      static_cast<__half*>(y_f16), S_dbg);
      break;
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

}  // extern "C"
