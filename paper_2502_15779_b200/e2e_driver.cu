// End-to-end decode step through the C ABI from a C++ host program (no interpreter in the loop): the four
// linears of a decoder layer, activations in page-locked host memory, results read back on the host after
// every step. Prints one JSON object. Used by bench.py beside its own end-to-end loop to show what part of
// that loop's time belongs to the Python binding.
//   e2e_driver <steps> <warmup> N1 K1 B1  N2 K2 B2 ...        (B: rotation block of the layer's input)
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <random>
#include <vector>

#include "../include/rcp.h"

#define CK(x) do { cudaError_t e__ = (x); if (e__ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e__)); return 2; } } while (0)

struct Layer {
  int N, K, B;
  uint32_t* words; __half* lut; __half* x_dev; uint8_t* xq; __half* scale; __half* y_dev; void* ws;
  __half* x_host; __half* y_host;
};

int main(int argc, char** argv) {
  if (argc < 6 || (argc - 3) % 3) { fprintf(stderr, "usage: e2e_driver steps warmup N K B ...\n"); return 1; }
  const int steps = atoi(argv[1]), warmup = atoi(argv[2]);
  std::vector<Layer> layers;
  std::mt19937 rng(250215779u);
  double bytes = 0;
  for (int a = 3; a + 2 < argc; a += 3) {
    Layer L{};
    L.N = atoi(argv[a]); L.K = atoi(argv[a + 1]); L.B = atoi(argv[a + 2]);
    const size_t nw = (size_t)L.N * (L.K / 16);
    std::vector<uint32_t> w(nw);
    for (auto& v : w) v = rng();
    std::vector<__half> lut((size_t)L.N * 4);
    for (size_t i = 0; i < lut.size(); i += 4) {
      float l[4];
      for (float& v : l) v = 0.02f * std::normal_distribution<float>()(rng);
      std::sort(l, l + 4);
      for (int c = 0; c < 4; c++) lut[i + c] = __float2half(l[c]);
    }
    CK(cudaMalloc(&L.words, nw * 4)); CK(cudaMemcpy(L.words, w.data(), nw * 4, cudaMemcpyHostToDevice));
    CK(cudaMalloc(&L.lut, lut.size() * 2)); CK(cudaMemcpy(L.lut, lut.data(), lut.size() * 2, cudaMemcpyHostToDevice));
    CK(cudaMalloc(&L.x_dev, (size_t)L.K * 2)); CK(cudaMalloc(&L.xq, L.K / 2)); CK(cudaMalloc(&L.scale, 2));
    CK(cudaMalloc(&L.y_dev, (size_t)L.N * 2));
    const size_t wsb = rcp_gemv_workspace_bytes(1, L.N, L.K);
    CK(cudaMalloc(&L.ws, wsb ? wsb : 16)); CK(cudaMemset(L.ws, 0, wsb ? wsb : 16));
    CK(cudaMallocHost(&L.x_host, (size_t)L.K * 2)); CK(cudaMallocHost(&L.y_host, (size_t)L.N * 2));
    for (int k = 0; k < L.K; k++) L.x_host[k] = __float2half(std::normal_distribution<float>()(rng));
    bytes += (double)L.N * L.K / 4 + 8.0 * L.N + L.K / 2 + 2.0 * L.N + 2.0 * L.K + 0.5 * L.K + 2;   // GEMV + quantizer bytes
    layers.push_back(L);
  }
  cudaStream_t st;
  CK(cudaStreamCreate(&st));
  auto step = [&]() -> int {
    for (auto& L : layers) {
      const int rc = rcp_linear_w2a4_host(L.x_host, 1, L.K, L.B, 1.0f, L.words, L.lut, L.N, L.y_host, L.x_dev, L.xq, L.scale,
                                          L.y_dev, L.ws, st);
      if (rc != RCP_OK) { fprintf(stderr, "rcp_linear_w2a4_host: %s\n", rcp_status_str(rc)); return rc; }
    }
    return cudaStreamSynchronize(st) == cudaSuccess ? 0 : -1;   // the host reads y before the next step
  };
  for (int i = 0; i < warmup; i++) if (step()) return 3;
  float checksum = 0.f;
  const auto t0 = std::chrono::steady_clock::now();
  for (int i = 0; i < steps; i++) {
    if (step()) return 3;
    checksum += __half2float(layers[0].y_host[i % layers[0].N]);
  }
  const auto t1 = std::chrono::steady_clock::now();
  const double us = std::chrono::duration<double, std::micro>(t1 - t0).count() / steps;
  printf("{\"steps\": %d, \"us_per_step\": %.3f, \"gbs\": %.2f, \"checksum\": %.6g}\n", steps, us, bytes / us / 1e3, checksum);
  return 0;
}
