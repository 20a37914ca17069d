// Rate and fragment layout of the binary tensor-core instruction (mma.sync m16n8k256 .b1, and.popc) on this GPU.
// With bit planes of the weights as A and bit planes of the int4 activations as B, three of these per KB of packed
// weights would replace all masks and dot products of the GEMV; the question is what one costs.
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <algorithm>

__device__ __forceinline__ void bmma(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// the 4-bit integer form (m16n8k64, u4 x s4): codes masked per nibble would halve the masks and take the int4
// activations as they are packed
__device__ __forceinline__ void imma4(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k64.row.col.s32.u4.s4.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NA, bool I4 = false>
__global__ void __launch_bounds__(512, 1) rate_kernel(uint32_t seed, int iters, int* sink, long long* clk) {
  int acc[NA][4];
#pragma unroll
  for (int a = 0; a < NA; a++)
#pragma unroll
    for (int r = 0; r < 4; r++) acc[a][r] = 0;
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; i++) w[i] = seed * (threadIdx.x + 1 + i);
  const uint32_t b0 = seed | 1, b1 = seed | 2;
  __syncthreads();
  const long long t0 = clock64();
  for (int it = 0; it < iters; it++) {
#pragma unroll
    for (int a = 0; a < NA; a++) {
      if (I4) imma4(acc[a], w[0], w[1], w[2], w[3], b0, b1);
      else bmma(acc[a], w[0], w[1], w[2], w[3], b0, b1);
    }
  }
  const long long t1 = clock64();
  int s = 0;
#pragma unroll
  for (int a = 0; a < NA; a++)
#pragma unroll
    for (int r = 0; r < 4; r++) s += acc[a][r];
  if (s == 0x12345678) sink[0] = s;
  if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}

// layout check: A [16][256] bits, B [8][256] bits; lane (g = lane >> 2, t = lane & 3)
__global__ void layout_kernel(const uint32_t* A, const uint32_t* B, int* D) {
  const int lane = threadIdx.x, g = lane >> 2, t = lane & 3;
  // A row r: 8 words; candidate layout: a0 = A[g][t], a1 = A[g+8][t], a2 = A[g][4+t], a3 = A[g+8][4+t]; b0 = B[g][t], b1 = B[g][4+t]
  int d[4] = {0, 0, 0, 0};
  bmma(d, A[g * 8 + t], A[(g + 8) * 8 + t], A[g * 8 + 4 + t], A[(g + 8) * 8 + 4 + t], B[g * 8 + t], B[g * 8 + 4 + t]);
  D[g * 8 + 2 * t] = d[0];
  D[g * 8 + 2 * t + 1] = d[1];
  D[(g + 8) * 8 + 2 * t] = d[2];
  D[(g + 8) * 8 + 2 * t + 1] = d[3];
}

template <int NA, bool I4 = false>
void run(int iters) {
  int* sink; long long* clk;
  cudaMalloc(&sink, 4); cudaMalloc(&clk, 148 * 8);
  rate_kernel<NA, I4><<<148, 512>>>(12345u, iters, sink, clk);
  cudaDeviceSynchronize();
  rate_kernel<NA, I4><<<148, 512>>>(12345u, iters, sink, clk);
  cudaError_t e = cudaDeviceSynchronize();
  std::vector<long long> h(148);
  cudaMemcpy(h.data(), clk, 148 * 8, cudaMemcpyDeviceToHost);
  long long mx = 0;
  for (auto v : h) mx = std::max(mx, v);
  const double per = (double)mx / iters / (16.0 * NA);   // clocks per instruction and SM (16 warps issue NA each per iteration)
  if (I4) printf("u4 x s4 m16n8k64  NA=%d  %s  clk per mma per SM %.3f\n", NA, cudaGetErrorString(e), per);
  else printf("b1 m16n8k256     NA=%d  %s  clk per mma per SM %.3f  (%.0f bit products per clk per SM)\n", NA, cudaGetErrorString(e), per, 16.0 * 8 * 256 / per);
  cudaFree(sink); cudaFree(clk);
}

int main() {
  // layout
  std::vector<uint32_t> A(16 * 8), B(8 * 8);
  srand(7);
  for (auto& v : A) v = (uint32_t)rand() * 2654435761u ^ (uint32_t)rand();
  for (auto& v : B) v = (uint32_t)rand() * 2246822519u ^ (uint32_t)rand();
  uint32_t *dA, *dB; int* dD;
  cudaMalloc(&dA, A.size() * 4); cudaMalloc(&dB, B.size() * 4); cudaMalloc(&dD, 16 * 8 * 4);
  cudaMemcpy(dA, A.data(), A.size() * 4, cudaMemcpyHostToDevice);
  cudaMemcpy(dB, B.data(), B.size() * 4, cudaMemcpyHostToDevice);
  layout_kernel<<<1, 32>>>(dA, dB, dD);
  cudaError_t e = cudaDeviceSynchronize();
  std::vector<int> D(16 * 8);
  cudaMemcpy(D.data(), dD, D.size() * 4, cudaMemcpyDeviceToHost);
  int bad = 0;
  for (int r = 0; r < 16; r++)
    for (int n = 0; n < 8; n++) {
      int ref = 0;
      for (int w = 0; w < 8; w++) ref += __builtin_popcount(A[r * 8 + w] & B[n * 8 + w]);
      if (ref != D[r * 8 + n]) bad++;
    }
  printf("layout check: %s, %d mismatches of 128\n", cudaGetErrorString(e), bad);
  run<1>(20000); run<2>(20000); run<3>(20000); run<6>(10000); run<12>(5000);
  run<1, true>(20000); run<3, true>(20000); run<6, true>(10000);
  return 0;
}
