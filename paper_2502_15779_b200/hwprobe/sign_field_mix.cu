// Instruction mix of the "two-bit field under the sign bit" formulation: per 4 words (rows g, g+8 x 2 k-words)
// 12 shifts + 16 adds + 32 logic ops + 12 int8 MMAs (u8 and s8 reading of the field, u8 of the product bit).
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdio>
#include <vector>
__device__ __forceinline__ void mma_u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// SH: 0 = C shifts (compiler's choice), 1 = multiply by a run-time power of two (IMAD)
// ZV: 0 = Z = F & (F + F); 1 = Z = lop3(w_p, w_p + w_p, 0x80808080)
template <int SH, int ZV>
__global__ void __launch_bounds__(512, 1) mix_kernel(const uint32_t* __restrict__ src, int iters, uint32_t m4, uint32_t m16,
                                                     uint32_t m64, int* sink, long long* clk) {
  __shared__ uint32_t sw[512 * 4];
  for (int i = threadIdx.x; i < 2048; i += 512) sw[i] = src[i];
  __syncthreads();
  int aU[4] = {0, 0, 0, 0}, aS[4] = {0, 0, 0, 0}, aZ[4] = {0, 0, 0, 0};
  const uint32_t b0 = 0x01020304u, b1 = 0x05060708u;
  const long long t0 = clock64();
  for (int it = 0; it < iters; it++) {
    const uint4 W = *reinterpret_cast<const uint4*>(&sw[((threadIdx.x + it) & 511) * 4]);
    const uint32_t w[4] = {W.x, W.y, W.z, W.w};
    uint32_t F[4][4], Z[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
      uint32_t s[4];
      s[3] = w[i];
      if (SH == 0) { s[2] = w[i] << 2; s[1] = w[i] << 4; s[0] = w[i] << 6; }
      else { s[2] = w[i] * m4; s[1] = w[i] * m16; s[0] = w[i] * m64; }
#pragma unroll
      for (int p = 0; p < 4; p++) {
        F[p][i] = s[p] & 0xC0C0C0C0u;
        if (ZV == 0) Z[p][i] = F[p][i] & (F[p][i] + F[p][i]);
        else asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(Z[p][i]) : "r"(s[p]), "r"(s[p] + s[p]), "r"(0x80808080u));
      }
    }
#pragma unroll
    for (int p = 0; p < 4; p++) {
      mma_u8(aU, F[p][0], F[p][1], F[p][2], F[p][3], b0, b1);
      mma_s8(aS, F[p][0], F[p][1], F[p][2], F[p][3], b0, b1);
      mma_u8(aZ, Z[p][0], Z[p][1], Z[p][2], Z[p][3], b0, b1);
    }
  }
  const long long t1 = clock64();
  int s = 0;
  for (int r = 0; r < 4; r++) s += aU[r] + aS[r] + aZ[r];
  if (s == 0x12345678) sink[0] = s;
  if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}
template <int SH, int ZV>
void run(const char* name, int iters, const uint32_t* src) {
  int* sink; long long* clk;
  cudaMalloc(&sink, 4); cudaMalloc(&clk, 148 * 8);
  mix_kernel<SH, ZV><<<148, 512>>>(src, iters, 4u, 16u, 64u, sink, clk);
  cudaDeviceSynchronize();
  mix_kernel<SH, ZV><<<148, 512>>>(src, iters, 4u, 16u, 64u, sink, clk);
  cudaError_t e = cudaDeviceSynchronize();
  std::vector<long long> h(148);
  cudaMemcpy(h.data(), clk, 148 * 8, cudaMemcpyDeviceToHost);
  long long mx = 0; for (auto v : h) mx = std::max(mx, v);
  // one warp-iteration = 4 word-sets = 512 B of weights; 16 warps -> 8 KB per SM-iteration
  printf("%-60s %s  %.1f clk per SM-iteration = %.1f clk per KB\n", name, cudaGetErrorString(e), (double)mx / iters, (double)mx / iters / 8.0);
}
int main() {
  std::vector<uint32_t> h(2048);
  for (size_t i = 0; i < h.size(); i++) h[i] = 2654435761u * (uint32_t)(i + 1);
  uint32_t* src; cudaMalloc(&src, 8192); cudaMemcpy(src, h.data(), 8192, cudaMemcpyHostToDevice);
  run<0, 0>("shifts by <<, Z = F & 2F", 20000, src);
  run<1, 0>("shifts by multiply, Z = F & 2F", 20000, src);
  run<0, 1>("shifts by <<, Z = lop3(s, 2s, 0x80..)", 20000, src);
  run<1, 1>("shifts by multiply, Z = lop3(s, 2s, 0x80..)", 20000, src);
  return 0;
}
