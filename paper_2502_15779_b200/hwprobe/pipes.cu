// Issue-rate experiments on one SM-filling grid: does int8 mma.sync overlap with LOP3 (a) from other warps of
// the same scheduler, (b) inside one warp with and without a dependency between the masks and the MMA.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lop(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm volatile("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ void dp4a(int& d, uint32_t a, uint32_t b) {
  asm volatile("dp4a.u32.s32 %0, %1, %2, %0;" : "+r"(d) : "r"(a), "r"(b));
}

// mode 0: every warp LOP3 only (NL independent chains)
// mode 1: every warp MMA only (NA independent accumulators)
// mode 2: even warps LOP3 only, odd warps MMA only
// mode 3: every warp: per iteration 12 LOP3 then 3 MMA, MMA operands do NOT depend on the LOP3 results
// mode 4: as 3 but the MMA operands are the LOP3 results of the same iteration
// mode 5: as 4 but the MMAs of iteration i use the masks made in iteration i-1 (software pipelined)
// mode 6: every warp dp4a only;  mode 7: 12 LOP3 + 12 dp4a dependent (the CUDA-core kernel's body)
template <int MODE, int NA>
__global__ void __launch_bounds__(512, 1) pipes_kernel(uint32_t seed, int iters, int* sink, long long* clk) {
  const int warp = threadIdx.x >> 5;
  uint32_t w[4], m[12], mp[12];
  int acc[NA][4];
#pragma unroll
  for (int i = 0; i < 4; i++) w[i] = seed * (threadIdx.x + 1 + i);
#pragma unroll
  for (int i = 0; i < 12; i++) { m[i] = seed + i; mp[i] = seed ^ i; }
#pragma unroll
  for (int a = 0; a < NA; a++)
#pragma unroll
    for (int r = 0; r < 4; r++) acc[a][r] = 0;
  const uint32_t b0 = seed | 1, b1 = seed | 2;
  __syncthreads();
  const long long t0 = clock64();
  for (int it0 = 0; it0 < iters; it0 += NA / 3) {
#pragma unroll
  for (int u = 0; u < NA / 3; u++) {
    const bool do_lop = MODE == 0 || (MODE == 2 && !(warp & 1)) || MODE >= 3;
    const bool do_mma = MODE == 1 || (MODE == 2 && (warp & 1)) || (MODE >= 3 && MODE <= 5);
    if (MODE == 6 || MODE == 7) {
      if (MODE == 7) {
#pragma unroll
        for (int i = 0; i < 12; i++) m[i] = lop(w[i & 3], m[i], 0x01010101u << (i & 7));
      }
#pragma unroll
      for (int i = 0; i < 12; i++) dp4a(acc[i % NA][i & 3], m[i], b0);
      continue;
    }
    if (MODE == 5) {
#pragma unroll
      for (int i = 0; i < 12; i++) mp[i] = m[i];
    }
    if (do_lop) {
#pragma unroll
      for (int i = 0; i < 12; i++) m[i] = lop(w[i & 3], m[i], 0x01010101u << (i & 7));
    }
    if (do_mma) {
#pragma unroll
      for (int j = 0; j < 3; j++) {
        if (MODE == 4) mma_u8s8(acc[u * 3 + j], m[4 * j], m[4 * j + 1], m[4 * j + 2], m[4 * j + 3], b0, b1);
        else if (MODE == 5) mma_u8s8(acc[u * 3 + j], mp[4 * j], mp[4 * j + 1], mp[4 * j + 2], mp[4 * j + 3], b0, b1);
        else mma_u8s8(acc[u * 3 + j], w[0], w[1], w[2], w[3], b0, b1);
      }
    }
  }
  }
  const long long t1 = clock64();
  int s = 0;
#pragma unroll
  for (int a = 0; a < NA; a++)
#pragma unroll
    for (int r = 0; r < 4; r++) s += acc[a][r];
#pragma unroll
  for (int i = 0; i < 12; i++) s += m[i];
  if (s == 0x12345678) sink[0] = s;
  if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}

template <int MODE, int NA>
void run(const char* name, int iters) {
  int* sink; long long* clk;
  cudaMalloc(&sink, 4); cudaMalloc(&clk, 148 * 8);
  pipes_kernel<MODE, NA><<<148, 512>>>(12345u, iters, sink, clk);
  cudaDeviceSynchronize();
  pipes_kernel<MODE, NA><<<148, 512>>>(12345u, iters, sink, clk);
  cudaError_t e = cudaDeviceSynchronize();
  std::vector<long long> h(148);
  cudaMemcpy(h.data(), clk, 148 * 8, cudaMemcpyDeviceToHost);
  long long mx = 0;
  for (auto v : h) mx = std::max(mx, v);
  // one iteration of one warp = the work for 32 words (128 bytes of packed weights); 16 warps per SM
  printf("%-46s NA=%d  %s  clk/iter/SM %.2f  (= %.1f clk per KB of weights at 128 B per warp-iteration)\n", name, NA,
         cudaGetErrorString(e), (double)mx / iters, (double)mx / iters / 2.0);
  cudaFree(sink); cudaFree(clk);
}

int main() {
  const int iters = 20000;
  run<0, 3>("0 LOP3 only (12 per warp-iter)", iters);
  run<1, 3>("1 MMA only (3 per warp-iter)", iters);
  run<1, 6>("1 MMA only", iters);
  run<1, 12>("1 MMA only", iters);
  run<2, 3>("2 even warps LOP3, odd warps MMA", iters);
  run<2, 6>("2 even warps LOP3, odd warps MMA", iters);
  run<3, 3>("3 LOP3 + MMA independent in every warp", iters);
  run<3, 6>("3 LOP3 + MMA independent in every warp", iters);
  run<3, 12>("3 LOP3 + MMA independent in every warp", iters);
  run<4, 3>("4 LOP3 -> MMA dependent", iters);
  run<4, 6>("4 LOP3 -> MMA dependent", iters);
  run<4, 12>("4 LOP3 -> MMA dependent", iters);
  run<5, 6>("5 LOP3 -> MMA one iteration later", iters);
  run<5, 12>("5 LOP3 -> MMA one iteration later", iters);
  run<6, 12>("6 dp4a only (12 per warp-iter)", iters);
  run<7, 12>("7 LOP3 -> dp4a dependent (12 + 12)", iters);
  return 0;
}
