// Rate of tcgen05.mma kind::i8 (M = 128, K = 32) as a function of N, A from tensor memory or from shared memory.
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>
constexpr uint32_t kSpin = 1u << 22;
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// mode 0: A in tensor memory; mode 1: A in shared memory
__global__ void __launch_bounds__(32, 1) rate_kernel(int N, int iters, int mode, long long* clk, int* err) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem);
  const uint32_t bar = smem_u32(smem + 16);
  const uint32_t sA = smem_u32(smem + 1024), sB = smem_u32(smem + 1024 + 4096);
  const int lane = threadIdx.x;
  for (int i = lane; i < (4096 + 8192) / 4; i += 32) reinterpret_cast<uint32_t*>(smem + 1024)[i] = 0x01020304u * (i + 1);
  if (lane == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(512) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  const uint32_t tbase = *s_tmem;
  // A columns: whatever tensor memory holds (integers: any bit pattern is a number); write them once to be defined
  {
    uint32_t v = 0x01010101u * (lane & 3);
    for (int c = 0; c < 8; c++)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(tbase + 256 + c), "r"(v) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncwarp();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  bool failed = false;
  long long t0 = clock64(), t1 = t0;
  if (lane == 0) {
    const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
    const uint64_t bd = make_desc(sB, 4096, 128);   // rows at 16-byte pitch, K halves 4096 apart
    const uint64_t ad = make_desc(sA, 2048, 128);
    for (int i = 0; i < iters; i++) {
      if (mode == 0)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5,%5,%5,%5}, p;\n\t}"
                     :: "r"(tbase), "r"(tbase + 256), "l"(bd), "r"(idesc), "r"(i > 0 ? 1 : 0), "r"(0) : "memory");
      else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5,%5,%5,%5}, p;\n\t}"
                     :: "r"(tbase), "l"(ad), "l"(bd), "r"(idesc), "r"(i > 0 ? 1 : 0), "r"(0) : "memory");
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    uint32_t n = 0;
    while (!mbar_try(bar, 0)) { if (++n > kSpin) { failed = true; break; } }
    t1 = clock64();
    if (failed) atomicExch(err, 1);
    clk[blockIdx.x] = t1 - t0;
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
}
int main() {
  long long* clk; int* err;
  cudaMalloc(&clk, 148 * 8); cudaMalloc(&err, 4); cudaMemset(err, 0, 4);
  const size_t smem = 1024 + 4096 + 8192;
  const int iters = 4096;
  for (int mode = 0; mode < 2; mode++)
    for (int N : {8, 16, 32, 64, 128, 256}) {
      rate_kernel<<<148, 32, smem>>>(N, iters, mode, clk, err);
      cudaError_t e = cudaDeviceSynchronize();
      std::vector<long long> h(148);
      cudaMemcpy(h.data(), clk, 148 * 8, cudaMemcpyDeviceToHost);
      int herr = 0; cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
      long long mx = 0; for (auto v : h) mx = std::max(mx, v);
      printf("A from %s  N=%3d  %s err=%d  %.1f clk per MMA (128 x N x 32 int8)\n", mode ? "smem" : "tmem", N, cudaGetErrorString(e), herr, (double)mx / iters);
      if (e != cudaSuccess || herr) return 1;
    }
  return 0;
}
