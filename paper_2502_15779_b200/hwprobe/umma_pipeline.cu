// The tcgen05 route for the W2A4 GEMV, measured: kind::i8 with the A operand written to tensor memory by the
// threads (two-bit fields moved under the sign bit and read once as unsigned and once as signed bytes, plus the
// b0*b1 bit, eight masked words per 16 codes), B (int8 activations) in shared memory, K-major without swizzle,
// rows aliased at 16-byte pitch so that one token costs K bytes. 128 rows per CTA, eight converter warps, one
// issuing thread. Checks the integer sums against the host (mode 0) and reports bytes of packed weights per
// clock and SM with no HBM traffic at all: mode 1 without issuing the MMAs (converters alone), mode 2 with the
// converters only signalling (MMAs alone).
// usage: umma_pipeline TOKENS ITERATIONS CTAS MODE
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

constexpr int kRows = 128;
constexpr int kChunkWords = 32;
constexpr uint32_t kSpin = 1u << 20;
constexpr int NSLOT = 6;      // A slots of 64 columns
constexpr int kAcols = 64;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpin; i++)
    if (mbar_try(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t and3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x80;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void umma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      :
      : "r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc), "r"(0)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// B descriptor: K-major, no swizzle; the two 16-byte K halves of a K-step are lbo bytes apart,
// 8-row groups sbo bytes apart (sm_100 descriptor version 1).
__device__ __forceinline__ uint64_t make_bdesc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}

struct Params {
  const uint32_t* words;   // [128][32] one chunk
  const int8_t* bperm;     // [32 units][M][16] permuted activations
  int M;                   // tokens (<= 8)
  int iters;               // groups per warpgroup
  int mode;                // 0: full, 1: no MMA issue (converter only), 2: MMA only (converters store once)
  uint32_t mul2, mul4, mul16, mul64;
  int32_t* out;            // [grid][6 tiles][128][8]
  long long* clocks;       // [grid][2]
  int* err;
};

__global__ void __launch_bounds__(288, 1) probe_kernel(const Params p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sW = smem;                                   // 16 KB
  uint8_t* sB = smem + 16384;                           // 32 units * M * 16 + 128
  const uint32_t bar0 = smem_u32(smem + 16384 + 32 * 16 * 8 + 128);
  const uint32_t full0 = bar0, empty0 = bar0 + 8 * NSLOT, dfull = bar0 + 16 * NSLOT;
  uint32_t* const s_tmem = reinterpret_cast<uint32_t*>(smem + 16384 + 32 * 16 * 8 + 128 + 8 * (2 * NSLOT + 1));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // fill shared memory: weights with the 128-byte swizzle a TMA box would have, activations as given
  for (int i = tid; i < kRows * 8; i += blockDim.x) {
    const int r = i >> 3, c = i & 7;
    const uint4 v = reinterpret_cast<const uint4*>(p.words)[r * 8 + c];
    *reinterpret_cast<uint4*>(sW + r * 128 + ((c ^ (r & 7)) << 4)) = v;
  }
  for (int i = tid; i < 32 * p.M + 8; i += blockDim.x) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (i < 32 * p.M) v = reinterpret_cast<const uint4*>(p.bperm)[i];
    *reinterpret_cast<uint4*>(sB + i * 16) = v;
  }
  if (warp == 8) {
    if (lane == 0) {
      for (int s = 0; s < NSLOT; s++) { mbar_init(full0 + 8 * s, 4); mbar_init(empty0 + 8 * s, 1); }
      mbar_init(dfull, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes of sB visible to the MMA's async proxy
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tbase = *s_tmem;
  const uint32_t Dbase = tbase;            // 6 tiles x 8 columns
  const uint32_t Abase = tbase + 64;       // NSLOT x 64 columns
  const int G = 2 * p.iters;               // groups in total
  bool failed = false;
  long long t0 = clock64();

  if (warp < 8) {
    const int wg = warp >> 2, row = (warp & 3) * 32 + lane;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t rowbase = smem_u32(sW) + row * 128;
    for (int it = 0; it < p.iters; it++) {
      const int g = it * 2 + wg, cs = g & 3, slot = g % NSLOT, use = g / NSLOT;
      if (p.mode == 2 && it > 0) {   // MMA-only timing: keep signalling full without new data
        if (use > 0 && !mbar_wait(empty0 + 8 * slot, (use - 1) & 1)) { failed = true; break; }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(full0 + 8 * slot);
        continue;
      }
      const uint4 U = lds128(rowbase + (((2 * cs) ^ (row & 7)) << 4));
      const uint4 V = lds128(rowbase + (((2 * cs + 1) ^ (row & 7)) << 4));
      const uint32_t w[8] = {U.x, U.y, U.z, U.w, V.x, V.y, V.z, V.w};
      uint32_t F[32], Z[32];
#pragma unroll
      for (int wi = 0; wi < 8; wi++) {
        const uint32_t x = w[wi];
        const uint32_t x1 = x * p.mul2;    // b0 moved onto b1's bit
        F[3 * 8 + wi] = x & 0xC0C0C0C0u;
        F[2 * 8 + wi] = (x * p.mul4) & 0xC0C0C0C0u;
        F[1 * 8 + wi] = (x * p.mul16) & 0xC0C0C0C0u;
        F[0 * 8 + wi] = (x * p.mul64) & 0xC0C0C0C0u;
#pragma unroll
        for (int pp = 0; pp < 4; pp++) Z[pp * 8 + wi] = and3(x, x1, 0x02020202u << (2 * pp));
      }
      if (use > 0 && !mbar_wait(empty0 + 8 * slot, (use - 1) & 1)) { failed = true; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_addr = Abase + lane_off + (uint32_t)slot * kAcols;
      tmem_st32(a_addr, F);
      tmem_st32(a_addr + 32, Z);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(full0 + 8 * slot);
    }
  } else if (lane == 0) {
    // MMA issuer
    const uint32_t idesc_u = (2u << 4) | (0u << 7) | (1u << 10) | ((8u >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t idesc_s = (2u << 4) | (1u << 7) | (1u << 10) | ((8u >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t lbo = (uint32_t)p.M * 16, sbo = 128;
    const uint32_t sBaddr = smem_u32(sB);
    for (int g = 0; g < G; g++) {
      const int cs = g & 3, slot = g % NSLOT, use = g / NSLOT;
      if (!mbar_wait(full0 + 8 * slot, use & 1)) { failed = true; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (p.mode != 1) {
        const uint32_t a_addr = Abase + (uint32_t)slot * kAcols;
#pragma unroll
        for (int pp = 0; pp < 4; pp++) {
          const uint64_t bd = make_bdesc(sBaddr + (uint32_t)((cs * 4 + pp) * 2) * lbo, lbo, sbo);
          const uint32_t acc = (g > 0 || pp > 0) ? 1u : 0u;
          umma_i8_ts(Dbase + 0, a_addr + pp * 8, bd, idesc_u, acc);
          umma_i8_ts(Dbase + 8, a_addr + pp * 8, bd, idesc_s, acc);
          umma_i8_ts(Dbase + 16 + 8 * pp, a_addr + 32 + pp * 8, bd, idesc_u, g > 0 ? 1u : 0u);
        }
      }
      umma_commit(empty0 + 8 * slot);
    }
    umma_commit(dfull);
  }
  long long t1 = clock64();
  __syncwarp();
  // results: warps 0..3 read the six accumulator tiles of their rows
  if (warp < 4) {
    if (!failed && !mbar_wait(dfull, 0)) failed = true;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    t1 = clock64();
    if (!failed) {
      const int row = warp * 32 + lane;
      for (int t = 0; t < 6; t++) {
        uint32_t r[8];
        tmem_ld8(Dbase + ((uint32_t)(warp * 32) << 16) + 8 * t, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        for (int n = 0; n < 8; n++) p.out[(((size_t)blockIdx.x * 6 + t) * 128 + row) * 8 + n] = (int32_t)r[n];
      }
    }
  }
  if (failed) atomicExch(p.err, 1 + warp);
  if (lane == 0 && (warp == 0 || warp == 8)) p.clocks[blockIdx.x * 2 + (warp == 8)] = t1 - t0;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
  }
}

#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e), __FILE__, __LINE__); return 1; } } while (0)

int main(int argc, char** argv) {
  const int M = argc > 1 ? atoi(argv[1]) : 1;
  const int iters = argc > 2 ? atoi(argv[2]) : 8;     // multiple of 2 so every 8-word piece is used equally often
  const int grid = argc > 3 ? atoi(argv[3]) : 1;
  const int mode = argc > 4 ? atoi(argv[4]) : 0;
  srand(1234);
  std::vector<uint32_t> words(kRows * kChunkWords);
  for (auto& w : words) w = ((uint32_t)rand() << 16) ^ (uint32_t)rand();
  std::vector<int8_t> q(8 * 512);
  for (auto& v : q) v = (int8_t)(rand() % 16 - 8);
  std::vector<int8_t> bperm(32 * M * 16);
  for (int cs = 0; cs < 4; cs++)
    for (int pp = 0; pp < 4; pp++)
      for (int half = 0; half < 2; half++)
        for (int m = 0; m < M; m++)
          for (int j = 0; j < 4; j++)
            for (int b = 0; b < 4; b++) {
              const int U = (cs * 4 + pp) * 2 + half, wi = half * 4 + j;
              bperm[((size_t)U * M + m) * 16 + j * 4 + b] = q[m * 512 + 16 * (cs * 8 + wi) + 4 * b + pp];
            }
  uint32_t* d_words; int8_t* d_b; int32_t* d_out; long long* d_clk; int* d_err;
  CK(cudaMalloc(&d_words, words.size() * 4));
  CK(cudaMalloc(&d_b, bperm.size()));
  CK(cudaMalloc(&d_out, (size_t)grid * 6 * 128 * 8 * 4));
  CK(cudaMalloc(&d_clk, grid * 2 * 8));
  CK(cudaMalloc(&d_err, 4));
  CK(cudaMemcpy(d_words, words.data(), words.size() * 4, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_b, bperm.data(), bperm.size(), cudaMemcpyHostToDevice));
  CK(cudaMemset(d_err, 0, 4));
  CK(cudaMemset(d_out, 0, (size_t)grid * 6 * 128 * 8 * 4));
  Params p{d_words, d_b, M, iters, mode, 2u, 4u, 16u, 64u, d_out, d_clk, d_err};
  const size_t smem = 16384 + 32 * 16 * 8 + 128 + 8 * (2 * NSLOT + 1) + 16;
  CK(cudaFuncSetAttribute(probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaEvent_t e0, e1;
  CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1));
  probe_kernel<<<grid, 288, smem>>>(p);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(e0));
  probe_kernel<<<grid, 288, smem>>>(p);
  CK(cudaEventRecord(e1));
  CK(cudaDeviceSynchronize());
  float ms = 0; CK(cudaEventElapsedTime(&ms, e0, e1));
  int err = 0; CK(cudaMemcpy(&err, d_err, 4, cudaMemcpyDeviceToHost));
  std::vector<int32_t> out((size_t)grid * 6 * 128 * 8);
  CK(cudaMemcpy(out.data(), d_out, out.size() * 4, cudaMemcpyDeviceToHost));
  std::vector<long long> clk(grid * 2);
  CK(cudaMemcpy(clk.data(), d_clk, clk.size() * 8, cudaMemcpyDeviceToHost));
  long long cmax = 0;
  for (int i = 0; i < grid; i++) cmax = std::max(cmax, clk[2 * i + 0]);
  const double bytes = (double)iters * 2 * 4096;   // packed weight bytes a CTA went through
  printf("M=%d iters=%d grid=%d mode=%d err=%d  kernel %.3f us  mma-warp clocks max %lld  -> %.2f B/clk/SM\n",
         M, iters, grid, mode, err, ms * 1e3, cmax, bytes / cmax);
  if (mode == 0 && err == 0) {
    // expected sums
    const int R = (2 * iters) / 4;
    long long bad = 0;
    for (int b = 0; b < grid; b++)
      for (int r = 0; r < 128; r++)
        for (int m = 0; m < M; m++) {
          long long T1 = 0, T2 = 0, T3p[4] = {0, 0, 0, 0};
          for (int k = 0; k < 512; k++) {
            const int c = (int)((words[r * 32 + k / 16] >> (2 * (k % 16))) & 3u);
            const int qq = q[m * 512 + k];
            T1 += (c & 1) * qq; T2 += (c >> 1) * qq; T3p[k % 4] += ((c & 1) & (c >> 1)) * qq;
          }
          const long long exp[6] = {R * (64 * T1 + 128 * T2), R * (64 * T1 - 128 * T2), R * 2 * T3p[0], R * 8 * T3p[1],
                                    R * 32 * T3p[2], R * 128 * T3p[3]};
          for (int t = 0; t < 6; t++) {
            const long long got = out[(((size_t)b * 6 + t) * 128 + r) * 8 + m];
            if (got != exp[t]) { if (bad < 8) printf("mismatch cta %d tile %d row %d tok %d: got %lld want %lld\n", b, t, r, m, got, exp[t]); bad++; }
          }
        }
    printf("check: %lld mismatches (R=%d)\n", bad, R);
    return bad ? 2 : 0;
  }
  return err ? 3 : 0;
}
