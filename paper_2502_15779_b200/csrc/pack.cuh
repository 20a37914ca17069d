// Weight-code packing: 16 two-bit codes per 32-bit word along K, least-significant first
// (Section 4.4: W_q is stored sub-byte packed along the input channel, prepared offline).
#pragma once
#include "common.cuh"

namespace rcp {

// One thread per output word: a 16-byte load of codes, one 4-byte store. Codes above 3 set *bad.
__global__ void __launch_bounds__(256) pack_weights_kernel(const uint4* __restrict__ codes16,
                                                           size_t nwords, uint32_t* __restrict__ words,
                                                           int* __restrict__ bad) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t step = (size_t)gridDim.x * blockDim.x;
  uint32_t any_bad = 0;
  for (; i < nwords; i += step) {
    const uint4 c = __ldg(codes16 + i);
    const uint32_t r[4] = {c.x, c.y, c.z, c.w};
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const uint32_t b = r[j];  // four codes, one per byte, lowest byte first
      any_bad |= b & 0xFCFCFCFCu;
      const uint32_t four = (b & 3u) | ((b >> 6) & 0xCu) | ((b >> 12) & 0x30u) | ((b >> 18) & 0xC0u);
      w |= four << (8 * j);
    }
    words[i] = w;
  }
  if (any_bad) atomicOr(bad, 1);
}

}  // namespace rcp
