// Bit-stream codec shared by the kernels: 32 consecutive N-bit codes occupy N
// consecutive 32-bit words (little-endian bit order, code j at stream bits
// [N*j, N*j + N)).
#pragma once
#include <stdint.h>

namespace eqat {

template <int BITS>
__device__ __forceinline__ void pack32(const uint32_t (&c)[32], uint32_t (&w)[BITS]) {
#pragma unroll
  for (int i = 0; i < BITS; ++i) w[i] = 0u;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int bit = BITS * j, word = bit >> 5, off = bit & 31;
    w[word] |= c[j] << off;
    if (off + BITS > 32) w[word + 1] |= c[j] >> (32 - off);
  }
}

template <int BITS>
__device__ __forceinline__ void unpack32(const uint32_t (&w)[BITS], uint32_t (&c)[32]) {
  constexpr uint32_t mask = (1u << BITS) - 1u;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int bit = BITS * j, word = bit >> 5, off = bit & 31;
    uint32_t x = w[word] >> off;
    if (off + BITS > 32) x |= w[word + 1] << (32 - off);
    c[j] = x & mask;
  }
}

}  // namespace eqat
