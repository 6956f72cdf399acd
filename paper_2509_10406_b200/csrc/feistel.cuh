// Seeded integer shuffle shared by the strided start of the clustering and by the streaming pass.
#pragma once
#include <stdint.h>

namespace muse {

__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Seeded bijection of [0, N): 4-round Feistel network on the smallest even-width power of two
// that covers N, cycle-walked into range (the "shuffle with a fixed random seed" of Appendix
// "Centroid Computation", step 1).
__device__ __forceinline__ int feistel_permute(int x0, int N, uint64_t seed, uint64_t stream) {
  int bits = 32 - __clz(max(N - 1, 1));
  if (bits < 2) bits = 2;
  bits += bits & 1;
  const int half = bits / 2;
  const uint64_t mask = (1ull << half) - 1ull;
  uint64_t x = (uint64_t)x0;
  for (int guard = 0; guard < 1 << 20; ++guard) {
    uint64_t L = x >> half, R = x & mask;
#pragma unroll
    for (uint64_t r = 0; r < 4; ++r) {
      uint64_t f = splitmix64(seed ^ (stream << 32) ^ (r << 56) ^ R) & mask;
      uint64_t nl = R; R = L ^ f; L = nl;
    }
    x = (L << half) | R;
    if (x < (uint64_t)N) break;
  }
  return (int)x;
}

}  // namespace muse
