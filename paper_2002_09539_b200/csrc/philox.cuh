// Philox4x32-10, implemented from its published definition (Salmon, Moraes, Dror, Shaw,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11, Section 3.3 and the Philox4x32 row
// of its constants table): ten rounds of
//   (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0))
// with the key bumped by the two Weyl constants before every round but the first; and the
// minibatch index rule built on it.
#pragma once

#include <cstdint>

namespace olsgd {

struct U4 { uint32_t w[4]; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += W0; k1 += W1; }
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  U4 r; r.w[0] = c0; r.w[1] = c1; r.w[2] = c2; r.w[3] = c3;
  return r;
}

constexpr uint32_t kStreamMinibatch = 1;
constexpr uint32_t kStreamPartition = 2;
constexpr uint32_t kStreamEpoch = 3;

// Slot j of global worker `worker` at iteration k, with replacement: word j % 4 of the Philox
// block with counter (j / 4, k, worker, 1) and key (seed lo, seed hi), scaled to [0, n).
__device__ __forceinline__ int32_t minibatch_index(uint32_t k0, uint32_t k1, uint32_t k,
                                                   uint32_t worker, int j, uint32_t n) {
  const U4 r = philox4x32_10((uint32_t)(j >> 2), k, worker, kStreamMinibatch, k0, k1);
  return (int32_t)__umulhi(r.w[j & 3], n);
}

}  // namespace olsgd
