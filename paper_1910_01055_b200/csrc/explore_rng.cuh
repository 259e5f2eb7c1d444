// Counter-based exploration noise for acting policies (paper Section 5, experimental set-up: a
// Gaussian noise layer on the actor's policy output).  The paper does not say how the draws are
// made; here row b, column n of a call with seed s gets
//   (x0, x1, x2, x3) = Philox-4x32-10(counter = (b mod 2^32, b div 2^32, n div 4, 0), key = (s mod 2^32, s div 2^32))
//   pair (x0, x1) for columns 4j, 4j + 1 and (x2, x3) for 4j + 2, 4j + 3 of block j = n div 4:
//   u1 = ((xa >> 9) + 1/2) 2^-23,  u2 = ((xb >> 9) + 1/2) 2^-23      (exact in binary32)
//   z = sqrt(-2 ln u1) * (cos(2 pi u2) for even n, sin(2 pi u2) for odd n)      (Box-Muller)
// so a row's noise depends on (seed, absolute row, column) only, not on the batch it travels in.
// Philox-4x32-10: Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11),
// written out from its definition: ten rounds of two 32 x 32 -> 64-bit multiplications with a Weyl
// key schedule.
#pragma once
#include <stdint.h>

namespace actorq {

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&x)[4]) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  x[0] = c0; x[1] = c1; x[2] = c2; x[3] = c3;
}

// the standard normal draw of (seed, row, column)
__device__ __forceinline__ float exploration_normal(uint32_t seed_lo, uint32_t seed_hi, long long row, int col) {
  uint32_t x[4];
  philox4x32_10((uint32_t)((unsigned long long)row & 0xffffffffull), (uint32_t)((unsigned long long)row >> 32), (uint32_t)(col >> 2), 0u,
                seed_lo, seed_hi, x);
  const uint32_t xa = (col & 2) ? x[2] : x[0], xb = (col & 2) ? x[3] : x[1];
  const float u1 = __fmul_rn(__fadd_rn((float)(xa >> 9), 0.5f), 0x1p-23f);
  const float two_u2 = __fmul_rn(__fadd_rn((float)(xb >> 9), 0.5f), 0x1p-22f);
  const float radius = sqrtf(-2.0f * logf(u1));
  float sn, cs;
  sincospif(two_u2, &sn, &cs);
  return radius * ((col & 1) ? sn : cs);
}

}  // namespace actorq
