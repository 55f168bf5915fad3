// Counter-based Philox4x32-10 and the map (seed, logical scale index) -> z ~ N(0,1).
//
// The paper regenerates the Gaussian direction z from a stored seed instead of keeping
// it (Sec. 3.1, the MeZO seed trick; Algorithm 1 resets the generator with seed s before
// every sweep).  Here z_i is a pure function of (seed, i):
//   key = (lo32(seed), hi32(seed)); counter = (lo32(i>>2), hi32(i>>2), 0, 0); lane = i & 3
//   U(x) = ((x >> 9) + 0.5) * 2^-23
//   lanes 0,1 = sqrt(-2 ln U(r0)) * (cos, sin)(2 pi U(r1)); lanes 2,3 likewise from (r2, r3)
// The same device functions serve the GEMM prologue and the scale update, so both see
// bit-identical z.
#pragma once
#include <stdint.h>

namespace qzo {

struct Philox4 { uint32_t r0, r1, r2, r3; };

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += W0; k1 += W1;
  }
  return Philox4{c0, c1, c2, c3};
}

// Words of the counter block that holds logical index i.
__device__ __forceinline__ Philox4 philox_block(uint64_t seed, uint64_t block) {
  return philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), 0u, 0u,
                       (uint32_t)seed, (uint32_t)(seed >> 32));
}

__device__ __forceinline__ float uniform_from_word(uint32_t x) {
  return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f;   // exact: 24 significant bits
}

// The four normals of one counter block (indices 4*block .. 4*block+3).
__device__ __forceinline__ void normals_of_block(uint64_t seed, uint64_t block, float z[4]) {
  const Philox4 p = philox_block(seed, block);
  const float rho0 = sqrtf(-2.0f * logf(uniform_from_word(p.r0)));
  const float rho1 = sqrtf(-2.0f * logf(uniform_from_word(p.r2)));
  float s0, c0, s1, c1;
  sincospif(2.0f * uniform_from_word(p.r1), &s0, &c0);
  sincospif(2.0f * uniform_from_word(p.r3), &s1, &c1);
  z[0] = rho0 * c0; z[1] = rho0 * s0; z[2] = rho1 * c1; z[3] = rho1 * s1;
}

}  // namespace qzo
