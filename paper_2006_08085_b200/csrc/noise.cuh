// Counter-based standard-normal noise of the stochastic gradient oracle.
//
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel Random Numbers: As Easy as 1, 2, 3",
// SC'11) with key (seed low word, seed high word) and counter (j low word, j high word,
// i / 4, step) gives four words r0..r3 for the workers 4q..4q+3 (q = i / 4) at global
// coordinate j.  (r0, r1) and (r2, r3) each feed one Box-Muller transform:
//   u_rad = ((r_even >> 9) + 0.5) * 2^-23 in (0,1),  u_ang = (r_odd >> 8) * 2^-24 in [0,1)
//   rad = sqrt(-2 ln u_rad);  first = rad cos(2 pi u_ang);  second = rad sin(2 pi u_ang)
// Both uniforms are exactly representable in float32, so the only float32 error is in the
// elementary functions (accurate logf / sqrtf / sincospif: about 1e-7 relative).
#ifndef DETAG_NOISE_CUH
#define DETAG_NOISE_CUH

#include <cstdint>

namespace detag {

struct Philox4 {
  uint32_t r0, r1, r2, r3;
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1) {
  constexpr uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u, kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(kM0, c0), lo0 = kM0 * c0;
    const uint32_t hi1 = __umulhi(kM1, c2), lo1 = kM1 * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += kW0;
    k1 += kW1;
  }
  return Philox4{c0, c1, c2, c3};
}

__device__ __forceinline__ void box_muller(uint32_t r_even, uint32_t r_odd, float& first, float& second) {
  const float u_rad = (static_cast<float>(r_even >> 9) + 0.5f) * 0x1p-23f;
  const float u_ang = static_cast<float>(r_odd >> 8) * 0x1p-24f;
  const float rad = sqrtf(-2.0f * logf(u_rad));
  float s, c;
  sincospif(2.0f * u_ang, &s, &c);
  first = rad * c;
  second = rad * s;
}

// Standard normals of workers 4q..4q+3 at global coordinate j and noise step t.
__device__ __forceinline__ void normal_quad(uint32_t seed_lo, uint32_t seed_hi, unsigned long long j, uint32_t q,
                                            uint32_t t, float xi[4]) {
  const Philox4 r = philox4x32_10(static_cast<uint32_t>(j), static_cast<uint32_t>(j >> 32), q, t, seed_lo, seed_hi);
  box_muller(r.r0, r.r1, xi[0], xi[1]);
  box_muller(r.r2, r.r3, xi[2], xi[3]);
}

}  // namespace detag
#endif  // DETAG_NOISE_CUH
