// Counter-based standard-normal noise of the stochastic gradient oracle.
//
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel Random Numbers: As Easy as 1, 2, 3",
// SC'11) with key (seed low word, seed high word) and counter (j low word, j high word,
// i / 4, step) gives four words r0..r3 for the workers 4q..4q+3 (q = i / 4) at global
// coordinate j.  (r0, r1) and (r2, r3) each feed one Box-Muller transform:
//   u_rad = (2 (r_even >> 9) + 1) * 2^-24 in (0,1),  u_ang = (r_odd >> 9) * 2^-23 in [0,1)
//   rad = sqrt(-2 ln u_rad);  first = rad cos(2 pi u_ang);  second = rad sin(2 pi u_ang)
// Both uniforms are exactly representable in float32 and are built with bit operations, no
// integer-to-float conversion.  The logarithm is an own float32 routine (exponent split, degree-7
// polynomial of ln(1+f)/..., relative error < 1.2e-7 over all 2^23 inputs); the square root uses the
// reciprocal-square-root unit and sine/cosine the special-function unit on an argument reduced
// exactly to [-pi, pi).  Resulting absolute error of a normal: about 1e-6 (1 + |xi|).
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
    const unsigned long long p0 = static_cast<unsigned long long>(kM0) * c0;  // one wide multiply: hi and lo
    const unsigned long long p1 = static_cast<unsigned long long>(kM1) * c2;
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    c0 = hi1 ^ c1 ^ (k0 + static_cast<uint32_t>(round) * kW0);
    c1 = lo1;
    c2 = hi0 ^ c3 ^ (k1 + static_cast<uint32_t>(round) * kW1);
    c3 = lo0;
  }
  return Philox4{c0, c1, c2, c3};
}

// -2 ln(u) for u = (2k+1) 2^-24, k = r >> 9.
__device__ __forceinline__ float neg2_ln_unit(uint32_t r) {
  const float v = __uint_as_float(0x3f800000u | (r >> 9));  // 1 + k 2^-23
  const float u = v - 0x1.fffffep-1f;                        // (2k+1) 2^-24, exact
  const int bits = __float_as_int(u);
  const int e = (bits - 0x3f2aaaab) >> 23;                   // u = m 2^e with m in [2/3, 4/3)
  const float m = __int_as_float(bits - (e << 23));
  const float f = m - 1.0f;
  // ln(1+f) = f + f^2 r(f) on |f| <= 1/3 (Chebyshev fit of (ln(1+f) - f)/f^2, degree 7)
  float r7 = 0.13756538927555084f;
  r7 = fmaf(r7, f, -0.1504942923784256f);
  r7 = fmaf(r7, f, 0.1405421793460846f);
  r7 = fmaf(r7, f, -0.16481579840183258f);
  r7 = fmaf(r7, f, 0.2000732272863388f);
  r7 = fmaf(r7, f, -0.25004205107688904f);
  r7 = fmaf(r7, f, 0.33333271741867065f);
  r7 = fmaf(r7, f, -0.49999985098838806f);
  float ln = fmaf(f * f, r7, f);
  const float ef = __int_as_float(0x4b400000 + e) - 12582912.0f;  // e as a float, no conversion instruction
  ln = fmaf(ef, 1.42860677e-06f, ln);
  ln = fmaf(ef, 0.693145751953125f, ln);
  return -2.0f * ln;
}

__device__ __forceinline__ void box_muller(uint32_t r_even, uint32_t r_odd, float& first, float& second) {
  const float t = neg2_ln_unit(r_even);                                   // > 0
  const float rad = t * rsqrtf(t);
  const float w = __uint_as_float(0x3f800000u | (r_odd >> 9)) - 1.5f;     // u_ang - 1/2 in [-1/2, 1/2), exact
  const float theta = w * 6.283185307179586f;                             // 2 pi u_ang - pi
  first = -rad * __cosf(theta);                                           // cos(2 pi u) = -cos(2 pi u - pi)
  second = -rad * __sinf(theta);
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
