// Real Fourier basis of the R-cycle (R = 4 or 8), q(p, r): orthonormal rows, used by the block-circulant step
// kernel (as compile-time constants) and by the host code that builds its per-frequency blocks.
//   p = 0            constant row, frequency 0
//   p = 2f-1, 2f     cosine and sine rows of frequency f = 1 .. R/2 - 1
//   p = R-1          alternating row, frequency R/2
#ifndef DETAG_TORUS_BASIS_H
#define DETAG_TORUS_BASIS_H

#ifdef __CUDACC__
#define DETAG_HD __host__ __device__
#else
#define DETAG_HD
#endif

namespace detag {

// cos(2 pi k / R) for R = 4, 8 with exact zeros and halves
DETAG_HD constexpr double torus_cos(int R, int k) {
  const int m = ((k % R) + R) % R;
  if (R == 4) return m == 0 ? 1.0 : m == 2 ? -1.0 : 0.0;
  // R == 8
  return m == 0 ? 1.0
       : m == 4 ? -1.0
       : (m == 2 || m == 6) ? 0.0
       : (m == 1 || m == 7) ? 0.70710678118654752440 : -0.70710678118654752440;
}

DETAG_HD constexpr int torus_frequency(int R, int p) { return p == 0 ? 0 : p == R - 1 ? R / 2 : (p + 1) / 2; }

DETAG_HD constexpr double torus_q(int R, int p, int r) {
  const double single = R == 4 ? 0.5 : 0.35355339059327376220;  // 1 / sqrt(R)
  const double pair = R == 4 ? 0.70710678118654752440 : 0.5;    // sqrt(2 / R)
  if (p == 0) return single;
  if (p == R - 1) return (r % 2 == 0) ? single : -single;
  const int f = (p + 1) / 2;
  const bool sine = (p % 2) == 0;
  return pair * torus_cos(R, f * r - (sine ? R / 4 : 0));  // sin(t) = cos(t - pi/2)
}

}  // namespace detag
#endif  // DETAG_TORUS_BASIS_H
