// Gradient oracle of the zero-chain objective of the lower-bound construction (proof of Theorem 1, "Setting 1"):
// every worker holds fhat(u) = sum_{i=0}^{T-1} [Psi(-u_i) Phi(-u_{i+1}) - Psi(u_i) Phi(u_{i+1})] with u_0 := 1,
//     Psi(z) = exp(1 - 1/(2z-1)^2) for z > 1/2, else 0;   Phi(z) = sqrt(e) * int_{-inf}^{z} exp(-t^2/2) dt,
// rescaled as f(x) = (L lambda^2 / l_1) fhat(x / lambda), and the oracle multiplies the partial derivatives beyond
// the progress of x (its last non-zero coordinate) by z / p, z ~ Bernoulli(p), one draw per worker and step.
// (The integrand of Phi is printed with the opposite sign of the exponent, which diverges; the bounds the proof
// quotes hold for the function above.)  Coordinates are coupled to their neighbours, so the whole chain of a worker
// must live in one array; everything is evaluated in float64 and rounded once.
//
// Two passes: the progress of every worker (an atomic maximum over its non-zero coordinates), then the gradient.
// The result goes to any [n][ld] array, typically the one registered with detag_set_gradient_source.
#include <cuda_runtime.h>

#include <cmath>

#include "detag_internal.h"
#include "noise.cuh"

namespace detag {

namespace {

constexpr int kZcThreads = 256;

__global__ void __launch_bounds__(kZcThreads) zero_chain_progress_kernel(int n, long long d, long long ld, const float* x,
                                                                         int* progress) {
  const long long items = static_cast<long long>(n) * d;
  for (long long it = blockIdx.x * static_cast<long long>(kZcThreads) + threadIdx.x; it < items;
       it += static_cast<long long>(gridDim.x) * kZcThreads) {
    const long long i = it / d, j = it - i * d;
    if (x[i * ld + j] != 0.f) atomicMax(&progress[i], static_cast<int>(j + 1));
  }
}

__device__ __forceinline__ double zc_psi(double z) {
  if (!(z > 0.5)) return 0.0;
  const double u = 2.0 * z - 1.0;
  return exp(1.0 - 1.0 / (u * u));
}

__device__ __forceinline__ double zc_psi_prime(double z) {
  if (!(z > 0.5)) return 0.0;
  const double u = 2.0 * z - 1.0;
  return exp(1.0 - 1.0 / (u * u)) * 4.0 / (u * u * u);
}

__device__ __forceinline__ double zc_phi(double z) {  // sqrt(2 pi e) * N(z)
  return 4.1327313541224930 * 0.5 * erfc(-z * 0.70710678118654752440);
}

__device__ __forceinline__ double zc_phi_prime(double z) { return 1.6487212707001282 * exp(-0.5 * z * z); }

__global__ void __launch_bounds__(kZcThreads) zero_chain_gradient_kernel(int n, long long d, long long ld, const float* x,
                                                                         float* g, const int* progress, double inv_lambda,
                                                                         double gain, double p, uint32_t seed_lo,
                                                                         uint32_t seed_hi, uint32_t t) {
  const long long items = static_cast<long long>(n) * d;
  for (long long it = blockIdx.x * static_cast<long long>(kZcThreads) + threadIdx.x; it < items;
       it += static_cast<long long>(gridDim.x) * kZcThreads) {
    const long long i = it / d, j = it - i * d;
    const float* row = x + i * ld;
    const double u = static_cast<double>(row[j]) * inv_lambda;
    const double left = j > 0 ? static_cast<double>(row[j - 1]) * inv_lambda : 1.0;  // u_0 := 1
    // the term in which this coordinate is the argument of Phi ...
    double gr = -(zc_psi(-left) * zc_phi_prime(-u) + zc_psi(left) * zc_phi_prime(u));
    // ... and the one in which it is the argument of Psi
    if (j + 1 < d) {
      const double right = static_cast<double>(row[j + 1]) * inv_lambda;
      gr -= zc_psi_prime(-u) * zc_phi(-right) + zc_psi_prime(u) * zc_phi(right);
    }
    if (j + 1 > progress[i]) {  // beyond the progress of this worker's model: times z / p
      const Philox4 r = philox4x32_10(static_cast<uint32_t>(i), 0u, 0xB0B0B0B0u, t, seed_lo, seed_hi);
      const double uni = (static_cast<double>(r.r0) + 0.5) * 2.3283064365386963e-10;  // 2^-32
      gr *= uni < p ? 1.0 / p : 0.0;
    }
    g[i * ld + j] = static_cast<float>(gain * gr);
  }
}

}  // namespace

}  // namespace detag

extern "C" int detag_zero_chain_gradient(int n, int64_t d, int64_t ld, const float* x, float* g_out, double lambda,
                                         double gain, double p, uint64_t seed, int64_t t, int32_t* scratch,
                                         void* stream) {
  if (n <= 0 || d <= 0 || ld < d || !x || !g_out || !scratch) return DETAG_ERR_ARG;
  if (!(lambda > 0.0) || !std::isfinite(lambda) || !std::isfinite(gain) || !(p > 0.0) || !(p <= 1.0) || t < 0)
    return DETAG_ERR_ARG;
  if (n > detag::kMaxWorkers || d > 0x7fffffffLL) return DETAG_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(scratch, 0, static_cast<size_t>(n) * sizeof(int32_t), st) != cudaSuccess) return DETAG_ERR_CUDA;
  int device = 0, sms = 0;
  if (cudaGetDevice(&device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return DETAG_ERR_CUDA;
  const long long items = static_cast<long long>(n) * d;
  long long grid = (items + detag::kZcThreads - 1) / detag::kZcThreads;
  if (grid > static_cast<long long>(sms) * 16) grid = static_cast<long long>(sms) * 16;
  detag::zero_chain_progress_kernel<<<static_cast<unsigned>(grid), detag::kZcThreads, 0, st>>>(n, d, ld, x, scratch);
  if (cudaGetLastError() != cudaSuccess) return DETAG_ERR_CUDA;
  detag::zero_chain_gradient_kernel<<<static_cast<unsigned>(grid), detag::kZcThreads, 0, st>>>(
      n, d, ld, x, g_out, scratch, 1.0 / lambda, gain, p, static_cast<uint32_t>(seed & 0xffffffffu),
      static_cast<uint32_t>(seed >> 32), static_cast<uint32_t>(t));
  return cudaGetLastError() == cudaSuccess ? DETAG_OK : DETAG_ERR_CUDA;
}
