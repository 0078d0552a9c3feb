// Stand-alone kernels around the step: the stochastic gradient of the synthetic objective
// (used for the initial state) and the consensus-error reduction.
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"

namespace detag {

namespace {

constexpr int kAuxThreads = 256;

// g = a (x - c) + sigma xi_t and y = g: the initial state y_0 = g(x_0) of the tracker.
// One thread handles the four workers 4q..4q+3 of one coordinate (one Philox call).
__global__ void __launch_bounds__(kAuxThreads) init_gradient_kernel(const StepParams p) {
  const int nq = (p.n + 3) >> 2;
  const long long items = static_cast<long long>(nq) * p.d;
  const double sigma = p.sigma;
  for (long long it = blockIdx.x * static_cast<long long>(kAuxThreads) + threadIdx.x; it < items;
       it += static_cast<long long>(gridDim.x) * kAuxThreads) {
    const int q = static_cast<int>(it / p.d);
    const long long j = it - static_cast<long long>(q) * p.d;
    float xi[4] = {0.f, 0.f, 0.f, 0.f};
    if (sigma != 0.0)
      normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j), q, p.t_noise, xi);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int i = 4 * q + w;
      if (i < p.n) {
        const long long off = static_cast<long long>(i) * p.ld + j;
        const double g = fma(static_cast<double>(p.a[off]),
                             static_cast<double>(p.x[off]) - static_cast<double>(p.c[off]),
                             sigma * static_cast<double>(xi[w]));
        const float gf = static_cast<float>(g);
        p.g[off] = gf;
        if (p.mode != kModeDpsgd) p.y[off] = gf;  // D-PSGD keeps no tracker
      }
    }
  }
}

// Caller-written gradients: the initial state is y_0 = g_old = the caller's gradient at x_0, so that the first
// tracker update of Algorithm 2 (y + g_new - g_old with g_new = g_old) changes nothing.
__global__ void __launch_bounds__(kAuxThreads) init_external_kernel(const StepParams p) {
  const long long items = static_cast<long long>(p.n) * p.d;
  for (long long it = blockIdx.x * static_cast<long long>(kAuxThreads) + threadIdx.x; it < items;
       it += static_cast<long long>(gridDim.x) * kAuxThreads) {
    const long long i = it / p.d, j = it - i * p.d;
    const long long off = i * p.ld + j;
    const float gv = p.g_ext[off];
    p.g[off] = gv;
    p.y[off] = gv;
  }
}

// Failure-detection self test: one thread waits, through the kernels' own bounded wait, on a barrier that nobody
// ever arrives at.  After `polls` polls the wait gives up, the status word is set and the kernel returns normally.
__global__ void expire_wait_kernel(int* status, unsigned polls) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    bar_init(&bar, 1);
    fence_barrier_init();
    if (!bar_wait(&bar, 0, polls)) atomicExch(status, 1);
  }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  return v;
}

// Per coordinate: mean over workers, then the sum of squared deviations (two passes, float64).
// Per CTA: warp-shuffle tree, then a fixed-order sum over the warps -> partials[blockIdx.x].
__global__ void __launch_bounds__(kAuxThreads) consensus_partial_kernel(const StepParams p, double* partials) {
  __shared__ double warp_part[kAuxThreads / 32];
  double acc = 0.0;
  const double inv_n = 1.0 / static_cast<double>(p.n);
  for (long long j = blockIdx.x * static_cast<long long>(kAuxThreads) + threadIdx.x; j < p.d;
       j += static_cast<long long>(gridDim.x) * kAuxThreads) {
    double sum = 0.0;
    for (int i = 0; i < p.n; ++i) sum += static_cast<double>(p.x[static_cast<long long>(i) * p.ld + j]);
    const double mean = sum * inv_n;
    double ss = 0.0;
    for (int i = 0; i < p.n; ++i) {
      const double dev = static_cast<double>(p.x[static_cast<long long>(i) * p.ld + j]) - mean;
      ss = fma(dev, dev, ss);
    }
    acc += ss;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kAuxThreads / 32; ++w) s += warp_part[w];
    partials[blockIdx.x] = s;
  }
}

// Single CTA: fixed-order sum of the partials.
__global__ void __launch_bounds__(kAuxThreads) consensus_final_kernel(const double* partials, int count,
                                                                      double* result) {
  __shared__ double warp_part[kAuxThreads / 32];
  double acc = 0.0;
  for (int k = threadIdx.x; k < count; k += kAuxThreads) acc += partials[k];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kAuxThreads / 32; ++w) s += warp_part[w];
    *result = s;
  }
}

}  // namespace

int launch_init_gradient(const StepParams& p, int sm_count, cudaStream_t stream) {
  const long long items = static_cast<long long>((p.n + 3) / 4) * p.d;
  if (items <= 0) return 0;
  long long grid = (items + kAuxThreads - 1) / kAuxThreads;
  const long long cap = static_cast<long long>(sm_count) * 16;
  if (grid > cap) grid = cap;
  init_gradient_kernel<<<static_cast<unsigned>(grid), kAuxThreads, 0, stream>>>(p);
  return static_cast<int>(cudaGetLastError());
}

int launch_init_external(const StepParams& p, int sm_count, cudaStream_t stream) {
  const long long items = static_cast<long long>(p.n) * p.d;
  if (items <= 0) return 0;
  long long grid = (items + kAuxThreads - 1) / kAuxThreads;
  const long long cap = static_cast<long long>(sm_count) * 16;
  if (grid > cap) grid = cap;
  init_external_kernel<<<static_cast<unsigned>(grid), kAuxThreads, 0, stream>>>(p);
  return static_cast<int>(cudaGetLastError());
}

int launch_expire_wait(int* status, unsigned polls, cudaStream_t stream) {
  expire_wait_kernel<<<1, 32, 0, stream>>>(status, polls);
  return static_cast<int>(cudaGetLastError());
}

int ensure_dynamic_smem(const void* kernel, int bytes) {
  struct Entry {
    const void* kernel;
    int device, bytes;
  };
  static std::mutex mu;
  static std::vector<Entry> done;  // the largest size configured so far per kernel and device
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return static_cast<int>(e);
  std::lock_guard<std::mutex> lock(mu);
  Entry* hit = nullptr;
  for (auto& en : done)
    if (en.kernel == kernel && en.device == device) hit = &en;
  if (hit != nullptr && hit->bytes >= bytes) return 0;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return static_cast<int>(e);
  if (hit != nullptr)
    hit->bytes = bytes;
  else
    done.push_back(Entry{kernel, device, bytes});
  return 0;
}

int launch_consensus_error(const StepParams& p, double* partials, double* result, int sm_count,
                           cudaStream_t stream) {
  long long grid = (p.d + kAuxThreads - 1) / kAuxThreads;
  long long cap = static_cast<long long>(sm_count) * 8;
  if (cap > kMaxPartials) cap = kMaxPartials;
  if (grid > cap) grid = cap;
  if (grid < 1) grid = 1;
  consensus_partial_kernel<<<static_cast<unsigned>(grid), kAuxThreads, 0, stream>>>(p, partials);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return static_cast<int>(e);
  consensus_final_kernel<<<1, kAuxThreads, 0, stream>>>(partials, static_cast<int>(grid), result);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag

// ---------------------------------------------------------------------------------------------------
// Consensus error without any caller-provided or allocated scratch.
//
// The partial sums live in this file-scope device array, which every GPU that loads the library keeps
// until the process exits (1 MiB + one result slot).  One partial per block of 256 coordinates, so the
// array bounds the problem size: d <= kStaticMaxCoords.  Host code may not hand the array's NAME to a
// kernel (on the host it is only a stand-in symbol); the device address is looked up once per device
// with cudaGetSymbolAddress and cached.
namespace {

constexpr int kStaticPartials = 131072;                                   // 1 MiB of float64 partial sums
constexpr long long kStaticMaxCoords = static_cast<long long>(kStaticPartials) * 256;  // 33,554,432
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) double g_static_consensus_scratch[kStaticPartials + 32];

double* g_static_scratch_addr[kStaticMaxDevices] = {nullptr};

}  // namespace

extern "C" int detag_consensus_error_static(int n, int64_t d, int64_t ld, const float* x, void* stream,
                                            double* host_out) {
  if (n <= 0 || d <= 0 || ld < d || !x || !host_out) return DETAG_ERR_ARG;
  if (n > detag::kMaxWorkers || d > kStaticMaxCoords) return DETAG_ERR_UNSUPPORTED;  // beyond the static scratch
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return DETAG_ERR_CUDA;
  if (device < 0 || device >= kStaticMaxDevices) return DETAG_ERR_UNSUPPORTED;
  if (g_static_scratch_addr[device] == nullptr) {  // first call on this device: resolve the array's device address
    double* addr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_static_consensus_scratch) != cudaSuccess || !addr)
      return DETAG_ERR_CUDA;
    g_static_scratch_addr[device] = addr;
  }
  double* partials = g_static_scratch_addr[device];
  double* result = partials + kStaticPartials;
  detag::StepParams p{};
  p.n = n;
  p.d = d;
  p.ld = ld;
  p.x = const_cast<float*>(x);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // One CTA per 256 coordinates: every partial slot in [0, grid) is overwritten, and so is the result
  // slot, so nothing left over from an earlier call is ever read and nothing needs clearing.
  const int grid = static_cast<int>((d + detag::kAuxThreads - 1) / detag::kAuxThreads);
  detag::consensus_partial_kernel<<<static_cast<unsigned>(grid), detag::kAuxThreads, 0, st>>>(p, partials);
  if (cudaGetLastError() != cudaSuccess) return DETAG_ERR_CUDA;
  detag::consensus_final_kernel<<<1, detag::kAuxThreads, 0, st>>>(partials, grid, result);
  if (cudaGetLastError() != cudaSuccess) return DETAG_ERR_CUDA;
  if (cudaMemcpyAsync(host_out, result, sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return DETAG_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DETAG_ERR_CUDA;
  return DETAG_OK;
}
