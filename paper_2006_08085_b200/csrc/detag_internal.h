// Internal declarations shared by the host API and the kernel launchers of libdetag.
#ifndef DETAG_INTERNAL_H
#define DETAG_INTERNAL_H

#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

#include "detag.h"

typedef struct CUstream_st* cudaStream_t;

namespace detag {

constexpr int kMaxWorkers = 1024;       // detag_create limit on n
constexpr int kMaxDenseWorkers = 64;    // dense-polynomial kernels with P in shared memory: limit on n
constexpr int kMaxWideWorkers = 128;    // dense-polynomial kernel with P in registers: limit on n
constexpr int kMaxPartials = 2048;      // per-CTA partial sums of the consensus-error reduction
constexpr size_t kWsAlign = 256;

// Everything a step / init / reduction kernel needs, passed by value.
struct StepParams {
  int n;
  int nnz;
  int K;
  int S;           // slab width in coordinates (power of two)
  int log2S;
  int csr_sub;     // generic rounds kernel: independent pieces the slab is cut into
  int csr_threads; // generic rounds kernel: threads per block (1024, or 512 with two blocks per SM)
  long long d;
  long long ld;
  long long num_slabs;
  long long coord_offset;  // global index of column 0 (noise counter)
  float* x;
  float* y;
  float* g;
  const float* a;
  const float* c;
  float* y_obs;  // optional gossiped-tracker output, may be null
  const int32_t* row_ptr;
  const int32_t* col_idx;
  const double* vals;
  const double* poly;  // dense P_K(M), row-major n x n (null when n > kMaxDenseWorkers)
  const double* circ_row;  // circulant kernel, dense mode: the first row of P_K(M) (or null)
  const double* wide;  // register-resident dense kernel (64 < n <= 128): the warp strips of P_K(M) in fragment order (or null)
  const double* torus; // block-circulant kernel: per-frequency 8 x 8 polynomial blocks in fragment order (or null)
  double eta;
  double alpha;
  double sigma;
  uint32_t seed_lo, seed_hi;
  uint32_t t_noise;  // step index that enters the noise counter
  int grad_at_start;  // nonzero: the gradient is taken at the model the step started from (Algorithm 2 as printed)
  int steps;          // consecutive steps in one launch (multi-step kernel only)
  int mode;           // kModeDetag, kModeExternal or kModeDpsgd
  const float* g_ext; // kModeExternal: the caller's newest stochastic gradient, [n][ld]
  unsigned spin_limit;    // polls after which a device-side wait gives up
  long long stall_after;  // failure-detection self test: a CTA's producer stops loading after this many tiles (< 0: off)
  int* status;
};

// What a step computes (the `mode` of StepParams)
constexpr int kModeDetag = 0;     // DeTAG with the library's own synthetic gradient (y holds the folded tracker)
constexpr int kModeExternal = 1;  // DeTAG with caller-written gradients: fold, gossip, model update; no gradient evaluation
constexpr int kModeDpsgd = 2;     // D-PSGD: x' = AG_K(x) - alpha g, g' = synthetic gradient at x'; no tracker

// Room for the tensor maps of one launch (eight 128-byte CUtensorMap objects), built once per set of bound
// buffers and kept in the state.
struct alignas(64) TensorMapSet {
  unsigned char bytes[8 * 128];
};

// host helpers (spectral.cpp)
int validate_csr(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals);
void csr_to_dense(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals, std::vector<double>& m);
bool is_symmetric(int n, const std::vector<double>& m, double tol);
void jacobi_eigenvalues(int n, std::vector<double>& a, std::vector<double>& ev);
double eta_from_lambda(double lam);

// kernel launchers; each returns a cudaError_t value as int (0 = success)
int launch_init_gradient(const StepParams& p, int sm_count, cudaStream_t stream);
int plan_step_csr(StepParams& p, int smem_optin_bytes);  // chooses S; DETAG_ERR_UNSUPPORTED if nothing fits
int launch_step_csr(const StepParams& p, int sm_count, cudaStream_t stream);
bool dense_variant_available(int n);  // n <= kMaxDenseWorkers and the driver offers tensor-map encoding
// Tensor-path kernels: build_* fills the tensor maps for the buffers in `p` (false: the driver refused one);
// launch_* takes the maps built for exactly those buffers.
bool build_maps_mma(const StepParams& p, TensorMapSet* maps);
int launch_step_mma(StepParams p, const TensorMapSet& maps, int sm_count, cudaStream_t stream);       // n <= 32
int launch_step_mma_many(StepParams p, const TensorMapSet& maps, int sm_count, cudaStream_t stream);  // p.steps steps
bool dense_window_available(int n);                // the band kernel's dense mode: 32 < n <= 64
bool build_maps_band(const StepParams& p, TensorMapSet* maps);
int launch_step_band(StepParams p, const TensorMapSet& maps, const double* band /* null: dense mode */, int sm_count,
                     cudaStream_t stream);
// circulant kernel (step_ring.cu): n % 32 == 0, 64 <= n <= 1024; band mode for half-band <= 16, dense mode for n <= 256
bool ring_variant_available(int n, int half_band);
bool ring_dense_available(int n);
bool build_maps_ring(const StepParams& p, TensorMapSet* maps);  // p.d a multiple of 64
int launch_step_ring(StepParams p, const TensorMapSet& maps, const double* band /* null: dense mode */,
                     const double* p_row /* device: first row of P, dense mode */, int sm_count, cudaStream_t stream);
bool torus_variant_available(int n);               // block-circulant kernel: n = 32 or 64 (4 or 8 blocks of 8)
bool build_maps_torus(const StepParams& p, TensorMapSet* maps);
int launch_step_torus(StepParams p, const TensorMapSet& maps, const double* phat_frag /* device */, int sm_count,
                      cudaStream_t stream);
// dense polynomial held in registers (step_wide.cu): 64 < n <= 128, p.d a multiple of 32, DeTAG step only
bool wide_variant_available(int n);
void wide_fragments(int n, const std::vector<double>& poly, std::vector<double>& frag);
bool build_maps_wide(const StepParams& p, TensorMapSet* maps);
int launch_step_wide(StepParams p, const TensorMapSet& maps, const double* p_frag /* device */, int sm_count,
                     cudaStream_t stream);
int launch_consensus_error(const StepParams& p, double* partials, double* result, int sm_count, cudaStream_t stream);
int launch_init_external(const StepParams& p, int sm_count, cudaStream_t stream);  // y = g = g_ext
int launch_expire_wait(int* status, unsigned polls, cudaStream_t stream);          // a wait nobody ends (self test)
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device; returns a cudaError_t value.
int ensure_dynamic_smem(const void* kernel, int bytes);

}  // namespace detag

struct detag_state {
  int n = 0;
  long long d = 0;
  int K = 0;
  double eta = 0.0, alpha = 0.0;
  std::vector<int32_t> row_ptr, col_idx;
  std::vector<double> vals;
  std::vector<double> poly;  // P_K(M) when n <= kMaxDenseWorkers
  bool circulant = false;    // every row of M is the previous one shifted by one
  int half_band = 0;         // of the circulant P_K(M): P[i][(i+delta) mod n] = 0 for |delta| > half_band
  double band[33] = {0};     // p(delta) at index delta + 16, valid when circulant and half_band <= 16
  std::vector<double> circ_row;  // first row of the circulant P_K(M) (kept when n <= 256)
  // block-circulant structure with 8-worker blocks, symmetric in the block distance (tori): the per-frequency
  // 8 x 8 polynomial blocks in MMA fragment order
  bool torus = false;
  std::vector<double> torus_frag;
  std::vector<double> wide_frag;  // 64 < n <= 128: P_K(M) as the warp strips of the register-resident kernel
  int variant_forced = DETAG_VARIANT_AUTO;
  int gradient_point = DETAG_GRADIENT_AT_NEW_MODEL;
  int algorithm = DETAG_ALGORITHM_DETAG;
  int gradient_source = DETAG_GRADIENT_SYNTHETIC;
  const float* g_ext = nullptr;
  unsigned spin_limit = 1u << 20;
  long long stall_after = -1;

  bool bound = false;
  long long ld = 0;
  float *x = nullptr, *y = nullptr, *g = nullptr;
  const float *a = nullptr, *c = nullptr;
  float* y_obs = nullptr;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int* d_status = nullptr;
  int* d_status_host = nullptr;  // status word of the staging area the last detag_step_host used
  double* d_result = nullptr;
  int32_t* d_row_ptr = nullptr;
  int32_t* d_col_idx = nullptr;
  double* d_vals = nullptr;
  double* d_poly = nullptr;
  double* d_torus = nullptr;
  double* d_circ_row = nullptr;
  double* d_wide = nullptr;
  double* d_partials = nullptr;

  double sigma = 0.0;
  uint64_t seed = 0;
  long long coord_offset = 0;
  long long t = 0;

  // host-resident stepping: two internal streams and their events, created on first use
  cudaStream_t host_stream[2] = {nullptr, nullptr};
  struct CUevent_st* host_event[3] = {nullptr, nullptr, nullptr};

  // tensor maps of the launches seen so far, keyed by kernel family and buffers (a few entries, round robin)
  struct MapEntry {
    int family = 0;
    const void* ptr[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    long long d = 0, ld = 0;
    detag::TensorMapSet maps;
  };
  std::vector<MapEntry> map_cache;
  size_t map_next = 0;

  int device = -1;
  int sm_count = 0;
  int smem_optin = 0;
  std::string err;
};

#endif  // DETAG_INTERNAL_H
