// Generic DeTAG step kernel: K accelerated-gossip rounds as neighbour-indexed sums over the CSR
// rows of M, on a coordinate slab of all n workers that is staged once in shared memory.
//
// Per slab of S coordinates a CTA
//   1. loads x and y for all n workers, widened to float64, into the "current" and "previous"
//      buffers (Algorithm 3 starts with z_{-1} = z_0),
//   2. runs K rounds  z_{r+1,i} = (1+eta) sum_j M[i][j] z_{r,j} - eta z_{r-1,i}  for both arrays;
//      the new value overwrites the previous-round slot of the same element, so two buffers
//      per array suffice and one barrier per round orders them,
//   3. finishes the step element-wise (Algorithm 2): x' = x~ - alpha y~, the stochastic gradient
//      g' = a (x' - c) + sigma xi at the new model, and the tracker fold y' = y~ + g' - g with the
//      float32 value of g' that is stored, so that the stored tracker telescopes exactly
//      against the stored gradients.
// All on-chip arithmetic is float64; each result is rounded once when it is stored.
//
// Modes: with caller-written gradients step 1 also applies Algorithm 2's tracker update, y + g_new - g_old, and
// step 3 stores the gossiped tracker and copies g_new over g_old instead of evaluating a gradient; in D-PSGD
// mode only the model is gossiped and x' = x~ - alpha g.
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"

namespace detag {

namespace {

constexpr int kCsrThreads = 256;

__host__ __device__ inline size_t csr_smem_bytes(int n, int nnz, int S) {
  // four slab buffers (x/y, current/previous) + values + row pointers + columns
  return static_cast<size_t>(4) * n * S * sizeof(double) + static_cast<size_t>(nnz) * sizeof(double) +
         static_cast<size_t>(n + 1 + nnz) * sizeof(int32_t);
}

__global__ void __launch_bounds__(kCsrThreads) step_csr_kernel(const StepParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n = p.n, S = p.S, NS = n * S, tid = threadIdx.x;
  double* cur_x = reinterpret_cast<double*>(smem_raw);
  double* cur_y = cur_x + NS;
  double* prv_x = cur_y + NS;
  double* prv_y = prv_x + NS;
  double* s_val = prv_y + NS;
  int32_t* s_row = reinterpret_cast<int32_t*>(s_val + p.nnz);
  int32_t* s_col = s_row + (n + 1);

  for (int k = tid; k < p.nnz; k += kCsrThreads) {
    s_val[k] = p.vals[k];
    s_col[k] = p.col_idx[k];
  }
  for (int k = tid; k <= n; k += kCsrThreads) s_row[k] = p.row_ptr[k];

  const double one_plus_eta = 1.0 + p.eta, eta = p.eta, alpha = p.alpha, sigma = p.sigma;
  const int nq = (n + 3) >> 2;

  for (long long slab = blockIdx.x; slab < p.num_slabs; slab += gridDim.x) {
    const long long j0 = slab * S;
    const int width = static_cast<int>(min(static_cast<long long>(S), p.d - j0));
    __syncthreads();  // the previous slab's epilogue has finished reading the buffers

    for (int e = tid; e < NS; e += kCsrThreads) {
      const int i = e >> p.log2S, col = e & (S - 1);
      double vx = 0.0, vy = 0.0;
      if (col < width) {
        const long long off = static_cast<long long>(i) * p.ld + j0 + col;
        vx = static_cast<double>(p.x[off]);
        if (p.mode != kModeDpsgd) vy = static_cast<double>(p.y[off]);
        if (p.mode == kModeExternal)  // Algorithm 2's tracker update with the caller's newest gradient
          vy += static_cast<double>(p.g_ext[off]) - static_cast<double>(p.g[off]);
      }
      cur_x[e] = vx;
      prv_x[e] = vx;
      cur_y[e] = vy;
      prv_y[e] = vy;
    }
    __syncthreads();

    double *cx = cur_x, *cy = cur_y, *px = prv_x, *py = prv_y;
    for (int r = 0; r < p.K; ++r) {
      for (int e = tid; e < NS; e += kCsrThreads) {
        const int i = e >> p.log2S, col = e & (S - 1);
        double ax = 0.0, ay = 0.0;
        const int k_end = s_row[i + 1];
        for (int k = s_row[i]; k < k_end; ++k) {
          const double w = s_val[k];
          const int src = (s_col[k] << p.log2S) + col;
          ax = fma(w, cx[src], ax);
          ay = fma(w, cy[src], ay);
        }
        px[e] = fma(one_plus_eta, ax, -eta * px[e]);
        py[e] = fma(one_plus_eta, ay, -eta * py[e]);  // D-PSGD: an all-zero slab, never stored
      }
      __syncthreads();
      double* t;
      t = cx; cx = px; px = t;
      t = cy; cy = py; py = t;
    }

    // element-wise tail of the step; a thread takes the four workers 4q..4q+3 of one coordinate
    for (int it = tid; it < nq * S; it += kCsrThreads) {
      const int q = it >> p.log2S, col = it & (S - 1);
      if (col >= width) continue;
      const long long j = j0 + col;
      float xi[4] = {0.f, 0.f, 0.f, 0.f};
      if (sigma != 0.0 && p.mode != kModeExternal)
        normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j), q, p.t_noise, xi);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int i = 4 * q + w;
        if (i < n) {
          const long long off = static_cast<long long>(i) * p.ld + j;
          if (p.mode == kModeExternal) {
            const double y_gossip = cy[i * S + col];
            p.x[off] = static_cast<float>(cx[i * S + col] - alpha * y_gossip);
            p.y[off] = static_cast<float>(y_gossip);
            p.g[off] = p.g_ext[off];  // the gradient just folded is the next step's g_old
            if (p.y_obs != nullptr) p.y_obs[off] = static_cast<float>(y_gossip);
            continue;
          }
          if (p.mode == kModeDpsgd) {
            const double x_new = cx[i * S + col] - alpha * static_cast<double>(p.g[off]);
            const float x_new_f = static_cast<float>(x_new);
            const double g_new = fma(static_cast<double>(p.a[off]), x_new - static_cast<double>(p.c[off]),
                                     sigma * static_cast<double>(xi[w]));
            p.x[off] = x_new_f;
            p.g[off] = static_cast<float>(g_new);
            continue;
          }
          const double y_gossip = cy[i * S + col];
          const double x_new = cx[i * S + col] - alpha * y_gossip;
          // gradient point: the new model, or (Algorithm 2 as printed) the model this step started from,
          // which is still in global memory because this thread overwrites it only below
          const double x_at = p.grad_at_start ? static_cast<double>(p.x[off]) : x_new;
          const double g_new = fma(static_cast<double>(p.a[off]), x_at - static_cast<double>(p.c[off]),
                                   sigma * static_cast<double>(xi[w]));
          const float g_new_f = static_cast<float>(g_new);
          const double y_new = y_gossip + (static_cast<double>(g_new_f) - static_cast<double>(p.g[off]));
          p.x[off] = static_cast<float>(x_new);
          p.y[off] = static_cast<float>(y_new);
          p.g[off] = g_new_f;
          if (p.y_obs != nullptr) p.y_obs[off] = static_cast<float>(y_gossip);
        }
      }
    }
  }
}

}  // namespace

int plan_step_csr(StepParams& p, int smem_optin_bytes) {
  // Largest power-of-two slab (<= 128 coordinates) whose buffers leave room for two CTAs per SM;
  // fall back to one CTA per SM with the widest slab that fits at all.
  const size_t two_cta_budget = 110 * 1024;
  int best = 0;
  for (int S = 128; S >= 4; S >>= 1)
    if (csr_smem_bytes(p.n, p.nnz, S) <= two_cta_budget) { best = S; break; }
  if (best < 16) {
    for (int S = 16; S >= 4; S >>= 1)
      if (csr_smem_bytes(p.n, p.nnz, S) <= static_cast<size_t>(smem_optin_bytes)) { best = S; break; }
  }
  if (best == 0) return DETAG_ERR_UNSUPPORTED;
  p.S = best;
  p.log2S = 0;
  while ((1 << p.log2S) < best) ++p.log2S;
  p.num_slabs = (p.d + best - 1) / best;
  return DETAG_OK;
}

int launch_step_csr(const StepParams& p, int sm_count, cudaStream_t stream) {
  const size_t smem = csr_smem_bytes(p.n, p.nnz, p.S);
  const int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(step_csr_kernel), static_cast<int>(smem));
  if (rc != 0) return rc;
  int per_sm = 1;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, step_csr_kernel, kCsrThreads, smem);
  if (e != cudaSuccess) return static_cast<int>(e);
  if (per_sm < 1) per_sm = 1;
  const long long grid = p.num_slabs < static_cast<long long>(sm_count) * per_sm
                             ? p.num_slabs
                             : static_cast<long long>(sm_count) * per_sm;
  if (grid <= 0) return 0;
  step_csr_kernel<<<static_cast<unsigned>(grid), kCsrThreads, smem, stream>>>(p);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
