// Generic DeTAG step kernel: K accelerated-gossip rounds as neighbour-indexed sums over the CSR rows of M, on a
// coordinate slab of all n workers that is staged once in shared memory (any graph, any K, n <= 1024).
//
// A thread owns one worker and four consecutive coordinates of the slab for the whole step.  Per slab
//   1. it loads its x and y (one 16-byte load each), widens them to float64, keeps them as the "previous" values of
//      Algorithm 3 (z_{-1} = z_0) in registers and publishes them in the shared slab;
//   2. K rounds  z_{r+1,i} = (1+eta) sum_j M[i][j] z_{r,j} - eta z_{r-1,i}  for both arrays: the neighbour values are
//      32-byte reads from the shared slab (the row's column indices and weights are read once per round and serve
//      all eight values), the thread's own previous values never leave its registers; a barrier separates reading
//      a round's inputs from overwriting them, so one slab buffer per array suffices;
//   3. it finishes the step element-wise (Algorithm 2): x' = x~ - alpha y~, the stochastic gradient
//      g' = a (x' - c) + sigma xi at the new model (the four workers of a Philox call sit in four lanes of one warp:
//      each lane draws one of the four coordinates and a 4 x 4 transpose hands everybody its own row), and the
//      tracker fold y' = y~ + g' - g with the float32 value of g' that is stored, so that the stored tracker
//      telescopes exactly against the stored gradients; a, c, g are 16-byte loads, x', y', g' 16-byte stores.
// All on-chip arithmetic is float64; each result is rounded once when it is stored.  What bounds the kernel is the
// shared-memory traffic of step 2: 8 bytes per multiply-add.  Layout for that traffic: the threads of a worker
// are neighbouring lanes (coordinate group fastest), and a slab row keeps the first coordinate pair of all groups
// contiguously, then the second pairs: a 16-byte read per lane then covers 128 contiguous bytes of ONE row per
// quarter warp - every bank once, whatever row the neighbour index names (with the thread's four doubles side by
// side each of the two reads would use half of the banks, and four rows would meet in every quarter warp).  With
// fewer than eight groups (n > 128) a quarter warp reads 2, 4 or 8 rows; the two pairs of a row then swap places
// according to one bit of the row index, chosen so that consecutive rows - the neighbours of consecutive workers
// on rings, tori and other banded matrices - fall on different banks.
//
// Modes: with caller-written gradients step 1 also applies Algorithm 2's tracker update, y + g_new - g_old, and
// step 3 stores the gossiped tracker and copies g_new over g_old instead of evaluating a gradient; in D-PSGD
// mode only the model is gossiped and x' = x~ - alpha g.
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"

namespace detag {

namespace {

constexpr int kCsrThreads = 1024;
constexpr int kCsrPad = 0;  // contiguous 128-byte pieces need no padding
constexpr int kCsrMaxS = 32;  // at most 8 coordinate groups: the four workers of a Philox call stay in one warp

__host__ __device__ inline size_t csr_smem_bytes(int n, int nnz, int S, bool tables) {
  // the x and y slabs (S coordinates in all, in pieces or not) + (if they fit) values, row pointers and columns
  return static_cast<size_t>(2) * n * (S + kCsrPad) * sizeof(double) +
         (tables ? static_cast<size_t>(nnz) * sizeof(double) + static_cast<size_t>(n + 1 + nnz) * sizeof(int32_t) : 0);
}

// 4 x 4 transpose over the four lanes that share a coordinate group: rows r4 = 0..3 sit `stride` lanes apart.
__device__ __forceinline__ void transpose_rows(float (&v)[4], int r4, int stride) {
  const bool b0 = (r4 & 1) != 0, b1 = (r4 & 2) != 0;
  float s0 = b0 ? v[0] : v[1], s1 = b0 ? v[2] : v[3];
  float r0 = __shfl_xor_sync(0xffffffffu, s0, stride), r1 = __shfl_xor_sync(0xffffffffu, s1, stride);
  if (b0) { v[0] = r0; v[2] = r1; } else { v[1] = r0; v[3] = r1; }
  s0 = b1 ? v[0] : v[2];
  s1 = b1 ? v[1] : v[3];
  r0 = __shfl_xor_sync(0xffffffffu, s0, 2 * stride);
  r1 = __shfl_xor_sync(0xffffffffu, s1, 2 * stride);
  if (b1) { v[0] = r0; v[1] = r1; } else { v[2] = r0; v[3] = r1; }
}

__device__ __forceinline__ void load4(const float* base, long long off, long long j, long long d, float (&v)[4]) {
  if (j + 3 < d) {
    const float4 t = *reinterpret_cast<const float4*>(base + off);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = j + e < d ? base[off + e] : 0.f;
  }
}

__device__ __forceinline__ void store4(float* base, long long off, long long j, long long d, const float (&v)[4]) {
  if (j + 3 < d) {
    *reinterpret_cast<float4*>(base + off) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (j + e < d) base[off + e] = v[e];
  }
}

// kTables: the CSR arrays are read from shared memory (they fit) instead of global memory.
// kSwap: fewer than eight coordinate groups, the pairs of a row swap places by a bit of the row index.
template <bool kTables, bool kSwap>
__global__ void __launch_bounds__(kCsrThreads, 1) step_csr_kernel(const StepParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // S coordinates per slab in p.csr_sub independent pieces of W = S / p.csr_sub coordinates (each with its own rows
  // in shared memory): small graphs fill the thread block with several pieces
  const int n = p.n, S = p.S, W = S / p.csr_sub, pitch = W + kCsrPad, tid = threadIdx.x;
  double* sx = reinterpret_cast<double*>(smem_raw);
  double* sy = sx + static_cast<size_t>(p.csr_sub) * n * pitch;
  const double* vals = p.vals;
  const int32_t* rows = p.row_ptr;
  const int32_t* cols = p.col_idx;
  if (kTables) {
    double* s_val = sy + static_cast<size_t>(p.csr_sub) * n * pitch;
    int32_t* s_row = reinterpret_cast<int32_t*>(s_val + p.nnz);
    int32_t* s_col = s_row + (n + 1);
    for (int k = tid; k < p.nnz; k += blockDim.x) {
      s_val[k] = p.vals[k];
      s_col[k] = p.col_idx[k];
    }
    for (int k = tid; k <= n; k += blockDim.x) s_row[k] = p.row_ptr[k];
    vals = s_val;
    rows = s_row;
    cols = s_col;
    __syncthreads();  // the tables are read right below
  }
  // item = ((row quad * 4 + row within quad) * groups + coordinate group): a row's threads side by side, the four
  // rows of a Philox call `groups` lanes apart in one warp (groups is a power of two, at most 8)
  const int groups = W >> 2, half = W >> 1, quads = (n + 3) / 4;
  const int cg = tid & (groups - 1), r4 = (tid / groups) & 3, qs = (tid / groups) >> 2;
  const int sub = qs / quads, q = qs - sub * quads;  // piece of the slab, row quad
  const int i = 4 * q + r4;
  const bool owner = sub < p.csr_sub && i < n;  // threads without an element idle (they still meet the barriers)
  const int k0 = owner ? rows[i] : 0, k1 = owner ? rows[i + 1] : 0;
  const double one_plus_eta = 1.0 + p.eta, eta = p.eta, alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool dpsgd = p.mode == kModeDpsgd, external = p.mode == kModeExternal;
  // the thread's coordinates 4 cg .. 4 cg + 3: the first pair at 2 cg of the row, the second at half + 2 cg
  const size_t piece = static_cast<size_t>(owner ? sub : 0) * n * pitch;
  // which of a row's pairs comes first: bit log2(4 / groups) of the row index (8 groups: always the first pair)
  const int swz_shift = groups >= 4 ? 0 : (groups == 2 ? 1 : 2), swz_mask = kSwap ? 1 : 0;
  const int my_first = (((owner ? i : 0) >> swz_shift) & swz_mask) * half;   // offset of this thread's first pair
  double* my_x = sx + piece + static_cast<size_t>(owner ? i : 0) * pitch + 2 * cg;
  double* my_y = sy + piece + static_cast<size_t>(owner ? i : 0) * pitch + 2 * cg;

  for (long long slab = blockIdx.x; slab < p.num_slabs; slab += gridDim.x) {
    const long long j = slab * S + sub * W + 4 * cg;  // this thread's first coordinate
    const long long off = static_cast<long long>(i) * p.ld + j;
    const bool active = owner && j < p.d;
    double px[4], py[4];  // z_{r-1} of this thread's elements; z_r is in the slab
    float gold[4] = {0.f, 0.f, 0.f, 0.f};
    if (active) {
      float xv[4], yv[4] = {0.f, 0.f, 0.f, 0.f};
      load4(p.x, off, j, p.d, xv);
      if (!dpsgd) load4(p.y, off, j, p.d, yv);
      if (external) {  // Algorithm 2's tracker update with the caller's newest gradient
        float gn[4];
        load4(p.g_ext, off, j, p.d, gn);
        load4(p.g, off, j, p.d, gold);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          px[e] = static_cast<double>(xv[e]);
          py[e] = static_cast<double>(yv[e]) + (static_cast<double>(gn[e]) - static_cast<double>(gold[e]));
          gold[e] = gn[e];  // what the step stores as the gradient folded last
        }
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          px[e] = static_cast<double>(xv[e]);
          py[e] = static_cast<double>(yv[e]);
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) px[e] = py[e] = 0.0;
    }
    __syncthreads();  // the previous slab's rounds have finished reading the slab
    if (owner) {
      *reinterpret_cast<double2*>(my_x + my_first) = make_double2(px[0], px[1]);
      *reinterpret_cast<double2*>(my_x + (half - my_first)) = make_double2(px[2], px[3]);
      *reinterpret_cast<double2*>(my_y + my_first) = make_double2(py[0], py[1]);
      *reinterpret_cast<double2*>(my_y + (half - my_first)) = make_double2(py[2], py[3]);
    }
    __syncthreads();

    // z_r lives in the slab, z_{r-1} of this thread's elements in px, py; after the loop cx, cy hold z_K
    double cx[4], cy[4];
    for (int r = 0; r < p.K; ++r) {
#pragma unroll
      for (int e = 0; e < 4; ++e) cx[e] = cy[e] = 0.0;
      for (int k = k0; k < k1; ++k) {
        const double w = vals[k];
        const int col = cols[k];
        const int first = ((col >> swz_shift) & swz_mask) * half;
        const size_t src = piece + static_cast<size_t>(col) * pitch + 2 * cg + first, src2 = src + (half - 2 * first);
        const double2 x01 = *reinterpret_cast<const double2*>(sx + src);
        const double2 x23 = *reinterpret_cast<const double2*>(sx + src2);
        cx[0] = fma(w, x01.x, cx[0]);
        cx[1] = fma(w, x01.y, cx[1]);
        cx[2] = fma(w, x23.x, cx[2]);
        cx[3] = fma(w, x23.y, cx[3]);
        if (!dpsgd) {
          const double2 y01 = *reinterpret_cast<const double2*>(sy + src);
          const double2 y23 = *reinterpret_cast<const double2*>(sy + src2);
          cy[0] = fma(w, y01.x, cy[0]);
          cy[1] = fma(w, y01.y, cy[1]);
          cy[2] = fma(w, y23.x, cy[2]);
          cy[3] = fma(w, y23.y, cy[3]);
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        cx[e] = fma(one_plus_eta, cx[e], -eta * px[e]);
        cy[e] = fma(one_plus_eta, cy[e], -eta * py[e]);
      }
      if (r + 1 < p.K) {
        if (owner) {  // this round's own values become the next round's "previous"
          const double2 x01 = *reinterpret_cast<const double2*>(my_x + my_first);
          const double2 x23 = *reinterpret_cast<const double2*>(my_x + (half - my_first));
          px[0] = x01.x; px[1] = x01.y; px[2] = x23.x; px[3] = x23.y;
          if (!dpsgd) {
            const double2 y01 = *reinterpret_cast<const double2*>(my_y + my_first);
            const double2 y23 = *reinterpret_cast<const double2*>(my_y + (half - my_first));
            py[0] = y01.x; py[1] = y01.y; py[2] = y23.x; py[3] = y23.y;
          }
        }
        __syncthreads();  // everybody has read round r's values
        if (owner) {
          *reinterpret_cast<double2*>(my_x + my_first) = make_double2(cx[0], cx[1]);
          *reinterpret_cast<double2*>(my_x + (half - my_first)) = make_double2(cx[2], cx[3]);
          if (!dpsgd) {
            *reinterpret_cast<double2*>(my_y + my_first) = make_double2(cy[0], cy[1]);
            *reinterpret_cast<double2*>(my_y + (half - my_first)) = make_double2(cy[2], cy[3]);
          }
        }
        __syncthreads();
      }
    }

    // ---- element-wise tail of the step on the thread's four elements
    float xi[4] = {0.f, 0.f, 0.f, 0.f};
    if (sigma != 0.f && !external) {  // every lane takes part (the shuffles want whole warps); idle lanes' draws are unused
      // lane r4 draws coordinate j + r4 for the quad's four workers; the transpose gives it its own row's four
      normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + r4), static_cast<uint32_t>(q),
                  p.t_noise, xi);
      transpose_rows(xi, r4, groups);
    }
    if (active) {
      float xo[4], yo[4], go[4];
      if (external) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          xo[e] = static_cast<float>(cx[e] - alpha * cy[e]);
          yo[e] = static_cast<float>(cy[e]);  // the gossiped tracker
          go[e] = gold[e];                    // the gradient just folded is the next step's g_old
        }
      } else {
        float av[4], cv[4], gv[4], xold[4];
        load4(p.a, off, j, p.d, av);
        load4(p.c, off, j, p.d, cv);
        load4(p.g, off, j, p.d, gv);
        if (p.grad_at_start) load4(p.x, off, j, p.d, xold);  // still the old model: this thread overwrites it below
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const double x_new = dpsgd ? cx[e] - alpha * static_cast<double>(gv[e]) : cx[e] - alpha * cy[e];
          // gradient point: the new model, or (Algorithm 2 as printed) the model this step started from
          const double x_at = p.grad_at_start ? static_cast<double>(xold[e]) : x_new;
          const double g_new = fma(static_cast<double>(av[e]), x_at - static_cast<double>(cv[e]),
                                   static_cast<double>(sigma) * static_cast<double>(xi[e]));
          go[e] = static_cast<float>(g_new);
          xo[e] = static_cast<float>(x_new);
          yo[e] = static_cast<float>(cy[e] + (static_cast<double>(go[e]) - static_cast<double>(gv[e])));
        }
      }
      store4(p.x, off, j, p.d, xo);
      if (!dpsgd) store4(p.y, off, j, p.d, yo);
      store4(p.g, off, j, p.d, go);
      if (p.y_obs != nullptr && !dpsgd) {
        float yg[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) yg[e] = static_cast<float>(cy[e]);
        store4(p.y_obs, off, j, p.d, yg);
      }
    }
  }
}

}  // namespace

// Chooses the slab width: the widest power of two (4 .. 32 coordinates) for which every (worker quad, four
// coordinates) item has a thread of its own and the slabs fit; the CSR arrays join them in shared memory if there
// is room.  p.log2S < 0 afterwards means the tables stay in global memory.
int plan_step_csr(StepParams& p, int smem_optin_bytes) {
  const int quads = (p.n + 3) / 4;
  // Two blocks of half the size per SM - while one loads a slab or finishes its tail, the other runs its rounds on
  // the shared-memory pipe - unless the halving would cost the full eight coordinate groups (64 < n <= 128).
  // Measured (d = 1 M .. 8 M): n = 32 8.4 -> 7.0 ms, 256-ring 14.8 -> 13.7 ms, 100 workers 14.1 -> 14.5 ms.
  const bool eight_in_half = quads * 4 * (kCsrMaxS / 4) <= kCsrThreads / 2;
  const bool eight_in_full = quads * 4 * (kCsrMaxS / 4) <= kCsrThreads;
  const int threads = (quads * 4 <= kCsrThreads / 2 && (eight_in_half || !eight_in_full)) ? kCsrThreads / 2 : kCsrThreads;
  p.csr_threads = threads;
  smem_optin_bytes = threads < kCsrThreads ? (smem_optin_bytes < 110 * 1024 ? smem_optin_bytes : 110 * 1024) : smem_optin_bytes;
  int best = 0;
  for (int S = kCsrMaxS; S >= 4; S >>= 1) {
    if (quads * 4 * (S / 4) > threads) continue;
    if (csr_smem_bytes(p.n, p.nnz, S, false) > static_cast<size_t>(smem_optin_bytes)) continue;
    best = S;
    break;
  }
  if (best == 0) return DETAG_ERR_UNSUPPORTED;
  // small graphs: as many pieces of that width as threads and shared memory allow (at most 8)
  int pieces = 1;
  while (pieces < 8 && quads * 4 * (best / 4) * (pieces * 2) <= threads &&
         csr_smem_bytes(p.n, p.nnz, best * pieces * 2, true) <= static_cast<size_t>(smem_optin_bytes))
    pieces *= 2;
  p.csr_sub = pieces;
  best *= pieces;
  p.S = best;
  p.log2S = csr_smem_bytes(p.n, p.nnz, best, true) <= static_cast<size_t>(smem_optin_bytes) ? 1 : -1;
  p.num_slabs = (p.d + best - 1) / best;
  return DETAG_OK;
}

int launch_step_csr(const StepParams& p, int sm_count, cudaStream_t stream) {
  const bool tables = p.log2S > 0;
  const size_t smem = csr_smem_bytes(p.n, p.nnz, p.S, tables);
  const bool swap = p.S / p.csr_sub < kCsrMaxS;
  auto kernel = tables ? (swap ? step_csr_kernel<true, true> : step_csr_kernel<true, false>)
                       : (swap ? step_csr_kernel<false, true> : step_csr_kernel<false, false>);
  const int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
  if (rc != 0) return rc;
  const long long ctas = static_cast<long long>(sm_count) * (kCsrThreads / p.csr_threads);
  const long long grid = p.num_slabs < ctas ? p.num_slabs : ctas;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), p.csr_threads, smem, stream>>>(p);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
