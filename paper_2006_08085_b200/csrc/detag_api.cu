// Host side of the C ABI declared in include/detag.h: argument checking, the host-side numerics
// (momentum, polynomial of the gossip matrix), workspace layout and kernel launches.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "detag_internal.h"
#include "torus_basis.h"

using detag::StepParams;

namespace {

size_t align_up(size_t v) { return (v + detag::kWsAlign - 1) / detag::kWsAlign * detag::kWsAlign; }

struct WsLayout {
  size_t status, result, row_ptr, col_idx, vals, poly, torus, circ_row, wide, partials, total;
};

WsLayout ws_layout(const detag_state* s) {
  WsLayout l{};
  size_t off = 0;
  l.status = off;
  l.result = off + 64;
  off += detag::kWsAlign;
  l.row_ptr = off;
  off += align_up((s->n + 1) * sizeof(int32_t));
  l.col_idx = off;
  off += align_up(s->col_idx.size() * sizeof(int32_t));
  l.vals = off;
  off += align_up(s->vals.size() * sizeof(double));
  l.poly = off;
  off += align_up(s->poly.size() * sizeof(double));
  l.torus = off;
  off += align_up(s->torus_frag.size() * sizeof(double));
  l.circ_row = off;
  off += align_up(s->circ_row.size() * sizeof(double));
  l.wide = off;
  off += align_up(s->wide_frag.size() * sizeof(double));
  l.partials = off;
  off += align_up(detag::kMaxPartials * sizeof(double));
  l.total = off;
  return l;
}

int fail(detag_state* s, int code, const char* what) {
  if (s) s->err = what;
  return code;
}

int fail_cuda(detag_state* s, int cuda_code, const char* where) {
  if (s) {
    char buf[256];
    std::snprintf(buf, sizeof buf, "%s: %s", where, cudaGetErrorString(static_cast<cudaError_t>(cuda_code)));
    s->err = buf;
  }
  return DETAG_ERR_CUDA;
}

// P_K(M) by the matrix form of Algorithm 3: P_{-1} = P_0 = I, P_{r+1} = (1+eta) M P_r - eta P_{r-1}.
void gossip_polynomial(const detag_state* s, std::vector<double>& out) {
  const int n = s->n;
  std::vector<double> prev(static_cast<size_t>(n) * n, 0.0), cur, next(static_cast<size_t>(n) * n);
  for (int i = 0; i < n; ++i) prev[static_cast<size_t>(i) * n + i] = 1.0;
  cur = prev;
  for (int r = 0; r < s->K; ++r) {
    for (int i = 0; i < n; ++i) {
      for (int j = 0; j < n; ++j) {
        double acc = 0.0;
        for (int k = s->row_ptr[i]; k < s->row_ptr[i + 1]; ++k)
          acc += s->vals[k] * cur[static_cast<size_t>(s->col_idx[k]) * n + j];
        next[static_cast<size_t>(i) * n + j] = (1.0 + s->eta) * acc - s->eta * prev[static_cast<size_t>(i) * n + j];
      }
    }
    prev.swap(cur);
    cur.swap(next);
  }
  out = cur;
}

// Circulant M (row i = row 0 shifted by i): then P_K(M) is circulant too; its row 0 is computed with the
// recursion of Algorithm 3 on a single row and stored as a band around the diagonal.
void analyse_circulant(detag_state* s) {
  const int n = s->n;
  std::vector<double> row0(n, 0.0);
  for (int k = s->row_ptr[0]; k < s->row_ptr[1]; ++k) row0[s->col_idx[k]] = s->vals[k];
  for (int i = 1; i < n; ++i) {
    if (s->row_ptr[i + 1] - s->row_ptr[i] != s->row_ptr[1] - s->row_ptr[0]) return;
    for (int k = s->row_ptr[i]; k < s->row_ptr[i + 1]; ++k)
      if (s->vals[k] != row0[((s->col_idx[k] - i) % n + n) % n]) return;
  }
  s->circulant = true;
  // row 0 of P_r: q_{r+1}[j] = (1+eta) sum_k M[0][k] q_r[(j - k) mod n] - eta q_{r-1}[j]   (circulant product)
  std::vector<double> prev(n, 0.0), cur, next(n);
  prev[0] = 1.0;
  cur = prev;
  for (int r = 0; r < s->K; ++r) {
    for (int j = 0; j < n; ++j) {
      double acc = 0.0;
      for (int k = s->row_ptr[0]; k < s->row_ptr[1]; ++k)
        acc += s->vals[k] * cur[((j - s->col_idx[k]) % n + n) % n];
      next[j] = (1.0 + s->eta) * acc - s->eta * prev[j];
    }
    prev.swap(cur);
    cur.swap(next);
  }
  int hb = 0;
  for (int j = 0; j < n; ++j)
    if (cur[j] != 0.0) {
      const int delta = j <= n / 2 ? j : n - j;
      if (delta > hb) hb = delta;
    }
  s->half_band = hb;
  if (n <= 256) s->circ_row = cur;  // p(0 .. n-1): the dense mode of the circulant kernel looks its fragments up here
  if (hb <= 16 && n >= 2 * hb + 1)
    for (int delta = -16; delta <= 16; ++delta)
      s->band[delta + 16] = (delta >= -hb && delta <= hb) ? cur[((delta % n) + n) % n] : 0.0;
}

// Block-circulant M with 8-worker blocks whose block (r, r') depends on the distance (r' - r) mod R only, equal for
// +k and -k (tori): the real Fourier basis Q of the R-cycle block-diagonalises every polynomial of M,
//     P_K(M) = sum_p (q_p q_p^T) (x) P_K(Mhat_p) ,   Mhat_p = sum_k cos(2 pi f_p k / R) G_k .
// The 8 x 8 blocks P_K(Mhat_p) come from the recursion of Algorithm 3 on Mhat_p; the result is accepted only if it
// reproduces the dense polynomial.
void analyse_torus(detag_state* s) {
  const int n = s->n, C = 8;
  if (s->poly.empty() || n % C != 0 || !detag::torus_variant_available(n)) return;
  const int R = n / C;
  std::vector<double> m;
  detag::csr_to_dense(n, s->row_ptr.data(), s->col_idx.data(), s->vals.data(), m);
  auto M = [&](int r, int c, int r2, int c2) { return m[static_cast<size_t>(r * C + c) * n + (r2 * C + c2)]; };
  for (int r = 0; r < R; ++r)
    for (int k = 0; k < R; ++k)
      for (int c = 0; c < C; ++c)
        for (int c2 = 0; c2 < C; ++c2) {
          if (M(r, c, (r + k) % R, c2) != M(0, c, k, c2)) return;        // block circulant
          if (M(0, c, k, c2) != M(0, c, (R - k) % R, c2)) return;        // the same block at distance +k and -k
        }
  const double kPi = 3.14159265358979323846;
  std::vector<double> q(static_cast<size_t>(R) * R);  // the kernel's basis, row p = basis vector p
  std::vector<int> freq(R);
  for (int p = 0; p < R; ++p) {
    freq[p] = detag::torus_frequency(R, p);
    for (int r = 0; r < R; ++r) q[p * R + r] = detag::torus_q(R, p, r);
  }
  std::vector<double> phat(static_cast<size_t>(R) * C * C);
  for (int p = 0; p < R; ++p) {
    double mh[8][8], prev[8][8], cur[8][8], next[8][8];
    for (int c = 0; c < C; ++c)
      for (int c2 = 0; c2 < C; ++c2) {
        double acc = 0.0;
        for (int k = 0; k < R; ++k) acc += std::cos(2.0 * kPi * freq[p] * k / R) * M(0, c, k, c2);
        mh[c][c2] = acc;
        prev[c][c2] = cur[c][c2] = c == c2 ? 1.0 : 0.0;
      }
    for (int round = 0; round < s->K; ++round) {  // P_{r+1} = (1+eta) Mhat P_r - eta P_{r-1}
      for (int c = 0; c < C; ++c)
        for (int c2 = 0; c2 < C; ++c2) {
          double acc = 0.0;
          for (int k = 0; k < C; ++k) acc += mh[c][k] * cur[k][c2];
          next[c][c2] = (1.0 + s->eta) * acc - s->eta * prev[c][c2];
        }
      std::memcpy(prev, cur, sizeof cur);
      std::memcpy(cur, next, sizeof cur);
    }
    for (int c = 0; c < C; ++c)
      for (int c2 = 0; c2 < C; ++c2) phat[(static_cast<size_t>(p) * C + c) * C + c2] = cur[c][c2];
  }
  // the decomposition must give back the dense polynomial
  double worst = 0.0, scale = 0.0;
  for (int r = 0; r < R; ++r)
    for (int r2 = 0; r2 < R; ++r2)
      for (int c = 0; c < C; ++c)
        for (int c2 = 0; c2 < C; ++c2) {
          double acc = 0.0;
          for (int p = 0; p < R; ++p) acc += q[p * R + r] * q[p * R + r2] * phat[(static_cast<size_t>(p) * C + c) * C + c2];
          const double want = s->poly[static_cast<size_t>(r * C + c) * n + (r2 * C + c2)];
          worst = std::fmax(worst, std::fabs(acc - want));
          scale = std::fmax(scale, std::fabs(want));
        }
  if (!(worst <= 1e-13 * std::fmax(1.0, scale))) return;
  s->torus = true;
  // fragment order of the kernel: entry (p, k-step s, lane) is Phat_p[c'][c] with the contraction index
  // c = lane % 4 + 4 s and the output position c' = pi(lane / 4), pi(2 q + e) = q + 4 e (see step_torus.cu)
  s->torus_frag.resize(static_cast<size_t>(R) * 2 * 32);
  // For R = 8 the kernel's butterflies leave out the basis' normalisation (1/sqrt(8) for the constant and the
  // alternating vector, 1/2 for the others) on the way in and on the way out: both factors go into the block.
  for (int p = 0; p < R; ++p) {
    const double scale = R == 8 ? ((p == 0 || p == R - 1) ? 0.125 : 0.25) : 1.0;
    for (int st = 0; st < 2; ++st)
      for (int lane = 0; lane < 32; ++lane)
        s->torus_frag[(static_cast<size_t>(p) * 2 + st) * 32 + lane] =
            scale * phat[(static_cast<size_t>(p) * C + ((lane / 4) >> 1) + 4 * ((lane / 4) & 1)) * C + (lane % 4) + 4 * st];
  }
}

bool torus_ok(const detag_state* s) { return s->torus && s->d <= 0x7fffffffLL; }

// The circulant kernel: band mode while the polynomial's half-band is at most 16, dense mode (n <= 256) beyond.
bool ring_band(const detag_state* s) { return detag::ring_variant_available(s->n, s->half_band); }

bool band_ok(const detag_state* s) {
  return s->circulant && s->d <= 0x7fffffffLL && (ring_band(s) || detag::ring_dense_available(s->n));
}

int step_mode(const detag_state* s) {
  if (s->algorithm == DETAG_ALGORITHM_DPSGD) return detag::kModeDpsgd;
  return s->gradient_source == DETAG_GRADIENT_EXTERNAL ? detag::kModeExternal : detag::kModeDetag;
}

StepParams make_params(const detag_state* s) {
  StepParams p{};
  p.n = s->n;
  p.nnz = static_cast<int>(s->col_idx.size());
  p.K = s->K;
  p.d = s->d;
  p.ld = s->ld;
  p.coord_offset = s->coord_offset;
  p.x = s->x;
  p.y = s->y;
  p.g = s->g;
  p.a = s->a;
  p.c = s->c;
  p.y_obs = s->y_obs;
  p.row_ptr = s->d_row_ptr;
  p.col_idx = s->d_col_idx;
  p.vals = s->d_vals;
  p.poly = s->d_poly;
  p.torus = s->d_torus;
  p.circ_row = s->d_circ_row;
  p.wide = s->d_wide;
  p.eta = s->eta;
  p.alpha = s->alpha;
  p.sigma = s->sigma;
  p.seed_lo = static_cast<uint32_t>(s->seed & 0xffffffffu);
  p.seed_hi = static_cast<uint32_t>(s->seed >> 32);
  p.status = s->d_status;
  p.grad_at_start = s->gradient_point == DETAG_GRADIENT_AT_PHASE_START ? 1 : 0;
  p.mode = step_mode(s);
  p.g_ext = s->g_ext;
  p.spin_limit = s->spin_limit;
  p.stall_after = s->stall_after;
  return p;
}

bool dense_ok(const detag_state* s) {
  if (s->d > 0x7fffffffLL) return false;
  return (!s->poly.empty() && detag::dense_variant_available(s->n)) ||
         (!s->wide_frag.empty() && detag::wide_variant_available(s->n));
}

// Host cost model.  The dense product needs n multiply-adds per element and array against the sparse
// rounds' K*(nnz per row), but keeps its outputs in registers and needs no barriers; it wins for every
// n it supports - except that for 32 < n <= 64 a circulant matrix with a narrow band is cheaper through the
// band kernel (80 instead of 128 MMAs per tile).  Caller-written gradients and D-PSGD run on the dense
// kernel for n <= 32 and on the generic rounds kernel otherwise.
// for 32 < n <= 64 a block-circulant matrix (torus) takes the transform kernel: 24 multiply-adds per element
// and array instead of 64.
bool variant_runs_mode(const detag_state* s, int variant) {
  if (step_mode(s) == detag::kModeDetag) return true;
  if (variant == DETAG_VARIANT_RING) return step_mode(s) == detag::kModeDpsgd;
  return variant == DETAG_VARIANT_CSR || (variant == DETAG_VARIANT_DENSE && s->n <= 32);  // n > 32: DeTAG step only
}

int resolve_variant(const detag_state* s) {
  if (s->variant_forced != DETAG_VARIANT_AUTO) return s->variant_forced;
  // a ring whose band fits takes the circulant kernel from n = 64 on; with a dense polynomial only beyond the
  // reach of the 64-row dense kernel
  const bool ring = band_ok(s) && (ring_band(s) || s->n > detag::kMaxDenseWorkers);
  if (step_mode(s) == detag::kModeDpsgd && s->n > 32 && ring) return DETAG_VARIANT_RING;
  if (step_mode(s) != detag::kModeDetag) return (s->n <= 32 && dense_ok(s)) ? DETAG_VARIANT_DENSE : DETAG_VARIANT_CSR;
  if (s->n > 32 && ring) return DETAG_VARIANT_RING;
  if (s->n > 32 && torus_ok(s)) return DETAG_VARIANT_TORUS;
  if (dense_ok(s)) {
    if (s->n > detag::kMaxDenseWorkers) {
      // Register-resident polynomial against the sparse rounds, both measured at d = 2 M (ms): the dense kernel is
      // bound by one warp scheduler's share of the MMAs - blocks / 4 strips (the next multiple of four when one
      // scheduler is a block short) of n / 4 k-steps - the rounds kernel by a per-worker part and K * nnz
      // shared-memory gathers.  The rounds win at one or two rounds on graphs of degree four.
      const int blocks = (s->n + 7) / 8, blocks_eff = blocks % 4 == 3 ? blocks + 1 : blocks;
      const double dense_ms = 0.0412 * blocks_eff * blocks / 2.0;
      const double rounds_ms = 0.024 * s->n + 0.00155 * s->K * static_cast<double>(s->col_idx.size());
      if (rounds_ms < dense_ms) return DETAG_VARIANT_CSR;
    }
    return DETAG_VARIANT_DENSE;
  }
  return DETAG_VARIANT_CSR;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int query_device(detag_state* s) {
  cudaError_t e = cudaGetDevice(&s->device);
  if (e != cudaSuccess) return fail_cuda(s, e, "cudaGetDevice");
  e = cudaDeviceGetAttribute(&s->sm_count, cudaDevAttrMultiProcessorCount, s->device);
  if (e != cudaSuccess) return fail_cuda(s, e, "cudaDeviceGetAttribute(sm count)");
  e = cudaDeviceGetAttribute(&s->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, s->device);
  if (e != cudaSuccess) return fail_cuda(s, e, "cudaDeviceGetAttribute(shared memory)");
  return DETAG_OK;
}

// Kernel families that take tensor maps.
enum { kFamilyMma = 1, kFamilyBand = 2, kFamilyTorus = 3, kFamilyRing = 4, kFamilyWide = 5 };

// Tensor maps for the buffers in `p`: built on first use, then found again by buffer addresses and sizes
// (detag_step always hits; detag_step_host cycles through its two chunk slots and the ragged last chunk).
const detag::TensorMapSet* maps_for(detag_state* s, int family, const StepParams& p) {
  const void* slot_a = p.mode == detag::kModeExternal ? static_cast<const void*>(p.g_ext) : p.a;
  const void* key[5] = {p.x, p.mode == detag::kModeDpsgd ? nullptr : p.y, p.g, slot_a,
                        p.mode == detag::kModeExternal ? nullptr : p.c};
  for (auto& en : s->map_cache) {
    if (en.family == family && en.d == p.d && en.ld == p.ld && std::memcmp(en.ptr, key, sizeof key) == 0)
      return &en.maps;
  }
  constexpr size_t kEntries = 6;
  detag_state::MapEntry* slot;
  if (s->map_cache.size() < kEntries) {
    s->map_cache.emplace_back();
    slot = &s->map_cache.back();
  } else {
    slot = &s->map_cache[s->map_next];
    s->map_next = (s->map_next + 1) % kEntries;
  }
  detag_state::MapEntry& en = *slot;
  en.family = 0;  // invalid until built
  const bool ok = family == kFamilyMma    ? detag::build_maps_mma(p, &en.maps)
                  : family == kFamilyBand ? detag::build_maps_band(p, &en.maps)
                  : family == kFamilyRing ? detag::build_maps_ring(p, &en.maps)
                  : family == kFamilyWide ? detag::build_maps_wide(p, &en.maps)
                                          : detag::build_maps_torus(p, &en.maps);
  if (!ok) return nullptr;
  en.family = family;
  en.d = p.d;
  en.ld = p.ld;
  std::memcpy(en.ptr, key, sizeof key);
  return &en.maps;
}

// The columns from `first` on through the generic rounds kernel (the tensor-path kernels that take whole 32- or
// 64-coordinate pieces hand their remainder here, in the same call).
int launch_tail_columns(detag_state* s, const StepParams& p, long long first, cudaStream_t stream, int* cuda_error) {
  StepParams pt = p;
  pt.d = p.d - first;
  pt.coord_offset = p.coord_offset + first;
  pt.x = p.x + first;
  pt.y = p.y + first;
  pt.g = p.g + first;
  pt.a = p.a + first;
  pt.c = p.c + first;
  if (p.y_obs) pt.y_obs = p.y_obs + first;
  const int rc = detag::plan_step_csr(pt, s->smem_optin);
  if (rc != DETAG_OK) return fail(s, rc, "graph too large for the shared-memory plan");
  *cuda_error = detag::launch_step_csr(pt, s->sm_count, stream);
  return DETAG_OK;
}

// Picks the kernel variant, plans it for the sizes in `p` and launches it.
int launch_step(detag_state* s, StepParams& p, cudaStream_t stream) {
  int e = 0;
  const int variant = resolve_variant(s);
  if (!variant_runs_mode(s, variant))
    return fail(s, DETAG_ERR_UNSUPPORTED,
                "this kernel variant runs the DeTAG step with the synthetic gradient only; use AUTO or CSR");
  if (p.mode != detag::kModeExternal && (!p.a || !p.c))
    return fail(s, DETAG_ERR_UNBOUND, "the synthetic gradient needs the objective arrays a and c");
  if (p.mode == detag::kModeExternal && !p.g_ext)
    return fail(s, DETAG_ERR_UNBOUND, "caller-written gradients selected but no gradient array given");
  switch (variant) {
    case DETAG_VARIANT_DENSE: {
      if (p.n > detag::kMaxDenseWorkers) {
        // the register-resident polynomial takes whole 32-coordinate halves; the last d % 32 columns go to the generic kernel
        const long long d_main = p.d & ~31LL;
        if (d_main > 0) {
          StepParams pm = p;
          pm.d = d_main;
          const detag::TensorMapSet* maps = maps_for(s, kFamilyWide, pm);
          if (!maps) return fail(s, DETAG_ERR_CUDA, "tensor map encoding failed");
          e = detag::launch_step_wide(pm, *maps, p.wide, s->sm_count, stream);
          if (e != 0) return fail_cuda(s, e, "step kernel launch");
        }
        if (d_main < p.d) {
          const int rc = launch_tail_columns(s, p, d_main, stream, &e);
          if (rc != DETAG_OK) return rc;
        }
        break;
      }
      const bool mma = p.n <= 32;
      const detag::TensorMapSet* maps = maps_for(s, mma ? kFamilyMma : kFamilyBand, p);
      if (!maps) return fail(s, DETAG_ERR_CUDA, "tensor map encoding failed");
      e = mma ? detag::launch_step_mma(p, *maps, s->sm_count, stream)
              : detag::launch_step_band(p, *maps, nullptr, s->sm_count, stream);
      break;
    }
    case DETAG_VARIANT_RING: {
      // the circulant kernel takes whole 64-coordinate slabs; the last d % 64 columns go to the generic kernel
      const long long d_main = p.d & ~63LL;
      if (d_main > 0) {
        StepParams pm = p;
        pm.d = d_main;
        const detag::TensorMapSet* maps = maps_for(s, kFamilyRing, pm);
        if (!maps) return fail(s, DETAG_ERR_CUDA, "tensor map encoding failed");
        e = detag::launch_step_ring(pm, *maps, ring_band(s) ? s->band : nullptr, p.circ_row, s->sm_count, stream);
        if (e != 0) return fail_cuda(s, e, "step kernel launch");
      }
      if (d_main < p.d) {
        const int rc = launch_tail_columns(s, p, d_main, stream, &e);
        if (rc != DETAG_OK) return rc;
      }
      break;
    }
    case DETAG_VARIANT_TORUS: {
      const detag::TensorMapSet* maps = maps_for(s, kFamilyTorus, p);
      if (!maps) return fail(s, DETAG_ERR_CUDA, "tensor map encoding failed");
      e = detag::launch_step_torus(p, *maps, p.torus, s->sm_count, stream);
      break;
    }
    case DETAG_VARIANT_CSR:
    default: {
      const int rc = detag::plan_step_csr(p, s->smem_optin);
      if (rc != DETAG_OK) return fail(s, rc, "graph too large for the shared-memory plan");
      e = detag::launch_step_csr(p, s->sm_count, stream);
    }
  }
  if (e != 0) return fail_cuda(s, e, "step kernel launch");
  return DETAG_OK;
}

}  // namespace

extern "C" {

int detag_create(detag_state** out, int n, int64_t d, const int32_t* row_ptr, const int32_t* col_idx,
                 const double* vals, int K, double eta, double alpha) {
  if (!out) return DETAG_ERR_ARG;
  *out = nullptr;
  if (n <= 0 || d <= 0 || K < 1 || !std::isfinite(alpha)) return DETAG_ERR_ARG;
  int rc = detag::validate_csr(n, row_ptr, col_idx, vals);
  if (rc != DETAG_OK) return rc;
  if (n > detag::kMaxWorkers) return DETAG_ERR_UNSUPPORTED;
  const int nnz = row_ptr[n];
  // doubly stochastic: every row and column sums to one
  std::vector<double> col_sum(n, 0.0);
  for (int i = 0; i < n; ++i) {
    double row_sum = 0.0;
    for (int k = row_ptr[i]; k < row_ptr[i + 1]; ++k) {
      row_sum += vals[k];
      col_sum[col_idx[k]] += vals[k];
    }
    if (std::fabs(row_sum - 1.0) > 1e-9) return DETAG_ERR_NOT_STOCHASTIC;
  }
  for (int j = 0; j < n; ++j)
    if (std::fabs(col_sum[j] - 1.0) > 1e-9) return DETAG_ERR_NOT_STOCHASTIC;

  if (std::isnan(eta)) {
    double lam = 0.0;
    rc = detag_spectral(n, row_ptr, col_idx, vals, nullptr, nullptr, &lam, &eta);
    if (rc != DETAG_OK) return rc;
  } else if (!std::isfinite(eta)) {
    return DETAG_ERR_ARG;
  }

  detag_state* s = new (std::nothrow) detag_state();
  if (!s) return DETAG_ERR_ARG;
  s->n = n;
  s->d = d;
  s->K = K;
  s->eta = eta;
  s->alpha = alpha;
  s->row_ptr.assign(row_ptr, row_ptr + n + 1);
  s->col_idx.assign(col_idx, col_idx + nnz);
  s->vals.assign(vals, vals + nnz);
  if (n <= detag::kMaxDenseWorkers) {
    gossip_polynomial(s, s->poly);
  } else if (n <= detag::kMaxWideWorkers) {  // kept as the warp strips of the register-resident kernel only
    std::vector<double> poly;
    gossip_polynomial(s, poly);
    detag::wide_fragments(n, poly, s->wide_frag);
  }
  analyse_circulant(s);
  analyse_torus(s);
  s->map_cache.reserve(8);
  *out = s;
  return DETAG_OK;
}

int detag_workspace_bytes(const detag_state* s, size_t* bytes) {
  if (!s || !bytes) return DETAG_ERR_ARG;
  *bytes = ws_layout(s).total;
  return DETAG_OK;
}

int detag_bind(detag_state* s, int64_t ld, float* x, float* y, float* g, const float* a, const float* c,
               void* workspace, size_t workspace_bytes) {
  if (!s) return DETAG_ERR_ARG;
  if (!x || !y || !g || !workspace) return fail(s, DETAG_ERR_ARG, "detag_bind: null buffer");
  if (ld < s->d || (ld & 3) != 0) return fail(s, DETAG_ERR_ARG, "detag_bind: ld must be >= d and a multiple of 4");
  if (!aligned16(x) || !aligned16(y) || !aligned16(g) || !aligned16(a) || !aligned16(c))  // NULL counts as aligned
    return fail(s, DETAG_ERR_ARG, "detag_bind: state arrays must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(workspace) % detag::kWsAlign) != 0)
    return fail(s, DETAG_ERR_ARG, "detag_bind: workspace must be 256-byte aligned");
  const WsLayout l = ws_layout(s);
  if (workspace_bytes < l.total) return fail(s, DETAG_ERR_ARG, "detag_bind: workspace too small");

  const int qrc = query_device(s);
  if (qrc != DETAG_OK) return qrc;
  cudaError_t e = cudaSuccess;

  unsigned char* base = static_cast<unsigned char*>(workspace);
  s->d_status = reinterpret_cast<int*>(base + l.status);
  s->d_result = reinterpret_cast<double*>(base + l.result);
  s->d_row_ptr = reinterpret_cast<int32_t*>(base + l.row_ptr);
  s->d_col_idx = reinterpret_cast<int32_t*>(base + l.col_idx);
  s->d_vals = reinterpret_cast<double*>(base + l.vals);
  s->d_poly = s->poly.empty() ? nullptr : reinterpret_cast<double*>(base + l.poly);
  s->d_torus = s->torus_frag.empty() ? nullptr : reinterpret_cast<double*>(base + l.torus);
  s->d_circ_row = s->circ_row.empty() ? nullptr : reinterpret_cast<double*>(base + l.circ_row);
  s->d_wide = s->wide_frag.empty() ? nullptr : reinterpret_cast<double*>(base + l.wide);
  s->d_partials = reinterpret_cast<double*>(base + l.partials);

  e = cudaMemset(base, 0, detag::kWsAlign);
  if (e == cudaSuccess)
    e = cudaMemcpy(s->d_row_ptr, s->row_ptr.data(), s->row_ptr.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(s->d_col_idx, s->col_idx.data(), s->col_idx.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(s->d_vals, s->vals.data(), s->vals.size() * sizeof(double), cudaMemcpyHostToDevice);
  if (e == cudaSuccess && s->d_poly)
    e = cudaMemcpy(s->d_poly, s->poly.data(), s->poly.size() * sizeof(double), cudaMemcpyHostToDevice);
  if (e == cudaSuccess && s->d_torus)
    e = cudaMemcpy(s->d_torus, s->torus_frag.data(), s->torus_frag.size() * sizeof(double), cudaMemcpyHostToDevice);
  if (e == cudaSuccess && s->d_circ_row)
    e = cudaMemcpy(s->d_circ_row, s->circ_row.data(), s->circ_row.size() * sizeof(double), cudaMemcpyHostToDevice);
  if (e == cudaSuccess && s->d_wide)
    e = cudaMemcpy(s->d_wide, s->wide_frag.data(), s->wide_frag.size() * sizeof(double), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return fail_cuda(s, e, "detag_bind: workspace upload");

  s->ld = ld;
  s->x = x;
  s->y = y;
  s->g = g;
  s->a = a;
  s->c = c;
  s->ws = workspace;
  s->ws_bytes = workspace_bytes;
  s->bound = true;
  return DETAG_OK;
}

int detag_observe_gossiped_tracker(detag_state* s, float* y_gossip) {
  if (!s) return DETAG_ERR_ARG;
  if (y_gossip && !aligned16(y_gossip)) return fail(s, DETAG_ERR_ARG, "observer buffer must be 16-byte aligned");
  s->y_obs = y_gossip;
  return DETAG_OK;
}

int detag_set_noise(detag_state* s, double sigma, uint64_t seed, int64_t coord_offset) {
  if (!s) return DETAG_ERR_ARG;
  if (!std::isfinite(sigma) || sigma < 0.0 || coord_offset < 0)
    return fail(s, DETAG_ERR_ARG, "detag_set_noise: bad value");
  s->sigma = sigma;
  s->seed = seed;
  s->coord_offset = coord_offset;
  return DETAG_OK;
}

int detag_set_variant(detag_state* s, int variant) {
  if (!s) return DETAG_ERR_ARG;
  switch (variant) {
    case DETAG_VARIANT_AUTO:
    case DETAG_VARIANT_CSR:
      break;
    case DETAG_VARIANT_DENSE:
      if (!dense_ok(s)) return fail(s, DETAG_ERR_UNSUPPORTED, "detag_set_variant: dense variant needs n <= 128");
      break;
    case DETAG_VARIANT_TORUS:
      if (!torus_ok(s))
        return fail(s, DETAG_ERR_UNSUPPORTED,
                    "detag_set_variant: torus variant needs n = 32 or 64 and a matrix that is block circulant in "
                    "8-worker blocks, symmetric in the block distance");
      break;
    case DETAG_VARIANT_RING:
      if (!band_ok(s))
        return fail(s, DETAG_ERR_UNSUPPORTED,
                    "detag_set_variant: ring variant needs a circulant matrix, n a multiple of 32, n >= 64, and K*bandwidth <= 16 or n <= 256");
      break;
    default:
      return fail(s, DETAG_ERR_ARG, "detag_set_variant: unknown variant");
  }
  s->variant_forced = variant;
  return DETAG_OK;
}

int detag_get_variant(const detag_state* s, int* variant) {
  if (!s || !variant) return DETAG_ERR_ARG;
  *variant = resolve_variant(s);
  return DETAG_OK;
}

int detag_set_gradient_point(detag_state* s, int where) {
  if (!s) return DETAG_ERR_ARG;
  if (where != DETAG_GRADIENT_AT_NEW_MODEL && where != DETAG_GRADIENT_AT_PHASE_START)
    return fail(s, DETAG_ERR_ARG, "detag_set_gradient_point: unknown value");
  s->gradient_point = where;
  return DETAG_OK;
}

int detag_get_gradient_point(const detag_state* s, int* where) {
  if (!s || !where) return DETAG_ERR_ARG;
  *where = s->gradient_point;
  return DETAG_OK;
}

int detag_set_algorithm(detag_state* s, int algorithm) {
  if (!s) return DETAG_ERR_ARG;
  if (algorithm != DETAG_ALGORITHM_DETAG && algorithm != DETAG_ALGORITHM_DPSGD)
    return fail(s, DETAG_ERR_ARG, "detag_set_algorithm: unknown value");
  if (algorithm == DETAG_ALGORITHM_DPSGD && s->gradient_source == DETAG_GRADIENT_EXTERNAL)
    return fail(s, DETAG_ERR_UNSUPPORTED, "detag_set_algorithm: D-PSGD runs with the synthetic gradient only");
  s->algorithm = algorithm;
  return DETAG_OK;
}

int detag_get_algorithm(const detag_state* s, int* algorithm) {
  if (!s || !algorithm) return DETAG_ERR_ARG;
  *algorithm = s->algorithm;
  return DETAG_OK;
}

int detag_set_gradient_source(detag_state* s, int source, const float* g_new) {
  if (!s) return DETAG_ERR_ARG;
  if (source == DETAG_GRADIENT_SYNTHETIC) {
    s->gradient_source = source;
    s->g_ext = nullptr;
    return DETAG_OK;
  }
  if (source != DETAG_GRADIENT_EXTERNAL) return fail(s, DETAG_ERR_ARG, "detag_set_gradient_source: unknown value");
  if (!g_new || !aligned16(g_new))
    return fail(s, DETAG_ERR_ARG, "detag_set_gradient_source: the gradient array must be non-null and 16-byte aligned");
  if (s->algorithm == DETAG_ALGORITHM_DPSGD)
    return fail(s, DETAG_ERR_UNSUPPORTED, "detag_set_gradient_source: D-PSGD runs with the synthetic gradient only");
  s->gradient_source = source;
  s->g_ext = g_new;
  return DETAG_OK;
}

int detag_debug_inject_stall(detag_state* s, int64_t after_tiles, uint32_t poll_limit) {
  if (!s) return DETAG_ERR_ARG;
  if (after_tiles < 0) {  // back to normal
    s->stall_after = -1;
    s->spin_limit = 1u << 20;
    return DETAG_OK;
  }
  if (poll_limit < 16 || poll_limit > (1u << 20))
    return fail(s, DETAG_ERR_ARG, "detag_debug_inject_stall: poll limit outside [16, 2^20]");
  s->stall_after = after_tiles;
  s->spin_limit = poll_limit;
  return DETAG_OK;
}

int detag_debug_expire_wait(detag_state* s, uint32_t polls, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (!s->bound) return fail(s, DETAG_ERR_UNBOUND, "detag_debug_expire_wait before detag_bind");
  if (polls < 1 || polls > (1u << 20)) return fail(s, DETAG_ERR_ARG, "detag_debug_expire_wait: polls outside [1, 2^20]");
  const int e = detag::launch_expire_wait(s->d_status, polls, static_cast<cudaStream_t>(stream));
  if (e != 0) return fail_cuda(s, e, "detag_debug_expire_wait launch");
  return DETAG_OK;
}

int detag_phase_length(int n, double lambda, double varsigma0_sq, double T, double delta_L, int* R) {
  if (!R || n < 1 || !(lambda >= 0.0) || !(lambda < 1.0)) return DETAG_ERR_ARG;
  double num = 0.5 * std::log(static_cast<double>(n));
  if (varsigma0_sq > 0.0 && T > 0.0 && delta_L > 0.0) {
    const double second = 0.5 * std::log(varsigma0_sq * T / delta_L);
    if (second > num) num = second;
  }
  const double r = std::ceil(num / std::sqrt(1.0 - lambda));
  *R = r < 1.0 ? 1 : (r > 2147483647.0 ? 2147483647 : static_cast<int>(r));
  return DETAG_OK;
}

int detag_init(detag_state* s, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (!s->bound) return fail(s, DETAG_ERR_UNBOUND, "detag_init before detag_bind");
  StepParams p = make_params(s);
  p.t_noise = 0;
  int e;
  if (p.mode == detag::kModeExternal) {
    if (!p.g_ext) return fail(s, DETAG_ERR_UNBOUND, "caller-written gradients selected but no gradient array given");
    e = detag::launch_init_external(p, s->sm_count, static_cast<cudaStream_t>(stream));
  } else {
    if (!p.a || !p.c) return fail(s, DETAG_ERR_UNBOUND, "the synthetic gradient needs the objective arrays a and c");
    e = detag::launch_init_gradient(p, s->sm_count, static_cast<cudaStream_t>(stream));
  }
  if (e != 0) return fail_cuda(s, e, "detag_init launch");
  s->t = 0;
  return DETAG_OK;
}

int detag_step(detag_state* s, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (!s->bound) return fail(s, DETAG_ERR_UNBOUND, "detag_step before detag_bind");
  StepParams p = make_params(s);
  p.t_noise = static_cast<uint32_t>(s->t + 1);
  const int rc = launch_step(s, p, static_cast<cudaStream_t>(stream));
  if (rc != DETAG_OK) return rc;
  s->t += 1;
  return DETAG_OK;
}

int detag_step_many(detag_state* s, int count, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (count < 1) return fail(s, DETAG_ERR_ARG, "detag_step_many: count must be at least 1");
  if (!s->bound) return fail(s, DETAG_ERR_UNBOUND, "detag_step_many before detag_bind");
  if (count >= 2 && step_mode(s) == detag::kModeExternal)
    return fail(s, DETAG_ERR_ARG, "detag_step_many: caller-written gradients need one call per step");
  // the fused kernel exists for the dense polynomial with n <= 32; the observer wants every step's tracker
  if (count >= 2 && resolve_variant(s) == DETAG_VARIANT_DENSE && s->n <= 32 && s->y_obs == nullptr &&
      step_mode(s) == detag::kModeDetag) {
    // A launch is cut off at kMaxFusedSteps so that no thread of the kernel waits on a peer for longer than its
    // bounded waits allow (a tile of 1024 steps takes some tens of milliseconds; the waits give up after seconds).
    constexpr int kMaxFusedSteps = 1024;
    for (int done = 0; done < count;) {
      const int now = count - done < kMaxFusedSteps ? count - done : kMaxFusedSteps;
      StepParams p = make_params(s);
      p.t_noise = static_cast<uint32_t>(s->t + 1);
      p.steps = now;
      if (!p.a || !p.c) return fail(s, DETAG_ERR_UNBOUND, "the synthetic gradient needs the objective arrays a and c");
      const detag::TensorMapSet* maps = maps_for(s, kFamilyMma, p);
      if (!maps) return fail(s, DETAG_ERR_CUDA, "tensor map encoding failed");
      const int e = detag::launch_step_mma_many(p, *maps, s->sm_count, static_cast<cudaStream_t>(stream));
      if (e != 0) return fail_cuda(s, e, "detag_step_many launch");
      s->t += now;
      done += now;
    }
    return DETAG_OK;
  }
  for (int i = 0; i < count; ++i) {
    const int rc = detag_step(s, stream);
    if (rc != DETAG_OK) return rc;
  }
  return DETAG_OK;
}

int detag_host_staging_bytes(const detag_state* s, int64_t chunk_coords, size_t* bytes) {
  if (!s || !bytes || chunk_coords < 128 || (chunk_coords % 128) != 0) return DETAG_ERR_ARG;
  *bytes = ws_layout(s).total + static_cast<size_t>(2) * 5 * s->n * static_cast<size_t>(chunk_coords) * sizeof(float);
  return DETAG_OK;
}

int detag_step_host(detag_state* s, int64_t ld_host, float* x, float* y, float* g, const float* a, const float* c,
                    void* staging, size_t staging_bytes, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (!x || !y || !g || !a || !c || !staging) return fail(s, DETAG_ERR_ARG, "detag_step_host: null buffer");
  if (step_mode(s) == detag::kModeExternal)
    return fail(s, DETAG_ERR_UNSUPPORTED, "detag_step_host: caller-written gradients are not offered on host-resident state");
  if (ld_host < s->d) return fail(s, DETAG_ERR_ARG, "detag_step_host: ld_host < d");
  if ((reinterpret_cast<uintptr_t>(staging) % detag::kWsAlign) != 0)
    return fail(s, DETAG_ERR_ARG, "detag_step_host: staging must be 256-byte aligned");
  const WsLayout l = ws_layout(s);
  const size_t per_coord = static_cast<size_t>(2) * 5 * s->n * sizeof(float);
  if (staging_bytes < l.total + per_coord * 128)
    return fail(s, DETAG_ERR_ARG, "detag_step_host: staging too small for a 128-coordinate chunk");
  long long chunk = static_cast<long long>((staging_bytes - l.total) / per_coord) / 128 * 128;
  const long long d_up = (s->d + 127) / 128 * 128;
  if (chunk > d_up) chunk = d_up;

  int rc = query_device(s);
  if (rc != DETAG_OK) return rc;
  cudaError_t e = cudaSuccess;
  for (int k = 0; k < 2 && e == cudaSuccess; ++k)
    if (!s->host_stream[k]) e = cudaStreamCreateWithFlags(&s->host_stream[k], cudaStreamNonBlocking);
  for (int k = 0; k < 3 && e == cudaSuccess; ++k)
    if (!s->host_event[k]) e = cudaEventCreateWithFlags(&s->host_event[k], cudaEventDisableTiming);
  if (e != cudaSuccess) return fail_cuda(s, e, "detag_step_host: stream/event creation");

  cudaStream_t user = static_cast<cudaStream_t>(stream);
  unsigned char* base = static_cast<unsigned char*>(staging);
  // Graph tables at the head of the staging area, ordered on the caller's stream.  The status word there is
  // cleared when a staging area is first used, not on every call: a time-out stays visible to detag_status.
  int* status_word = reinterpret_cast<int*>(base + l.status);
  if (s->d_status_host != status_word) e = cudaMemsetAsync(base, 0, detag::kWsAlign, user);
  s->d_status_host = status_word;
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(base + l.row_ptr, s->row_ptr.data(), s->row_ptr.size() * sizeof(int32_t),
                        cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(base + l.col_idx, s->col_idx.data(), s->col_idx.size() * sizeof(int32_t),
                        cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(base + l.vals, s->vals.data(), s->vals.size() * sizeof(double), cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess && !s->poly.empty())
    e = cudaMemcpyAsync(base + l.poly, s->poly.data(), s->poly.size() * sizeof(double), cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess && !s->torus_frag.empty())
    e = cudaMemcpyAsync(base + l.torus, s->torus_frag.data(), s->torus_frag.size() * sizeof(double),
                        cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess && !s->circ_row.empty())
    e = cudaMemcpyAsync(base + l.circ_row, s->circ_row.data(), s->circ_row.size() * sizeof(double),
                        cudaMemcpyHostToDevice, user);
  if (e == cudaSuccess && !s->wide_frag.empty())
    e = cudaMemcpyAsync(base + l.wide, s->wide_frag.data(), s->wide_frag.size() * sizeof(double), cudaMemcpyHostToDevice,
                        user);
  if (e == cudaSuccess) e = cudaEventRecord(s->host_event[2], user);
  for (int k = 0; k < 2 && e == cudaSuccess; ++k) e = cudaStreamWaitEvent(s->host_stream[k], s->host_event[2], 0);
  if (e != cudaSuccess) return fail_cuda(s, e, "detag_step_host: table upload");

  StepParams p = make_params(s);
  p.row_ptr = reinterpret_cast<int32_t*>(base + l.row_ptr);
  p.col_idx = reinterpret_cast<int32_t*>(base + l.col_idx);
  p.vals = reinterpret_cast<double*>(base + l.vals);
  p.poly = s->poly.empty() ? nullptr : reinterpret_cast<double*>(base + l.poly);
  p.torus = s->torus_frag.empty() ? nullptr : reinterpret_cast<double*>(base + l.torus);
  p.circ_row = s->circ_row.empty() ? nullptr : reinterpret_cast<double*>(base + l.circ_row);
  p.wide = s->wide_frag.empty() ? nullptr : reinterpret_cast<double*>(base + l.wide);
  p.status = status_word;
  p.y_obs = nullptr;
  p.t_noise = static_cast<uint32_t>(s->t + 1);
  p.ld = chunk;
  float* slots = reinterpret_cast<float*>(base + l.total);
  const size_t arr = static_cast<size_t>(s->n) * chunk;  // elements of one staged array
  const size_t hp = static_cast<size_t>(ld_host) * sizeof(float), dp = static_cast<size_t>(chunk) * sizeof(float);

  long long k = 0;
  for (long long j0 = 0; j0 < s->d; j0 += chunk, ++k) {
    const long long w = (s->d - j0 < chunk) ? s->d - j0 : chunk;
    cudaStream_t st = s->host_stream[k & 1];
    float* sx = slots + (k & 1) * 5 * arr;
    float *sy = sx + arr, *sg = sy + arr, *sa = sg + arr, *sc = sa + arr;
    const size_t wb = static_cast<size_t>(w) * sizeof(float);
    e = cudaMemcpy2DAsync(sx, dp, x + j0, hp, wb, s->n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(sy, dp, y + j0, hp, wb, s->n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(sg, dp, g + j0, hp, wb, s->n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(sa, dp, a + j0, hp, wb, s->n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(sc, dp, c + j0, hp, wb, s->n, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail_cuda(s, e, "detag_step_host: host-to-device copy");
    p.x = sx; p.y = sy; p.g = sg; p.a = sa; p.c = sc;
    p.d = w;
    p.coord_offset = s->coord_offset + j0;
    rc = launch_step(s, p, st);
    if (rc != DETAG_OK) return rc;
    e = cudaMemcpy2DAsync(x + j0, hp, sx, dp, wb, s->n, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(y + j0, hp, sy, dp, wb, s->n, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpy2DAsync(g + j0, hp, sg, dp, wb, s->n, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail_cuda(s, e, "detag_step_host: device-to-host copy");
  }
  for (int q = 0; q < 2 && e == cudaSuccess; ++q) {
    e = cudaEventRecord(s->host_event[q], s->host_stream[q]);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, s->host_event[q], 0);
  }
  if (e != cudaSuccess) return fail_cuda(s, e, "detag_step_host: join");
  s->t += 1;
  return DETAG_OK;
}

int detag_consensus_error(detag_state* s, void* stream, double* host_out) {
  if (!s || !host_out) return DETAG_ERR_ARG;
  if (!s->bound) return fail(s, DETAG_ERR_UNBOUND, "detag_consensus_error before detag_bind");
  const StepParams p = make_params(s);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int e = detag::launch_consensus_error(p, s->d_partials, s->d_result, s->sm_count, st);
  if (e != 0) return fail_cuda(s, e, "detag_consensus_error launch");
  cudaError_t ce = cudaMemcpyAsync(host_out, s->d_result, sizeof(double), cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) return fail_cuda(s, ce, "detag_consensus_error copy");
  return DETAG_OK;
}

int detag_get_step(const detag_state* s, int64_t* t) {
  if (!s || !t) return DETAG_ERR_ARG;
  *t = s->t;
  return DETAG_OK;
}

int detag_set_step(detag_state* s, int64_t t) {
  if (!s || t < 0) return DETAG_ERR_ARG;
  s->t = t;
  return DETAG_OK;
}

int detag_status(detag_state* s, void* stream) {
  if (!s) return DETAG_ERR_ARG;
  if (!s->bound && !s->d_status_host) return fail(s, DETAG_ERR_UNBOUND, "detag_status before detag_bind or detag_step_host");
  int word[2] = {0, 0};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  if (s->bound) e = cudaMemcpyAsync(&word[0], s->d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess && s->d_status_host)
    e = cudaMemcpyAsync(&word[1], s->d_status_host, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail_cuda(s, e, "detag_status");
  if (word[0] == 2 || word[1] == 2) return fail(s, DETAG_ERR_CUDA, "a kernel found its shared memory misaligned");
  if (word[0] != 0 || word[1] != 0) return fail(s, DETAG_ERR_TIMEOUT, "a device-side wait gave up");
  s->d_status_host = nullptr;  // read and clean: the staging area is not referred to again until the next host step
  return DETAG_OK;
}

const char* detag_last_error(const detag_state* s) { return s ? s->err.c_str() : ""; }

int detag_destroy(detag_state* s) {
  if (!s) return DETAG_ERR_ARG;
  for (int k = 0; k < 2; ++k)
    if (s->host_stream[k]) {
      cudaStreamSynchronize(s->host_stream[k]);
      cudaStreamDestroy(s->host_stream[k]);
    }
  for (int k = 0; k < 3; ++k)
    if (s->host_event[k]) cudaEventDestroy(s->host_event[k]);
  delete s;
  return DETAG_OK;
}

}  // extern "C"
