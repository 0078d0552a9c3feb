// Host-side spectral routine: eigenvalues of a symmetric gossip matrix by cyclic Jacobi
// rotations in float64, then lambda = max(|lambda_2|, |lambda_n|) (paper, Section "Protocol
// Layer") and the accelerated-gossip momentum eta of Algorithm 3.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "detag_internal.h"

namespace detag {

int validate_csr(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals) {
  if (n <= 0 || !row_ptr || !col_idx || !vals) return DETAG_ERR_ARG;
  if (row_ptr[0] != 0) return DETAG_ERR_CSR;
  for (int i = 0; i < n; ++i) {
    if (row_ptr[i + 1] < row_ptr[i]) return DETAG_ERR_CSR;
    for (int k = row_ptr[i]; k < row_ptr[i + 1]; ++k) {
      if (col_idx[k] < 0 || col_idx[k] >= n) return DETAG_ERR_CSR;
      if (k > row_ptr[i] && col_idx[k] <= col_idx[k - 1]) return DETAG_ERR_CSR;  // unsorted or duplicate
      if (!std::isfinite(vals[k])) return DETAG_ERR_ARG;
    }
  }
  return DETAG_OK;
}

void csr_to_dense(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals, std::vector<double>& m) {
  m.assign(static_cast<size_t>(n) * n, 0.0);
  for (int i = 0; i < n; ++i)
    for (int k = row_ptr[i]; k < row_ptr[i + 1]; ++k) m[static_cast<size_t>(i) * n + col_idx[k]] = vals[k];
}

bool is_symmetric(int n, const std::vector<double>& m, double tol) {
  for (int i = 0; i < n; ++i)
    for (int j = i + 1; j < n; ++j)
      if (std::fabs(m[static_cast<size_t>(i) * n + j] - m[static_cast<size_t>(j) * n + i]) > tol) return false;
  return true;
}

// Eigenvalues (ascending) of the symmetric matrix `a` (destroyed) by cyclic Jacobi sweeps.
void jacobi_eigenvalues(int n, std::vector<double>& a, std::vector<double>& ev) {
  auto at = [&](int i, int j) -> double& { return a[static_cast<size_t>(i) * n + j]; };
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0.0, diag = 0.0;
    for (int i = 0; i < n; ++i) {
      diag += at(i, i) * at(i, i);
      for (int j = i + 1; j < n; ++j) off += at(i, j) * at(i, j);
    }
    if (off <= 1e-30 * std::max(diag, 1e-300)) break;
    for (int p = 0; p < n - 1; ++p) {
      for (int q = p + 1; q < n; ++q) {
        const double apq = at(p, q);
        if (apq == 0.0) continue;
        // rotation angle that zeroes a_pq: tan(2 theta) = 2 a_pq / (a_qq - a_pp)
        const double theta = (at(q, q) - at(p, p)) / (2.0 * apq);
        const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
        const double c = 1.0 / std::sqrt(t * t + 1.0), s = t * c;
        for (int k = 0; k < n; ++k) {  // columns p, q
          const double akp = at(k, p), akq = at(k, q);
          at(k, p) = c * akp - s * akq;
          at(k, q) = s * akp + c * akq;
        }
        for (int k = 0; k < n; ++k) {  // rows p, q
          const double apk = at(p, k), aqk = at(q, k);
          at(p, k) = c * apk - s * aqk;
          at(q, k) = s * apk + c * aqk;
        }
      }
    }
  }
  ev.resize(n);
  for (int i = 0; i < n; ++i) ev[i] = at(i, i);
  std::sort(ev.begin(), ev.end());
}

double eta_from_lambda(double lam) {
  const double s = std::sqrt(std::max(0.0, 1.0 - lam * lam));
  return (1.0 - s) / (1.0 + s);
}

}  // namespace detag

extern "C" int detag_spectral(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals,
                              double* lambda2, double* lambda_min, double* lambda, double* eta) {
  int rc = detag::validate_csr(n, row_ptr, col_idx, vals);
  if (rc != DETAG_OK) return rc;
  if (n > 2048) return DETAG_ERR_UNSUPPORTED;
  std::vector<double> m, ev;
  detag::csr_to_dense(n, row_ptr, col_idx, vals, m);
  if (!detag::is_symmetric(n, m, 1e-12)) return DETAG_ERR_NOT_SYMMETRIC;
  detag::jacobi_eigenvalues(n, m, ev);
  const double l2 = n >= 2 ? ev[n - 2] : 0.0;
  const double lmin = ev[0];
  const double lam = n >= 2 ? std::max(std::fabs(l2), std::fabs(lmin)) : 0.0;
  if (lambda2) *lambda2 = l2;
  if (lambda_min) *lambda_min = lmin;
  if (lambda) *lambda = lam;
  if (lam >= 1.0 - 1e-13) return DETAG_ERR_SPECTRUM;
  if (eta) *eta = detag::eta_from_lambda(lam);
  return DETAG_OK;
}
