/*
 * detag.h - C ABI of the B200 (sm_100a) DeTAG step library.
 *
 * DeTAG = decentralized stochastic gradient tracking with by-phase accelerated gossip
 * (arXiv 2006.08085, Algorithms 2 and 3).  The library applies one DeTAG iteration at once
 * to all n simulated workers, each holding a flat float32 parameter vector of length d, on
 * one GPU.
 *
 * Conventions used by every entry point
 *   - Return value: DETAG_OK (0) or a negative DETAG_ERR_* code.  Nothing throws, traps or
 *     exits; detag_last_error() gives a text for the last failure on a state.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global memory of
 *     the device that is current when the call is made.  The library allocates no device
 *     memory: the caller owns every device buffer (state arrays and the workspace) and
 *     keeps it alive and unaliased while it is bound.  detag_destroy frees host memory only.
 *   - `stream` is a CUDA stream handle (cudaStream_t / CUstream) passed as void*; NULL is
 *     the legacy default stream.  Calls documented "asynchronous" only enqueue work.
 *   - State arrays are row-major [n][ld] float32: worker i's vector starts at element
 *     i*ld; ld >= d, ld a multiple of 4, base addresses 16-byte aligned.
 *   - A state is used by one host thread at a time.
 *
 * One step, in the order the kernels execute it (Algorithm 2; gradient evaluated at the new
 * model, folded into the tracker before the next gossip):
 *     y~  = AG_K(y)                      Algorithm 3 on the tracker
 *     x~  = AG_K(x)                      Algorithm 3 on the model
 *     x'  = x~ - alpha * y~              model update of Algorithm 2
 *     g'  = a o (x' - c) + sigma * xi    stochastic gradient of f_i(x) = 1/2 sum_j a_ij (x_j - c_ij)^2
 *     y'  = y~ + g' - g                  tracker update of Algorithm 2 (with the stored float32 g')
 * so the `y` buffer always holds the tracker with the newest gradient already folded in,
 * and each of x, y, g, a, c is read once and x, y, g written once per step.
 */
#ifndef DETAG_H
#define DETAG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct detag_state detag_state; /* opaque, lives in host memory */

enum {
  DETAG_OK = 0,
  DETAG_ERR_ARG = -1,            /* null pointer, non-positive size, misaligned or too small buffer */
  DETAG_ERR_CSR = -2,            /* row_ptr not monotone, column out of range, unsorted or duplicate */
  DETAG_ERR_NOT_STOCHASTIC = -3, /* some row or column sum differs from 1 by more than 1e-9 */
  DETAG_ERR_NOT_SYMMETRIC = -4,  /* eta had to be derived but the matrix is not symmetric */
  DETAG_ERR_UNSUPPORTED = -5,    /* n or nnz beyond what the kernels' shared-memory plan holds */
  DETAG_ERR_UNBOUND = -6,        /* a call that needs buffers came before detag_bind */
  DETAG_ERR_CUDA = -7,           /* a CUDA runtime call or launch failed (text in detag_last_error) */
  DETAG_ERR_TIMEOUT = -8,        /* a bounded device-side wait gave up (reported by detag_status) */
  DETAG_ERR_SPECTRUM = -9        /* lambda >= 1: disconnected or bipartite graph, no valid eta */
};

/* Kernel variants of the gossip part of the step; all compute the same result. */
enum {
  DETAG_VARIANT_AUTO = 0,  /* host cost model picks */
  DETAG_VARIANT_CSR = 1,   /* K rounds of neighbour-indexed sums over the CSR rows, slab staged on chip: any graph, n <= 1024 */
  DETAG_VARIANT_DENSE = 2, /* one product with the host-precomputed polynomial P_K(M), n <= 128 (any M); for 64 < n <= 128
                              the last d % 32 coordinates run through the CSR kernel in the same call */
  DETAG_VARIANT_RING = 3,  /* circulant M (rings), n % 32 == 0, 64 <= n <= 1024: the circulant polynomial P_K(M) as a band
                              while K * bandwidth <= 16, as a dense circulant (n <= 256) beyond, e.g. at Theorem 3's phase
                              length; the last d % 64 coordinates run through the CSR kernel in the same call */
  DETAG_VARIANT_TORUS = 4  /* block-circulant M with 8-worker blocks, symmetric in the block distance (R x 8 tori, n = 32 or 64):
                              Fourier transform along the block axis, one 8 x 8 polynomial block per frequency, transform back */
};
/* Caller-written gradients run on DENSE (n <= 32) and CSR, D-PSGD on DENSE (n <= 32), RING and CSR; AUTO picks among
   those, a forced variant outside them makes detag_step return DETAG_ERR_UNSUPPORTED. */

/* The point at which a step queries the stochastic gradient oracle. */
enum {
  DETAG_GRADIENT_AT_NEW_MODEL = 0,   /* at x', the model the step produces (default; the step listing above) */
  DETAG_GRADIENT_AT_PHASE_START = 1  /* at x, the model the step started from: Algorithm 2 as printed */
};

/* Which decentralized algorithm a step runs. */
enum {
  DETAG_ALGORITHM_DETAG = 0, /* Algorithm 2 with Algorithm 3 as the gossip (default) */
  DETAG_ALGORITHM_DPSGD = 1  /* D-PSGD, the paper's main baseline: no gradient tracker */
};

/* Who evaluates the stochastic gradient. */
enum {
  DETAG_GRADIENT_SYNTHETIC = 0, /* the library: g = a o (x - c) + sigma xi of the synthetic objective (default) */
  DETAG_GRADIENT_EXTERNAL = 1   /* the caller (e.g. back-propagation) writes it into a device array before each step */
};

/*
 * Spectrum of a symmetric gossip matrix and the accelerated-gossip momentum.
 * Paper: Section "Protocol Layer" (lambda = max(|lambda_2|, |lambda_n|)) and Algorithm 3
 * (eta = (1 - sqrt(1 - lambda^2)) / (1 + sqrt(1 - lambda^2))).
 * Host only.  The matrix is n x n in CSR (host pointers: row_ptr[n+1], col_idx[nnz], vals[nnz]).
 * Any output pointer may be NULL.  Errors: ARG, CSR, NOT_SYMMETRIC, UNSUPPORTED (n > 2048),
 * SPECTRUM (lambda >= 1; the eigenvalue outputs are still written).
 */
int detag_spectral(int n, const int32_t* row_ptr, const int32_t* col_idx, const double* vals,
                   double* lambda2, double* lambda_min, double* lambda, double* eta);

/*
 * Create a state for n workers with d coordinates each.
 * The CSR arrays (host; copied) describe the matrix M that a gossip round applies row-wise,
 * z'_i = sum_j M[i][j] z_j, i.e. M[i][j] is the paper's W_ji (Eq. "gossip update",
 * Algorithm 3).  Columns sorted and unique within a row; M doubly stochastic.
 * K >= 1 is the number of accelerated-gossip rounds per step (the paper's phase length R),
 * alpha the step size of Algorithm 2, eta the momentum of Algorithm 3; pass NaN to have it
 * derived from the spectrum (needs a symmetric M).  Host only; no device work.
 * Errors: ARG, CSR, NOT_STOCHASTIC, NOT_SYMMETRIC, SPECTRUM, UNSUPPORTED (n > 1024).
 */
int detag_create(detag_state** out, int n, int64_t d, const int32_t* row_ptr, const int32_t* col_idx,
                 const double* vals, int K, double eta, double alpha);

/* Bytes of device workspace detag_bind needs for this state (graph tables, polynomial, partial sums). */
int detag_workspace_bytes(const detag_state* s, size_t* bytes);

/*
 * Bind the caller's device buffers (see the layout conventions above):
 *   x, y, g : state, read and written by detag_init / detag_step
 *   a, c    : objective data, read only; both may be NULL when every gradient comes from the caller
 *             (detag_set_gradient_source), otherwise init and step return DETAG_ERR_UNBOUND
 *   workspace: at least detag_workspace_bytes() bytes, 256-byte aligned; the call fills it with
 *              the graph tables (synchronous copies on the current device).
 * Rebinding is allowed (e.g. to step another coordinate shard with the same graph).
 * Errors: ARG, CUDA.
 */
int detag_bind(detag_state* s, int64_t ld, float* x, float* y, float* g, const float* a, const float* c,
               void* workspace, size_t workspace_bytes);

/*
 * Optional observer: when y_gossip (device, [n][ld] float32) is non-NULL, every later step also
 * stores the tracker right after its gossip (y~ above, the value Algorithm 2 uses in the model
 * update).  NULL (the default) switches it off.  Costs one extra array write per step.
 */
int detag_observe_gossiped_tracker(detag_state* s, float* y_gossip);

/*
 * Noise of the stochastic gradient oracle (Section "Setting", oracle class): xi is standard
 * normal, a pure function of (seed, step, worker, global coordinate); sigma = 0 gives the exact
 * gradient.  coord_offset is the global index of column 0 of the bound arrays (for coordinate
 * shards).  Defaults: sigma 0, seed 0, offset 0.
 */
int detag_set_noise(detag_state* s, double sigma, uint64_t seed, int64_t coord_offset);

/* Force a kernel variant (DETAG_VARIANT_*).  Errors: ARG, UNSUPPORTED (variant not applicable to this M). */
int detag_set_variant(detag_state* s, int variant);
/* The variant the next detag_step will run (never AUTO). */
int detag_get_variant(const detag_state* s, int* variant);

/*
 * Where the stochastic gradient of a step is evaluated (DETAG_GRADIENT_AT_*).
 * Algorithm 2 as printed queries the oracle during the K gossip rounds of a phase, at the point x_k
 * the phase started from, and folds g_(k) - g_(k-1) into the tracker at the end of the phase; its
 * gradients are therefore one phase older than with the default, which evaluates at the new model:
 *     g'  = a o (x - c) + sigma * xi     (x = the model before this step's update)
 * Everything else in the step listing at the top is unchanged, and so is detag_init.  Errors: ARG.
 */
int detag_set_gradient_point(detag_state* s, int where);
int detag_get_gradient_point(const detag_state* s, int* where);

/*
 * D-PSGD (the baseline of the paper's Section "Experiments"; update rule in its Section "Related work":
 * every worker averages its neighbours' models with the gossip matrix and takes a step along its own
 * stochastic gradient).  With DETAG_ALGORITHM_DPSGD a step is
 *     x'  = AG_K(x) - alpha * g          (plain D-PSGD is K = 1, eta = 0: x' = M x - alpha g)
 *     g'  = a o (x' - c) + sigma * xi    (the gradient the NEXT step uses, evaluated at the new model)
 * on the same kernels, with one contraction and no tracker: the y buffer is neither read nor written, and
 * 24 bytes per worker-coordinate cross HBM instead of 32.  detag_init then sets g = gradient at the bound x only.
 * Synthetic gradient only.  Errors: ARG, UNSUPPORTED (combined with caller-written gradients).
 */
int detag_set_algorithm(detag_state* s, int algorithm);
int detag_get_algorithm(const detag_state* s, int* algorithm);

/*
 * Caller-written stochastic gradients.  In the paper the gradient oracle of Algorithm 2 (Section "Setting",
 * oracle class; the line of Algorithm 2 that spends the query budget) is back-propagation on a mini-batch, not
 * a formula.  With DETAG_GRADIENT_EXTERNAL the library evaluates no gradient: before detag_init and before every
 * detag_step the caller writes the stochastic gradient at the CURRENT model x into g_new (device, [n][ld]
 * float32, 16-byte aligned, caller-owned, must stay valid), and a step is Algorithm 2 without the query:
 *     y   = y + g_new - g                tracker update (g = the gradient folded by the previous step)
 *     y'  = AG_K(y) ;  x' = AG_K(x) - alpha * y'
 *     g   = g_new                        the library keeps the folded gradient for the next update
 * so here the y buffer holds the gossiped tracker itself (not the early-folded one of the default mode), and
 * 28 bytes per worker-coordinate cross HBM.  detag_init sets y = g = g_new (the first update is then the
 * identity).  a, c, the noise settings and the gradient point are not used.  detag_step_many accepts count = 1
 * only; detag_step_host is not offered.  DETAG_GRADIENT_SYNTHETIC switches back (g_new is ignored).
 * Errors: ARG (unknown source, null or misaligned g_new), UNSUPPORTED (combined with D-PSGD).
 */
int detag_set_gradient_source(detag_state* s, int source, const float* g_new);

/*
 * Stochastic gradient of the zero-chain objective of the paper's lower-bound construction (proof of Theorem 1:
 * the equation defining the base function fhat, and "Setting 1": every worker holds fhat, rescaled as
 * f(x) = (L lambda^2 / l_1) fhat(x / lambda); the oracle multiplies the partial derivatives beyond the progress of
 * x - its last non-zero coordinate - by z / p with z ~ Bernoulli(p), one draw per worker and step):
 *     g_out[i][j] = gain * d_j fhat(x_i / lambda) * (j > prog(x_i) ? z_i / p : 1)          gain = L lambda / l_1
 *     fhat(u) = sum_{i=0}^{d-1} [Psi(-u_i) Phi(-u_{i+1}) - Psi(u_i) Phi(u_{i+1})],  u_0 := 1,
 *     Psi(z) = exp(1 - 1/(2z-1)^2) for z > 1/2 (else 0),  Phi(z) = sqrt(e) int_{-inf}^z exp(-t^2/2) dt.
 * The chain runs over all d coordinates of a worker, which are coupled to their neighbours: unlike the diagonal
 * objective this gradient cannot be evaluated shard by shard.  z_i is a pure function of (seed, t, i).
 * x, g_out: device, [n][ld] float32 (may not alias); scratch: device, n int32 (per-worker progress, overwritten).
 * Meant to be used with detag_set_gradient_source(DETAG_GRADIENT_EXTERNAL): write g_out = the registered array
 * before each detag_step.  Asynchronous on `stream`.  No detag_state is involved.
 * Errors: ARG (null pointers, ld < d, lambda <= 0, p outside (0, 1], t < 0), UNSUPPORTED (n > 1024, d >= 2^31), CUDA.
 */
int detag_zero_chain_gradient(int n, int64_t d, int64_t ld, const float* x, float* g_out, double lambda, double gain,
                              double p, uint64_t seed, int64_t t, int32_t* scratch, void* stream);

/*
 * Phase length of Theorem 3: R = max(1/2 ln n, 1/2 ln(varsigma0_sq * T / delta_L)) / sqrt(1 - lambda),
 * rounded up to a whole number of gossip rounds, at least 1.  lambda as returned by detag_spectral,
 * varsigma0_sq the bound on the gradient dissimilarity at the origin (Section "Setting"), T the
 * number of iterations, delta_L the product Delta * L; the second term is left out when any of
 * varsigma0_sq, T, delta_L is not positive.  Host only.  Errors: ARG (n < 1, lambda outside [0, 1), null R).
 */
int detag_phase_length(int n, double lambda, double varsigma0_sq, double T, double delta_L, int* R);

/*
 * Initial state of Algorithm 2 (which leaves the tracker's start open): g = stochastic gradient at the bound x
 * (noise of step 0), y = g.  Sets the step counter to 0.  Asynchronous.  Errors: UNBOUND, CUDA.
 */
int detag_init(detag_state* s, void* stream);

/*
 * One DeTAG iteration for all workers (Algorithm 2 with Algorithm 3 as the gossip; see the
 * step listing at the top).  Asynchronous; the step counter advances by one at enqueue time.
 * Errors: UNBOUND, CUDA (launch failure).  Device-side problems surface in detag_status.
 */
int detag_step(detag_state* s, void* stream);

/*
 * `count` consecutive DeTAG iterations: the same result, bit for bit, as `count` calls of detag_step.
 * The iteration never mixes coordinates (Algorithm 3 mixes workers only, the synthetic objective is
 * diagonal), so where the kernel variant allows it (dense polynomial, n <= 32, no observer buffer) all
 * `count` iterations of a coordinate slab run on chip in one launch and the state crosses HBM once per
 * call instead of once per iteration; otherwise the call enqueues `count` single steps.
 * Asynchronous; the step counter advances by `count`.  Errors: ARG (count < 1), UNBOUND, CUDA.
 */
int detag_step_many(detag_state* s, int count, void* stream);

/*
 * Consensus error of the model, ||X - Xbar 1^T||_F^2 = sum_j sum_i (x_ij - mean_i x_ij)^2
 * (the quantity bounded in the proof of Theorem 3), accumulated in float64 in a fixed order.
 * Enqueues on `stream`, waits for it, writes *host_out.  Errors: ARG, UNBOUND, CUDA.
 */
int detag_consensus_error(detag_state* s, void* stream, double* host_out);

/*
 * One DeTAG iteration (same arithmetic as detag_step) on state that lives in HOST memory: x, y, g
 * (read and written) and a, c (read) are host arrays [n][ld_host] float32, page-locked if the
 * copies are to overlap.  The coordinate axis is cut into chunks; each chunk is copied to the
 * device, stepped and copied back, two chunks in flight on two internal streams (the step never
 * mixes coordinates, so chunks are independent).  `staging` is caller-owned device memory of
 * `staging_bytes` >= detag_host_staging_bytes(s, chunk_coords): it holds the graph tables and two
 * chunk slots; buffers bound with detag_bind are not touched and need not exist.
 * Ordering: the work starts after everything enqueued on `stream` so far and `stream` waits for
 * it; the call itself returns without waiting.  The step counter advances by one.
 * Errors: ARG (null/misaligned pointers, staging too small for a 128-coordinate chunk), CUDA.
 */
int detag_step_host(detag_state* s, int64_t ld_host, float* x, float* y, float* g, const float* a, const float* c,
                    void* staging, size_t staging_bytes, void* stream);
/* Device bytes detag_step_host needs to run with chunks of `chunk_coords` coordinates (a multiple of 128). */
int detag_host_staging_bytes(const detag_state* s, int64_t chunk_coords, size_t* bytes);

/*
 * Consensus error (same definition and kernels as detag_consensus_error) for callers that cannot
 * give the library any scratch memory.  The paper has no counterpart: this entry point exists for
 * the sake of its callers only.
 *
 * Who needs it: code that must not allocate device memory at the point where it wants the number,
 * and has no workspace at hand either - for example a monitoring hook that runs while a CUDA graph
 * is being replayed or inside a memory-pool region where cudaMalloc would synchronise the device,
 * a plug-in that is handed only the model buffer, or a process whose allocator has already given all
 * device memory to the training job.  It takes no detag_state and no workspace: only the input
 * x (device, [n][ld] float32, ld >= d) and the output *host_out (host).
 *
 * The partial sums go to an array that is compiled into the library (1 MiB + one result slot per
 * GPU that loads it, held until the process exits), one float64 partial per 256 coordinates.  That
 * fixes the limit: d <= 33,554,432 (and n <= 1024); larger sizes return DETAG_ERR_UNSUPPORTED and
 * do nothing.  The call allocates and frees nothing, on the device or through any library.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 * caches it; make that first call outside any stream capture.  All calls on a device share the one
 * array.  Every slot a call reads is written by that call first, so leftovers of earlier calls do
 * no harm and nothing has to be cleared; but two calls that overlap on the GPU (different streams,
 * or different host threads) race on it and both results are then garbage: serialise them.
 * Enqueues on `stream`, waits for it, writes *host_out.
 * Errors: ARG, UNSUPPORTED (size beyond the built-in array, device ordinal >= 64), CUDA.
 */
int detag_consensus_error_static(int n, int64_t d, int64_t ld, const float* x, void* stream, double* host_out);

/* Step counter t (number of completed steps; enters the noise counter).  set_step is for resume. */
int detag_get_step(const detag_state* s, int64_t* t);
int detag_set_step(detag_state* s, int64_t t);

/*
 * Waits for `stream`, then reads the device status words - the one in the bound workspace and, if
 * detag_step_host has run since the last clean detag_status, the one at the head of its staging area
 * (which must therefore still be allocated) - and returns DETAG_OK, DETAG_ERR_TIMEOUT (a bounded
 * device-side wait gave up; the state arrays are then not to be trusted) or DETAG_ERR_CUDA.  A state that
 * has only ever stepped host-resident needs no detag_bind for this call.  The words are sticky: detag_bind
 * clears the workspace's, a staging area's is cleared when detag_step_host first uses it.
 * Errors: UNBOUND (neither bound nor stepped host-resident), CUDA, TIMEOUT.
 */
int detag_status(detag_state* s, void* stream);

/*
 * Failure-detection self tests.  The paper has no counterpart (its algorithm is synchronous and assumes
 * no failures); these exist so that the bounded waits of the kernels, their wind-down and DETAG_ERR_TIMEOUT
 * can be exercised without faulting, trapping or hanging the GPU.
 *
 * detag_debug_inject_stall: from now on the loading thread of every CTA of the tensor-path step kernels stops
 * issuing loads after `after_tiles` tiles, and every device-side wait gives up after `poll_limit` polls
 * (16 .. 2^20; a poll suspends for at most about two microseconds).  The CTAs' waiters then time out one
 * after the other, set the status word and return; the launch ends normally and detag_status reports
 * DETAG_ERR_TIMEOUT.  The state arrays are left partly updated.  after_tiles < 0 restores normal operation
 * (no stall, default limit).  Host only.  Errors: ARG.
 *
 * detag_debug_expire_wait: launches one thread that waits, through the same bounded wait, on a barrier that
 * nothing ever arrives at, with a limit of `polls` polls (1 .. 2^20); it gives up, sets the workspace's status
 * word and returns.  Asynchronous.  Errors: ARG, UNBOUND, CUDA.
 */
int detag_debug_inject_stall(detag_state* s, int64_t after_tiles, uint32_t poll_limit);
int detag_debug_expire_wait(detag_state* s, uint32_t polls, void* stream);

/* Text of the last error on this state ("" if none).  Owned by the state. */
const char* detag_last_error(const detag_state* s);

/* Frees the host-side state.  Device buffers stay the caller's. */
int detag_destroy(detag_state* s);

#ifdef __cplusplus
}
#endif
#endif /* DETAG_H */
