// DeTAG step for block-circulant gossip matrices with 8-worker blocks (the R x 8 torus): the K-round accelerated
// gossip as "transform along the block axis, one 8 x 8 product per frequency, transform back".
//
// Workers are numbered i = 8 r + c (block r = 0..R-1, position c = 0..7).  When M[(r,c)][(r',c')] depends on the
// block distance (r' - r) mod R only, and equally for +k and -k (every torus with uniform or Metropolis weights:
// the blocks are the rings of one axis, the block distance runs along the other), M - and with it every
// polynomial of M, in particular P = P_K(M) of Algorithm 3 - is block-diagonalised by the real Fourier basis Q
// of the R-cycle:
//     P = sum_p (q_p q_p^T) (x) Phat_p ,      Phat_p = P_K(Mhat_p) ,  Mhat_p = sum_k cos(2 pi f_p k / R) G_k
// (G_k the 8 x 8 block at distance k, f_p the frequency of basis vector q_p; all built by the host in float64
// and checked there against the dense polynomial).  Applying P to a slab then costs, per worker-coordinate and
// array, a transform along r, 8 multiply-adds for the block product and the transform back: about 13 operations
// for R = 8 (butterflies) instead of the 64 of the dense 64 x 64 product.
//
// Mapping onto the float64 tensor instruction (mma m8n8k4): the eight coordinates of a warp's tile are the M
// index, the position c is the contraction index (two k-steps of four, c = kq + 4 s) and the output position c'
// the N index, with the N columns permuted (column 2 kq + e stands for c' = kq + 4 e):
//     D[coord][c'] = sum_c Zhat_p[coord][c] Phat_p[c'][c] .
// The A fragment a lane supplies and the C fragment it receives are then the SAME worker positions: lane
// (coord = lane / 4, kq = lane % 4) owns workers 8 r + kq + 4 e (r = 0..R-1, e = 0, 1) of one coordinate for input
// and output alike.  So the transforms along r run inside the lane over its own registers, the tail of the step
// (model update, noise, gradient, tracker fold) is lane-local, and every lane writes its results over the very
// elements it read: the output needs no tile of its own.
//
// Shared memory holds tiles of [64 or 32 workers][64 coordinates], loaded by ONE three-dimensional TMA box per
// array and slab - {32 coordinates, 2 halves, all rows}, 128-byte swizzle - so that every row is fetched as one
// contiguous 256-byte piece (boxes of 32 coordinates fetched on their own reach 0.71 of the HBM copy rate with
// this access pattern, 256-byte pieces 0.88).  With the ownership above every warp-wide access hits 32 different
// banks, and the TMA stores undo the swizzle on the way out.  The box walks whole 32-coordinate halves: the last
// d % 32 columns of the arrays are patched into the stage, and written back, by the lanes that own them.
// Roles of the persistent CTA (one per SM):
//   loaders   two threads: per slab one box each of x, y into one of two short-lived stages (handed back as soon as
//             the tracker contraction has read its operands), and one box each of g, a, c into one of three
//             long-lived stages (read in the tail, then overwritten with g', x', y');
//   consumers 16 warps in two groups taking alternate slabs; a warp owns 8 coordinates x all workers;
//   storer    one thread: when a group's 8 warps have written their results, three TMA stores send the stage's
//             tiles out; once they have been read the stage goes back to its loader.
// Arithmetic: float64 on chip, every stored value rounded once; x' = P (x - alpha y) by linearity of AG_K, the
// tracker fold as (y~ - g) + fl32(g') like the other kernels.  Every wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"
#include "tma.cuh"
#include "torus_basis.h"

namespace detag {

namespace {

constexpr int kC = 8;                  // workers per block = MMA contraction and N extent
constexpr int kTS = 64;                // coordinates per slab
constexpr int kHalfCols = 32;          // coordinates per 128-byte swizzle row
constexpr int kXYStages = 2, kEStages = 3;
constexpr int kTGroups = 2, kTGroupWarps = kTS / 8;
constexpr int kTConsumerWarps = kTGroups * kTGroupWarps;
constexpr int kTLoadXYWarp = kTConsumerWarps, kTStoreWarp = kTConsumerWarps + 1, kTLoadEWarp = kTConsumerWarps + 2;
constexpr int kTThreads = (kTConsumerWarps + 3) * 32;

template <int R>
struct TorusPlan {
  static constexpr int kRows = R * kC;
  static constexpr int kTileFloats = kRows * kTS;          // one array of one slab: [row][half][32]
  static constexpr int kTileBytes = kTileFloats * 4;
  static constexpr int kXYBytes = 2 * kTileBytes, kEBytes = 3 * kTileBytes;
  static constexpr int kFragDoubles = R * 2 * 32;          // Phat in fragment order: [p][k-step][lane]
  static constexpr size_t kBarrierOffset =
      static_cast<size_t>(kXYStages) * kXYBytes + static_cast<size_t>(kEStages) * kEBytes + kFragDoubles * 8;
  static constexpr size_t kSmemBytes = kBarrierOffset + 128 + 1024;  // + barriers, + slack to align the tiles to 1 KiB
  static_assert((2 * kXYStages + 3 * kEStages) * 8 + kTGroups * 4 <= 128, "barrier area");
  static_assert(kSmemBytes <= 232448, "shared memory plan");
};

struct TorusMaps {
  CUtensorMap x, y, g, a, c;  // loads: boxes {32 coordinates, 2 halves, all rows}, 128-byte swizzle, zero fill
  CUtensorMap xs, ys, gs;     // stores: the same boxes
};
static_assert(sizeof(TorusMaps) <= sizeof(TensorMapSet), "tensor map storage");

// Transform of one worker column (this lane's R values along the block axis) into the Fourier components of the
// block cycle, and back.  R = 8: butterflies of the real 8-point transform WITHOUT normalisation (20 operations
// instead of 48; the host folds the two missing factors 1/8 resp. 1/4 into the per-frequency blocks).  Other R:
// dense product with the orthonormal basis.  Component order as in torus_basis.h.
template <int R>
__device__ __forceinline__ void torus_forward(const double (&z)[R], double (&w)[R]) {
  if (R == 8) {
    constexpr double c = 0.70710678118654752440;
    const double s0 = z[0] + z[4], d0 = z[0] - z[4], s1 = z[1] + z[5], d1 = z[1] - z[5];
    const double s2 = z[2] + z[6], d2 = z[2] - z[6], s3 = z[3] + z[7], d3 = z[3] - z[7];
    const double t0 = s0 + s2, t1 = s1 + s3, u = d1 - d3, v = d1 + d3;
    w[0] = t0 + t1;            // frequency 0
    w[R - 1] = t0 - t1;        // frequency 4
    w[1] = fma(c, u, d0);      // frequency 1: cosine, sine
    w[2] = fma(c, v, d2);
    w[3] = s0 - s2;            // frequency 2
    w[4] = s1 - s3;
    w[R - 3] = fma(-c, u, d0); // frequency 3
    w[R - 2] = fma(c, v, -d2);
  } else {
#pragma unroll
    for (int pf = 0; pf < R; ++pf) {
      double acc = 0.0;
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (torus_q(R, pf, r) != 0.0) acc = fma(torus_q(R, pf, r), z[r], acc);
      w[pf] = acc;
    }
  }
}

template <int R>
__device__ __forceinline__ void torus_backward(const double (&w)[R], double (&z)[R]) {
  if (R == 8) {
    constexpr double c = 0.70710678118654752440;
    const double e0 = w[0] + w[R - 1], e1 = w[0] - w[R - 1];
    const double p1 = w[1] + w[R - 3], p2 = w[2] - w[R - 2];  // C1 + C3, S1 - S3
    const double q1 = w[1] - w[R - 3], q2 = w[2] + w[R - 2];  // C1 - C3, S1 + S3
    const double a0 = e0 + w[3], a1 = e0 - w[3], b0 = e1 + w[4], b1 = e1 - w[4];
    const double m0 = q1 + q2, m1 = q2 - q1;
    z[0] = a0 + p1;
    z[4] = a0 - p1;
    z[2] = a1 + p2;
    z[R - 2] = a1 - p2;
    z[1] = fma(c, m0, b0);
    z[R - 3] = fma(-c, m0, b0);
    z[3] = fma(c, m1, b1);
    z[R - 1] = fma(-c, m1, b1);
  } else {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      double acc = 0.0;
#pragma unroll
      for (int pf = 0; pf < R; ++pf)
        if (torus_q(R, pf, r) != 0.0) acc = fma(torus_q(R, pf, r), w[pf], acc);
      z[r] = acc;
    }
  }
}

// P applied to this lane's two worker columns: forward transform of each (column(s, z) supplies column c = 2 kq + s),
// one float64 MMA pair per frequency (contraction over the position inside the block, all four lanes of a coordinate
// together) - torus_contract - then the transform back of the columns c' = 2 kq + e - torus_finish.
template <int R, typename Column>
__device__ __forceinline__ void torus_contract(double (&acc)[R][2], const double* frag, int lane, Column column) {
#pragma unroll
  for (int pf = 0; pf < R; ++pf) acc[pf][0] = acc[pf][1] = 0.0;
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    double z[R], w[R];
    asm volatile("" ::: "memory");  // keeps the second column's loads behind the first column's arithmetic (registers)
    column(s, z);
    torus_forward<R>(z, w);
#pragma unroll
    for (int pf = 0; pf < R; ++pf) dmma(acc[pf], w[pf], frag[(pf * 2 + s) * 32 + lane]);
  }
}

template <int R>
__device__ __forceinline__ void torus_finish(const double (&acc)[R][2], int e, double (&out)[R]) {
  double w[R];
#pragma unroll
  for (int pf = 0; pf < R; ++pf) w[pf] = acc[pf][e];
  torus_backward<R>(w, out);
}


// Gradient phase of a lane: g' = a (x_at - c) + sigma xi for its 2R elements (element (r, e) at off + r * 512 + e * 256),
// written over c in the stage (c is not needed again; the tracker phase picks g' up from there).  x_at: the model
// at which the gradient is taken.  Noise: the lane's workers 8 r + 4 e + kq are position kq of the Philox quads
// 2 r + e, which the four lanes of a coordinate share: each draws every fourth quad (all four normals of it) and a
// 4 x 4 transpose over the lanes hands everybody its own position.
template <int R>
__device__ __forceinline__ void torus_gradient(const StepParams& p, const float* sa, float* sc, int off,
                                               const float (&x_at)[2][R], int kq, long long j, float sigma, bool noisy) {
  unsigned long long jn = static_cast<unsigned long long>(p.coord_offset + j);
#pragma unroll
  for (int t = 0; t < R / 2; ++t) {  // quads 4 t .. 4 t + 3: blocks r = 2 t, 2 t + 1
    float xi[4] = {0.f, 0.f, 0.f, 0.f};
    if (noisy) {
      normal_quad(p.seed_lo, p.seed_hi, jn, static_cast<uint32_t>(4 * t + kq), p.t_noise, xi);
      transpose_quad(xi, kq);  // xi[i]: this lane's position of quad 4 t + i, i.e. r = 2 t + (i >> 1), e = i & 1
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = 2 * t + (i >> 1), e = i & 1, o = off + r * 512 + e * 256;
      sc[o] = fmaf(sa[o], x_at[e][r] - sc[o], sigma * xi[i]);
    }
  }
}

template <int R, bool kAtStart>
__global__ void __launch_bounds__(kTThreads, 1)
step_torus_kernel(const StepParams p, const __grid_constant__ TorusMaps maps, const double* __restrict__ phat_frag) {
  using Plan = TorusPlan<R>;
  extern __shared__ unsigned char smem_unaligned[];
  // the swizzle pattern is a function of the shared-memory address: tiles start on 1 KiB boundaries
  unsigned char* smem_raw = smem_unaligned + ((1024u - (s_addr(smem_unaligned) & 1023u)) & 1023u);
  float* xy_mem = reinterpret_cast<float*>(smem_raw);                                   // [stage][x | y]
  float* e_mem = xy_mem + kXYStages * 2 * Plan::kTileFloats;                            // [stage][g | a | c]
  double* frag = reinterpret_cast<double*>(e_mem + kEStages * 3 * Plan::kTileFloats);   // [p][k-step][lane]
  uint64_t* xy_full = reinterpret_cast<uint64_t*>(smem_raw + Plan::kBarrierOffset);
  uint64_t* xy_empty = xy_full + kXYStages;
  uint64_t* e_full = xy_empty + kXYStages;
  uint64_t* e_empty = e_full + kEStages;
  uint64_t* out_ready = e_empty + kEStages;
  unsigned* seen = reinterpret_cast<unsigned*>(out_ready + kEStages);  // [group]: 1 + last slab whose g, a, c it saw

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < Plan::kFragDoubles; e += kTThreads) frag[e] = phat_frag[e];
  if (tid == 0) {
    for (int g = 0; g < kTGroups; ++g) seen[g] = 0;
    for (int s = 0; s < kXYStages; ++s) {
      bar_init(&xy_full[s], 1);
      bar_init(&xy_empty[s], kTGroupWarps);
    }
    for (int s = 0; s < kEStages; ++s) {
      bar_init(&e_full[s], 1);
      bar_init(&e_empty[s], 1);
      bar_init(&out_ready[s], kTGroupWarps);
    }
    fence_barrier_init();
  }
  fence_async_shared();
  __syncthreads();

  // this CTA takes slabs blockIdx.x, blockIdx.x + gridDim.x, ...; k counts them
  const long long my_slabs = blockIdx.x < p.num_slabs ? (p.num_slabs - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const unsigned limit = p.spin_limit;
  const long long d32 = p.d & ~31LL;  // columns below this travel by TMA, the rest by the lanes that own them
  const int halves = static_cast<int>(d32 / kHalfCols);

  if (warp == kTLoadXYWarp) {
    // ---------------------------------------------------------------- x, y loader: runs ahead of the other one
    if (lane == 0) {
      long long k = 0;
      bool ok = true;
      for (; k < my_slabs; ++k) {
        if (p.stall_after >= 0 && k >= p.stall_after) return;  // self test: the loads stop, every waiter times out
        const int sx = static_cast<int>(k % kXYStages);
        if (k >= kXYStages) ok = bar_wait(&xy_empty[sx], ((k / kXYStages) - 1) & 1, limit);
        if (!ok) break;
        const int half = static_cast<int>((blockIdx.x + k * gridDim.x) * 2);
        float* tx = xy_mem + static_cast<size_t>(sx) * 2 * Plan::kTileFloats;
        const bool any = half < halves;  // a slab without a whole half is served entirely by its lanes
        bar_expect_tx(&xy_full[sx], any ? Plan::kXYBytes : 0u);
        if (any) {
          rows_load(tx, &maps.x, half, 0, &xy_full[sx]);
          rows_load(tx + Plan::kTileFloats, &maps.y, half, 0, &xy_full[sx]);
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (long long back = 1; back <= kXYStages && back <= k; ++back) {  // drain copies still in flight (bounded)
          const long long q = k - back;
          bar_wait(&xy_full[q % kXYStages], (q / kXYStages) & 1, limit);
        }
      }
    }
    return;
  }
  if (warp == kTLoadEWarp) {
    // ---------------------------------------------------------------- g, a, c loader
    if (lane == 0) {
      long long k = 0;
      bool ok = true;
      for (; k < my_slabs; ++k) {
        if (p.stall_after >= 0 && k >= p.stall_after) return;
        const int se = static_cast<int>(k % kEStages);
        if (k >= kEStages) ok = bar_wait(&e_empty[se], ((k / kEStages) - 1) & 1, limit);
        if (!ok) break;
        const int half = static_cast<int>((blockIdx.x + k * gridDim.x) * 2);
        float* te = e_mem + static_cast<size_t>(se) * 3 * Plan::kTileFloats;
        const bool any = half < halves;
        bar_expect_tx(&e_full[se], any ? Plan::kEBytes : 0u);
        if (any) {
          rows_load(te, &maps.g, half, 0, &e_full[se]);
          rows_load(te + Plan::kTileFloats, &maps.a, half, 0, &e_full[se]);
          rows_load(te + 2 * Plan::kTileFloats, &maps.c, half, 0, &e_full[se]);
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (long long back = 1; back <= kEStages && back <= k; ++back) {
          const long long q = k - back;
          bar_wait(&e_full[q % kEStages], (q / kEStages) & 1, limit);
        }
      }
    }
    return;
  }
  if (warp == kTStoreWarp) {
    if (lane == 0) {
      for (long long k = 0; k < my_slabs; ++k) {
        const int se = static_cast<int>(k % kEStages);
        if (!bar_wait(&out_ready[se], (k / kEStages) & 1, limit)) {
          atomicExch(p.status, 1);
          break;
        }
        const float* te = e_mem + static_cast<size_t>(se) * 3 * Plan::kTileFloats;  // now [g' | x' | y']
        const int half = static_cast<int>((blockIdx.x + k * gridDim.x) * 2);
        if (half < halves) {  // the stores clip at the last whole half
          rows_store(&maps.gs, half, 0, te);
          rows_store(&maps.xs, half, 0, te + Plan::kTileFloats);
          rows_store(&maps.ys, half, 0, te + 2 * Plan::kTileFloats);
        }
        store_commit();
        store_wait_read();  // the stage may be refilled now
        bar_arrive(&e_empty[se]);
      }
      store_wait_all();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int kq = lane & 3, crow = lane >> 2;  // crow: this lane's coordinate within the warp's 8
  const int group = warp / kTGroupWarps, tile = warp % kTGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  // Float offset of this lane's element (r = 0, e = 0) inside an array's tile; element (r, e) - worker
  // 8 r + kq + 4 e - lies r * 512 + e * 256 further.  Tile = [row][half][32]; the 16-byte chunk index is XORed with
  // the low three bits of the 128-byte row number 2 * row + half (the tensor maps' swizzle), which for this lane's
  // rows is always 2 kq + half.
  const int half_of_tile = tile >> 2;
  const int chunk = 2 * (tile & 3) + (crow >> 2);
  const int off = kq * kTS + half_of_tile * kHalfCols + (((chunk ^ ((2 * kq + half_of_tile) & 7)) << 2) | (crow & 3));

  for (long long k = group; k < my_slabs; k += kTGroups) {
    const int sx = static_cast<int>(k % kXYStages), se = static_cast<int>(k % kEStages);
    bool ok = true;
    if (lane == 0) ok = bar_wait(&xy_full[sx], (k / kXYStages) & 1, limit);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    float* sxp = xy_mem + static_cast<size_t>(sx) * 2 * Plan::kTileFloats;
    float* syp = sxp + Plan::kTileFloats;
    float* sg = e_mem + static_cast<size_t>(se) * 3 * Plan::kTileFloats;
    float* sa = sg + Plan::kTileFloats;
    float* sc = sa + Plan::kTileFloats;
    const long long slab = blockIdx.x + k * gridDim.x;
    const long long j = slab * kTS + tile * 8 + crow;  // this lane's coordinate
    const bool active = slab * kTS + tile * 8 < p.d;   // a tile wholly beyond column d computes nothing
    const bool mine = j >= d32 && j < p.d;             // a column the TMA boxes do not reach: this lane moves it
    if (mine) {
#pragma unroll
      for (int e = 0; e < 2; ++e)
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const long long g_off = static_cast<long long>(8 * r + kq + 4 * e) * p.ld + j;
          sxp[off + r * 512 + e * 256] = p.x[g_off];
          syp[off + r * 512 + e * 256] = p.y[g_off];
        }
    }

    // Registers are the scarce resource here (2R values per array and lane, float64 accumulators): the phases below
    // run one after the other, read their operands from the stages when they need them and park what a later
    // phase needs in the lane's own slots - g' over c, x' over a (both read just before), finally g' over g and y'
    // over c.
    float xv[2][R];  // x'
    if (active) {
      // ---- model: x' = P (x - alpha y), by linearity of AG_K
      double acc[R][2];
      torus_contract<R>(acc, frag, lane, [&](int s, double (&z)[R]) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int o = off + r * 512 + s * 256;
          z[r] = fma(-alpha, static_cast<double>(syp[o]), static_cast<double>(sxp[o]));
        }
      });
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        double out[R];
        torus_finish<R>(acc, e, out);
#pragma unroll
        for (int r = 0; r < R; ++r) xv[e][r] = static_cast<float>(out[r]);  // rounded once
      }
    }
    // g, a, c are needed from here on; their loads had the model contraction to arrive in
    if (lane == 0) {
      // The stage last held slab k - 3, which belongs to the other group (odd stage count): a parity wait must not
      // start before that phase has completed, or it could not tell the two apart.
      if (k >= kEStages) ok = count_wait(&seen[(k - kEStages) % kTGroups], static_cast<unsigned>(k - kEStages + 1), limit);
      if (ok) ok = bar_wait(&e_full[se], (k / kEStages) & 1, limit);
      if (ok && tile == 0) count_publish(&seen[group], static_cast<unsigned>(k + 1));
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    if (mine) {
#pragma unroll
      for (int e = 0; e < 2; ++e)
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const long long g_off = static_cast<long long>(8 * r + kq + 4 * e) * p.ld + j;
          sg[off + r * 512 + e * 256] = p.g[g_off];
          sa[off + r * 512 + e * 256] = p.a[g_off];
          sc[off + r * 512 + e * 256] = p.c[g_off];
        }
    }
    if (active) {
      if (kAtStart) {  // Algorithm 2 as printed: the gradient at the model the step started from (still staged)
        float xold[2][R];
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int r = 0; r < R; ++r) xold[e][r] = sxp[off + r * 512 + e * 256];
        torus_gradient<R>(p, sa, sc, off, xold, kq, j, sigma, noisy);
      } else {
        torus_gradient<R>(p, sa, sc, off, xv, kq, j, sigma, noisy);
      }
#pragma unroll
      for (int e = 0; e < 2; ++e)
#pragma unroll
        for (int r = 0; r < R; ++r) sa[off + r * 512 + e * 256] = xv[e][r];  // x' takes a's place
    }
    // ---- tracker: y~ = P y, then the fold (y~ - g) + g'
    double acc[R][2];
    if (active) {
      torus_contract<R>(acc, frag, lane, [&](int s, double (&z)[R]) {
#pragma unroll
        for (int r = 0; r < R; ++r) z[r] = static_cast<double>(syp[off + r * 512 + s * 256]);
      });
    }
    if (mine) fence_async_shared();  // this lane wrote into the x, y stage: order that before the next load into it
    __syncwarp();
    if (lane == 0) bar_arrive(&xy_empty[sx]);  // that was the last read of the x, y stage: it can be refilled
    if (active) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        double out[R];
        torus_finish<R>(acc, e, out);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int o = off + r * 512 + e * 256;
          const float go = sc[o];  // g', parked there by the gradient phase
          const float yo = static_cast<float>((out[r] - static_cast<double>(sg[o])) + static_cast<double>(go));
          sg[o] = go;
          sc[o] = yo;
          if (p.y_obs != nullptr && j < p.d)  // optional observer: the gossiped tracker, stored directly
            p.y_obs[static_cast<long long>(8 * r + kq + 4 * e) * p.ld + j] = static_cast<float>(out[r]);
        }
      }
      if (mine) {  // the last d % 32 columns go out directly
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int o = off + r * 512 + e * 256;
            const long long g_off = static_cast<long long>(8 * r + kq + 4 * e) * p.ld + j;
            p.x[g_off] = sa[o];
            p.y[g_off] = sc[o];
            p.g[g_off] = sg[o];
          }
      }
    }
    fence_async_shared();  // results visible to the TMA stores
    __syncwarp();
    if (lane == 0) bar_arrive(&out_ready[se]);
  }
}

typedef void (*TorusKernel)(const StepParams, const TorusMaps, const double*);

}  // namespace

bool torus_variant_available(int n) { return (n == 32 || n == 64) && encode_tiled_fn() != nullptr; }

bool build_maps_torus(const StepParams& p, TensorMapSet* out) {
  TorusMaps& m = *reinterpret_cast<TorusMaps*>(out->bytes);
  if (!make_half_map(&m.x, p.x, p.n, p.d, p.ld, p.n) || !make_half_map(&m.y, p.y, p.n, p.d, p.ld, p.n) ||
      !make_half_map(&m.g, p.g, p.n, p.d, p.ld, p.n) || !make_half_map(&m.a, p.a, p.n, p.d, p.ld, p.n) ||
      !make_half_map(&m.c, p.c, p.n, p.d, p.ld, p.n))
    return false;
  m.xs = m.x;
  m.ys = m.y;
  m.gs = m.g;
  return true;
}

// phat_frag: device pointer to the R x 2 x 32 doubles of the per-frequency blocks in fragment order.
int launch_step_torus(StepParams p, const TensorMapSet& maps, const double* phat_frag, int sm_count,
                      cudaStream_t stream) {
  if (p.mode != kModeDetag || (p.n != 32 && p.n != 64)) return static_cast<int>(cudaErrorInvalidValue);
  const int R = p.n / kC;
  p.S = kTS;
  p.num_slabs = (p.d + kTS - 1) / kTS;
  TorusKernel kernel;
  size_t smem;
  if (R == 8) {
    kernel = p.grad_at_start ? step_torus_kernel<8, true> : step_torus_kernel<8, false>;
    smem = TorusPlan<8>::kSmemBytes;
  } else {
    kernel = p.grad_at_start ? step_torus_kernel<4, true> : step_torus_kernel<4, false>;
    smem = TorusPlan<4>::kSmemBytes;
  }
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kTThreads, smem, stream>>>(p, *reinterpret_cast<const TorusMaps*>(maps.bytes),
                                                                   phat_frag);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
