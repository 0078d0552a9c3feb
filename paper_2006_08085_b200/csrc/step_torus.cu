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
// array, R multiply-adds for the forward transform, 8 for the block product and R for the way back: 24 for
// R = 8 instead of the 64 of the dense 64 x 64 product.
//
// Mapping onto the float64 tensor instruction (mma m8n8k4): the eight coordinates of a warp's tile are the M
// index, the position c is the contraction index (two k-steps of four) and the output position c' the N index:
//     D[coord][c'] = sum_c Zhat_p[coord][c] Phat_p[c'][c] .
// With the k-steps taking c = 2 (lane % 4) + s, the A fragment a lane supplies and the C fragment it receives are
// the SAME worker positions: lane (coord = lane / 4, kq = lane % 4) owns workers 8 r + 2 kq + e (r = 0..R-1,
// e = 0, 1) of one coordinate for input and output alike.  So the transforms along r run inside the lane over its
// own registers (dense R x R with compile-time coefficients; a quarter of them are zero and cost nothing), the tail of the
// step (model update, noise, gradient, tracker fold) is lane-local, and every lane writes its results over the
// very elements it read: the output needs no tile of its own.
//
// Shared memory holds tiles of [64 or 32 workers][64 coordinates] as two 32-coordinate halves in the 128-byte
// swizzle of the tensor maps; with the ownership above every warp-wide access hits 32 different banks, and the
// TMA stores undo the swizzle on the way out.  Roles of the persistent CTA (one per SM):
//   producer  one thread: per slab two loads each of x, y into one of two short-lived stages (handed back as soon as
//             the tracker contraction has read its operands) and of g, a, c into one of three long-lived stages
//             (read in the tail, then overwritten with g', x', y');
//   consumers 16 warps in two groups taking alternate slabs; a warp owns 8 coordinates x all workers;
//   storer    one thread: when a group's 8 warps have written their results, six TMA stores send the stage's three
//             tiles out; once they have been read the stage goes back to the producer.
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
constexpr int kHalfCols = 32;          // coordinates per swizzled half tile (128 bytes)
constexpr int kXYStages = 2, kEStages = 3;
constexpr int kTGroups = 2, kTGroupWarps = kTS / 8;
constexpr int kTConsumerWarps = kTGroups * kTGroupWarps;
constexpr int kTProducerWarp = kTConsumerWarps, kTStoreWarp = kTConsumerWarps + 1;
constexpr int kTThreads = (kTConsumerWarps + 2) * 32;

template <int R>
struct TorusPlan {
  static constexpr int kRows = R * kC;
  static constexpr int kTileFloats = kRows * kTS;          // one array of one slab: two halves of [rows][32]
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
  CUtensorMap x, y, g, a, c;  // loads: boxes of [rows][32 coordinates], 128-byte swizzle, zero fill
  CUtensorMap xs, ys, gs;     // stores: the same boxes over the columns below d & ~3
};
static_assert(sizeof(TorusMaps) <= sizeof(TensorMapSet), "tensor map storage");

// [rows][32-coordinate box] tensor map with the 128-byte swizzle.
inline bool make_swizzled_map(CUtensorMap* m, const float* base, int n, long long d, long long ld, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(n)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * sizeof(float)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kHalfCols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Gradient phase of a lane: g' = a (x_at - c) + sigma xi for its 2R elements, written over c in the stage (c is not
// needed again; the tracker phase picks g' up from there).  x_at: the model at which the gradient is taken.
// Noise: the Philox call of (coordinate, workers 8 r + 4 (kq / 2) .. + 3) serves this lane and its neighbour
// kq ^ 1; each draws the calls of every other block r and they swap the word pairs they do not need themselves.
template <int R>
__device__ __forceinline__ void torus_gradient(const StepParams& p, const float* sa, float* sc, const int (&off_e)[2],
                                               const float (&x_at)[2][R], int kq, long long j, float sigma, bool noisy) {
  unsigned long long jn = static_cast<unsigned long long>(p.coord_offset + j);
  // Ties the counter to the model values so that the compiler cannot start the generator's integer work while the
  // contraction before this phase still holds its accumulators (it would spill them).
  asm volatile("" : "+l"(jn) : "f"(x_at[0][0]), "f"(x_at[1][R - 1]));
  const bool odd = (kq & 1) != 0;
#pragma unroll
  for (int h = 0; h < R / 2; ++h) {
    float xi[2][2] = {{0.f, 0.f}, {0.f, 0.f}};  // [e][block 2h, 2h + 1]
    if (noisy) {
      const int r_mine = 2 * h + (odd ? 1 : 0);
      const Philox4 w = philox4x32_10(static_cast<uint32_t>(jn), static_cast<uint32_t>(jn >> 32),
                                      static_cast<uint32_t>(2 * r_mine + (kq >> 1)), p.t_noise, p.seed_lo, p.seed_hi);
      // even kq owns the first pair of words (workers +0, +1 of the quad), odd kq the second (workers +2, +3)
      const uint32_t keep0 = odd ? w.r2 : w.r0, keep1 = odd ? w.r3 : w.r1;
      const uint32_t give0 = odd ? w.r0 : w.r2, give1 = odd ? w.r1 : w.r3;
      const uint32_t got0 = __shfl_xor_sync(0xffffffffu, give0, 1), got1 = __shfl_xor_sync(0xffffffffu, give1, 1);
      float n0, n1, m0, m1;
      box_muller(keep0, keep1, n0, n1);  // block r_mine
      box_muller(got0, got1, m0, m1);    // the neighbour's block
      xi[0][0] = odd ? m0 : n0;
      xi[1][0] = odd ? m1 : n1;
      xi[0][1] = odd ? n0 : m0;
      xi[1][1] = odd ? n1 : m1;
    }
#pragma unroll
    for (int b = 0; b < 2; ++b)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int r = 2 * h + b, o = off_e[e] + r * 256;
        sc[o] = fmaf(sa[o], x_at[e][r] - sc[o], sigma * xi[e][b]);
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

  if (warp == kTProducerWarp) {
    if (lane == 0) {
      long long k = 0;
      bool ok = true;
      for (; k < my_slabs; ++k) {
        if (p.stall_after >= 0 && k >= p.stall_after) return;  // self test: the loads stop, every waiter times out
        const int sx = static_cast<int>(k % kXYStages), se = static_cast<int>(k % kEStages);
        if (k >= kEStages) ok = bar_wait(&e_empty[se], ((k / kEStages) - 1) & 1, limit);
        if (ok && k >= kXYStages) ok = bar_wait(&xy_empty[sx], ((k / kXYStages) - 1) & 1, limit);
        if (!ok) break;
        const int col = static_cast<int>((blockIdx.x + k * gridDim.x) * kTS);
        float* tx = xy_mem + static_cast<size_t>(sx) * 2 * Plan::kTileFloats;
        float* te = e_mem + static_cast<size_t>(se) * 3 * Plan::kTileFloats;
        bar_expect_tx(&xy_full[sx], Plan::kXYBytes);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          tile_load(tx + h * (Plan::kTileFloats / 2), &maps.x, col + h * kHalfCols, 0, &xy_full[sx]);
          tile_load(tx + Plan::kTileFloats + h * (Plan::kTileFloats / 2), &maps.y, col + h * kHalfCols, 0, &xy_full[sx]);
        }
        bar_expect_tx(&e_full[se], Plan::kEBytes);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          tile_load(te + h * (Plan::kTileFloats / 2), &maps.g, col + h * kHalfCols, 0, &e_full[se]);
          tile_load(te + Plan::kTileFloats + h * (Plan::kTileFloats / 2), &maps.a, col + h * kHalfCols, 0, &e_full[se]);
          tile_load(te + 2 * Plan::kTileFloats + h * (Plan::kTileFloats / 2), &maps.c, col + h * kHalfCols, 0, &e_full[se]);
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (long long back = 1; back <= kEStages && back <= k; ++back) {  // drain copies still in flight (bounded)
          const long long q = k - back;
          bar_wait(&e_full[q % kEStages], (q / kEStages) & 1, limit);
          if (back <= kXYStages) bar_wait(&xy_full[q % kXYStages], (q / kXYStages) & 1, limit);
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
        const int col = static_cast<int>((blockIdx.x + k * gridDim.x) * kTS);
        const long long d_tma = p.d & ~3LL;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (col + h * kHalfCols < d_tma) {
            tile_store(&maps.gs, col + h * kHalfCols, 0, te + h * (Plan::kTileFloats / 2));
            tile_store(&maps.xs, col + h * kHalfCols, 0, te + Plan::kTileFloats + h * (Plan::kTileFloats / 2));
            tile_store(&maps.ys, col + h * kHalfCols, 0, te + 2 * Plan::kTileFloats + h * (Plan::kTileFloats / 2));
          }
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
  const long long d_tma = p.d & ~3LL;
  // Float offset of this lane's element (r = 0, e) inside an array's tile; element (r, e) lies r * 256 further.
  // Tile = [half][row][32]; 16-byte chunk index XOR (row & 7) is the tensor maps' 128-byte swizzle.
  int off_e[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int row7 = 2 * kq + e;  // (8 r + 2 kq + e) & 7
    const int chunk = 2 * (tile & 3) + (crow >> 2);
    off_e[e] = (tile >> 2) * (Plan::kTileFloats / 2) + row7 * kHalfCols + (((chunk ^ row7) << 2) | (crow & 3));
  }

  for (long long k = group; k < my_slabs; k += kTGroups) {
    const int sx = static_cast<int>(k % kXYStages), se = static_cast<int>(k % kEStages);
    bool ok = true;
    if (lane == 0) {
      ok = bar_wait(&xy_full[sx], (k / kXYStages) & 1, limit);
      // The g, a, c stage last held slab k - 3, which belongs to the other group (odd stage count): a parity wait
      // must not start before that phase has completed, or it could not tell the two apart.
      if (ok && k >= kEStages)
        ok = count_wait(&seen[(k - kEStages) % kTGroups], static_cast<unsigned>(k - kEStages + 1), limit);
      if (ok) ok = bar_wait(&e_full[se], (k / kEStages) & 1, limit);
      if (ok && tile == 0) count_publish(&seen[group], static_cast<unsigned>(k + 1));
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    const float* sxp = xy_mem + static_cast<size_t>(sx) * 2 * Plan::kTileFloats;
    const float* syp = sxp + Plan::kTileFloats;
    float* sg = e_mem + static_cast<size_t>(se) * 3 * Plan::kTileFloats;
    float* sa = sg + Plan::kTileFloats;
    float* sc = sa + Plan::kTileFloats;
    const long long slab = blockIdx.x + k * gridDim.x;
    const long long j = slab * kTS + tile * 8 + crow;  // this lane's coordinate
    const bool active = slab * kTS + tile * 8 < p.d;   // a tile wholly beyond column d computes nothing

    bool released = false;
    if (active) {
      // Registers are the scarce resource here (2R values per array and lane, float64 accumulators): the phases
      // below run one after the other, read their operands from the stages when they need them and park what a
      // later phase needs in the lane's own slots - x' over a, then g' over c (both read just before), finally g'
      // over g and y' over c.
      float xv[2][R];  // the model at which the gradient is taken, then x'
      if (kAtStart) {  // Algorithm 2 as printed: the gradient at the model the step started from
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int r = 0; r < R; ++r) xv[e][r] = sxp[off_e[e] + r * 256];
        torus_gradient<R>(p, sa, sc, off_e, xv, kq, j, sigma, noisy);
      }
      // ---- model: x' = P (x - alpha y), by linearity of AG_K
      {
        double acc[R][2];
#pragma unroll
        for (int pf = 0; pf < R; ++pf) acc[pf][0] = acc[pf][1] = 0.0;
#pragma unroll
        for (int s = 0; s < 2; ++s) {  // k-step s: this lane's worker column c = 2 kq + s
          double z[R];
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int o = off_e[s] + r * 256;
            z[r] = fma(-alpha, static_cast<double>(syp[o]), static_cast<double>(sxp[o]));
          }
#pragma unroll
          for (int pf = 0; pf < R; ++pf) {
            double zh = 0.0;  // forward transform: component pf of the column
#pragma unroll
            for (int r = 0; r < R; ++r) if (torus_q(R, pf, r) != 0.0) zh = fma(torus_q(R, pf, r), z[r], zh);
            dmma(acc[pf], zh, frag[(pf * 2 + s) * 32 + lane]);
          }
        }
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int r = 0; r < R; ++r) {
            double v = 0.0;  // transform back: worker (r, 2 kq + e)
#pragma unroll
            for (int pf = 0; pf < R; ++pf) if (torus_q(R, pf, r) != 0.0) v = fma(torus_q(R, pf, r), acc[pf][e], v);
            xv[e][r] = static_cast<float>(v);  // x', rounded once
          }
      }
      if (!kAtStart) torus_gradient<R>(p, sa, sc, off_e, xv, kq, j, sigma, noisy);  // at the new model
#pragma unroll
      for (int e = 0; e < 2; ++e)
#pragma unroll
        for (int r = 0; r < R; ++r) sa[off_e[e] + r * 256] = xv[e][r];  // x' takes a's place
      // ---- tracker: y~ = P y, then the fold (y~ - g) + g'
      {
        double acc[R][2];
#pragma unroll
        for (int pf = 0; pf < R; ++pf) acc[pf][0] = acc[pf][1] = 0.0;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          double z[R];
#pragma unroll
          for (int r = 0; r < R; ++r) z[r] = static_cast<double>(syp[off_e[s] + r * 256]);
          if (s == 1) {  // the last read of the x, y stage: it can be refilled
            __syncwarp();
            if (lane == 0) bar_arrive(&xy_empty[sx]);
            released = true;
          }
#pragma unroll
          for (int pf = 0; pf < R; ++pf) {
            double zh = 0.0;
#pragma unroll
            for (int r = 0; r < R; ++r) if (torus_q(R, pf, r) != 0.0) zh = fma(torus_q(R, pf, r), z[r], zh);
            dmma(acc[pf], zh, frag[(pf * 2 + s) * 32 + lane]);
          }
        }
        const bool in_d = j < p.d;
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int r = 0; r < R; ++r) {
            double v = 0.0;
#pragma unroll
            for (int pf = 0; pf < R; ++pf) if (torus_q(R, pf, r) != 0.0) v = fma(torus_q(R, pf, r), acc[pf][e], v);
            const int o = off_e[e] + r * 256;
            const float go = sc[o];  // g', parked there by the gradient phase
            const float yo = static_cast<float>((v - static_cast<double>(sg[o])) + static_cast<double>(go));
            sg[o] = go;
            sc[o] = yo;
            if (p.y_obs != nullptr && in_d)  // optional observer: the gossiped tracker, stored directly
              p.y_obs[static_cast<long long>(8 * r + 2 * kq + e) * p.ld + j] = static_cast<float>(v);
          }
        if (in_d && j >= d_tma) {  // TMA clips stores at 16-byte granularity: the last d % 4 columns go out directly
#pragma unroll
          for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int r = 0; r < R; ++r) {
              const int o = off_e[e] + r * 256;
              const long long off = static_cast<long long>(8 * r + 2 * kq + e) * p.ld + j;
              p.x[off] = sa[o];
              p.y[off] = sc[o];
              p.g[off] = sg[o];
            }
        }
      }
    }
    if (!released) {  // idle tile: same protocol, nothing computed
      __syncwarp();
      if (lane == 0) bar_arrive(&xy_empty[sx]);
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
  const long long d_tma = p.d & ~3LL;
  if (!make_swizzled_map(&m.x, p.x, p.n, p.d, p.ld, p.n) || !make_swizzled_map(&m.y, p.y, p.n, p.d, p.ld, p.n) ||
      !make_swizzled_map(&m.g, p.g, p.n, p.d, p.ld, p.n) || !make_swizzled_map(&m.a, p.a, p.n, p.d, p.ld, p.n) ||
      !make_swizzled_map(&m.c, p.c, p.n, p.d, p.ld, p.n))
    return false;
  if (d_tma > 0 && (!make_swizzled_map(&m.xs, p.x, p.n, d_tma, p.ld, p.n) ||
                    !make_swizzled_map(&m.ys, p.y, p.n, d_tma, p.ld, p.n) ||
                    !make_swizzled_map(&m.gs, p.g, p.n, d_tma, p.ld, p.n)))
    return false;
  if (d_tma == 0) m.xs = m.ys = m.gs = m.x;  // never used
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
