// Dense-polynomial DeTAG step on the FP64 tensor path (n <= 32).
//
// AG_K is linear, AG_K(z) = P z with P = P_K(M) built by the host in float64 from the matrix form of
// Algorithm 3.  For a slab of coordinates the step is therefore two small dense contractions
// (P times the tracker rows, P times the model rows) followed by Algorithm 2's element-wise updates.
// Here the contractions run as warp-level float64 matrix multiply-accumulates (mma m8n8k4, f64):
//   A (8 x 4) : a block of P.  The 4 x 8 blocks of the 32 x 32 matrix sit in shared memory in
//               fragment order (one conflict-free 8-byte load per lane and block).
//   B (4 x 8) : four workers x eight coordinates of the staged tracker / model slab, read from shared
//               memory once per warp (one 4-byte load + one widening per lane and block).
//   C (8 x 8) : float64 accumulators, 2 per lane and block.
// Row permutation: block t of P holds workers {4r + t : r = 0..7}, so lane (r = lane/4) ends up with
// workers 4r..4r+3 - exactly the four workers one Philox call serves - for its two coordinates.
//
// Warp roles of the persistent CTA (one per SM):
//   producer  one thread keeps three input stages in flight with five 2-D TMA tile loads each (all 32
//             worker rows x one slab of 64 coordinates of x, y, g, a, c), completion counted on the
//             stage's "full" mbarrier.  The tiles are loaded a few columns wider than the slab (72 for
//             x, y; 68 for g, a, c): TMA writes a tile densely, so the box width IS the row pitch in
//             shared memory, and 8 (mod 32) floats makes the B-fragment loads bank-conflict free.  The
//             extra columns belong to the next slab (read by its CTA at about the same time, so they
//             come from L2) and are not used.
//   consumers 16 warps in two groups that take alternate slabs; a warp owns 8 coordinates of the slab:
//             64 MMAs, then the element-wise tail (model update, Philox/Box-Muller noise, gradient,
//             tracker fold), results written to the group's dense output tile in shared memory.  The
//             tail's inputs (a, c) are copied to registers after the MMAs and the stage is handed back
//             to the producer before the tail starts: with three stages and two groups, a stage held
//             through the tail leaves a single stage of loads in flight, which is too little to cover
//             the HBM latency (measured: 5.27 -> 4.88 ms per step at n = 32, d = 25.6 M).
//   storer    one thread writes each finished output tile (x', y', g': 32 rows x 256 bytes) with three
//             TMA tile stores.  Row-contiguous 256-byte writes matter: storing straight from the
//             accumulator layout (32-byte pieces of 8 rows per instruction) halves the HBM throughput.
// Every mbarrier wait is bounded; a wait that gives up sets the status word and the CTA winds down.
//
// Modes (template parameter): the DeTAG step with the library's synthetic gradient (above); the DeTAG step with
// caller-written gradients (Algorithm 2's tracker update y + g_new - g_old forms the B operand of the tracker
// contraction, the tail only rounds and copies g_new over g_old); and D-PSGD (one contraction: x' = P x - alpha g,
// no tracker).
#include "mma_common.cuh"

namespace detag {

namespace {

// kMode: what the step computes (kModeDetag / kModeExternal / kModeDpsgd).
// kAtStart: the gradient is taken at the model the step started from (Algorithm 2 as printed) instead of the new one.
// kKs: number of 4-worker input blocks that can be non-zero, ceil(n / 4) rounded up to 2, 4 or 8; the MMAs of the
// all-zero blocks of the padded P are not issued.
template <int kMode, bool kAtStart, int kKs>
__global__ void __launch_bounds__(kMmaThreads, 1)
step_mma_kernel(const StepParams p, const __grid_constant__ MmaMaps maps) {
  // No static shared memory in this kernel: the dynamic array starts at the CTA's shared window, whose
  // 128-byte alignment (needed by the TMA tiles) is checked in the set-up rather than assumed.
  extern __shared__ __align__(128) unsigned char smem_raw[];
  MmaShared sm;
  if (!mma_setup(p, smem_raw, sm)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  const long long first = blockIdx.x, stride = gridDim.x;

  if (warp == kProducerWarp) {
    if (lane == 0) mma_producer<kMode>(p, maps, sm);
    return;
  }
  if (warp == kStoreWarp) {
    if (lane == 0) mma_storer<kMode>(p, maps, sm);
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int r = lane >> 2, kq = lane & 3;
  const int group = warp / kGroupWarps, tile = warp % kGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  float* ob = sm.out_mem + group * kOutFloats;
  const int cl = tile * 8;
  const long long d_tma = p.d & ~3LL;  // columns below this are written by the TMA stores

  long long use = 0;  // how many slabs this group has taken so far
  for (long long k = group, slab = first + group * stride; slab < p.num_slabs;
       slab += kWarpGroups * stride, k += kWarpGroups, ++use) {
    const int s = static_cast<int>(k % kMmaStages);
    if (!mma_wait_slab(p, sm, k, group, tile, lane)) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    const float* sx = sm.stage_mem + static_cast<size_t>(s) * kStageFloats;
    const float* sy = sx + kN * kPitchXY;
    const float* sg = sy + kN * kPitchXY;
    const float* sa = sg + kN * kPitchE;  // objective data a, or the caller's newest gradient
    const float* sc = sa + kN * kPitchE;
    const long long j0 = slab * kS;

    // A tile wholly beyond column d computes nothing but keeps the barrier protocol.
    bool released = false, out_ok = true;
    if (j0 + cl < p.d) {
      // The two contractions are arranged so that the element-wise tail needs a single float64 addition:
      //   cx accumulates P (x - alpha y) = x~ - alpha y~ = x'      (linearity of AG_K; Algorithm 2's model update)
      //   cy starts at -g and accumulates P y, ending as y~ - g    (so the fold is y' = cy + g')
      // Scalar float64 operations share the FP64 tensor pipe with the MMAs; every one issued from the tail
      // queues behind other warps' MMAs, so as many as possible are done here, where this warp holds the pipe.
      // Caller-written gradients: the tracker operand is folded here, y + (g_new - g_old), and cy starts at 0.
      // D-PSGD: cx starts at -alpha g and accumulates P x; there is no tracker.
      double cy[4][2], cx[4][2];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        cy[t][0] = cy[t][1] = 0.0;
        cx[t][0] = cx[t][1] = 0.0;
        if (kMode != kModeExternal) {
          const float2 gv = *reinterpret_cast<const float2*>(sg + (4 * r + t) * kPitchE + cl + 2 * kq);
          if (kMode == kModeDetag) {
            cy[t][0] = static_cast<double>(-gv.x);
            cy[t][1] = static_cast<double>(-gv.y);
          } else {
            cx[t][0] = -alpha * static_cast<double>(gv.x);
            cx[t][1] = -alpha * static_cast<double>(gv.y);
          }
        }
      }
#pragma unroll
      for (int ks = 0; ks < kKs; ++ks) {
        const int src = (4 * ks + kq) * kPitchXY + cl + r;
        double by = 0.0, bx;
        if (kMode == kModeDpsgd) {
          bx = static_cast<double>(sx[src]);
        } else {
          by = static_cast<double>(sy[src]);
          if (kMode == kModeExternal) {
            const int esrc = (4 * ks + kq) * kPitchE + cl + r;
            by += static_cast<double>(sa[esrc]) - static_cast<double>(sg[esrc]);  // Algorithm 2's tracker update
          }
          bx = fma(-alpha, by, static_cast<double>(sx[src]));
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const double a = sm.frag[(t * 8 + ks) * 32 + lane];
          if (kMode != kModeDpsgd) dmma(cy[t], a, by);
          dmma(cx[t], a, bx);
        }
      }
      // the tail's inputs move to registers so that the stage can be refilled while the tail runs
      float2 av4[4], cv4[4], gv4[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int eoff = (4 * r + t) * kPitchE + cl + 2 * kq;
        av4[t] = *reinterpret_cast<const float2*>(sa + eoff);
        if (kMode != kModeExternal) cv4[t] = *reinterpret_cast<const float2*>(sc + eoff);
        if (kMode == kModeDetag && p.y_obs != nullptr) gv4[t] = *reinterpret_cast<const float2*>(sg + eoff);
      }
      __syncwarp();
      if (lane == 0) {
        bar_arrive(&sm.empty[s]);
        released = true;
        if (use > 0 && !bar_wait(&sm.out_free[group], (use - 1) & 1, p.spin_limit)) out_ok = false;  // previous tile stored
      }
      out_ok = __shfl_sync(0xffffffffu, out_ok ? 1 : 0, 0) != 0;
      if (!out_ok) {
        if (lane == 0) atomicExch(p.status, 1);
        return;
      }
      // element-wise tail: workers 4r..4r+3 (index t), coordinates j, j+1
      const long long j = j0 + cl + 2 * kq;
      float xi[2][4];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        if (kMode != kModeExternal && noisy) {
          normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + e),
                      static_cast<uint32_t>(r), p.t_noise, xi[e]);
        } else {
          xi[e][0] = xi[e][1] = xi[e][2] = xi[e][3] = 0.f;
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int row = 4 * r + t;
        const float2 av = av4[t];
        float2 xo, yo, go;
        xo.x = static_cast<float>(cx[t][0]);                           // x' (float64 accumulator, rounded once)
        xo.y = static_cast<float>(cx[t][1]);
        if (kMode == kModeExternal) {
          go = av;                                                     // the gradient just folded becomes g_old
          yo.x = static_cast<float>(cy[t][0]);                         // the gossiped tracker
          yo.y = static_cast<float>(cy[t][1]);
        } else {
          const float2 cv = cv4[t];
          float2 x_at = xo;  // gradient point: the new model, or (Algorithm 2 as printed) the model before this step.
          if (kAtStart && row < n) {
            // The old model is still in global memory: this slab's stores are issued after all of its tails.
            const long long off = static_cast<long long>(row) * p.ld + j;
            x_at.x = j < p.d ? p.x[off] : 0.f;
            x_at.y = j + 1 < p.d ? p.x[off + 1] : 0.f;
          }
          go.x = fmaf(av.x, x_at.x - cv.x, sigma * xi[0][t]);            // stochastic gradient
          go.y = fmaf(av.y, x_at.y - cv.y, sigma * xi[1][t]);
          yo.x = static_cast<float>(cy[t][0] + static_cast<double>(go.x));  // fold: (y~ - g) + g', g' as stored
          yo.y = static_cast<float>(cy[t][1] + static_cast<double>(go.y));
        }
        const int ooff = row * kS + cl + 2 * kq;
        *reinterpret_cast<float2*>(ob + ooff) = xo;
        if (kMode != kModeDpsgd) *reinterpret_cast<float2*>(ob + kN * kS + ooff) = yo;
        *reinterpret_cast<float2*>(ob + 2 * kN * kS + ooff) = go;
        if (j >= d_tma && row < n) {
          // TMA clips a store at 16-byte granularity; the last d % 4 coordinates are written here so that
          // nothing beyond column d is touched
          const long long off = static_cast<long long>(row) * p.ld + j;
          if (j < p.d) {
            p.x[off] = xo.x;
            if (kMode != kModeDpsgd) p.y[off] = yo.x;
            p.g[off] = go.x;
          }
          if (j + 1 < p.d) {
            p.x[off + 1] = xo.y;
            if (kMode != kModeDpsgd) p.y[off + 1] = yo.y;
            p.g[off + 1] = go.y;
          }
        }
        if (kMode != kModeDpsgd && p.y_obs != nullptr && row < n) {  // optional observer: the gossiped tracker, stored directly
          const long long off = static_cast<long long>(row) * p.ld + j;
          float2 yg = yo;
          if (kMode == kModeDetag) {
            const float2 gv = gv4[t];
            yg = make_float2(static_cast<float>(cy[t][0] + static_cast<double>(gv.x)),
                             static_cast<float>(cy[t][1] + static_cast<double>(gv.y)));
          }
          if (j + 1 < p.d) {
            *reinterpret_cast<float2*>(p.y_obs + off) = yg;
          } else if (j < p.d) {
            p.y_obs[off] = yg.x;
          }
        }
      }
    }
    // outputs visible to the TMA store
    fence_async_shared();
    __syncwarp();
    if (!(j0 + cl < p.d)) {  // idle tile
      if (lane == 0 && use > 0 && !bar_wait(&sm.out_free[group], (use - 1) & 1, p.spin_limit)) atomicExch(p.status, 1);
    }
    if (lane == 0) {
      bar_arrive(&sm.out_ready[group]);
      if (!released) bar_arrive(&sm.empty[s]);
    }
  }
}

typedef void (*MmaKernel)(const StepParams, const MmaMaps);

template <int kKs>
MmaKernel pick_mode(const StepParams& p) {
  if (p.mode == kModeExternal) return step_mma_kernel<kModeExternal, false, kKs>;
  if (p.mode == kModeDpsgd) return step_mma_kernel<kModeDpsgd, false, kKs>;
  return p.grad_at_start ? step_mma_kernel<kModeDetag, true, kKs> : step_mma_kernel<kModeDetag, false, kKs>;
}

}  // namespace

// Tensor maps over the arrays in `p`; false when the driver refuses one.
bool build_maps_mma(const StepParams& p, TensorMapSet* out) {
  MmaMaps* maps = reinterpret_cast<MmaMaps*>(out->bytes);
  const float* slot_a = p.mode == kModeExternal ? p.g_ext : p.a;
  const float* slot_c = p.mode == kModeExternal ? p.g_ext : p.c;
  const float* y = p.mode == kModeDpsgd ? p.x : p.y;  // D-PSGD has no tracker: the map is never used
  if (!make_map(&maps->x, p.x, p.n, p.d, p.ld, kN, kPitchXY) || !make_map(&maps->y, y, p.n, p.d, p.ld, kN, kPitchXY) ||
      !make_map(&maps->g, p.g, p.n, p.d, p.ld, kN, kPitchE) || !make_map(&maps->a, slot_a, p.n, p.d, p.ld, kN, kPitchE) ||
      !make_map(&maps->c, slot_c, p.n, p.d, p.ld, kN, kPitchE))
    return false;
  const long long d_tma = p.d & ~3LL;  // the stores' tensor ends on a 16-byte boundary (see the kernels' tails)
  if (d_tma > 0 && (!make_map(&maps->xs, p.x, p.n, d_tma, p.ld, kN, kS) || !make_map(&maps->ys, y, p.n, d_tma, p.ld, kN, kS) ||
                    !make_map(&maps->gs, p.g, p.n, d_tma, p.ld, kN, kS)))
    return false;
  if (d_tma == 0) maps->xs = maps->ys = maps->gs = maps->x;  // never used: every slab lies beyond column 0
  return true;
}

int launch_step_mma(StepParams p, const TensorMapSet& maps, int sm_count, cudaStream_t stream) {
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  const MmaKernel kernel = p.n <= 8 ? pick_mode<2>(p) : p.n <= 16 ? pick_mode<4>(p) : pick_mode<8>(p);
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(kMmaSmemBytes));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kMmaThreads, kMmaSmemBytes, stream>>>(p, *reinterpret_cast<const MmaMaps*>(maps.bytes));
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
