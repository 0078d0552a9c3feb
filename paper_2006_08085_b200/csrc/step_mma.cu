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
#include "mma_common.cuh"

namespace detag {

namespace {

// kAtStart: the gradient is taken at the model the step started from (Algorithm 2 as printed) instead of the new one.
// kKs: number of 4-worker input blocks that can be non-zero, ceil(n / 4) rounded up to 2, 4 or 8; the MMAs of the
// all-zero blocks of the padded P are not issued.
template <bool kAtStart, int kKs>
__global__ void __launch_bounds__(kMmaThreads, 1)
step_mma_kernel(const StepParams p, const __grid_constant__ MmaMaps maps) {
  // No static shared memory in this kernel: the dynamic array starts at the CTA's shared window, whose
  // 128-byte alignment (needed by the TMA tiles) is checked below rather than assumed.
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* stage_mem = reinterpret_cast<float*>(smem_raw);
  float* out_mem = stage_mem + kMmaStages * kStageFloats;                             // [group][x', y', g'][32][kS]
  double* frag = reinterpret_cast<double*>(out_mem + kWarpGroups * kOutFloats);       // [t][ks][lane]
  uint64_t* full = reinterpret_cast<uint64_t*>(frag + 32 * 32);
  uint64_t* empty = full + kMmaStages;
  uint64_t* out_ready = empty + kMmaStages;      // [group]: the group's 8 warps have written their outputs
  uint64_t* out_free = out_ready + kWarpGroups;  // [group]: the stores have finished reading the tile
  unsigned* seen = reinterpret_cast<unsigned*>(out_free + kWarpGroups);  // [group]: 1 + last slab index whose data it saw
  if ((s_addr(smem_raw) & 127u) != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, 2);
    return;
  }

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  // P in fragment order: block (t, ks), lane (r, kq) holds P[4r + t][4ks + kq]
  for (int e = tid; e < 32 * 32; e += kMmaThreads) {
    const int l = e & 31, ks = (e >> 5) & 7, t = e >> 8;
    const int i = 4 * (l >> 2) + t, j = 4 * ks + (l & 3);
    frag[e] = (i < n && j < n) ? p.poly[static_cast<size_t>(i) * n + j] : 0.0;
  }
  if (tid == 0) {
    for (int g = 0; g < kWarpGroups; ++g) seen[g] = 0;
    for (int s = 0; s < kMmaStages; ++s) {
      bar_init(&full[s], 1);
      bar_init(&empty[s], kGroupWarps);
    }
    for (int g = 0; g < kWarpGroups; ++g) {
      bar_init(&out_ready[g], kGroupWarps);
      bar_init(&out_free[g], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;

  if (warp == kProducerWarp) {
    // ---------------------------------------------------------------- producer: one elected thread
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (long long slab = first; slab < p.num_slabs; slab += stride, ++issued) {
        const int s = issued % kMmaStages;
        if (issued >= kMmaStages) ok = bar_wait(&empty[s], ((issued / kMmaStages) - 1) & 1);
        if (!ok) break;
        float* st = stage_mem + static_cast<size_t>(s) * kStageFloats;
        const int col = static_cast<int>(slab * kS);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_addr(&full[s])),
                     "r"(static_cast<unsigned>(kStageBytes))
                     : "memory");
        tile_load(st, &maps.x, col, &full[s]);
        tile_load(st + kN * kPitchXY, &maps.y, col, &full[s]);
        float* se = st + 2 * kN * kPitchXY;
        tile_load(se, &maps.g, col, &full[s]);
        tile_load(se + kN * kPitchE, &maps.a, col, &full[s]);
        tile_load(se + 2 * kN * kPitchE, &maps.c, col, &full[s]);
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (int back = 1; back <= kMmaStages && back <= issued; ++back) {  // drain copies still in flight (bounded)
          const int k = issued - back;
          bar_wait(&full[k % kMmaStages], (k / kMmaStages) & 1);
        }
      }
    }
    return;
  }

  if (warp == kStoreWarp) {
    // ---------------------------------------------------------------- storer: one elected thread
    if (lane == 0) {
      long long k = 0;
      for (long long slab = first; slab < p.num_slabs; slab += stride, ++k) {
        const int g = static_cast<int>(k % kWarpGroups);
        if (!bar_wait(&out_ready[g], (k / kWarpGroups) & 1)) {
          atomicExch(p.status, 1);
          break;
        }
        const float* ob = out_mem + g * kOutFloats;
        const int col = static_cast<int>(slab * kS);
        if (col < (p.d & ~3LL)) {
          tile_store(&maps.xs, col, ob);
          tile_store(&maps.ys, col, ob + kN * kS);
          tile_store(&maps.gs, col, ob + 2 * kN * kS);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the tile may be overwritten now
        bar_arrive(&out_free[g]);
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // all global writes done before the CTA leaves
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int r = lane >> 2, kq = lane & 3;
  const int group = warp / kGroupWarps, tile = warp % kGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  float* ob = out_mem + group * kOutFloats;
  const int cl = tile * 8;
  const long long d_tma = p.d & ~3LL;  // columns below this are written by the TMA stores

  long long use = 0;  // how many slabs this group has taken so far
  for (long long k = group, slab = first + group * stride; slab < p.num_slabs;
       slab += kWarpGroups * stride, k += kWarpGroups, ++use) {
    const int s = static_cast<int>(k % kMmaStages);
    bool ok = true;
    if (lane == 0) {
      // The stage last held slab k - kMmaStages, which belongs to the other group when the stage count is odd.
      // A parity wait must not start before that phase has completed (it could not tell the two apart), and
      // it costs nothing to make sure: this slab cannot have been loaded before that one was consumed.
      if (kMmaStages % kWarpGroups != 0 && k >= kMmaStages)
        ok = count_wait(&seen[(k - kMmaStages) % kWarpGroups], static_cast<unsigned>(k - kMmaStages + 1));
      if (ok) ok = bar_wait(&full[s], (k / kMmaStages) & 1);
      if (ok && tile == 0) count_publish(&seen[group], static_cast<unsigned>(k + 1));
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    const float* sx = stage_mem + static_cast<size_t>(s) * kStageFloats;
    const float* sy = sx + kN * kPitchXY;
    const float* sg = sy + kN * kPitchXY;
    const float* sa = sg + kN * kPitchE;
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
      double cy[4][2], cx[4][2];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 gv = *reinterpret_cast<const float2*>(sg + (4 * r + t) * kPitchE + cl + 2 * kq);
        cy[t][0] = static_cast<double>(-gv.x);
        cy[t][1] = static_cast<double>(-gv.y);
        cx[t][0] = cx[t][1] = 0.0;
      }
#pragma unroll
      for (int ks = 0; ks < kKs; ++ks) {
        const int src = (4 * ks + kq) * kPitchXY + cl + r;
        const double by = static_cast<double>(sy[src]);
        const double bx = fma(-alpha, by, static_cast<double>(sx[src]));
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const double a = frag[(t * 8 + ks) * 32 + lane];
          dmma(cy[t], a, by);
          dmma(cx[t], a, bx);
        }
      }
      // the tail's inputs move to registers so that the stage can be refilled while the tail runs
      float2 av4[4], cv4[4], gv4[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int eoff = (4 * r + t) * kPitchE + cl + 2 * kq;
        av4[t] = *reinterpret_cast<const float2*>(sa + eoff);
        cv4[t] = *reinterpret_cast<const float2*>(sc + eoff);
        if (p.y_obs != nullptr) gv4[t] = *reinterpret_cast<const float2*>(sg + eoff);
      }
      __syncwarp();
      if (lane == 0) {
        bar_arrive(&empty[s]);
        released = true;
        if (use > 0 && !bar_wait(&out_free[group], (use - 1) & 1)) out_ok = false;  // previous tile stored
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
        if (noisy) {
          normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + e),
                      static_cast<uint32_t>(r), p.t_noise, xi[e]);
        } else {
          xi[e][0] = xi[e][1] = xi[e][2] = xi[e][3] = 0.f;
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int row = 4 * r + t;
        const int eoff = row * kPitchE + cl + 2 * kq;
        const float2 av = av4[t];
        const float2 cv = cv4[t];
        float2 xo, yo, go;
        xo.x = static_cast<float>(cx[t][0]);                           // x' (float64 accumulator, rounded once)
        xo.y = static_cast<float>(cx[t][1]);
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
        const int ooff = row * kS + cl + 2 * kq;
        *reinterpret_cast<float2*>(ob + ooff) = xo;
        *reinterpret_cast<float2*>(ob + kN * kS + ooff) = yo;
        *reinterpret_cast<float2*>(ob + 2 * kN * kS + ooff) = go;
        if (j >= d_tma && row < n) {
          // TMA clips a store at 16-byte granularity; the last d % 4 coordinates are written here so that
          // nothing beyond column d is touched
          const long long off = static_cast<long long>(row) * p.ld + j;
          if (j < p.d) {
            p.x[off] = xo.x;
            p.y[off] = yo.x;
            p.g[off] = go.x;
          }
          if (j + 1 < p.d) {
            p.x[off + 1] = xo.y;
            p.y[off + 1] = yo.y;
            p.g[off + 1] = go.y;
          }
        }
        if (p.y_obs != nullptr && row < n) {  // optional observer: the gossiped tracker, stored directly
          const long long off = static_cast<long long>(row) * p.ld + j;
          const float2 gv = gv4[t];
          if (j + 1 < p.d) {
            *reinterpret_cast<float2*>(p.y_obs + off) =
                make_float2(static_cast<float>(cy[t][0] + static_cast<double>(gv.x)),
                            static_cast<float>(cy[t][1] + static_cast<double>(gv.y)));
          } else if (j < p.d) {
            p.y_obs[off] = static_cast<float>(cy[t][0] + static_cast<double>(gv.x));
          }
        }
      }
    }
    // outputs visible to the TMA store
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (!(j0 + cl < p.d)) {  // idle tile
      if (lane == 0 && use > 0 && !bar_wait(&out_free[group], (use - 1) & 1)) atomicExch(p.status, 1);
    }
    if (lane == 0) {
      bar_arrive(&out_ready[group]);
      if (!released) bar_arrive(&empty[s]);
    }
  }
}

}  // namespace

int launch_step_mma(StepParams p, int sm_count, cudaStream_t stream) {
  MmaMaps maps;
  if (!make_mma_maps(&maps, p)) return static_cast<int>(cudaErrorInvalidValue);
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  void (*kernel)(const StepParams, const MmaMaps);
  if (p.n <= 8)
    kernel = p.grad_at_start ? step_mma_kernel<true, 2> : step_mma_kernel<false, 2>;
  else if (p.n <= 16)
    kernel = p.grad_at_start ? step_mma_kernel<true, 4> : step_mma_kernel<false, 4>;
  else
    kernel = p.grad_at_start ? step_mma_kernel<true, 8> : step_mma_kernel<false, 8>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kMmaSmemBytes));
  if (e != cudaSuccess) return static_cast<int>(e);
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kMmaThreads, kMmaSmemBytes, stream>>>(p, maps);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
