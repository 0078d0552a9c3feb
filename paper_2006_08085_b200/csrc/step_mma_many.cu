// Several consecutive DeTAG steps in one launch (dense polynomial on the FP64 tensor path, n <= 32).
//
// The step never mixes coordinates: each coordinate's n-vector of models, trackers and gradients evolves on its
// own (the gossip mixes workers, the synthetic objective is diagonal, the noise is a pure function of
// (step, worker, coordinate)).  So a warp that holds the 32 x 8 tile of a slab can run `steps` iterations on it
// without meeting any other warp: the state is read from HBM once, stepped `steps` times on chip and written
// once.  The HBM traffic of a run of T steps drops from 32 T to 32 bytes per worker-coordinate, and what bounds
// the kernel is the FP64 tensor pipe (64 multiply-adds per worker-coordinate and step) instead of HBM.
//
// Same roles, pipeline and arithmetic as the one-step kernel (step_mma.cu): the results are bit-identical to
// `steps` launches of it.  Differences: the stage is kept for all steps and a tile's intermediate x', y', g' are
// written back into the stage, into the warp's own eight columns (the B-fragment loads of the next step read
// them there); only the last step writes the dense output tile that the TMA stores send out.  The noise index of
// step i of the launch is t_noise + i.
#include "mma_common.cuh"

namespace detag {

namespace {

// kKs: number of 4-worker input blocks that can be non-zero, ceil(n / 4) rounded up to 2, 4 or 8; the MMAs of the
// all-zero blocks of the padded P are not issued.
template <bool kAtStart, int kKs>
__global__ void __launch_bounds__(kMmaThreads, 1)
step_mma_many_kernel(const StepParams p, const __grid_constant__ MmaMaps maps) {
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
  const int steps = p.steps;

  long long use = 0;  // how many slabs this group has taken so far
  for (long long k = group, slab = first + group * stride; slab < p.num_slabs;
       slab += kWarpGroups * stride, k += kWarpGroups, ++use) {
    const int s = static_cast<int>(k % kMmaStages);
    bool ok = true;
    if (lane == 0) {
      // see step_mma.cu: a parity wait on a stage shared with the other group must not start a phase early
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
    float* sx = stage_mem + static_cast<size_t>(s) * kStageFloats;
    float* sy = sx + kN * kPitchXY;
    float* sg = sy + kN * kPitchXY;
    const float* sa = sg + kN * kPitchE;
    const float* sc = sa + kN * kPitchE;
    const long long j0 = slab * kS;
    const long long j = j0 + cl + 2 * kq;

    if (j0 + cl < p.d) {
      for (int step = 0; step < steps; ++step) {
        const bool final_step = step == steps - 1;
        // the two contractions, exactly as in the one-step kernel: cx = P (x - alpha y) = x', cy = P y - g = y~ - g
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
        if (final_step && use > 0) {  // the group's output tile must have been read by the previous stores
          if (lane == 0) ok = bar_wait(&out_free[group], (use - 1) & 1);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) {
            if (lane == 0) atomicExch(p.status, 1);
            return;
          }
        }
        // element-wise tail: workers 4r..4r+3 (index t), coordinates j, j+1
        float xi[2][4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          if (noisy) {
            normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + e),
                        static_cast<uint32_t>(r), p.t_noise + static_cast<uint32_t>(step), xi[e]);
          } else {
            xi[e][0] = xi[e][1] = xi[e][2] = xi[e][3] = 0.f;
          }
        }
        __syncwarp();  // every lane has read its B fragments of x and y before anyone overwrites them below
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int row = 4 * r + t;
          const int eoff = row * kPitchE + cl + 2 * kq;
          const int xoff = row * kPitchXY + cl + 2 * kq;
          const float2 av = *reinterpret_cast<const float2*>(sa + eoff);
          const float2 cv = *reinterpret_cast<const float2*>(sc + eoff);
          float2 xo, yo, go;
          xo.x = static_cast<float>(cx[t][0]);                           // x' (float64 accumulator, rounded once)
          xo.y = static_cast<float>(cx[t][1]);
          // gradient point: the new model, or (Algorithm 2 as printed) the staged model this step started from
          const float2 x_at = kAtStart ? *reinterpret_cast<const float2*>(sx + xoff) : xo;
          go.x = fmaf(av.x, x_at.x - cv.x, sigma * xi[0][t]);            // stochastic gradient
          go.y = fmaf(av.y, x_at.y - cv.y, sigma * xi[1][t]);
          yo.x = static_cast<float>(cy[t][0] + static_cast<double>(go.x));  // fold: (y~ - g) + g', g' as stored
          yo.y = static_cast<float>(cy[t][1] + static_cast<double>(go.y));
          if (!final_step) {
            // the next step of this tile reads its state where this one found it: this warp's own eight columns
            *reinterpret_cast<float2*>(sx + xoff) = xo;
            *reinterpret_cast<float2*>(sy + xoff) = yo;
            *reinterpret_cast<float2*>(sg + eoff) = go;
          } else {
            const int ooff = row * kS + cl + 2 * kq;
            *reinterpret_cast<float2*>(ob + ooff) = xo;
            *reinterpret_cast<float2*>(ob + kN * kS + ooff) = yo;
            *reinterpret_cast<float2*>(ob + 2 * kN * kS + ooff) = go;
            if (j >= d_tma && row < n) {
              // TMA clips a store at 16-byte granularity; the last d % 4 coordinates are written here
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
          }
        }
        __syncwarp();  // the new state is in place before the next step's fragment loads
      }
    } else if (use > 0) {  // idle tile: same protocol, nothing computed
      if (lane == 0 && !bar_wait(&out_free[group], (use - 1) & 1)) atomicExch(p.status, 1);
    }
    // outputs visible to the TMA store, input stage no longer read or written by this warp
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
      bar_arrive(&out_ready[group]);
      bar_arrive(&empty[s]);
    }
  }
}

}  // namespace

int launch_step_mma_many(StepParams p, int sm_count, cudaStream_t stream) {
  MmaMaps maps;
  if (p.steps < 1 || !make_mma_maps(&maps, p)) return static_cast<int>(cudaErrorInvalidValue);
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  void (*kernel)(const StepParams, const MmaMaps);
  if (p.n <= 8)
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 2> : step_mma_many_kernel<false, 2>;
  else if (p.n <= 16)
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 4> : step_mma_many_kernel<false, 4>;
  else
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 8> : step_mma_many_kernel<false, 8>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kMmaSmemBytes));
  if (e != cudaSuccess) return static_cast<int>(e);
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kMmaThreads, kMmaSmemBytes, stream>>>(p, maps);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
