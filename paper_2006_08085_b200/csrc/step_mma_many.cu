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
  // 128-byte alignment (needed by the TMA tiles) is checked in the set-up rather than assumed.
  extern __shared__ __align__(128) unsigned char smem_raw[];
  MmaShared sm;
  if (!mma_setup(p, smem_raw, sm)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  const long long first = blockIdx.x, stride = gridDim.x;
  float* const stage_mem = sm.stage_mem;
  uint64_t* const empty = sm.empty;
  uint64_t* const out_ready = sm.out_ready;
  uint64_t* const out_free = sm.out_free;
  const double* const frag = sm.frag;

  if (warp == kProducerWarp) {
    if (lane == 0) mma_producer<kModeDetag>(p, maps, sm);
    return;
  }
  if (warp == kStoreWarp) {
    if (lane == 0) mma_storer<kModeDetag>(p, maps, sm);
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
  const int steps = p.steps;

  long long use = 0;  // how many slabs this group has taken so far
  for (long long k = group, slab = first + group * stride; slab < p.num_slabs;
       slab += kWarpGroups * stride, k += kWarpGroups, ++use) {
    const int s = static_cast<int>(k % kMmaStages);
    bool ok = true;
    if (!mma_wait_slab(p, sm, k, group, tile, lane)) {
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
          if (lane == 0) ok = bar_wait(&out_free[group], (use - 1) & 1, p.spin_limit);
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
      if (lane == 0 && !bar_wait(&out_free[group], (use - 1) & 1, p.spin_limit)) atomicExch(p.status, 1);
    }
    // outputs visible to the TMA store, input stage no longer read or written by this warp
    fence_async_shared();
    __syncwarp();
    if (lane == 0) {
      bar_arrive(&out_ready[group]);
      bar_arrive(&empty[s]);
    }
  }
}

}  // namespace

int launch_step_mma_many(StepParams p, const TensorMapSet& maps, int sm_count, cudaStream_t stream) {
  if (p.steps < 1 || p.mode != kModeDetag) return static_cast<int>(cudaErrorInvalidValue);
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  void (*kernel)(const StepParams, const MmaMaps);
  if (p.n <= 8)
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 2> : step_mma_many_kernel<false, 2>;
  else if (p.n <= 16)
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 4> : step_mma_many_kernel<false, 4>;
  else
    kernel = p.grad_at_start ? step_mma_many_kernel<true, 8> : step_mma_many_kernel<false, 8>;
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(kMmaSmemBytes));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kMmaThreads, kMmaSmemBytes, stream>>>(p, *reinterpret_cast<const MmaMaps*>(maps.bytes));
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
