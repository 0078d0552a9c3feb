// Dense-polynomial DeTAG step on the FP64 tensor path (n <= 32).
//
// AG_K is linear, AG_K(z) = P z with P = P_K(M) built by the host in float64 from the matrix form of
// Algorithm 3.  For a slab of coordinates the step is therefore two small dense contractions
// (P times the tracker rows, P times the model rows) followed by Algorithm 2's element-wise updates.
// Here the contractions run as warp-level float64 matrix multiply-accumulates (mma m8n8k4, f64):
//   A (8 x 4) : a block of P.  All 4 x 8 blocks of the 32 x 32 matrix stay in registers for the
//               whole kernel (32 doubles per lane).
//   B (4 x 8) : four workers x eight coordinates of the staged tracker / model slab, read from shared
//               memory once per warp (one 4-byte load + one widening per lane and block).
//   C (8 x 8) : float64 accumulators, 2 per lane and block.
// Row permutation: block t of P holds workers {4r + t : r = 0..7}, so lane (r = lane/4) ends up with
// workers 4r..4r+3 - exactly the four workers one Philox call serves - for its two coordinates.
//
// Data movement: a producer warp fills three stages with bulk asynchronous copies, one 384-byte row per
// (array, worker) and lane, completion counted on the stage's "full" mbarrier.  Rows are laid out with
// a padded pitch (S+8 floats for x, y; S+4 for g, a, c) so the B-fragment loads are bank-conflict free.
// Consumer warps hand a stage back with one arrive per warp on its "empty" mbarrier.  Results go to
// global memory straight from the accumulator layout (32-byte row segments, whole sectors).
// Every mbarrier wait is bounded; a wait that gives up sets the status word and the CTA winds down.
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"

namespace detag {

namespace {

constexpr int kN = 32;           // padded worker count
constexpr int kS = 96;           // coordinates per stage: 12 tiles of 8, one per consumer warp
constexpr int kPitchXY = kS + 8; // floats; 8 mod 32 -> the four workers of a B fragment hit disjoint banks
constexpr int kPitchE = kS + 4;  // floats; rows of g, a, c (read in the accumulator layout)
constexpr int kStageFloats = 2 * kN * kPitchXY + 3 * kN * kPitchE;
constexpr int kStageBytes = kStageFloats * 4;
constexpr int kMmaStages = 3;
constexpr int kConsumerWarps = 12;
constexpr int kMmaThreads = (kConsumerWarps + 1) * 32;
constexpr int kTilesPerStage = kS / 8;
constexpr unsigned kMmaSpinLimit = 1u << 22;
constexpr size_t kMmaSmemBytes = 128 + static_cast<size_t>(kMmaStages) * kStageBytes + 64;

__device__ __forceinline__ uint32_t s_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool bar_wait(uint64_t* bar, unsigned parity) {
  const uint32_t addr = s_addr(bar);
  for (unsigned spin = 0; spin < kMmaSpinLimit; ++spin) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

__device__ __forceinline__ void bulk_row(float* dst, const float* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   s_addr(dst)),
               "l"(src), "r"(bytes), "r"(s_addr(bar))
               : "memory");
}

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

__global__ void __launch_bounds__(kMmaThreads, 1) step_mma_kernel(const StepParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  float* stage_mem = reinterpret_cast<float*>(base);
  uint64_t* full = reinterpret_cast<uint64_t*>(base + static_cast<size_t>(kMmaStages) * kStageBytes);
  uint64_t* empty = full + kMmaStages;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  // rows >= n and slab tails are never written by the copies: give them a finite value once
  for (int e = tid; e < kMmaStages * kStageFloats; e += kMmaThreads) stage_mem[e] = 0.f;
  if (tid == 0) {
    for (int s = 0; s < kMmaStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_addr(&full[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_addr(&empty[s])), "r"(kConsumerWarps));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the zero fill above went through the generic proxy; order it before the async-proxy copies
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;

  if (warp == kConsumerWarps) {
    // ---------------------------------------------------------------- producer warp: lane = worker row
    int issued = 0;
    bool ok = true;
    for (long long slab = first; slab < p.num_slabs; slab += stride, ++issued) {
      const int s = issued % kMmaStages;
      if (issued >= kMmaStages) {
        if (lane == 0) ok = bar_wait(&empty[s], ((issued / kMmaStages) - 1) & 1);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      }
      if (!ok) break;
      const long long j0 = slab * kS;
      const long long width = (p.d - j0 < kS) ? p.d - j0 : kS;
      const unsigned row_bytes = static_cast<unsigned>((width + 3) / 4 * 16);  // ld >= d rounded up to 4: in bounds
      if (lane == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_addr(&full[s])),
                     "r"(row_bytes * 5u * static_cast<unsigned>(n))
                     : "memory");
      }
      __syncwarp();
      if (lane < n) {
        float* st = stage_mem + static_cast<size_t>(s) * kStageFloats;
        const long long off = static_cast<long long>(lane) * p.ld + j0;
        bulk_row(st + lane * kPitchXY, p.x + off, row_bytes, &full[s]);
        bulk_row(st + kN * kPitchXY + lane * kPitchXY, p.y + off, row_bytes, &full[s]);
        float* se = st + 2 * kN * kPitchXY;
        bulk_row(se + lane * kPitchE, p.g + off, row_bytes, &full[s]);
        bulk_row(se + kN * kPitchE + lane * kPitchE, p.a + off, row_bytes, &full[s]);
        bulk_row(se + 2 * kN * kPitchE + lane * kPitchE, p.c + off, row_bytes, &full[s]);
      }
    }
    if (!ok && lane == 0) {
      atomicExch(p.status, 1);
      for (int back = 1; back <= kMmaStages && back <= issued; ++back) {  // drain copies still in flight (bounded)
        const int k = issued - back;
        bar_wait(&full[k % kMmaStages], (k / kMmaStages) & 1);
      }
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int r = lane >> 2, kq = lane & 3;
  // A fragments: block (t, s) element [r][kq] = P[4r + t][4s + kq]
  double afrag[4][8];
#pragma unroll
  for (int t = 0; t < 4; ++t)
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const int i = 4 * r + t, j = 4 * s + kq;
      afrag[t][s] = (i < n && j < n) ? p.poly[static_cast<size_t>(i) * n + j] : 0.0;
    }
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;

  int k = 0;
  for (long long slab = first; slab < p.num_slabs; slab += stride, ++k) {
    const int s = k % kMmaStages;
    bool ok = true;
    if (lane == 0) ok = bar_wait(&full[s], (k / kMmaStages) & 1);
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

    for (int tile = warp; tile < kTilesPerStage; tile += kConsumerWarps) {
      const int cl = tile * 8;
      if (j0 + cl >= p.d) break;
      double cy[4][2], cx[4][2];
#pragma unroll
      for (int t = 0; t < 4; ++t) cy[t][0] = cy[t][1] = cx[t][0] = cx[t][1] = 0.0;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int src = (4 * ks + kq) * kPitchXY + cl + r;
        const double by = static_cast<double>(sy[src]);
        const double bx = static_cast<double>(sx[src]);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          dmma(cy[t], afrag[t][ks], by);
          dmma(cx[t], afrag[t][ks], bx);
        }
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
      const bool in0 = j < p.d, in1 = j + 1 < p.d;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int row = 4 * r + t;
        const int eoff = row * kPitchE + cl + 2 * kq;
        const float2 gv = *reinterpret_cast<const float2*>(sg + eoff);
        const float2 av = *reinterpret_cast<const float2*>(sa + eoff);
        const float2 cv = *reinterpret_cast<const float2*>(sc + eoff);
        float2 xo, yo, go, yg;
        {
          const float x_new = static_cast<float>(fma(-alpha, cy[t][0], cx[t][0]));
          const float g_new = fmaf(av.x, x_new - cv.x, sigma * xi[0][t]);
          xo.x = x_new;
          go.x = g_new;
          yo.x = static_cast<float>(cy[t][0] + (static_cast<double>(g_new) - static_cast<double>(gv.x)));
          yg.x = static_cast<float>(cy[t][0]);
        }
        {
          const float x_new = static_cast<float>(fma(-alpha, cy[t][1], cx[t][1]));
          const float g_new = fmaf(av.y, x_new - cv.y, sigma * xi[1][t]);
          xo.y = x_new;
          go.y = g_new;
          yo.y = static_cast<float>(cy[t][1] + (static_cast<double>(g_new) - static_cast<double>(gv.y)));
          yg.y = static_cast<float>(cy[t][1]);
        }
        if (row < n) {
          const long long off = static_cast<long long>(row) * p.ld + j;
          if (in1) {
            *reinterpret_cast<float2*>(p.x + off) = xo;
            *reinterpret_cast<float2*>(p.y + off) = yo;
            *reinterpret_cast<float2*>(p.g + off) = go;
            if (p.y_obs != nullptr) *reinterpret_cast<float2*>(p.y_obs + off) = yg;
          } else if (in0) {
            p.x[off] = xo.x;
            p.y[off] = yo.x;
            p.g[off] = go.x;
            if (p.y_obs != nullptr) p.y_obs[off] = yg.x;
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0)
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_addr(&empty[s])) : "memory");
  }
}

}  // namespace

int launch_step_mma(StepParams p, int sm_count, cudaStream_t stream) {
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  cudaError_t e = cudaFuncSetAttribute(step_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kMmaSmemBytes));
  if (e != cudaSuccess) return static_cast<int>(e);
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  step_mma_kernel<<<static_cast<unsigned>(grid), kMmaThreads, kMmaSmemBytes, stream>>>(p);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
