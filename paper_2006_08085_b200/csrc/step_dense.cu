// Dense-polynomial DeTAG step kernel (n <= 64) with a TMA + mbarrier load pipeline.
//
// K rounds of Algorithm 3 are linear in their input: AG_K(z) = P z with P = P_K(M), the polynomial the
// host builds in float64 from the matrix form of the recursion (P_{-1} = P_0 = I,
// P_{r+1} = (1+eta) M P_r - eta P_{r-1}).  For small n one product with the dense n x n matrix P costs
// about as many multiply-adds as the K sparse rounds and needs no barriers and ~7x less shared-memory
// traffic, because a thread keeps an 8-worker x 2-coordinate block of outputs in registers.
//
// Structure of a CTA (persistent, one per SM):
//   warp 0        producer: for each slab of S = 4096/N coordinates, five 2-D TMA tile loads
//                 (x, y, g, a, c: all N worker rows x S coordinates, float32) into one of two stages,
//                 completion counted on the stage's "full" mbarrier;
//   warps 1..8    consumers: thread (row group rg, column group cg) accumulates
//                 y~[8][2] in float64 (DFMA) and x~[8][2] in float32 from the staged x, y and the
//                 transposed P held in shared memory, then finishes the step for its 16 elements
//                 (model update, Philox/Box-Muller noise, gradient, tracker fold) and stores x', y', g'
//                 straight from registers (8-byte stores, 256 contiguous bytes per warp and row);
//                 one arrive per warp on the stage's "empty" mbarrier hands the stage back.
// Precision: the tracker product and the fold run in float64 (inputs up to ~1e3 cancel to ~0 and the
// result must be good to 1e-5 absolute); the model product, whose result is not a cancellation, and
// the gradient run in float32.  Every mbarrier wait is bounded: when it gives up the kernel records
// DETAG_ERR_TIMEOUT in the status word, the producer drains its outstanding copies (bounded), and the
// CTA returns.
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kStages = 2;
constexpr int kTileRows = 8;   // workers per thread
constexpr int kTileCols = 2;   // coordinates per thread
constexpr unsigned kSpinLimit = 1u << 22;  // polls of try_wait before a wait gives up

struct DenseMaps {
  CUtensorMap x, y, g, a, c;
};

template <int N>
struct DenseShape {
  static constexpr int S = (4096 / N) > 256 ? 256 : (4096 / N);  // coordinates per stage (TMA box <= 256)
  static constexpr int kRowGroups = N / kTileRows;
  static constexpr int kColGroups = S / kTileCols;
  static constexpr int kConsumers = kRowGroups * kColGroups;  // threads
  static constexpr int kThreads = kConsumers + 32;
  static constexpr int kArrayFloats = N * S;
  static constexpr int kStageBytes = 5 * kArrayFloats * 4;
  static constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + static_cast<size_t>(kStages) * kStageBytes +
                                       static_cast<size_t>(N) * N * (sizeof(double) + sizeof(float)) + 64;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Bounded wait for the phase with the given parity; false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
  const uint32_t addr = smem_u32(bar);
  for (unsigned spin = 0; spin < kSpinLimit; ++spin) {
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

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

template <int N>
__global__ void __launch_bounds__(DenseShape<N>::kThreads, 1)
step_dense_kernel(const StepParams p, const __grid_constant__ DenseMaps maps) {
  using Sh = DenseShape<N>;
  constexpr int S = Sh::S;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* stage_mem = reinterpret_cast<float*>(base);
  double* pt_d = reinterpret_cast<double*>(base + static_cast<size_t>(kStages) * Sh::kStageBytes);  // Pt[j][i] = P[i][j]
  float* pt_f = reinterpret_cast<float*>(pt_d + N * N);
  uint64_t* bars = reinterpret_cast<uint64_t*>(pt_f + N * N);  // full[kStages], empty[kStages]
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;

  const int tid = threadIdx.x;
  const int n = p.n;
  for (int e = tid; e < N * N; e += Sh::kThreads) {
    const int j = e / N, i = e - j * N;
    const double v = (i < n && j < n) ? p.poly[static_cast<size_t>(i) * n + j] : 0.0;
    pt_d[e] = v;
    pt_f[e] = static_cast<float>(v);
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], Sh::kConsumers / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;

  if (tid < 32) {
    // ------------------------------------------------------------------ producer warp
    if (tid == 0) {
      int issued = 0;
      bool ok = true;
      for (long long slab = first; slab < p.num_slabs && ok; slab += stride, ++issued) {
        const int s = issued % kStages;
        if (issued >= kStages) ok = mbar_wait(&empty[s], ((issued / kStages) - 1) & 1);
        if (!ok) break;
        float* dst = stage_mem + static_cast<size_t>(s) * 5 * Sh::kArrayFloats;
        const int col = static_cast<int>(slab * S);
        mbar_expect_tx(&full[s], Sh::kStageBytes);
        tma_load_2d(dst + 0 * Sh::kArrayFloats, &maps.x, col, 0, &full[s]);
        tma_load_2d(dst + 1 * Sh::kArrayFloats, &maps.y, col, 0, &full[s]);
        tma_load_2d(dst + 2 * Sh::kArrayFloats, &maps.g, col, 0, &full[s]);
        tma_load_2d(dst + 3 * Sh::kArrayFloats, &maps.a, col, 0, &full[s]);
        tma_load_2d(dst + 4 * Sh::kArrayFloats, &maps.c, col, 0, &full[s]);
      }
      if (!ok) {
        atomicExch(p.status, 1);
        // the consumers may have left: wait (bounded) for the copies still in flight before returning
        for (int back = 1; back <= kStages && back <= issued; ++back) {
          const int k = issued - back;
          mbar_wait(&full[k % kStages], (k / kStages) & 1);
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int ct = tid - 32;
  const int cg = ct % Sh::kColGroups;  // column group: coordinates 2cg, 2cg+1 of the slab
  const int rg = ct / Sh::kColGroups;  // row group: workers 8rg .. 8rg+7 (uniform within a warp)
  const float alpha_unused = 0.f;
  (void)alpha_unused;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;

  int k = 0;
  for (long long slab = first; slab < p.num_slabs; slab += stride, ++k) {
    const int s = k % kStages;
    if (!mbar_wait(&full[s], (k / kStages) & 1)) {
      atomicExch(p.status, 1);
      return;
    }
    const float* sx = stage_mem + static_cast<size_t>(s) * 5 * Sh::kArrayFloats;
    const float* sy = sx + Sh::kArrayFloats;
    const float* sg = sy + Sh::kArrayFloats;
    const float* sa = sg + Sh::kArrayFloats;
    const float* sc = sa + Sh::kArrayFloats;

    double accy[kTileRows][kTileCols];
    float accx[kTileRows][kTileCols];
#pragma unroll
    for (int i = 0; i < kTileRows; ++i) {
      accy[i][0] = accy[i][1] = 0.0;
      accx[i][0] = accx[i][1] = 0.f;
    }
#pragma unroll 4
    for (int j = 0; j < N; ++j) {
      const float2 xv = *reinterpret_cast<const float2*>(sx + j * S + 2 * cg);
      const float2 yv = *reinterpret_cast<const float2*>(sy + j * S + 2 * cg);
      const double y0 = static_cast<double>(yv.x), y1 = static_cast<double>(yv.y);
      const double2* pd = reinterpret_cast<const double2*>(pt_d + j * N + kTileRows * rg);
      const float4* pf = reinterpret_cast<const float4*>(pt_f + j * N + kTileRows * rg);
      double wd[kTileRows];
      float wf[kTileRows];
#pragma unroll
      for (int h = 0; h < kTileRows / 2; ++h) {
        const double2 t = pd[h];
        wd[2 * h] = t.x;
        wd[2 * h + 1] = t.y;
      }
#pragma unroll
      for (int h = 0; h < kTileRows / 4; ++h) {
        const float4 t = pf[h];
        wf[4 * h] = t.x;
        wf[4 * h + 1] = t.y;
        wf[4 * h + 2] = t.z;
        wf[4 * h + 3] = t.w;
      }
#pragma unroll
      for (int i = 0; i < kTileRows; ++i) {
        accy[i][0] = fma(wd[i], y0, accy[i][0]);
        accy[i][1] = fma(wd[i], y1, accy[i][1]);
        accx[i][0] = fmaf(wf[i], xv.x, accx[i][0]);
        accx[i][1] = fmaf(wf[i], xv.y, accx[i][1]);
      }
    }

    // ---- element-wise tail for rows 8rg..8rg+7 (quads 2rg, 2rg+1) and coordinates j, j+1
    const long long j = slab * S + 2 * cg;
    float xi[kTileCols][kTileRows];
#pragma unroll
    for (int cc = 0; cc < kTileCols; ++cc) {
#pragma unroll
      for (int h = 0; h < kTileRows / 4; ++h) {
        if (noisy) {
          normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + cc),
                      static_cast<uint32_t>(2 * rg + h), p.t_noise, &xi[cc][4 * h]);
        } else {
          xi[cc][4 * h] = xi[cc][4 * h + 1] = xi[cc][4 * h + 2] = xi[cc][4 * h + 3] = 0.f;
        }
      }
    }
    const bool in0 = j < p.d, in1 = j + 1 < p.d;
#pragma unroll
    for (int i = 0; i < kTileRows; ++i) {
      const int row = kTileRows * rg + i;
      const float2 av = *reinterpret_cast<const float2*>(sa + row * S + 2 * cg);
      const float2 cv = *reinterpret_cast<const float2*>(sc + row * S + 2 * cg);
      const float2 gv = *reinterpret_cast<const float2*>(sg + row * S + 2 * cg);
      float2 xo, yo, go, yg;
      // gradient point: the new model, or (Algorithm 2 as printed) the staged model this step started from
      float2 x_at = make_float2(0.f, 0.f);
      if (p.grad_at_start) x_at = *reinterpret_cast<const float2*>(sx + row * S + 2 * cg);
      {
        const float x_new = accx[i][0] - static_cast<float>(alpha * accy[i][0]);
        const float g_new = fmaf(av.x, (p.grad_at_start ? x_at.x : x_new) - cv.x, sigma * xi[0][i]);
        xo.x = x_new;
        go.x = g_new;
        yo.x = static_cast<float>(accy[i][0] + (static_cast<double>(g_new) - static_cast<double>(gv.x)));
        yg.x = static_cast<float>(accy[i][0]);
      }
      {
        const float x_new = accx[i][1] - static_cast<float>(alpha * accy[i][1]);
        const float g_new = fmaf(av.y, (p.grad_at_start ? x_at.y : x_new) - cv.y, sigma * xi[1][i]);
        xo.y = x_new;
        go.y = g_new;
        yo.y = static_cast<float>(accy[i][1] + (static_cast<double>(g_new) - static_cast<double>(gv.y)));
        yg.y = static_cast<float>(accy[i][1]);
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
    // this warp no longer reads the stage: hand it back (one arrive per consumer warp)
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive(&empty[s]);
  }
}

template <int N>
int launch_dense(StepParams p, int sm_count, cudaStream_t stream) {
  using Sh = DenseShape<N>;
  DenseMaps maps;
  if (!make_map(&maps.x, p.x, p.n, p.d, p.ld, N, Sh::S) || !make_map(&maps.y, p.y, p.n, p.d, p.ld, N, Sh::S) ||
      !make_map(&maps.g, p.g, p.n, p.d, p.ld, N, Sh::S) || !make_map(&maps.a, p.a, p.n, p.d, p.ld, N, Sh::S) ||
      !make_map(&maps.c, p.c, p.n, p.d, p.ld, N, Sh::S))
    return static_cast<int>(cudaErrorInvalidValue);
  p.S = Sh::S;
  p.num_slabs = (p.d + Sh::S - 1) / Sh::S;
  cudaError_t e = cudaFuncSetAttribute(step_dense_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(Sh::kSmemBytes));
  if (e != cudaSuccess) return static_cast<int>(e);
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  step_dense_kernel<N><<<static_cast<unsigned>(grid), Sh::kThreads, Sh::kSmemBytes, stream>>>(p, maps);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace

bool dense_variant_available(int n) { return n >= 1 && n <= kMaxDenseWorkers && encode_tiled_fn() != nullptr; }

int launch_step_dense(const StepParams& p, int sm_count, cudaStream_t stream) {
  return launch_dense<64>(p, sm_count, stream);
}

}  // namespace detag
