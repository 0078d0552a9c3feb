// DeTAG step with the dense polynomial for 32 < n <= 64 workers (any gossip matrix) on the FP64 tensor path.
//
// AG_K(z) = P z with P = P_K(M) built by the host in float64.  One unit of work ("tile") is 32 output rows x 64
// coordinates; its window is all 64 rows (rows >= n are zero-filled by the loads), every one of the 16 x 4 blocks of
// the 32 x 64 slice of P is issued (128 float64 MMAs m8n8k4 per 8-coordinate tile for tracker and model together)
// and the A fragments come from shared memory (32 KB for the two slices).
//
// A CTA owns whole slabs of 64 coordinates and walks the two row blocks of a slab in order.  Warp roles, mbarrier
// pipeline, padded TMA input tiles (box = row pitch), dense output tile + TMA tile stores, tail inputs in registers
// and the stage handed back before the tail: as in the dense kernel for n <= 32.  The x, y window is fetched as four
// 16-row boxes; g, a, c are needed for the 32 output rows only.  The window is read twice (once per row block);
// the second read comes from L2.
//
// The step updates x and y in place, and the second tile's window contains the rows the first tile overwrites: the
// results of row block 0 are stored only after the window of block 1 has landed in shared memory (a signalling
// thread publishes a "tiles landed" counter; the storing thread, and the warps that write the d % 4 tail columns
// directly, wait for it).  Different slabs share no coordinates.
//
// Output rows are the natural blocks 8t + r, so the four workers of one Philox call sit in four lanes: each lane
// draws the calls of one block and a 4 x 4 transpose over those lanes (two shuffle stages) hands every lane its
// own workers' normals.  Every mbarrier wait is bounded; a wait that gives up sets the status word and the CTA
// winds down.  (Circulant matrices with n >= 64 have their own kernel, step_ring.cu; tori step_torus.cu.)
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kR = 32;             // output rows per tile
constexpr int kW = 64;             // window rows: all (padded) workers
constexpr int kS = 64;             // coordinates per tile: 8 MMA tiles of 8, one per consumer warp of a group
constexpr int kPitchXY = kS + 8;   // floats; 8 mod 32 -> the four window rows of a B fragment hit disjoint banks
constexpr int kPitchE = kS + 8;    // floats; rows of g, a, c: consecutive rows 8t + r of the accumulator layout
                                   // land 8 banks apart, so those loads are conflict-free as well
constexpr int kStageFloats = 2 * kW * kPitchXY + 3 * kR * kPitchE;
constexpr int kStageBytes = kStageFloats * 4;
constexpr int kStages = 2;
constexpr int kWarpGroups = 2;     // consumer groups take alternate tiles
constexpr int kGroupWarps = kS / 8;
constexpr int kConsumerWarps = kGroupWarps * kWarpGroups;
constexpr int kProducerWarp = kConsumerWarps, kStoreWarp = kConsumerWarps + 1, kSignalWarp = kConsumerWarps + 2;
constexpr int kThreads = (kConsumerWarps + 3) * 32;
constexpr int kOutFloats = 3 * kR * kS;
constexpr size_t kSmemBytes =
    static_cast<size_t>(kStages) * kStageBytes + kWarpGroups * kOutFloats * 4 + 128;  // + barriers, counters
constexpr int kDenseFragBytes = 2 * (kW / 4) * 4 * 32 * 8;  // dense mode: [row block][window step][t][lane] doubles
static_assert(kSmemBytes + kDenseFragBytes <= 232448, "shared memory plan");

struct BandMaps {
  CUtensorMap x16, y16;        // loads, 16-row boxes of width kPitchXY
  CUtensorMap g16, a16, c16;   // loads, 16-row boxes of width kPitchE
  CUtensorMap xs, ys, gs;      // stores, 32-row boxes of width kS
};

static_assert(sizeof(BandMaps) <= sizeof(TensorMapSet), "tensor map storage");

// 4 x 4 transpose over the four lanes {lane ^ 0, 4, 8, 12} (lane bits 2 and 3): lane with index q = (lane >> 2) & 3
// gives row q = v[0..3] and receives column q.
__device__ __forceinline__ void transpose4(float (&v)[4], int q) {
  const bool b0 = (q & 1) != 0, b1 = (q & 2) != 0;
  float s0 = b0 ? v[0] : v[1], s1 = b0 ? v[2] : v[3];
  float r0 = __shfl_xor_sync(0xffffffffu, s0, 4), r1 = __shfl_xor_sync(0xffffffffu, s1, 4);
  if (b0) { v[0] = r0; v[2] = r1; } else { v[1] = r0; v[3] = r1; }
  s0 = b1 ? v[0] : v[2];
  s1 = b1 ? v[1] : v[3];
  r0 = __shfl_xor_sync(0xffffffffu, s0, 8);
  r1 = __shfl_xor_sync(0xffffffffu, s1, 8);
  if (b1) { v[0] = r0; v[1] = r1; } else { v[2] = r0; v[3] = r1; }
}

__global__ void __launch_bounds__(kThreads, 1)
step_band_kernel(const StepParams p, const __grid_constant__ BandMaps maps) {
  // No static shared memory: the dynamic array starts at the CTA's shared window; its alignment is checked.
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* stage_mem = reinterpret_cast<float*>(smem_raw);
  float* out_mem = stage_mem + kStages * kStageFloats;   // [group][x', y', g'][32][kS]
  uint64_t* full = reinterpret_cast<uint64_t*>(out_mem + kWarpGroups * kOutFloats);
  uint64_t* empty = full + kStages;
  uint64_t* out_ready = empty + kStages;
  uint64_t* out_free = out_ready + kWarpGroups;
  unsigned* landed = reinterpret_cast<unsigned*>(out_free + kWarpGroups);  // tiles whose window is in shared memory
  unsigned* seen = landed + 1;  // [group]: 1 + index of the last tile whose data the group has seen
  double* frag = reinterpret_cast<double*>(smem_raw + kSmemBytes);  // dense mode only (the launch adds the bytes)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  constexpr int row_blocks = 2;  // 64 padded rows
  if ((s_addr(smem_raw) & 127u) != 0) {
    if (tid == 0) atomicExch(p.status, 2);
    return;
  }
  {
    // slice rb of P in fragment order: block (ws, t), lane (r, kq) holds P[32 rb + 8t + r][4 ws + kq]
    for (int e = tid; e < 2 * (kW / 4) * 4 * 32; e += kThreads) {
      const int l = e & 31, t = (e >> 5) & 3, ws = (e >> 7) % (kW / 4), b = e / (32 * 4 * (kW / 4));
      const int i = kR * b + 8 * t + (l >> 2), j = 4 * ws + (l & 3);
      frag[e] = (i < n && j < n) ? p.poly[static_cast<size_t>(i) * n + j] : 0.0;
    }
  }
  if (tid == 0) {
    *landed = 0;
    for (int g = 0; g < kWarpGroups; ++g) seen[g] = 0;
    for (int s = 0; s < kStages; ++s) {
      bar_init(&full[s], 1);
      bar_init(&empty[s], kGroupWarps + 1);  // the group's warps + the signalling thread
    }
    for (int g = 0; g < kWarpGroups; ++g) {
      bar_init(&out_ready[g], kGroupWarps);
      bar_init(&out_free[g], 1);
    }
    fence_barrier_init();
  }
  fence_async_shared();
  __syncthreads();

  // this CTA takes slabs blockIdx.x, blockIdx.x + gridDim.x, ...; tile k is row block k % row_blocks of its
  // (k / row_blocks)-th slab
  const long long my_slabs = blockIdx.x < p.num_slabs ? (p.num_slabs - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const long long num_tiles = my_slabs * row_blocks;

  if (warp == kSignalWarp) {
    // publishes how many tiles (in order) have their window in shared memory
    if (lane == 0) {
      for (long long k = 0; k < num_tiles; ++k) {
        const int s = static_cast<int>(k % kStages);
        if (!bar_wait(&full[s], (k / kStages) & 1, p.spin_limit)) {
          atomicExch(p.status, 1);
          break;
        }
        count_publish(landed, static_cast<unsigned>(k + 1));
        bar_arrive(&empty[s]);  // keeps the stage's phase from running ahead of this thread
      }
    }
    return;
  }
  if (warp == kProducerWarp) {
    if (lane == 0) {
      long long issued = 0;
      bool ok = true;
      for (; issued < num_tiles; ++issued) {
        if (p.stall_after >= 0 && issued >= p.stall_after) return;  // self test: the loads stop, every waiter times out
        const int s = static_cast<int>(issued % kStages);
        if (issued >= kStages) ok = bar_wait(&empty[s], ((issued / kStages) - 1) & 1, p.spin_limit);
        if (!ok) break;
        const long long slab_no = issued / row_blocks;
        const int rb = static_cast<int>(issued % row_blocks);
        const long long slab = blockIdx.x + slab_no * gridDim.x;
        float* st = stage_mem + static_cast<size_t>(s) * kStageFloats;
        const int col = static_cast<int>(slab * kS);
        bar_expect_tx(&full[s], static_cast<unsigned>(kStageBytes));
#pragma unroll
        for (int q = 0; q < kW / 16; ++q) {  // the window = all 64 rows, in 16-row pieces
          const int row = 16 * q;
          tile_load(st + q * 16 * kPitchXY, &maps.x16, col, row, &full[s]);
          tile_load(st + kW * kPitchXY + q * 16 * kPitchXY, &maps.y16, col, row, &full[s]);
        }
        float* se = st + 2 * kW * kPitchXY;
#pragma unroll
        for (int q = 0; q < kR / 16; ++q) {
          const int row = rb * kR + 16 * q;
          tile_load(se + q * 16 * kPitchE, &maps.g16, col, row, &full[s]);
          tile_load(se + kR * kPitchE + q * 16 * kPitchE, &maps.a16, col, row, &full[s]);
          tile_load(se + 2 * kR * kPitchE + q * 16 * kPitchE, &maps.c16, col, row, &full[s]);
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (long long back = 1; back <= kStages && back <= issued; ++back) {  // drain copies still in flight (bounded)
          const long long k = issued - back;
          bar_wait(&full[k % kStages], (k / kStages) & 1, p.spin_limit);
        }
      }
    }
    return;
  }
  if (warp == kStoreWarp) {
    if (lane == 0) {
      for (long long k = 0; k < num_tiles; ++k) {
        const int g = static_cast<int>(k % kWarpGroups);
        if (!bar_wait(&out_ready[g], (k / kWarpGroups) & 1, p.spin_limit)) {
          atomicExch(p.status, 1);
          break;
        }
        const long long slab_no = k / row_blocks;
        const int rb = static_cast<int>(k % row_blocks);
        // in-place update: the next block's window (it contains this block's last rows) must have landed
        if (rb + 1 < row_blocks && !count_wait(landed, static_cast<unsigned>(k + 2), p.spin_limit)) {
          atomicExch(p.status, 1);
          break;
        }
        const float* ob = out_mem + g * kOutFloats;
        const int col = static_cast<int>((blockIdx.x + slab_no * gridDim.x) * kS);
        if (col < (p.d & ~3LL)) {
          tile_store(&maps.xs, col, rb * kR, ob);
          tile_store(&maps.ys, col, rb * kR, ob + kR * kS);
          tile_store(&maps.gs, col, rb * kR, ob + 2 * kR * kS);
        }
        store_commit();
        store_wait_read();
        bar_arrive(&out_free[g]);
      }
      store_wait_all();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int r = lane >> 2, kq = lane & 3;
  const int group = warp / kGroupWarps, mtile = warp % kGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  float* ob = out_mem + group * kOutFloats;
  const int cl = mtile * 8;
  const long long d_tma = p.d & ~3LL;
  const int pos = r & 3, half = r >> 2;  // this lane's worker is number `pos` of its Philox quad

  // 32-bit bookkeeping: the launcher admits this kernel only for d < 2^31, so tile and slab counts fit easily
  const int tiles = static_cast<int>(num_tiles);
  int use = 0;
  for (int k = group; k < tiles; k += kWarpGroups, ++use) {
    const int s = k % kStages;
    const int slab_no = k / row_blocks;
    const int rb = k - slab_no * row_blocks;
    const long long slab = blockIdx.x + static_cast<long long>(slab_no) * gridDim.x;
    bool ok = true;
    if (lane == 0) {
      // with an odd stage count the stage last served the other group: a parity wait must not start before
      // that phase has completed (it could not tell the two apart); the counter says when it has
      if (kStages % kWarpGroups != 0 && k >= kStages)
        ok = count_wait(&seen[(k - kStages) % kWarpGroups], static_cast<unsigned>(k - kStages + 1), p.spin_limit);
      if (ok) ok = bar_wait(&full[s], (k / kStages) & 1, p.spin_limit);
      if (ok && mtile == 0) count_publish(&seen[group], static_cast<unsigned>(k + 1));
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    const float* sx = stage_mem + static_cast<size_t>(s) * kStageFloats;
    const float* sy = sx + kW * kPitchXY;
    const float* sg = sy + kW * kPitchXY;
    const float* sa = sg + kR * kPitchE;
    const float* sc = sa + kR * kPitchE;
    const long long j0 = slab * kS;
    const long long j = j0 + cl + 2 * kq;
    const bool active = j0 + cl < p.d;  // a tile wholly beyond column d computes nothing but keeps the protocol

    // cx accumulates P (x - alpha y) = x' and cy starts at -g, ending as y~ - g: the tail then needs a single
    // float64 addition (scalar float64 work queues behind other warps' MMAs on the shared FP64 pipe)
    double cy[4][2], cx[4][2];
    float2 av4[4], cv4[4];
    if (active) {
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 gv = *reinterpret_cast<const float2*>(sg + (8 * t + r) * kPitchE + cl + 2 * kq);
        cy[t][0] = static_cast<double>(-gv.x);
        cy[t][1] = static_cast<double>(-gv.y);
        cx[t][0] = cx[t][1] = 0.0;
      }
#pragma unroll
      for (int ws = 0; ws < kW / 4; ++ws) {  // window steps of four rows
        const int src = (4 * ws + kq) * kPitchXY + cl + r;
        const double by = static_cast<double>(sy[src]);
        const double bx = fma(-alpha, by, static_cast<double>(sx[src]));
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const double a = frag[((rb * (kW / 4) + ws) * 4 + t) * 32 + lane];
          dmma(cy[t], a, by);
          dmma(cx[t], a, bx);
        }
      }
      // the tail's inputs move to registers so that the stage can be refilled while the tail runs
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int eoff = (8 * t + r) * kPitchE + cl + 2 * kq;
        av4[t] = *reinterpret_cast<const float2*>(sa + eoff);
        cv4[t] = *reinterpret_cast<const float2*>(sc + eoff);
      }
    }
    __syncwarp();
    if (lane == 0) {
      bar_arrive(&empty[s]);  // stage no longer read by this warp
      if (use > 0) ok = bar_wait(&out_free[group], (use - 1) & 1, p.spin_limit);  // previous tile of this group stored
      // The d % 4 tail columns are stored directly (not by the storing thread): same in-place rule for them.  The
      // window of the previous block holds this block's first rows as well, and two stages' loads may complete out
      // of order, so the slab's last block (which has no next window to wait for) waits until every tile up to
      // its own has landed.
      if (ok && j0 + kS > d_tma && p.d != d_tma)
        ok = count_wait(landed, static_cast<unsigned>(k + (rb + 1 < row_blocks ? 2 : 1)), p.spin_limit);
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }

    if (active) {
      // noise: this lane draws the two calls (coordinates j, j+1) of block t = pos for its half, then the
      // 4 x 4 transposes over the lanes of the quad give it the normals of its own worker for t = 0..3
      float xi[2][4];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        if (noisy) {
          const uint32_t quad = static_cast<uint32_t>((rb * kR + 8 * pos) / 4 + half);
          normal_quad(p.seed_lo, p.seed_hi, static_cast<unsigned long long>(p.coord_offset + j + e), quad, p.t_noise,
                      xi[e]);
          transpose4(xi[e], pos);
        } else {
          xi[e][0] = xi[e][1] = xi[e][2] = xi[e][3] = 0.f;
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int orow = 8 * t + r;  // output row within the tile
        const float2 av = av4[t], cv = cv4[t];
        float2 xo, yo, go;
        xo.x = static_cast<float>(cx[t][0]);                              // x' (Algorithm 2's model update)
        xo.y = static_cast<float>(cx[t][1]);
        const bool row_ok = rb * kR + orow < n;  // dense mode pads n up to 64: padded rows exist on chip only
        const long long off = static_cast<long long>(rb * kR + orow) * p.ld + j;
        // Gradient point: the new model, or (Algorithm 2 as printed) the model before this step.  The old x and g
        // of this tile are still in global memory: its stores are issued after all of its warps are done.
        float2 x_at = xo;
        if (p.grad_at_start && row_ok) {
          x_at.x = j < p.d ? p.x[off] : 0.f;
          x_at.y = j + 1 < p.d ? p.x[off + 1] : 0.f;
        }
        go.x = fmaf(av.x, x_at.x - cv.x, sigma * xi[0][t]);               // stochastic gradient
        go.y = fmaf(av.y, x_at.y - cv.y, sigma * xi[1][t]);
        yo.x = static_cast<float>(cy[t][0] + static_cast<double>(go.x));  // fold: (y~ - g) + g', g' as stored
        yo.y = static_cast<float>(cy[t][1] + static_cast<double>(go.y));
        const int ooff = orow * kS + cl + 2 * kq;
        *reinterpret_cast<float2*>(ob + ooff) = xo;
        *reinterpret_cast<float2*>(ob + kR * kS + ooff) = yo;
        *reinterpret_cast<float2*>(ob + 2 * kR * kS + ooff) = go;
        if (p.y_obs != nullptr && row_ok) {  // optional observer: the gossiped tracker y~ = (y~ - g) + g, stored directly
          if (j < p.d) p.y_obs[off] = static_cast<float>(cy[t][0] + static_cast<double>(p.g[off]));
          if (j + 1 < p.d) p.y_obs[off + 1] = static_cast<float>(cy[t][1] + static_cast<double>(p.g[off + 1]));
        }
        if (j >= d_tma && row_ok) {  // the last d % 4 coordinates: TMA clips stores at 16-byte granularity
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
    fence_async_shared();  // outputs visible to the TMA store
    __syncwarp();
    if (lane == 0) bar_arrive(&out_ready[group]);
  }
}

}  // namespace

bool dense_window_available(int n) { return n > kR && n <= kW && encode_tiled_fn() != nullptr; }

bool dense_variant_available(int n) { return n >= 1 && n <= kMaxDenseWorkers && encode_tiled_fn() != nullptr; }

bool build_maps_band(const StepParams& p, TensorMapSet* out) {
  BandMaps& maps = *reinterpret_cast<BandMaps*>(out->bytes);
  const long long d_tma = p.d & ~3LL;
  if (!make_map(&maps.x16, p.x, p.n, p.d, p.ld, 16, kPitchXY) || !make_map(&maps.y16, p.y, p.n, p.d, p.ld, 16, kPitchXY) ||
      !make_map(&maps.g16, p.g, p.n, p.d, p.ld, 16, kPitchE) || !make_map(&maps.a16, p.a, p.n, p.d, p.ld, 16, kPitchE) ||
      !make_map(&maps.c16, p.c, p.n, p.d, p.ld, 16, kPitchE))
    return false;
  if (d_tma > 0 && (!make_map(&maps.xs, p.x, p.n, d_tma, p.ld, kR, kS) || !make_map(&maps.ys, p.y, p.n, d_tma, p.ld, kR, kS) ||
                    !make_map(&maps.gs, p.g, p.n, d_tma, p.ld, kR, kS)))
    return false;
  if (d_tma == 0) maps.xs = maps.ys = maps.gs = maps.x16;  // never used
  return true;
}

// 32 < n <= 64, p.poly holds P_K(M); `band` must be null (kept for the launcher's signature).
int launch_step_band(StepParams p, const TensorMapSet& maps, const double* band, int sm_count, cudaStream_t stream) {
  if (p.mode != kModeDetag || band != nullptr) return static_cast<int>(cudaErrorInvalidValue);
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  auto kernel = step_band_kernel;
  const size_t smem = kSmemBytes + kDenseFragBytes;
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kThreads, smem, stream>>>(p, *reinterpret_cast<const BandMaps*>(maps.bytes));
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
