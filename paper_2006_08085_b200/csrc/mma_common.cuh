// Pieces shared by the dense-polynomial kernels for n <= 32 (step_mma.cu, step_mma_many.cu): tile geometry, the
// shared-memory plan, the set-up, producer and storing roles of the persistent CTA, and the tensor maps.
#ifndef DETAG_MMA_COMMON_CUH
#define DETAG_MMA_COMMON_CUH

#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kN = 32;            // padded worker count
constexpr int kS = 64;            // coordinates per slab: 8 tiles of 8, one per consumer warp of a group
constexpr int kPitchXY = kS + 8;  // floats; 8 mod 32 -> the four workers of a B fragment hit disjoint banks
constexpr int kPitchE = kS + 4;   // floats; rows of g, a, c (read in the accumulator layout)
constexpr int kStageFloats = 2 * kN * kPitchXY + 3 * kN * kPitchE;
constexpr int kStageBytes = kStageFloats * 4;
constexpr int kMmaStages = 3;
constexpr int kWarpGroups = 2;    // consumer groups take alternate slabs, so their phases interleave
constexpr int kGroupWarps = kS / 8;
constexpr int kConsumerWarps = kGroupWarps * kWarpGroups;
constexpr int kProducerWarp = kConsumerWarps, kStoreWarp = kConsumerWarps + 1;
constexpr int kMmaThreads = (kConsumerWarps + 2) * 32;
constexpr int kOutFloats = 3 * kN * kS;       // x', y', g' tiles of one slab, dense rows
constexpr int kFragBytes = 32 * 32 * 8;       // P in fragment order
constexpr size_t kMmaSmemBytes =
    static_cast<size_t>(kMmaStages) * kStageBytes + kWarpGroups * kOutFloats * 4 + kFragBytes + 128;
// the last 128 bytes hold the mbarriers (full, empty per stage; ready, free per output tile) and the group counters
static_assert((2 * kMmaStages + 2 * kWarpGroups) * 8 + kWarpGroups * 4 <= 128, "barrier area");
static_assert(kMmaSmemBytes <= 232448, "shared memory plan");

// Loads (padded boxes): x, y, g and two more arrays - the objective data a, c, or (caller-written gradients) the
// newest gradient in the `a` slot.  Stores (exact slab width): x', y', g'.
struct MmaMaps {
  CUtensorMap x, y, g, a, c;
  CUtensorMap xs, ys, gs;
};
static_assert(sizeof(MmaMaps) <= sizeof(TensorMapSet), "tensor map storage");

// Pointers into the CTA's dynamic shared memory.
struct MmaShared {
  float* stage_mem;     // [stage][x | y | g | a | c]
  float* out_mem;       // [group][x', y', g'][32][kS]
  double* frag;         // P in fragment order: [t][ks][lane]
  uint64_t* full;       // [stage]: the stage's loads have landed
  uint64_t* empty;      // [stage]: the group's warps no longer read the stage
  uint64_t* out_ready;  // [group]: the group's 8 warps have written their outputs
  uint64_t* out_free;   // [group]: the stores have finished reading the tile
  unsigned* seen;       // [group]: 1 + last slab index whose data the group saw
};

// Carves up the shared memory, writes P in fragment order and initialises the barriers.  Returns false (and
// sets status 2) when the shared window is not 128-byte aligned, which the TMA tiles need.  All threads call it.
__device__ __forceinline__ bool mma_setup(const StepParams& p, unsigned char* smem_raw, MmaShared& sm) {
  sm.stage_mem = reinterpret_cast<float*>(smem_raw);
  sm.out_mem = sm.stage_mem + kMmaStages * kStageFloats;
  sm.frag = reinterpret_cast<double*>(sm.out_mem + kWarpGroups * kOutFloats);
  sm.full = reinterpret_cast<uint64_t*>(sm.frag + 32 * 32);
  sm.empty = sm.full + kMmaStages;
  sm.out_ready = sm.empty + kMmaStages;
  sm.out_free = sm.out_ready + kWarpGroups;
  sm.seen = reinterpret_cast<unsigned*>(sm.out_free + kWarpGroups);
  if ((s_addr(smem_raw) & 127u) != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, 2);
    return false;
  }
  const int tid = threadIdx.x, n = p.n;
  // block (t, ks), lane (r, kq) holds P[4r + t][4ks + kq]
  for (int e = tid; e < 32 * 32; e += kMmaThreads) {
    const int l = e & 31, ks = (e >> 5) & 7, t = e >> 8;
    const int i = 4 * (l >> 2) + t, j = 4 * ks + (l & 3);
    sm.frag[e] = (i < n && j < n) ? p.poly[static_cast<size_t>(i) * n + j] : 0.0;
  }
  if (tid == 0) {
    for (int g = 0; g < kWarpGroups; ++g) sm.seen[g] = 0;
    for (int s = 0; s < kMmaStages; ++s) {
      bar_init(&sm.full[s], 1);
      bar_init(&sm.empty[s], kGroupWarps);
    }
    for (int g = 0; g < kWarpGroups; ++g) {
      bar_init(&sm.out_ready[g], kGroupWarps);
      bar_init(&sm.out_free[g], 1);
    }
    fence_barrier_init();
  }
  fence_async_shared();
  __syncthreads();
  return true;
}

// Producer role (one thread): keeps kMmaStages slabs in flight.  kMode selects which arrays a stage holds.
template <int kMode>
__device__ __forceinline__ void mma_producer(const StepParams& p, const MmaMaps& maps, const MmaShared& sm) {
  constexpr unsigned kBytes = static_cast<unsigned>(kStageBytes) -
                              (kMode == kModeDpsgd ? kN * kPitchXY * 4u : 0u) -   // no tracker
                              (kMode == kModeExternal ? kN * kPitchE * 4u : 0u);  // no objective data
  const long long first = blockIdx.x, stride = gridDim.x;
  long long issued = 0;
  bool ok = true;
  for (long long slab = first; slab < p.num_slabs; slab += stride, ++issued) {
    if (p.stall_after >= 0 && issued >= p.stall_after) return;  // self test: the loads stop, every waiter times out
    const int s = static_cast<int>(issued % kMmaStages);
    if (issued >= kMmaStages) ok = bar_wait(&sm.empty[s], ((issued / kMmaStages) - 1) & 1, p.spin_limit);
    if (!ok) break;
    float* st = sm.stage_mem + static_cast<size_t>(s) * kStageFloats;
    const int col = static_cast<int>(slab * kS);
    bar_expect_tx(&sm.full[s], kBytes);
    tile_load(st, &maps.x, col, 0, &sm.full[s]);
    if (kMode != kModeDpsgd) tile_load(st + kN * kPitchXY, &maps.y, col, 0, &sm.full[s]);
    float* se = st + 2 * kN * kPitchXY;
    tile_load(se, &maps.g, col, 0, &sm.full[s]);
    tile_load(se + kN * kPitchE, &maps.a, col, 0, &sm.full[s]);
    if (kMode != kModeExternal) tile_load(se + 2 * kN * kPitchE, &maps.c, col, 0, &sm.full[s]);
  }
  if (!ok) {
    atomicExch(p.status, 1);
    for (long long back = 1; back <= kMmaStages && back <= issued; ++back) {  // drain copies still in flight (bounded)
      const long long k = issued - back;
      bar_wait(&sm.full[k % kMmaStages], (k / kMmaStages) & 1, p.spin_limit);
    }
  }
}

// Storing role (one thread): each finished output tile goes out with one TMA tile store per array.
template <int kMode>
__device__ __forceinline__ void mma_storer(const StepParams& p, const MmaMaps& maps, const MmaShared& sm) {
  const long long first = blockIdx.x, stride = gridDim.x;
  long long k = 0;
  for (long long slab = first; slab < p.num_slabs; slab += stride, ++k) {
    const int g = static_cast<int>(k % kWarpGroups);
    if (!bar_wait(&sm.out_ready[g], (k / kWarpGroups) & 1, p.spin_limit)) {
      atomicExch(p.status, 1);
      break;
    }
    const float* ob = sm.out_mem + g * kOutFloats;
    const int col = static_cast<int>(slab * kS);
    if (col < (p.d & ~3LL)) {
      tile_store(&maps.xs, col, 0, ob);
      if (kMode != kModeDpsgd) tile_store(&maps.ys, col, 0, ob + kN * kS);
      tile_store(&maps.gs, col, 0, ob + 2 * kN * kS);
    }
    store_commit();
    store_wait_read();  // the tile may be overwritten now
    bar_arrive(&sm.out_free[g]);
  }
  store_wait_all();  // all global writes done before the CTA leaves
}

// Consumer side: waits until slab k (stage s) of this CTA has landed.  Lane 0 polls, the warp gets the verdict.
__device__ __forceinline__ bool mma_wait_slab(const StepParams& p, const MmaShared& sm, long long k, int group,
                                              int tile, int lane) {
  bool ok = true;
  if (lane == 0) {
    const int s = static_cast<int>(k % kMmaStages);
    // The stage last held slab k - kMmaStages, which belongs to the other group when the stage count is odd.
    // A parity wait must not start before that phase has completed (it could not tell the two apart), and
    // it costs nothing to make sure: this slab cannot have been loaded before that one was consumed.
    if (kMmaStages % kWarpGroups != 0 && k >= kMmaStages)
      ok = count_wait(&sm.seen[(k - kMmaStages) % kWarpGroups], static_cast<unsigned>(k - kMmaStages + 1), p.spin_limit);
    if (ok) ok = bar_wait(&sm.full[s], (k / kMmaStages) & 1, p.spin_limit);
    if (ok && tile == 0) count_publish(&sm.seen[group], static_cast<unsigned>(k + 1));
  }
  return __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
}

}  // namespace

}  // namespace detag
#endif  // DETAG_MMA_COMMON_CUH
