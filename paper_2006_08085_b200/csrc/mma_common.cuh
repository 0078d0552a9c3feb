// Pieces shared by the dense-polynomial kernels for n <= 32 (step_mma.cu, step_mma_many.cu): tile geometry, the
// shared-memory plan, mbarrier / TMA / FP64-MMA wrappers and the tensor maps with their host-side set-up.
#ifndef DETAG_MMA_COMMON_CUH
#define DETAG_MMA_COMMON_CUH

#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
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
constexpr unsigned kMmaSpinLimit = 1u << 20;  // polls before a wait gives up (each may suspend ~kSuspendHintNs)
constexpr unsigned kSuspendHintNs = 2000;
constexpr size_t kMmaSmemBytes =
    static_cast<size_t>(kMmaStages) * kStageBytes + kWarpGroups * kOutFloats * 4 + kFragBytes + 128;
// the last 128 bytes hold the mbarriers (full, empty per stage; ready, free per output tile) and the group counters
static_assert((2 * kMmaStages + 2 * kWarpGroups) * 8 + kWarpGroups * 4 <= 128, "barrier area");
static_assert(kMmaSmemBytes <= 232448, "shared memory plan");

struct MmaMaps {
  CUtensorMap x, y, g, a, c;  // loads (padded boxes)
  CUtensorMap xs, ys, gs;     // stores (exact slab width)
};

__device__ __forceinline__ uint32_t s_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool bar_wait(uint64_t* bar, unsigned parity) {
  const uint32_t addr = s_addr(bar);
  for (unsigned spin = 0; spin < kMmaSpinLimit; ++spin) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    if (done) return true;
  }
  return false;
}

// Monotonic progress counter in shared memory (release/acquire at CTA scope), bounded wait.
__device__ __forceinline__ void count_publish(unsigned* counter, unsigned value) {
  asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(s_addr(counter)), "r"(value) : "memory");
}

__device__ __forceinline__ bool count_wait(const unsigned* counter, unsigned at_least) {
  const uint32_t addr = s_addr(counter);
  for (unsigned spin = 0; spin < kMmaSpinLimit; ++spin) {
    unsigned v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    if (v >= at_least) return true;
    __nanosleep(100);
  }
  return false;
}

__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_addr(bar)) : "memory");
}

__device__ __forceinline__ void bar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_addr(bar)), "r"(count));
}

__device__ __forceinline__ void tile_load(float* dst, const CUtensorMap* map, int col, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          s_addr(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(col), "r"(0), "r"(s_addr(bar))
      : "memory");
}

__device__ __forceinline__ void tile_store(const CUtensorMap* map, int col, const float* src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(col), "r"(0), "r"(s_addr(src))
               : "memory");
}

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

// Tensor maps over the bound arrays; false when the driver refuses one.
inline bool make_mma_maps(MmaMaps* maps, const StepParams& p) {
  if (!make_map(&maps->x, p.x, p.n, p.d, p.ld, kN, kPitchXY) || !make_map(&maps->y, p.y, p.n, p.d, p.ld, kN, kPitchXY) ||
      !make_map(&maps->g, p.g, p.n, p.d, p.ld, kN, kPitchE) || !make_map(&maps->a, p.a, p.n, p.d, p.ld, kN, kPitchE) ||
      !make_map(&maps->c, p.c, p.n, p.d, p.ld, kN, kPitchE))
    return false;
  const long long d_tma = p.d & ~3LL;  // the stores' tensor ends on a 16-byte boundary (see the kernels' tails)
  if (d_tma > 0 && (!make_map(&maps->xs, p.x, p.n, d_tma, p.ld, kN, kS) || !make_map(&maps->ys, p.y, p.n, d_tma, p.ld, kN, kS) ||
                    !make_map(&maps->gs, p.g, p.n, d_tma, p.ld, kN, kS)))
    return false;
  if (d_tma == 0) maps->xs = maps->ys = maps->gs = maps->x;  // never used: every slab lies beyond column 0
  return true;
}

}  // namespace

}  // namespace detag
#endif  // DETAG_MMA_COMMON_CUH
