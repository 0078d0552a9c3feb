// Device-side building blocks shared by the tensor-path step kernels: bounded mbarrier and counter waits,
// TMA tile loads and stores, the float64 warp-level multiply-accumulate, a 4 x 4 transpose over lanes.
//
// Every wait is bounded by a poll limit that the launch passes in (StepParams::spin_limit): a wait that runs out
// returns false, the caller sets the status word and winds down.  Nothing here traps or spins without a limit.
#ifndef DETAG_PIPELINE_CUH
#define DETAG_PIPELINE_CUH

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace detag {

namespace {

constexpr unsigned kDefaultSpinLimit = 1u << 20;  // polls before a wait gives up (each may suspend ~kSuspendHintNs)
constexpr unsigned kSuspendHintNs = 2000;

__device__ __forceinline__ uint32_t s_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool bar_wait(uint64_t* bar, unsigned parity, unsigned limit) {
  const uint32_t addr = s_addr(bar);
  for (unsigned spin = 0; spin < limit; ++spin) {
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

// Non-blocking test of a phase: for phases already known to be complete (through a progress counter), where the
// caller only needs the ordering that observing the barrier gives; no suspension, no polling.
__device__ __forceinline__ bool bar_test(uint64_t* bar, unsigned parity) {
  unsigned done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(s_addr(bar)), "r"(parity)
      : "memory");
  return done != 0;
}

// Monotonic progress counter in this CTA's shared memory (release/acquire at CTA scope), bounded wait.
__device__ __forceinline__ void count_publish(unsigned* counter, unsigned value) {
  asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(s_addr(counter)), "r"(value) : "memory");
}

__device__ __forceinline__ bool count_wait(const unsigned* counter, unsigned at_least, unsigned limit) {
  const uint32_t addr = s_addr(counter);
  for (unsigned spin = 0; spin < limit; ++spin) {
    unsigned v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    if (v >= at_least) return true;
    __nanosleep(100);
  }
  return false;
}

// The same wait with relaxed loads: for callers that follow it up with a test of the barrier the counter stands
// for (the test is what orders them after the data); an acquiring load costs several hundred cycles each time.
__device__ __forceinline__ bool count_wait_relaxed(const unsigned* counter, unsigned at_least, unsigned limit) {
  const uint32_t addr = s_addr(counter);
  for (unsigned spin = 0; spin < limit; ++spin) {
    unsigned v;
    asm volatile("ld.relaxed.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    if (v >= at_least) return true;
    __nanosleep(100);
  }
  return false;
}

// Waits until each of `count` consecutive counters has reached `at_least`: relaxed loads issued together, one
// acquire fence at the end (an acquiring load per counter would cost several hundred cycles each).
__device__ __forceinline__ bool counters_wait(const unsigned* counters, int count, unsigned at_least, unsigned limit) {
  const uint32_t addr = s_addr(counters);
  for (unsigned spin = 0; spin < limit; ++spin) {
    unsigned lowest = 0xffffffffu;
    for (int k = 0; k < count; ++k) {
      unsigned v;
      asm volatile("ld.relaxed.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr + 4u * k) : "memory");
      lowest = v < lowest ? v : lowest;
    }
    if (lowest >= at_least) {
      asm volatile("fence.acq_rel.cta;" ::: "memory");
      return true;
    }
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

__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_addr(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Orders generic-proxy writes to shared memory before later async-proxy (TMA) reads of it, and vice versa.
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Tile [box rows][box columns] at (row, col) of a 2-D tensor map -> dense tile in shared memory.
__device__ __forceinline__ void tile_load(float* dst, const CUtensorMap* map, int col, int row, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          s_addr(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(col), "r"(row), "r"(s_addr(bar))
      : "memory");
}

__device__ __forceinline__ void tile_store(const CUtensorMap* map, int col, int row, const float* src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(col), "r"(row), "r"(s_addr(src))
               : "memory");
}

// Box {32 coordinates, 2 halves, box rows} at (half, row) of a three-dimensional map (make_half_map) -> tile
// [row][half][32] in shared memory, 16-byte chunks swizzled within each 1 KiB; and the store of such a tile.
__device__ __forceinline__ void rows_load(float* dst, const CUtensorMap* map, int half, int row, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          s_addr(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(half), "r"(row), "r"(s_addr(bar))
      : "memory");
}

__device__ __forceinline__ void rows_store(const CUtensorMap* map, int half, int row, const float* src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(0), "r"(half), "r"(row), "r"(s_addr(src))
               : "memory");
}

__device__ __forceinline__ void store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// The committed stores have finished READING shared memory (the tile may be overwritten).
__device__ __forceinline__ void store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// The committed stores are complete (their global writes are done).
__device__ __forceinline__ void store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// C (8 x 8, float64, 2 per lane) += A (8 x 4, row-major fragment: lane holds A[lane/4][lane%4])
//                                  x B (4 x 8, column fragment: lane holds B[lane%4][lane/4]);
// lane holds C[lane/4][2 (lane%4)] and C[lane/4][2 (lane%4) + 1].
__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

// 4 x 4 transpose over four neighbouring lanes (lane bits 0 and 1): lane kq gives row kq = v[0..3] and receives
// column kq.
__device__ __forceinline__ void transpose_quad(float (&v)[4], int kq) {
  const bool b0 = (kq & 1) != 0, b1 = (kq & 2) != 0;
  float s0 = b0 ? v[0] : v[1], s1 = b0 ? v[2] : v[3];
  float r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
  if (b0) { v[0] = r0; v[2] = r1; } else { v[1] = r0; v[3] = r1; }
  s0 = b1 ? v[0] : v[2];
  s1 = b1 ? v[1] : v[3];
  r0 = __shfl_xor_sync(0xffffffffu, s0, 2);
  r1 = __shfl_xor_sync(0xffffffffu, s1, 2);
  if (b1) { v[0] = r0; v[1] = r1; } else { v[2] = r0; v[3] = r1; }
}

}  // namespace

}  // namespace detag
#endif  // DETAG_PIPELINE_CUH
