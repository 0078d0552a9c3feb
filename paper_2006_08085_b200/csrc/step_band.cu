// DeTAG step for circulant gossip matrices (rings) with many workers: banded polynomial on the FP64 tensor path.
//
// For a circulant M (every row is the previous one shifted by one: the ring with uniform weights, the paper's
// Metropolis ring and its slack matrices) the K-round accelerated gossip AG_K(z) = P z has a circulant
// P = P_K(M) whose row is a band: P[i][j] = p((j - i) mod n), p(delta) = 0 for |delta| > K * (bandwidth of M).
// The dense product needs n multiply-adds per element, the K sparse rounds 3K dependent ones; the band needs
// 2K+1, and it can be applied to a block of output rows from a window of input rows:
//     out rows [R, R+32)  <-  window rows [R-16, R+48)   (mod n),   half-band <= 16.
// Per 8-coordinate tile that is, for each of the four 8-row output blocks t, the ten 4-row window steps
// s = 2t .. 2t+9 (all other blocks of the 32 x 64 band matrix are zero): 80 float64 MMAs (m8n8k4) for the
// tracker and the model together, and because P is circulant the A fragment depends on s - 2t only:
// ten doubles per lane, kept in registers, for every tile of the run.
//
// A CTA works on tiles (32 output rows x 64 coordinates).  Warp roles, mbarrier pipeline, padded TMA input
// tiles (box = row pitch), dense output tile + TMA tile stores: as in the dense kernel for n <= 32.  The
// window rows wrap around the ring, so the x, y windows are fetched as four 16-row boxes each at row
// (R - 16 + 16 q) mod n; g, a, c are needed for the 32 output rows only.
//
// The step updates x and y in place, and a tile's window contains rows that neighbouring row blocks
// overwrite.  So the n/32 row blocks of one slab are processed by the CTAs of one thread-block cluster
// (cluster rank = row block), and no CTA stores its results of a slab before every CTA of the cluster has
// its window of that slab in shared memory: a signalling thread publishes "slab k landed" into a per-peer
// counter in every peer's shared memory (st.release.cluster), and the storing thread polls its local copy of
// all peers' counters before it issues the slab's TMA stores.  Halo rows of neighbouring row blocks are read
// by CTAs of the same cluster at about the same time, so they come from L2.
//
// Output rows are the natural blocks 8t + r (a permuted block would widen the band), so the four workers of
// one Philox call sit in four lanes: each lane draws the calls of one block and a 4 x 4 transpose over those
// lanes (two shuffle stages) hands every lane its own workers' normals.
// Every mbarrier wait is bounded; a wait that gives up sets the status word and the CTA winds down.
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kR = 32;             // output rows per tile
constexpr int kHalo = 16;          // window rows on each side = largest supported half-band
constexpr int kW = kR + 2 * kHalo; // window rows
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
constexpr int kMaxCluster = 8;     // portable cluster size: n <= 256
constexpr int kOutFloats = 3 * kR * kS;
constexpr int kBandSteps = 10;     // 4-row window steps that meet an 8-row output block: (2*16 + 8) / 4
constexpr unsigned kSpinLimit = 1u << 20;
constexpr unsigned kSuspendHintNs = 2000;
constexpr size_t kSmemBytes = static_cast<size_t>(kStages) * kStageBytes + kWarpGroups * kOutFloats * 4 + 128;  // barriers + peer counters

struct BandMaps {
  CUtensorMap x16, y16;        // loads, 16-row boxes of width kPitchXY
  CUtensorMap g16, a16, c16;   // loads, 16-row boxes of width kPitchE
  CUtensorMap xs, ys, gs;      // stores, 32-row boxes of width kS
};

struct BandCoef {
  double p[2 * kHalo + 1];  // p[delta + kHalo] = P[i][(i + delta) mod n]
};

__device__ __forceinline__ uint32_t s_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool bar_wait(uint64_t* bar, unsigned parity) {
  const uint32_t addr = s_addr(bar);
  for (unsigned spin = 0; spin < kSpinLimit; ++spin) {
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

__device__ __forceinline__ unsigned cluster_rank() {
  unsigned v;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(v));
  return v;
}

__device__ __forceinline__ void cluster_sync_all() {  // every thread of every CTA of the cluster
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}

// Writes `value` into the counter at the same shared-memory offset in CTA `peer` of the cluster.
__device__ __forceinline__ void publish_to_peer(unsigned* local_counter, unsigned peer, unsigned value) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(s_addr(local_counter)), "r"(peer));
  asm volatile("st.release.cluster.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"(value) : "memory");
}

// Bounded wait until all `count` counters (written by the peers) have reached `at_least`.
__device__ __forceinline__ bool peers_wait(const unsigned* counters, int count, unsigned at_least) {
  for (unsigned spin = 0; spin < kSpinLimit; ++spin) {
    bool all = true;
    for (int q = 0; q < count; ++q) {
      unsigned v;
      asm volatile("ld.acquire.cluster.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(s_addr(counters + q)) : "memory");
      all = all && v >= at_least;
    }
    if (all) return true;
    __nanosleep(200);
  }
  return false;
}

// Monotonic progress counter in this CTA's shared memory (release/acquire at CTA scope), bounded wait.
__device__ __forceinline__ void count_publish(unsigned* counter, unsigned value) {
  asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(s_addr(counter)), "r"(value) : "memory");
}

__device__ __forceinline__ bool count_wait(const unsigned* counter, unsigned at_least) {
  const uint32_t addr = s_addr(counter);
  for (unsigned spin = 0; spin < kSpinLimit; ++spin) {
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

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

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
step_band_kernel(const StepParams p, const __grid_constant__ BandMaps maps, const __grid_constant__ BandCoef coef) {
  // No static shared memory: the dynamic array starts at the CTA's shared window; its alignment is checked.
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* stage_mem = reinterpret_cast<float*>(smem_raw);
  float* out_mem = stage_mem + kStages * kStageFloats;  // [group][x', y', g'][32][kS]
  uint64_t* full = reinterpret_cast<uint64_t*>(out_mem + kWarpGroups * kOutFloats);
  uint64_t* empty = full + kStages;
  uint64_t* out_ready = empty + kStages;
  uint64_t* out_free = out_ready + kWarpGroups;
  unsigned* landed = reinterpret_cast<unsigned*>(out_free + kWarpGroups);  // [peer]: slabs whose window peer has loaded
  unsigned* seen = landed + kMaxCluster;  // [group]: 1 + index of the last slab whose data the group has seen
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  const int row_blocks = n / kR;             // = cluster size
  const int rb = static_cast<int>(cluster_rank());
  const bool aligned_ok = (s_addr(smem_raw) & 127u) == 0;
  if (tid == 0) {
    for (int q = 0; q < kMaxCluster; ++q) landed[q] = 0;
    for (int g = 0; g < kWarpGroups; ++g) seen[g] = 0;
    for (int s = 0; s < kStages; ++s) {
      bar_init(&full[s], 1);
      bar_init(&empty[s], kGroupWarps + 1);  // the group's warps + the signalling thread
    }
    for (int g = 0; g < kWarpGroups; ++g) {
      bar_init(&out_ready[g], kGroupWarps);
      bar_init(&out_free[g], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!aligned_ok) atomicExch(p.status, 2);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  cluster_sync_all();  // counters and barriers of every CTA of the cluster are initialised

  // the cluster takes slabs first, first + stride, ...; this CTA their row block rb
  const long long first = blockIdx.x / row_blocks, stride = gridDim.x / row_blocks;
  const long long num_tiles = aligned_ok ? p.num_slabs : 0;  // "tile" below = slab of this cluster

  if (warp == kSignalWarp) {
    // tells every CTA of the cluster (itself included) that this CTA's window of slab k is in shared memory
    if (lane == 0) {
      long long k = 0;
      for (long long tile = first; tile < num_tiles; tile += stride, ++k) {
        const int s = static_cast<int>(k % kStages);
        if (!bar_wait(&full[s], (k / kStages) & 1)) {
          atomicExch(p.status, 1);
          break;
        }
        for (int peer = 0; peer < row_blocks; ++peer) publish_to_peer(&landed[rb], peer, static_cast<unsigned>(k + 1));
        bar_arrive(&empty[s]);  // keeps the stage's phase from running ahead of this thread
      }
    }
  } else if (warp == kProducerWarp) {
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (long long tile = first; tile < num_tiles; tile += stride, ++issued) {
        const int s = issued % kStages;
        if (issued >= kStages) ok = bar_wait(&empty[s], ((issued / kStages) - 1) & 1);
        if (!ok) break;
        const long long slab = tile;
        float* st = stage_mem + static_cast<size_t>(s) * kStageFloats;
        const int col = static_cast<int>(slab * kS);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_addr(&full[s])),
                     "r"(static_cast<unsigned>(kStageBytes))
                     : "memory");
#pragma unroll
        for (int q = 0; q < kW / 16; ++q) {  // the window wraps around the ring in 16-row pieces
          const int row = ((rb * kR - kHalo + 16 * q) % n + n) % n;
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
        for (int back = 1; back <= kStages && back <= issued; ++back) {  // drain copies still in flight (bounded)
          const int k = issued - back;
          bar_wait(&full[k % kStages], (k / kStages) & 1);
        }
      }
    }
  } else if (warp == kStoreWarp) {
    if (lane == 0) {
      long long k = 0;
      for (long long tile = first; tile < num_tiles; tile += stride, ++k) {
        const int g = static_cast<int>(k % kWarpGroups);
        if (!bar_wait(&out_ready[g], (k / kWarpGroups) & 1)) {
          atomicExch(p.status, 1);
          break;
        }
        const long long slab = tile;
        // in-place update: every CTA of the cluster must hold its window of this slab before anyone overwrites it
        if (!peers_wait(landed, row_blocks, static_cast<unsigned>(k + 1))) {
          atomicExch(p.status, 1);
          break;
        }
        const float* ob = out_mem + g * kOutFloats;
        const int col = static_cast<int>(slab * kS);
        if (col < (p.d & ~3LL)) {
          tile_store(&maps.xs, col, rb * kR, ob);
          tile_store(&maps.ys, col, rb * kR, ob + kR * kS);
          tile_store(&maps.gs, col, rb * kR, ob + 2 * kR * kS);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        bar_arrive(&out_free[g]);
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
  } else {
  // ------------------------------------------------------------------ consumer warps
  const int r = lane >> 2, kq = lane & 3;
  const int group = warp / kGroupWarps, mtile = warp % kGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  float* ob = out_mem + group * kOutFloats;
  const int cl = mtile * 8;
  const long long d_tma = p.d & ~3LL;
  // A fragment of window step u = s - 2t: element [r][kq] = p(4u + kq - r - 16); the same for every block and tile
  double afrag[kBandSteps];
#pragma unroll
  for (int u = 0; u < kBandSteps; ++u) {
    const int delta = 4 * u + kq - r - kHalo;
    afrag[u] = (delta >= -kHalo && delta <= kHalo) ? coef.p[delta + kHalo] : 0.0;
  }
  const int pos = r & 3, half = r >> 2;  // this lane's worker is number `pos` of its Philox quad

  long long use = 0;
  for (long long k = group, tile = first + group * stride; tile < num_tiles;
       tile += kWarpGroups * stride, k += kWarpGroups, ++use) {
    const int s = static_cast<int>(k % kStages);
    bool ok = true;
    if (lane == 0) {
      // with an odd stage count the stage last served the other group: a parity wait must not start before
      // that phase has completed (it could not tell the two apart); the counter says when it has
      if (kStages % kWarpGroups != 0 && k >= kStages)
        ok = count_wait(&seen[(k - kStages) % kWarpGroups], static_cast<unsigned>(k - kStages + 1));
      if (ok) ok = bar_wait(&full[s], (k / kStages) & 1);
      if (ok && mtile == 0) count_publish(&seen[group], static_cast<unsigned>(k + 1));
      if (ok && use > 0) ok = bar_wait(&out_free[group], (use - 1) & 1);
    }
    const long long slab = tile;
    // the d % 4 tail columns are stored directly (not by the storing thread): same in-place rule for them
    if (lane == 0 && ok && slab * kS + kS > d_tma && p.d != d_tma)
      ok = peers_wait(landed, row_blocks, static_cast<unsigned>(k + 1));
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      break;
    }
    const float* sx = stage_mem + static_cast<size_t>(s) * kStageFloats;
    const float* sy = sx + kW * kPitchXY;
    const float* sg = sy + kW * kPitchXY;
    const float* sa = sg + kR * kPitchE;
    const float* sc = sa + kR * kPitchE;
    const long long j0 = slab * kS;

    if (j0 + cl < p.d) {
      // cx accumulates P (x - alpha y) = x' and cy starts at -g, ending as y~ - g: the tail then needs a single
      // float64 addition (scalar float64 work queues behind other warps' MMAs on the shared FP64 pipe)
      double cy[4][2], cx[4][2];
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
          const int u = ws - 2 * t;  // compile-time after unrolling: only the band's blocks are issued
          if (u >= 0 && u < kBandSteps) {
            dmma(cy[t], afrag[u], by);
            dmma(cx[t], afrag[u], bx);
          }
        }
      }
      // noise: this lane draws the two calls (coordinates j, j+1) of block t = pos for its half, then the
      // 4 x 4 transposes over the lanes of the quad give it the normals of its own worker for t = 0..3
      const long long j = j0 + cl + 2 * kq;
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
        const int eoff = orow * kPitchE + cl + 2 * kq;
        const float2 av = *reinterpret_cast<const float2*>(sa + eoff);
        const float2 cv = *reinterpret_cast<const float2*>(sc + eoff);
        float2 xo, yo, go;
        xo.x = static_cast<float>(cx[t][0]);                              // x' (Algorithm 2's model update)
        xo.y = static_cast<float>(cx[t][1]);
        float2 x_at = xo;  // gradient point: the new model, or (Algorithm 2 as printed) the model before this step,
        if (p.grad_at_start) {  // which sits in the window: output row orow is window row orow + kHalo
          const float* xw = sx + (orow + kHalo) * kPitchXY + cl + 2 * kq;
          x_at = make_float2(xw[0], xw[1]);
        }
        go.x = fmaf(av.x, x_at.x - cv.x, sigma * xi[0][t]);               // stochastic gradient
        go.y = fmaf(av.y, x_at.y - cv.y, sigma * xi[1][t]);
        yo.x = static_cast<float>(cy[t][0] + static_cast<double>(go.x));  // fold: (y~ - g) + g', g' as stored
        yo.y = static_cast<float>(cy[t][1] + static_cast<double>(go.y));
        const int ooff = orow * kS + cl + 2 * kq;
        *reinterpret_cast<float2*>(ob + ooff) = xo;
        *reinterpret_cast<float2*>(ob + kR * kS + ooff) = yo;
        *reinterpret_cast<float2*>(ob + 2 * kR * kS + ooff) = go;
        const long long off = static_cast<long long>(rb * kR + orow) * p.ld + j;
        if (j >= d_tma) {  // the last d % 4 coordinates: TMA clips stores at 16-byte granularity
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
        if (p.y_obs != nullptr) {  // optional observer: the gossiped tracker, stored directly
          const float2 gv = *reinterpret_cast<const float2*>(sg + eoff);
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
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
      bar_arrive(&out_ready[group]);
      bar_arrive(&empty[s]);
    }
  }
  }
  cluster_sync_all();  // no CTA leaves while a peer may still write its counters
}

}  // namespace

bool band_variant_available(int n, int half_band) {
  return n % kR == 0 && n >= kW && n / kR <= kMaxCluster && half_band <= kHalo && encode_tiled_fn() != nullptr;
}

int launch_step_band(StepParams p, const double* band /* 2*16+1 entries, p(delta) at index delta+16 */, int sm_count,
                     cudaStream_t stream) {
  BandMaps maps;
  BandCoef coef;
  for (int k = 0; k < 2 * kHalo + 1; ++k) coef.p[k] = band[k];
  const long long d_tma = p.d & ~3LL;
  if (!make_map(&maps.x16, p.x, p.n, p.d, p.ld, 16, kPitchXY) || !make_map(&maps.y16, p.y, p.n, p.d, p.ld, 16, kPitchXY) ||
      !make_map(&maps.g16, p.g, p.n, p.d, p.ld, 16, kPitchE) || !make_map(&maps.a16, p.a, p.n, p.d, p.ld, 16, kPitchE) ||
      !make_map(&maps.c16, p.c, p.n, p.d, p.ld, 16, kPitchE))
    return static_cast<int>(cudaErrorInvalidValue);
  if (d_tma > 0 && (!make_map(&maps.xs, p.x, p.n, d_tma, p.ld, kR, kS) || !make_map(&maps.ys, p.y, p.n, d_tma, p.ld, kR, kS) ||
                    !make_map(&maps.gs, p.g, p.n, d_tma, p.ld, kR, kS)))
    return static_cast<int>(cudaErrorInvalidValue);
  if (d_tma == 0) maps.xs = maps.ys = maps.gs = maps.x16;  // never used
  p.S = kS;
  p.num_slabs = (p.d + kS - 1) / kS;
  cudaError_t e = cudaFuncSetAttribute(step_band_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kSmemBytes));
  if (e != cudaSuccess) return static_cast<int>(e);
  e = cudaFuncSetAttribute(step_band_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 0);
  if (e != cudaSuccess) return static_cast<int>(e);
  const int row_blocks = p.n / kR;  // = cluster size: the CTAs of a cluster take the row blocks of one slab
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(row_blocks);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(static_cast<unsigned>(row_blocks));
  int max_clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&max_clusters, step_band_kernel, &cfg);
  if (e != cudaSuccess) return static_cast<int>(e);
  if (max_clusters < 1) return static_cast<int>(cudaErrorLaunchOutOfResources);
  (void)sm_count;
  const long long clusters = p.num_slabs < max_clusters ? p.num_slabs : max_clusters;
  if (clusters <= 0) return 0;
  cfg.gridDim = dim3(static_cast<unsigned>(clusters * row_blocks));
  e = cudaLaunchKernelEx(&cfg, step_band_kernel, p, maps, coef);
  return static_cast<int>(e != cudaSuccess ? e : cudaGetLastError());
}

}  // namespace detag
