// DeTAG step for circulant gossip matrices (rings) with many workers, n = 64 .. 1024 in multiples of 32.
//
// For a circulant M (every row is the previous one shifted by one: the ring with uniform weights, the paper's
// Metropolis ring and its slack matrices) the K-round accelerated gossip AG_K(z) = P z has a circulant
// P = P_K(M), P[i][j] = p((j - i) mod n).  Two modes:
//   band   p(delta) = 0 for |delta| > 16 (K times the bandwidth of M at most 16): 32 output rows need a window
//          of 64 input rows, and of the 16 x 4 blocks of that 64 x 32 slice only 10 per 8-row output block are
//          non-zero: 80 float64 MMAs (m8n8k4) per 8 coordinates x 32 workers for tracker and model together.
//   dense  any p (Theorem 3's phase length makes P dense): every output block contracts the whole ring, n / 4
//          k-steps, with the B fragments looked up in the one stored row of P.  n <= 256.
//
// Layout of the contraction: the eight coordinates of a warp's tile are the M index of the MMA, the input worker
// the contraction index (k-step s takes window rows 4 s + kq) and the output worker the N index, permuted so that
// column 2 kq + e of output block t stands for tile row 8 t + kq + 4 e.  A lane then supplies rows kq + 4 s and
// receives rows kq + 4 m (m = 0..7) of ONE coordinate: the element-wise tail of the step (model update, noise,
// gradient, tracker fold) is lane-local and its results replace, in shared memory, the very g, a, c elements the
// lane read.  The A operand is consumed k-step by k-step straight from shared memory; the accumulators of both
// arrays (16 doubles) are all that lives across the loop.
//
// A CTA owns whole slabs of 64 coordinates and walks the n / 32 row blocks ("tiles") of a slab in order.
//   x, y   travel in chunks of 16 rows, EACH LOADED ONCE into a ring of shared-memory slots that all tiles read
//          (a tile's window is four consecutive chunks): per slab the chunks n/16 - 1, 0, 1, .., n/16 - 1 in this
//          order, plus a second copy of chunk 0 in a side buffer, taken before anything of the slab is stored, for
//          the last tile, whose window wraps around to rows 0..15.  Since no row is fetched again after it was
//          fetched once (except those two, both handled), the in-place update of x and y needs no further care.
//          Dense mode: the chunks 0 .. n/16 - 1 of a slab all stay resident until its last tile is done.
//   g, a, c  of a tile's 32 rows go to one of four (dense: two) stages; the tail overwrites them with g', x', y'
//          and three TMA stores send the stage out.
// Every transfer is one three-dimensional TMA box {32 coordinates, 2 halves, rows} in the 128-byte swizzle: rows
// arrive as contiguous 256-byte pieces, and with the row ownership above every warp-wide shared-memory access hits
// 32 different banks.  The kernel takes whole slabs only: the host hands the last d % 64 columns to the generic
// kernel.
// Roles: 16 consumer warps in two groups taking alternate tiles; one thread loading x, y chunks, one loading
// g, a, c stages, one storing, one publishing how many chunks have landed (so that no consumer ever starts a
// parity wait on a slot whose previous phase is still open).  Every wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kRS = 64;                 // coordinates per slab
constexpr int kRHalf = 32;              // coordinates per 128-byte swizzle row
constexpr int kRT = 32;                 // output rows per tile
constexpr int kChunkRows = 16;
constexpr int kChunkFloats = kChunkRows * kRS;          // one array of one chunk: [row][half][32]
constexpr int kSlotFloats = 2 * kChunkFloats;           // x chunk, y chunk
constexpr int kEArrayFloats = kRT * kRS;
constexpr int kEStageFloats = 3 * kEArrayFloats;        // g | a | c  ->  g' | x' | y'
constexpr int kRHalo = 16, kBandSteps = 10;             // band mode: half-band limit; k-steps that meet an output block
constexpr int kRGroups = 2, kRGroupWarps = kRS / 8;
constexpr int kRConsumerWarps = kRGroups * kRGroupWarps;
constexpr int kLoadXYWarp = kRConsumerWarps, kLoadEWarp = kRConsumerWarps + 1, kRStoreWarp = kRConsumerWarps + 2,
              kRSignalWarp = kRConsumerWarps + 3;
constexpr int kRThreads = (kRConsumerWarps + 4) * 32;
constexpr int kMaxSlots = 16;

template <bool kDense>
struct RingPlan {
  static constexpr int kSlots = kDense ? 16 : 12;       // ring of x, y chunks
  static constexpr int kEStages = kDense ? 2 : 4;       // even: a stage always serves the same consumer group
  static constexpr int kSideFloats = kDense ? 0 : 2 * kSlotFloats;   // chunk 0 copies, one per slab parity
  static constexpr int kTableDoubles = kDense ? 256 : 0;             // the stored row of P
  static constexpr size_t kCtrlOffset = static_cast<size_t>(kSlots) * kSlotFloats * 4 + kSideFloats * 4 +
                                        static_cast<size_t>(kEStages) * kEStageFloats * 4 + kTableDoubles * 8;
  // control area: slot barriers, side barriers (2), stage barriers (full, empty, ready), counters
  static constexpr size_t kCtrlBytes = (kMaxSlots + 2 + 3 * 4) * 8 + (2 + kRConsumerWarps) * 4;
  static constexpr size_t kSmemBytes = kCtrlOffset + 512 + 1024;     // + slack to align the tiles to 1 KiB
  static_assert(kCtrlBytes <= 512, "control area");
  static_assert(kSmemBytes <= 232448, "shared memory plan");
};

struct RingMaps {
  CUtensorMap x, y;        // boxes {32, 2, 16 rows}
  CUtensorMap g, a, c;     // boxes {32, 2, 32 rows}: loads and (g, x, y arrays) stores
  CUtensorMap xs, ys;      // boxes {32, 2, 32 rows} over x and y, for the stores
};
static_assert(sizeof(RingMaps) <= sizeof(TensorMapSet), "tensor map storage");

struct RingCoef {
  double p[2 * kRHalo + 1];  // band mode: p[delta + 16] = P[i][(i + delta) mod n]
};

template <bool kDense>
__global__ void __launch_bounds__(kRThreads, 1)
step_ring_kernel(const StepParams p, const __grid_constant__ RingMaps maps, const __grid_constant__ RingCoef coef,
                 const double* __restrict__ p_row) {
  using Plan = RingPlan<kDense>;
  constexpr int kSlots = Plan::kSlots, kEStages = Plan::kEStages;
  extern __shared__ unsigned char smem_unaligned[];
  // the swizzle pattern is a function of the shared-memory address: tiles start on 1 KiB boundaries
  unsigned char* smem_raw = smem_unaligned + ((1024u - (s_addr(smem_unaligned) & 1023u)) & 1023u);
  float* ring_mem = reinterpret_cast<float*>(smem_raw);                 // [slot][x chunk | y chunk]
  float* side_mem = ring_mem + kSlots * kSlotFloats;                    // [slab parity][x chunk 0 | y chunk 0]
  float* e_mem = side_mem + Plan::kSideFloats;                          // [stage][g | a | c]
  double* table = reinterpret_cast<double*>(e_mem + kEStages * kEStageFloats);   // dense mode: p(0 .. n-1)
  uint64_t* slot_full = reinterpret_cast<uint64_t*>(smem_raw + Plan::kCtrlOffset);
  uint64_t* side_full = slot_full + kMaxSlots;
  uint64_t* e_full = side_full + 2;
  uint64_t* e_empty = e_full + 4;
  uint64_t* out_ready = e_empty + 4;
  unsigned* landed = reinterpret_cast<unsigned*>(out_ready + 4);   // chunks (in loading order) that are in shared memory
  unsigned* side_landed = landed + 1;                              // slabs whose side copy is in shared memory
  unsigned* released = side_landed + 1;                            // [consumer warp]: tiles whose x, y it is done reading

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.n;
  const int NB = n / kRT;                                    // tiles (row blocks) per slab
  const int NC = n / kChunkRows;                             // chunks per ring
  const int CPS = kDense ? NC : NC + 1;                      // chunk loads per slab into the slot ring
  if (kDense)
    for (int e = tid; e < n; e += kRThreads) table[e] = p_row[e];
  if (tid == 0) {
    *landed = 0;
    *side_landed = 0;
    for (int w = 0; w < kRConsumerWarps; ++w) released[w] = 0;
    for (int s = 0; s < kSlots; ++s) bar_init(&slot_full[s], 1);
    for (int s = 0; s < 2; ++s) bar_init(&side_full[s], 1);
    for (int s = 0; s < kEStages; ++s) {
      bar_init(&e_full[s], 1);
      bar_init(&e_empty[s], 1);
      bar_init(&out_ready[s], kRGroupWarps);
    }
    fence_barrier_init();
  }
  fence_async_shared();
  __syncthreads();

  // this CTA takes slabs blockIdx.x, blockIdx.x + gridDim.x, ...
  // 32-bit bookkeeping throughout: the launcher admits d < 2^31, so slab, tile and chunk counts of a CTA fit easily,
  // and nothing in the per-tile paths divides by a run-time value
  const int my_slabs =
      blockIdx.x < p.num_slabs ? static_cast<int>((p.num_slabs - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;
  const int num_tiles = my_slabs * NB;
  const unsigned limit = p.spin_limit;

  if (warp == kLoadXYWarp) {
    // ---------------------------------------------------------------- x, y chunks, each loaded once
    if (lane == 0) {
      int confirmed = 0;  // tiles 0 .. confirmed - 1 are known to be done with their x, y
      bool ok = true;
      // waits until every consumer warp has released all tiles up to and including `tile`
      auto wait_released = [&](int tile) {
        if (tile < confirmed) return true;
        for (int g = 0; g < kRGroups; ++g) {
          if (tile < g) continue;
          const unsigned need = static_cast<unsigned>((tile - g) / kRGroups + 1);  // tiles of group g among 0 .. tile
          if (!counters_wait(&released[g * kRGroupWarps], kRGroupWarps, need, limit)) return false;
        }
        confirmed = tile + 1;
        return true;
      };
      int Q = 0;
      // self test: the loads stop once the chunks of about `stall_after` tiles have gone out
      const long long stall_at = p.stall_after >= 0 ? 2 * p.stall_after : -1;
      for (int sl = 0; sl < my_slabs && ok; ++sl) {
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(sl) * gridDim.x) * 2);
        if (!kDense) {
          // second copy of chunk 0 for the slab's last tile; the buffer was last read by the last tile two slabs back
          if (sl >= 2) ok = wait_released((sl - 1) * NB - 1);
          if (!ok) break;
          if (stall_at >= 0 && Q >= stall_at) return;
          float* sd = side_mem + static_cast<size_t>(sl & 1) * kSlotFloats;
          bar_expect_tx(&side_full[sl & 1], kSlotFloats * 4);
          rows_load(sd, &maps.x, half, 0, &side_full[sl & 1]);
          rows_load(sd + kChunkFloats, &maps.y, half, 0, &side_full[sl & 1]);
        }
        for (int q = 0; q < CPS && ok; ++q, ++Q) {
          if (stall_at >= 0 && Q >= stall_at) return;
          const int slot = static_cast<int>(Q % kSlots);
          if (Q >= kSlots) {
            // the chunk that held this slot: position q_old of slab sl_old; its last reader is tile q_old / 2 of
            // that slab (dense mode: the slab's last tile)
            const int Qo = Q - kSlots, slo = Qo / CPS;
            const int qo = Qo - slo * CPS;
            const int last_reader = kDense ? NB - 1 : (qo / 2 < NB ? qo / 2 : NB - 1);
            ok = wait_released(slo * NB + last_reader);
            if (!ok) break;
          }
          const int chunk = kDense ? q : (q + NC - 1) % NC;  // band mode starts with the chunk before row 0
          float* st = ring_mem + static_cast<size_t>(slot) * kSlotFloats;
          bar_expect_tx(&slot_full[slot], kSlotFloats * 4);
          rows_load(st, &maps.x, half, chunk * kChunkRows, &slot_full[slot]);
          rows_load(st + kChunkFloats, &maps.y, half, chunk * kChunkRows, &slot_full[slot]);
        }
      }
      if (!ok) atomicExch(p.status, 1);
      // copies still in flight land in this CTA's shared memory: wait for them (bounded) before leaving
      for (int back = 1; back <= kSlots && back <= Q; ++back) {
        const int q = Q - back;
        bar_wait(&slot_full[q % kSlots], (q / kSlots) & 1, limit);
      }
    }
    return;
  }
  if (warp == kRSignalWarp) {
    // ---------------------------------------------------------------- publishes what has landed, strictly in order
    if (lane == 0) {
      int Q = 0;
      for (int sl = 0; sl < my_slabs; ++sl) {
        if (!kDense) {
          if (!bar_wait(&side_full[sl & 1], (sl >> 1) & 1, limit)) {
            atomicExch(p.status, 1);
            return;
          }
          count_publish(side_landed, static_cast<unsigned>(sl + 1));
        }
        for (int q = 0; q < CPS; ++q, ++Q) {
          if (!bar_wait(&slot_full[Q % kSlots], (Q / kSlots) & 1, limit)) {
            atomicExch(p.status, 1);
            return;
          }
          count_publish(landed, static_cast<unsigned>(Q + 1));
        }
      }
    }
    return;
  }
  if (warp == kLoadEWarp) {
    // ---------------------------------------------------------------- g, a, c of each tile
    if (lane == 0) {
      int T = 0, sl = 0, b = 0;
      bool ok = true;
      for (; T < num_tiles; ++T) {
        if (p.stall_after >= 0 && T >= p.stall_after) return;
        const int se = T % kEStages;
        if (T >= kEStages) ok = bar_wait(&e_empty[se], ((T / kEStages) - 1) & 1, limit);
        if (!ok) break;
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(sl) * gridDim.x) * 2);
        float* te = e_mem + static_cast<size_t>(se) * kEStageFloats;
        bar_expect_tx(&e_full[se], kEStageFloats * 4);
        rows_load(te, &maps.g, half, b * kRT, &e_full[se]);
        rows_load(te + kEArrayFloats, &maps.a, half, b * kRT, &e_full[se]);
        rows_load(te + 2 * kEArrayFloats, &maps.c, half, b * kRT, &e_full[se]);
        if (++b == NB) {
          b = 0;
          ++sl;
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (int back = 1; back <= kEStages && back <= T; ++back) {
          const int q = T - back;
          bar_wait(&e_full[q % kEStages], (q / kEStages) & 1, limit);
        }
      }
    }
    return;
  }
  if (warp == kRStoreWarp) {
    if (lane == 0) {
      for (int T = 0, sl = 0, b = 0; T < num_tiles; ++T, b = (b + 1 == NB ? 0 : b + 1), sl += (b == 0 ? 1 : 0)) {
        const int se = T % kEStages;
        if (!bar_wait(&out_ready[se], (T / kEStages) & 1, limit)) {
          atomicExch(p.status, 1);
          break;
        }
        // rows 0..15 are read once more, into the side buffer: nothing of the slab goes out before that copy is in
        if (!kDense && b == 0 && !count_wait(side_landed, static_cast<unsigned>(sl + 1), limit)) {
          atomicExch(p.status, 1);
          break;
        }
        const float* te = e_mem + static_cast<size_t>(se) * kEStageFloats;  // now [g' | x' | y']
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(sl) * gridDim.x) * 2);
        rows_store(&maps.g, half, b * kRT, te);
        rows_store(&maps.xs, half, b * kRT, te + kEArrayFloats);
        if (p.mode != kModeDpsgd) rows_store(&maps.ys, half, b * kRT, te + 2 * kEArrayFloats);
        store_commit();
        store_wait_read();  // the stage may be refilled now
        bar_arrive(&e_empty[se]);
      }
      store_wait_all();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int kq = lane & 3, crow = lane >> 2;  // crow: this lane's coordinate within the warp's 8
  const int group = warp / kRGroupWarps, ctile = warp % kRGroupWarps;
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool noisy = p.sigma != 0.0;
  const bool dpsgd = p.mode == kModeDpsgd;  // one contraction, x' = P x - alpha g, no tracker
  // Float offset of this lane's element in local row kq of a [row][half][32] array; the rows it touches are
  // kq + 4 i, 256 floats apart.  The 16-byte chunk index is XORed with the low three bits of the 128-byte row
  // number 2 * row + half (the tensor maps' swizzle), which for rows kq + 4 i is always 2 kq + half.
  const int half_of_tile = ctile >> 2;
  const int chunk16 = 2 * (ctile & 3) + (crow >> 2);
  const int off = kq * kRS + half_of_tile * kRHalf + (((chunk16 ^ ((2 * kq + half_of_tile) & 7)) << 2) | (crow & 3));
  // band mode: B fragment of window step u = s - 2t: entry [k = kq][column crow] = p(delta), delta = input row -
  // output row = (4 u + kq) - 16 - (crow / 2 + 4 (crow & 1)); the same for every tile
  double bfrag[kDense ? 1 : kBandSteps];
  const int out_pos = (crow >> 1) + 4 * (crow & 1);  // tile row (within its 8-row block) that MMA column `crow` stands for
  if (!kDense) {
#pragma unroll
    for (int u = 0; u < kBandSteps; ++u) {
      const int delta = 4 * u + kq - kRHalo - out_pos;
      bfrag[u] = (delta >= -kRHalo && delta <= kRHalo) ? coef.p[delta + kRHalo] : 0.0;
    }
  }

  unsigned done = 0;  // tiles this group has finished
  // tile T = row block b of this CTA's slab number sl; Qbase = loading position of the slab's first chunk
  int sl = group / NB, b = group % NB;
  for (int T = group; T < num_tiles; T += kRGroups, ++done, b += kRGroups) {
    if (b >= NB) {  // NB >= 2: at most one slab further
      b -= NB;
      ++sl;
    }
    const int Qbase = sl * CPS;
    const int se = T % kEStages;
    const long long j = (blockIdx.x + static_cast<long long>(sl) * gridDim.x) * kRS + ctile * 8 + crow;  // this lane's coordinate
    // The normals of this tile need no data: they are drawn first, while the tile's chunks may still be on their way.
    // This lane's workers 32 b + kq + 4 m are position kq of the Philox quads 8 b + m, shared by the four
    // lanes of a coordinate: each draws two of the eight quads and a 4 x 4 transpose hands everybody its position
    float xi[8];
    if (noisy) {
      const unsigned long long jn = static_cast<unsigned long long>(p.coord_offset + j);
#pragma unroll
      for (int hq = 0; hq < 2; ++hq) {
        float v[4];
        normal_quad(p.seed_lo, p.seed_hi, jn, static_cast<uint32_t>(8 * b + 4 * hq + kq), p.t_noise, v);
        transpose_quad(v, kq);  // v[i]: position kq of quad 8 b + 4 hq + i
#pragma unroll
        for (int i = 0; i < 4; ++i) xi[4 * hq + i] = v[i];
      }
    } else {
#pragma unroll
      for (int m = 0; m < 8; ++m) xi[m] = 0.f;
    }
    // ---- the window: band mode chunks at loading positions 2b .. 2b+3 (the last one of the slab's last tile is
    // the side copy of chunk 0); dense mode all NC chunks of the slab
    const int q_first = kDense ? 0 : 2 * b;
    const int q_last = kDense ? NC - 1 : (2 * b + 3 < CPS ? 2 * b + 3 : CPS - 1);
    const bool wraps = !kDense && 2 * b + 3 >= CPS;
    bool ok = true;
    if (lane == 0) {
      ok = count_wait_relaxed(landed, static_cast<unsigned>(Qbase + q_last + 1), limit);
      if (ok && wraps) ok = count_wait_relaxed(side_landed, static_cast<unsigned>(sl + 1), limit);
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    // The phases are known to be complete: a non-blocking test per barrier (one lane each, all at once) orders the
    // warp after the copies; should a test ever fail, the bounded wait takes over.
    if (ok) {
      const int q = q_first + lane;
      if (q <= q_last) {
        uint64_t* bar = &slot_full[(Qbase + q) % kSlots];
        const unsigned parity = ((Qbase + q) / kSlots) & 1;
        if (!bar_test(bar, parity)) ok = bar_wait(bar, parity, limit);
      }
      if (wraps && lane == 31 && !bar_test(&side_full[sl & 1], (sl >> 1) & 1))
        ok = bar_wait(&side_full[sl & 1], (sl >> 1) & 1, limit);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    double cx[4][2], cy[4][2];
#pragma unroll
    for (int t = 0; t < 4; ++t) cx[t][0] = cx[t][1] = cy[t][0] = cy[t][1] = 0.0;
    if (!kDense) {
      // cx accumulates P x, cy accumulates P y; the model update x' = x~ - alpha y~ happens in the tail
#pragma unroll
      for (int w = 0; w < 4; ++w) {  // window chunk w: rows 32 b - 16 + 16 w ..; the slab's last tile ends in the side copy
        const int q = 2 * b + w;
        const float* ch = (q < CPS) ? ring_mem + static_cast<size_t>((Qbase + q) % kSlots) * kSlotFloats
                                    : side_mem + static_cast<size_t>(sl & 1) * kSlotFloats;
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // k-step s = 4 w + i: window rows 4 s + kq
          const int s = 4 * w + i;
          const double zx = static_cast<double>(ch[off + i * 256]);
          const double zy = static_cast<double>(ch[kChunkFloats + off + i * 256]);
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const int u = s - 2 * t;  // compile-time after unrolling: only the band's blocks are issued
            if (u >= 0 && u < kBandSteps) {
              if (!dpsgd) dmma(cy[t], zy, bfrag[u]);
              dmma(cx[t], zx, bfrag[u]);
            }
          }
        }
      }
    } else {
      for (int c = 0; c < NC; ++c) {  // every chunk of the ring
        const float* ch = ring_mem + static_cast<size_t>((Qbase + c) % kSlots) * kSlotFloats;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int in_row = c * kChunkRows + 4 * i + kq;
          const float xv = ch[off + i * 256], yv = ch[kChunkFloats + off + i * 256];
          const double by = static_cast<double>(yv), bx = static_cast<double>(xv);
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            int delta = in_row - (b * kRT + 8 * t + out_pos);  // P[out][in] = p((in - out) mod n)
            delta += delta < 0 ? n : 0;
            const double bv = table[delta];
            if (!dpsgd) dmma(cy[t], by, bv);
            dmma(cx[t], bx, bv);
          }
        }
      }
    }
    // gradient point of Algorithm 2 as printed: this lane's own rows of the old model, still in their chunks
    float x_old[8];
    if (p.grad_at_start) {
      const int q_own = kDense ? 2 * b : 2 * b + 1;
#pragma unroll
      for (int m = 0; m < 8; ++m)
        x_old[m] = ring_mem[static_cast<size_t>((Qbase + q_own + (m >> 2)) % kSlots) * kSlotFloats + off + (m & 3) * 256];
    }
    __syncwarp();
    if (lane == 0) count_publish(&released[warp], done + 1);  // this warp is done with the tile's x, y chunks

    // ---- g, a, c: the stage serves this group only (even stage count), so its phases are waited for in order
    if (lane == 0) ok = bar_wait(&e_full[se], (T / kEStages) & 1, limit);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    float* sg = e_mem + static_cast<size_t>(se) * kEStageFloats;
    float* sa = sg + kEArrayFloats;
    float* sc = sa + kEArrayFloats;
    // All inputs of the tail are read before anything is written back: the stores below go to the same arrays, and
    // loads that had to stay behind them would run one element at a time.
    float gv[8], av[8], cv[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      gv[m] = sg[off + m * 256];
      av[m] = sa[off + m * 256];
      cv[m] = sc[off + m * 256];
    }
    // ---- element-wise tail on the lane's own eight elements (tile rows kq + 4 m); results replace the inputs
    float xo[8], yo[8], go[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int t = m >> 1, e = m & 1;
      // model update: x' = x~ - alpha y~ (D-PSGD: x~ - alpha g)
      xo[m] = static_cast<float>(fma(-alpha, dpsgd ? static_cast<double>(gv[m]) : cy[t][e], cx[t][e]));
      const float x_at = p.grad_at_start ? x_old[m] : xo[m];  // gradient point: new model, or the one the step started from
      go[m] = fmaf(av[m], x_at - cv[m], sigma * xi[m]);
      yo[m] = static_cast<float>((cy[t][e] - static_cast<double>(gv[m])) + static_cast<double>(go[m]));  // fold
    }
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int o = off + m * 256;
      sg[o] = go[m];
      sa[o] = xo[m];
      sc[o] = yo[m];
      if (p.y_obs != nullptr && !dpsgd)  // optional observer: the gossiped tracker, stored directly
        p.y_obs[static_cast<long long>(b * kRT + kq + 4 * m) * p.ld + j] = static_cast<float>(cy[m >> 1][m & 1]);
    }
    fence_async_shared();  // results visible to the TMA stores
    __syncwarp();
    if (lane == 0) bar_arrive(&out_ready[se]);
  }
}

}  // namespace

bool ring_variant_available(int n, int half_band) {
  return n % kRT == 0 && n >= 64 && n <= kMaxWorkers && half_band <= kRHalo && encode_tiled_fn() != nullptr;
}

bool ring_dense_available(int n) { return n % kRT == 0 && n >= 64 && n <= 256 && encode_tiled_fn() != nullptr; }

// p.d must be a multiple of 64 (the caller hands the remaining columns to the generic kernel).
bool build_maps_ring(const StepParams& p, TensorMapSet* out) {
  RingMaps& m = *reinterpret_cast<RingMaps*>(out->bytes);
  const float* y = p.mode == kModeDpsgd ? p.x : p.y;  // D-PSGD has no tracker: those maps are never used
  return make_half_map(&m.x, p.x, p.n, p.d, p.ld, kChunkRows) && make_half_map(&m.y, y, p.n, p.d, p.ld, kChunkRows) &&
         make_half_map(&m.g, p.g, p.n, p.d, p.ld, kRT) && make_half_map(&m.a, p.a, p.n, p.d, p.ld, kRT) &&
         make_half_map(&m.c, p.c, p.n, p.d, p.ld, kRT) && make_half_map(&m.xs, p.x, p.n, p.d, p.ld, kRT) &&
         make_half_map(&m.ys, y, p.n, p.d, p.ld, kRT);
}

// band != nullptr: band mode, the 33 entries p(delta) at index delta + 16.  band == nullptr: dense mode, p_row is a
// device pointer to the n entries p(0 .. n-1) of the first row of the circulant P.
int launch_step_ring(StepParams p, const TensorMapSet& maps, const double* band, const double* p_row, int sm_count,
                     cudaStream_t stream) {
  if (p.mode == kModeExternal || p.d % kRS != 0) return static_cast<int>(cudaErrorInvalidValue);
  RingCoef coef{};
  const bool dense = band == nullptr;
  if (!dense)
    for (int k = 0; k < 2 * kRHalo + 1; ++k) coef.p[k] = band[k];
  p.S = kRS;
  p.num_slabs = p.d / kRS;
  auto kernel = dense ? step_ring_kernel<true> : step_ring_kernel<false>;
  const size_t smem = dense ? RingPlan<true>::kSmemBytes : RingPlan<false>::kSmemBytes;
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), kRThreads, smem, stream>>>(p, *reinterpret_cast<const RingMaps*>(maps.bytes), coef,
                                                                   p_row);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
