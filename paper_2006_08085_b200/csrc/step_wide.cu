// DeTAG step with the dense polynomial for 64 < n <= 128 workers (any gossip matrix) on the FP64 tensor path.
//
// AG_K(z) = P z with P = P_K(M) built by the host in float64 from the matrix form of Algorithm 3; the step is then
// two dense contractions per slab (P times the model rows, P times the tracker rows) and Algorithm 2's element-wise
// updates.  At these sizes P no longer fits beside the slabs in shared memory (128 x 128 doubles are 128 KB), so it
// lives in REGISTERS, spread over the warps: warp b owns the 8 output workers 8b .. 8b+7 and keeps the whole
// 8 x n strip of P for them as the B fragments of its MMAs (one double per lane and 4-worker input block, at most 32).
//
// Mapping onto mma m8n8k4 (float64): the eight coordinates of a tile are the M index, the input worker the
// contraction index (k-step s covers workers 4s .. 4s+3) and the warp's output workers the N index, with the columns
// permuted so that column 2 kq + e stands for worker 8b + kq + 4e:
//     D[coord][w'] = sum_w Z[coord][w] P[w'][w] .
// A lane (coord = lane / 4, kq = lane % 4) therefore supplies the elements of workers kq + 4s of its coordinate and
// receives the results of workers 8b + kq, 8b + kq + 4: rows with the same residue mod 4, which in the swizzled tile
// [row][half][32] (one {32, 2, rows} TMA box per array and slab, rows fetched as contiguous 256-byte pieces) gives
// conflict-free accesses throughout.  Every warp reads all rows of the x, y tiles (each operand element is widened
// once per warp that uses it - the price of keeping P in registers); the tail of the step is lane-local and each
// lane writes g', x', y' over the g, a, c elements it read, so the output needs no tile of its own.
//
// A warp works through the slab two 8-coordinate tiles at a time: four independent accumulator chains (model and
// tracker of both tiles) of ceil(n / 4) MMAs each, then the tail of those 2 x 2 x 8 elements.  The four lanes of a
// coordinate share the Philox calls of the tail: the two tiles' two 4-worker quads make four calls, one per lane,
// handed round by a 4 x 4 transpose.  The FP64 MMA rate of each of the SM's four warp schedulers is what bounds the
// kernel (2 n multiply-adds per element against 32 bytes), so the blocks are dealt to the schedulers evenly: see
// wide_consumers().
//
// Roles of the persistent CTA (one per SM): ceil(n / 8) or a few more consumer warps; a loader for x, y (two stages, handed back when
// every warp has finished the slab's contractions); a loader for g, a, c (two stages while ten tiles fit in shared
// memory, n <= 88, else one); a storer that sends a finished stage out with three TMA stores.  Every wait is bounded.
//
// The kernel takes whole 32-coordinate halves (the boxes' granularity); the caller hands the last d % 32 columns to
// the generic kernel.
#include <cuda.h>
#include <cuda_runtime.h>

#include "detag_internal.h"
#include "noise.cuh"
#include "pipeline.cuh"
#include "tma.cuh"

namespace detag {

namespace {

constexpr int kWS = 64;              // coordinates per slab
constexpr int kWMaxRows = 128;       // n limit
constexpr int kWXYStages = 2;
constexpr int kWPairs = kWS / 16;    // pairs of 8-coordinate tiles per slab
constexpr size_t kWSmemLimit = 232448;

struct WideMaps {
  CUtensorMap x, y, g, a, c;  // boxes {32 coordinates, 2 halves, n rounded up to 8 rows}: loads and stores
};
static_assert(sizeof(WideMaps) <= sizeof(TensorMapSet), "tensor map storage");

// Consumer warps for B output blocks.  A warp scheduler's share of the MMAs is what bounds the kernel, and warps go to
// the four schedulers round robin: with B = 4m + 1 blocks the last block is shared by four warps (one pair of tiles
// each), with B = 4m + 2 the last two blocks by two warps each (two pairs each), so that every scheduler carries the
// same load; B = 4m + 3 is left as it is (one scheduler a quarter block short).
__host__ __device__ constexpr int wide_consumers(int blocks) { return blocks % 4 == 1 ? blocks + 3 : blocks % 4 == 2 ? blocks + 2 : blocks; }

struct WidePlan {
  int rows;       // n rounded up to a multiple of 8
  int warps;      // consumer warps
  int e_stages;   // 1 or 2
  int tile_floats;
  size_t ctrl_offset, smem_bytes;
};

inline WidePlan wide_plan(int n) {
  WidePlan w{};
  w.rows = (n + 7) / 8 * 8;
  w.warps = wide_consumers(w.rows / 8);
  w.tile_floats = w.rows * kWS;
  const size_t tile = static_cast<size_t>(w.tile_floats) * 4;
  w.e_stages = (2 * kWXYStages + 6) * tile + 128 + 1024 <= kWSmemLimit ? 2 : 1;
  w.ctrl_offset = (2 * kWXYStages + 3 * w.e_stages) * tile;
  w.smem_bytes = w.ctrl_offset + 128 + 1024;  // + barriers, + slack to align the tiles to 1 KiB
  return w;
}

// kKs: k-steps issued, ceil(n / 4) rounded up to an even number (the B fragments beyond n are zero).
template <int kKs>
__global__ void __launch_bounds__((wide_consumers(kKs / 2) + 3) * 32, 1)
step_wide_kernel(const StepParams p, const __grid_constant__ WideMaps maps, const double* __restrict__ p_frag,
                 const int rows, const int e_stages) {
  extern __shared__ unsigned char smem_unaligned[];
  // the swizzle pattern is a function of the shared-memory address: tiles start on 1 KiB boundaries
  unsigned char* smem_raw = smem_unaligned + ((1024u - (s_addr(smem_unaligned) & 1023u)) & 1023u);
  const int tile_floats = rows * kWS;
  constexpr int kBlocks = kKs / 2;                      // 8-worker output blocks
  constexpr int consumers = wide_consumers(kBlocks);
  // Tail of a pair of tiles in one instruction stream with the next pair's contractions: pays only at the smallest
  // size (measured, d = 2 M: 1.68 against 1.79 ms at n = 72; 2.09 against 2.06 at n = 80, 2.99 against 2.96 at n = 96),
  // and needs the 128 registers per thread that 16 warps leave.
  constexpr bool kPipelined = kKs <= 18;
  float* xy_mem = reinterpret_cast<float*>(smem_raw);            // [stage][x | y]
  float* e_mem = xy_mem + kWXYStages * 2 * tile_floats;          // [stage][g | a | c]
  uint64_t* xy_full = reinterpret_cast<uint64_t*>(e_mem + e_stages * 3 * tile_floats);
  uint64_t* xy_empty = xy_full + kWXYStages;
  uint64_t* e_full = xy_empty + kWXYStages;
  uint64_t* e_empty = e_full + 2;
  uint64_t* out_ready = e_empty + 2;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < kWXYStages; ++s) {
      bar_init(&xy_full[s], 1);
      bar_init(&xy_empty[s], consumers);
    }
    for (int s = 0; s < 2; ++s) {
      bar_init(&e_full[s], 1);
      bar_init(&e_empty[s], 1);
      bar_init(&out_ready[s], consumers);
    }
    fence_barrier_init();
  }
  fence_async_shared();
  __syncthreads();

  // this CTA takes slabs blockIdx.x, blockIdx.x + gridDim.x, ...; k counts them
  const int my_slabs =
      blockIdx.x < p.num_slabs ? static_cast<int>((p.num_slabs - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;
  const unsigned limit = p.spin_limit;
  const unsigned xy_bytes = 2u * tile_floats * 4u, e_bytes = 3u * tile_floats * 4u;

  if (warp == consumers) {
    // ---------------------------------------------------------------- x, y loader
    if (lane == 0) {
      int k = 0;
      bool ok = true;
      for (; k < my_slabs; ++k) {
        if (p.stall_after >= 0 && k >= p.stall_after) return;  // self test: the loads stop, every waiter times out
        const int sx = k % kWXYStages;
        if (k >= kWXYStages) ok = bar_wait(&xy_empty[sx], ((k / kWXYStages) - 1) & 1, limit);
        if (!ok) break;
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(k) * gridDim.x) * 2);
        float* tx = xy_mem + static_cast<size_t>(sx) * 2 * tile_floats;
        bar_expect_tx(&xy_full[sx], xy_bytes);
        rows_load(tx, &maps.x, half, 0, &xy_full[sx]);
        rows_load(tx + tile_floats, &maps.y, half, 0, &xy_full[sx]);
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (int back = 1; back <= kWXYStages && back <= k; ++back) {  // drain copies still in flight (bounded)
          const int q = k - back;
          bar_wait(&xy_full[q % kWXYStages], (q / kWXYStages) & 1, limit);
        }
      }
    }
    return;
  }
  if (warp == consumers + 1) {
    // ---------------------------------------------------------------- g, a, c loader
    if (lane == 0) {
      int k = 0;
      bool ok = true;
      for (; k < my_slabs; ++k) {
        if (p.stall_after >= 0 && k >= p.stall_after) return;
        const int se = k % e_stages;
        if (k >= e_stages) ok = bar_wait(&e_empty[se], ((k / e_stages) - 1) & 1, limit);
        if (!ok) break;
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(k) * gridDim.x) * 2);
        float* te = e_mem + static_cast<size_t>(se) * 3 * tile_floats;
        bar_expect_tx(&e_full[se], e_bytes);
        rows_load(te, &maps.g, half, 0, &e_full[se]);
        rows_load(te + tile_floats, &maps.a, half, 0, &e_full[se]);
        rows_load(te + 2 * tile_floats, &maps.c, half, 0, &e_full[se]);
      }
      if (!ok) {
        atomicExch(p.status, 1);
        for (int back = 1; back <= e_stages && back <= k; ++back) {
          const int q = k - back;
          bar_wait(&e_full[q % e_stages], (q / e_stages) & 1, limit);
        }
      }
    }
    return;
  }
  if (warp == consumers + 2) {
    // ---------------------------------------------------------------- storer
    if (lane == 0) {
      for (int k = 0; k < my_slabs; ++k) {
        const int se = k % e_stages;
        if (!bar_wait(&out_ready[se], (k / e_stages) & 1, limit)) {
          atomicExch(p.status, 1);
          break;
        }
        const float* te = e_mem + static_cast<size_t>(se) * 3 * tile_floats;  // now [g' | x' | y']
        const int half = static_cast<int>((blockIdx.x + static_cast<long long>(k) * gridDim.x) * 2);
        rows_store(&maps.g, half, 0, te);
        rows_store(&maps.x, half, 0, te + tile_floats);
        rows_store(&maps.y, half, 0, te + 2 * tile_floats);
        store_commit();
        store_wait_read();  // the stage may be refilled now
        bar_arrive(&e_empty[se]);
      }
      store_wait_all();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warp: output workers 8 block .. 8 block + 7
  // for num_pairs of the slab's four pairs of tiles, from first_pair on
  int block = warp, first_pair = 0, num_pairs = kWPairs;
  if (kBlocks % 4 == 1 && warp >= kBlocks - 1) {
    block = kBlocks - 1;
    first_pair = warp - (kBlocks - 1);
    num_pairs = 1;
  } else if (kBlocks % 4 == 2 && warp >= kBlocks - 2) {
    block = kBlocks - 2 + ((warp - (kBlocks - 2)) >> 1);
    first_pair = 2 * ((warp - (kBlocks - 2)) & 1);
    num_pairs = 2;
  }
  const int kq = lane & 3, crow = lane >> 2;  // crow: this lane's coordinate within an 8-coordinate tile
  double bf[kKs];                             // this warp's strip of P in fragment order
#pragma unroll
  for (int s = 0; s < kKs; ++s) bf[s] = p_frag[(static_cast<size_t>(block) * 32 + s) * 32 + lane];
  const double alpha = p.alpha;
  const float sigma = static_cast<float>(p.sigma);
  const bool at_start = p.grad_at_start != 0;
  const uint32_t quad = 2u * static_cast<uint32_t>(block) + (kq & 1);  // the Philox quad this lane draws for its coordinate group
  // Float offset, inside an array's tile, of this lane's element of row kq in 8-coordinate tile o: tile = [row][half][32],
  // the 16-byte chunk index XORed with the low three bits of the 128-byte row number 2 row + half (the tensor maps'
  // swizzle), which is 2 kq + half for every row kq + 4 m.  Row kq + 4 m lies m * 256 floats further.
  auto tile_off = [&](int o) {
    const int half = o >> 2, chunk = 2 * (o & 3) + (crow >> 2);
    return kq * kWS + half * 32 + (((chunk ^ ((2 * kq + half) & 7)) << 2) | (crow & 3));
  };

  for (int k = 0; k < my_slabs; ++k) {
    const int sx = k % kWXYStages, se = k % e_stages;
    bool ok = true;
    if (lane == 0) ok = bar_wait(&xy_full[sx], (k / kWXYStages) & 1, limit);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) atomicExch(p.status, 1);
      return;
    }
    const float* sxp = xy_mem + static_cast<size_t>(sx) * 2 * tile_floats;
    const float* syp = sxp + tile_floats;
    float* sg = e_mem + static_cast<size_t>(se) * 3 * tile_floats;
    float* sa = sg + tile_floats;
    float* sc = sa + tile_floats;
    const long long j0 = (blockIdx.x + static_cast<long long>(k) * gridDim.x) * kWS;
    // The four accumulator chains of a pair of tiles: model and tracker of both.
    auto contract = [&](int pair, double (&cx)[2][2], double (&cy)[2][2]) {
      const int off0 = tile_off(2 * pair), off1 = tile_off(2 * pair + 1);
      cx[0][0] = cx[0][1] = cx[1][0] = cx[1][1] = 0.0;
      cy[0][0] = cy[0][1] = cy[1][0] = cy[1][1] = 0.0;
#pragma unroll
      for (int s = 0; s < kKs; ++s) {
        const double ax0 = static_cast<double>(sxp[off0 + s * 256]), ay0 = static_cast<double>(syp[off0 + s * 256]);
        const double ax1 = static_cast<double>(sxp[off1 + s * 256]), ay1 = static_cast<double>(syp[off1 + s * 256]);
        dmma(cx[0], ax0, bf[s]);
        dmma(cy[0], ay0, bf[s]);
        dmma(cx[1], ax1, bf[s]);
        dmma(cy[1], ay1, bf[s]);
      }
    };
    // Normals of the pair's 2 tiles x 2 workers of this lane: lane kq draws quad 2 block + (kq & 1) at the coordinate of
    // tile (kq >> 1); the transpose hands lane kq position kq of all four, so that xi[i] belongs to worker
    // 8 block + 4 (i & 1) + kq in tile (i >> 1).
    auto draw = [&](int pair, float (&xi)[4]) {
      const unsigned long long jn = static_cast<unsigned long long>(p.coord_offset + j0 + pair * 16 + (kq >> 1) * 8 + crow);
      normal_quad(p.seed_lo, p.seed_hi, jn, quad, p.t_noise, xi);
      transpose_quad(xi, kq);
    };
    // Element-wise tail of the pair: model update, gradient, tracker fold; g', x', y' go over g, a, c.
    auto tail = [&](int pair, const double (&cx)[2][2], const double (&cy)[2][2], const float (&xi)[4]) {
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int off = tile_off(2 * pair + t) + block * 512;
        const long long j = j0 + pair * 16 + t * 8 + crow;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int o = off + e * 256;
          const double yt = cy[t][e];
          const float xo = static_cast<float>(fma(-alpha, yt, cx[t][e]));  // x' = x~ - alpha y~, rounded once
          const float x_at = at_start ? sxp[o] : xo;  // Algorithm 2 as printed: the gradient at the model the step started from
          const float gold = sg[o];
          const float go = fmaf(sa[o], x_at - sc[o], sigma * xi[2 * t + e]);
          const float yo = static_cast<float>((yt - static_cast<double>(gold)) + static_cast<double>(go));
          sg[o] = go;
          sa[o] = xo;
          sc[o] = yo;
          const int row = 8 * block + kq + 4 * e;
          if (p.y_obs != nullptr && row < p.n && j < p.d)  // optional observer: the gossiped tracker, stored directly
            p.y_obs[static_cast<long long>(row) * p.ld + j] = static_cast<float>(yt);
        }
      }
    };
    auto wait_e = [&]() {  // g, a, c are needed from the first tail on; their loads had the first contractions to arrive in
      bool got = true;
      if (lane == 0) got = bar_wait(&e_full[se], (k / e_stages) & 1, limit);
      return __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
    };

    // pairs of tiles of this slab that are this warp's: the slab has all four or (the last one, d a multiple of 32) two
    const int slab_pairs = p.d - j0 >= kWS ? kWPairs : kWPairs / 2;
    const int my_pairs = slab_pairs - first_pair < num_pairs ? slab_pairs - first_pair : num_pairs;
    double cx[2][2], cy[2][2];
    if (kPipelined && my_pairs == kWPairs) {
      // Software pipeline: the tail of a pair (a long dependent chain: Philox, Box-Muller, special-function unit)
      // shares straight-line code with the contractions of the next pair, whose MMAs fill its issue slots.
      contract(0, cx, cy);
      if (!wait_e()) {
        if (lane == 0) atomicExch(p.status, 1);
        return;
      }
#pragma unroll
      for (int pair = 1; pair <= kWPairs; ++pair) {
        float xi[4];
        draw(pair - 1, xi);
        double nx[2][2], ny[2][2];
        if (pair < kWPairs) contract(pair, nx, ny);
        tail(pair - 1, cx, cy, xi);
        if (pair < kWPairs) {
#pragma unroll
          for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              cx[t][e] = nx[t][e];
              cy[t][e] = ny[t][e];
            }
        }
      }
    } else {
      bool e_seen = false;
#pragma unroll 1
      for (int q = 0; q < my_pairs; ++q) {
        contract(first_pair + q, cx, cy);
        if (!e_seen) {
          e_seen = true;
          if (!wait_e()) {
            if (lane == 0) atomicExch(p.status, 1);
            return;
          }
        }
        float xi[4];
        draw(first_pair + q, xi);
        tail(first_pair + q, cx, cy, xi);
      }
      if (!e_seen && !wait_e()) {  // nothing of this slab is this warp's: keep the protocol
        if (lane == 0) atomicExch(p.status, 1);
        return;
      }
    }
    __syncwarp();
    if (lane == 0) bar_arrive(&xy_empty[sx]);  // the x, y stage can be refilled
    fence_async_shared();  // results visible to the TMA stores
    __syncwarp();
    if (lane == 0) bar_arrive(&out_ready[se]);
  }
}

typedef void (*WideKernel)(const StepParams, const WideMaps, const double*, int, int);

WideKernel pick_wide(int ks) {
  switch ((ks + 1) / 2 * 2) {
    case 18: return step_wide_kernel<18>;
    case 20: return step_wide_kernel<20>;
    case 22: return step_wide_kernel<22>;
    case 24: return step_wide_kernel<24>;
    case 26: return step_wide_kernel<26>;
    case 28: return step_wide_kernel<28>;
    case 30: return step_wide_kernel<30>;
    default: return step_wide_kernel<32>;
  }
}

}  // namespace

bool wide_variant_available(int n) { return n > 64 && n <= kWMaxRows && encode_tiled_fn() != nullptr; }

// The warp strips of P in fragment order: entry ((b * 32 + s) * 32 + lane) = P[8 b + pi(lane / 4)][4 s + lane % 4],
// pi(2 q + e) = q + 4 e, zero outside the matrix.  16 x 32 x 32 doubles.
void wide_fragments(int n, const std::vector<double>& poly, std::vector<double>& frag) {
  frag.assign(static_cast<size_t>(16) * 32 * 32, 0.0);
  for (int b = 0; b < (n + 7) / 8; ++b)
    for (int s = 0; s < (n + 3) / 4; ++s)
      for (int lane = 0; lane < 32; ++lane) {
        const int nn = lane / 4, out = 8 * b + (nn >> 1) + 4 * (nn & 1), in = 4 * s + lane % 4;
        if (out < n && in < n) frag[(static_cast<size_t>(b) * 32 + s) * 32 + lane] = poly[static_cast<size_t>(out) * n + in];
      }
}

// p.d must be a multiple of 32 (the caller hands the remaining columns to the generic kernel).
bool build_maps_wide(const StepParams& p, TensorMapSet* out) {
  WideMaps& m = *reinterpret_cast<WideMaps*>(out->bytes);
  const int rows = wide_plan(p.n).rows;
  return make_half_map(&m.x, p.x, p.n, p.d, p.ld, rows) && make_half_map(&m.y, p.y, p.n, p.d, p.ld, rows) &&
         make_half_map(&m.g, p.g, p.n, p.d, p.ld, rows) && make_half_map(&m.a, p.a, p.n, p.d, p.ld, rows) &&
         make_half_map(&m.c, p.c, p.n, p.d, p.ld, rows);
}

// p_frag: device pointer to the fragments of wide_fragments().
int launch_step_wide(StepParams p, const TensorMapSet& maps, const double* p_frag, int sm_count, cudaStream_t stream) {
  if (p.mode != kModeDetag || p.n <= 64 || p.n > kWMaxRows || (p.d & 31) != 0 || p_frag == nullptr)
    return static_cast<int>(cudaErrorInvalidValue);
  const WidePlan w = wide_plan(p.n);
  p.S = kWS;
  p.num_slabs = (p.d + kWS - 1) / kWS;
  const WideKernel kernel = pick_wide((p.n + 3) / 4);
  const int e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(w.smem_bytes));
  if (e != 0) return e;
  const long long grid = p.num_slabs < sm_count ? p.num_slabs : sm_count;
  if (grid <= 0) return 0;
  kernel<<<static_cast<unsigned>(grid), (w.warps + 3) * 32, w.smem_bytes, stream>>>(
      p, *reinterpret_cast<const WideMaps*>(maps.bytes), p_frag, w.rows, w.e_stages);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace detag
