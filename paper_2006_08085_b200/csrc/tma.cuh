// Host-side helpers for the TMA tensor maps over the [n][ld] float32 state arrays.
#ifndef DETAG_TMA_CUH
#define DETAG_TMA_CUH

#include <cuda.h>
#include <cuda_runtime.h>

namespace detag {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// [n rows][d columns] float32 with row pitch ld, tiles of box_rows x box_cols, zero fill outside.
inline bool make_map(CUtensorMap* m, const float* base, int n, long long d, long long ld, int box_rows, int box_cols) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(n)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * sizeof(float)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// View of an [n][ld] array as {32 coordinates, d / 32 halves at a stride of 128 bytes, n rows} with boxes of
// {32, 2, box_rows} and the 128-byte swizzle: a box is a slab of 64 coordinates whose rows are fetched as contiguous
// 256-byte pieces.  Only whole 32-coordinate halves are in the view; rows and halves outside read as zero and are
// not written.
inline bool make_half_map(CUtensorMap* m, const float* base, int n, long long d, long long ld, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  constexpr int kHalf = 32;
  const long long halves = d / kHalf;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(kHalf), static_cast<cuuint64_t>(halves > 0 ? halves : 1),
                              static_cast<cuuint64_t>(n)};
  const cuuint64_t strides[2] = {kHalf * sizeof(float), static_cast<cuuint64_t>(ld) * sizeof(float)};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(kHalf), 2, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace detag
#endif  // DETAG_TMA_CUH
