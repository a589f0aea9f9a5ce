// Host-side construction of TMA tensor maps without linking libcuda: the driver's encode function
// is looked up through the CUDA runtime at first use.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace hc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// 2-D bf16 tensor [rows][row_elems] (row pitch = pitch_elems), box = 64 columns x box_rows rows,
// 128-byte swizzle, out-of-range elements read as zero.  Returns false on failure.
inline bool make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t row_elems, uint64_t rows,
                              uint64_t pitch_elems, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_tiled();
  if (!fn) return false;
  cuuint64_t dims[2] = {row_elems, rows};
  cuuint64_t strides[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Unswizzled maps over a [rows][row_elems] bf16 tensor for plain tile movement (cache split / append): the box
// lands in shared memory as consecutive rows of box_cols elements, i.e. in the order a per-head buffer stores them.
//  - 2-D: box = box_cols columns x box_rows rows.
//  - grid view (3-D): the rows are tokens of frames laid out as grid rows of grid_w tokens; coordinates are
//    (column, x, grid row), box = box_cols x box_x x box_y - one rectangle of the token grid, row after row.
// Out-of-range elements read as zero.
inline bool make_tmap_bf16_rows(CUtensorMap* out, const void* base, uint64_t row_elems, uint64_t rows, uint32_t box_cols,
                                uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_tiled();
  if (!fn || box_cols > 256 || box_rows > 256) return false;
  cuuint64_t dims[2] = {row_elems, rows};
  cuuint64_t strides[1] = {row_elems * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool make_tmap_bf16_grid(CUtensorMap* out, const void* base, uint64_t row_elems, uint64_t rows, uint64_t grid_w,
                                uint32_t box_cols, uint32_t box_x, uint32_t box_y) {
  EncodeTiledFn fn = get_encode_tiled();
  if (!fn || box_cols > 256 || box_x > 256 || box_y > 256 || rows % grid_w != 0) return false;
  cuuint64_t dims[3] = {row_elems, grid_w, rows / grid_w};
  cuuint64_t strides[2] = {row_elems * 2, grid_w * row_elems * 2};
  cuuint32_t box[3] = {box_cols, box_x, box_y};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace hc
