// Host-side construction of TMA tensor maps.  The driver entry point is looked up through the
// runtime so that the library does not link against libcuda (it must load on machines without
// a GPU, where only the planner is used).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace mebptt {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 2-D row-major tensor [rows][cols] of 2- or 4-byte elements, 128-byte swizzle, zero fill
// outside.  box_cols * elem_bytes must be 128.  Returns false on failure.
inline bool make_tmap_2d(CUtensorMap* map, const void* base, int elem_bytes, uint64_t cols, uint64_t rows,
                         uint64_t row_stride_bytes, uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride_bytes & 15)) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstr[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  return fn(map, dt, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same 2-D array of 2-byte elements seen as [cols / 64][rows][64]: coordinate 0 runs inside a
// block of 64 columns (128 bytes), coordinate 1 over the rows, coordinate 2 over the blocks.  One
// box of (64, box_rows, box_blocks) then lands in shared memory as box_blocks consecutive tiles
// of [box_rows][128 B], 128-byte swizzled -- the layout a K-major MMA operand wants -- with a
// single copy instruction.  cols must be a multiple of 64 (a partial last block would read on into
// the next row instead of being zero-filled).
inline bool make_tmap_blocks64(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows,
                               uint64_t row_stride_bytes, uint32_t box_rows, uint32_t box_blocks) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || cols % 64 != 0 || box_blocks > 256 || box_rows > 256) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride_bytes & 15)) return false;
  cuuint64_t gdim[3] = {64, rows, cols / 64};
  cuuint64_t gstr[2] = {row_stride_bytes, 128};
  cuuint32_t box[3] = {64, box_rows, box_blocks};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace mebptt
