// Host-side helper: tensor map of a dense row-major bf16 matrix [rows, cols] for tiled TMA loads of boxes of 64
// columns (128 bytes, the swizzle span) by `box_rows` rows in the 128-byte swizzled shared-memory layout; elements
// outside the matrix arrive as zeros.  The driver's encoder is looked up through the runtime, so the library does not
// link against libcuda.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace laser {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// False when the encoder is missing or refuses the shape (cols must be a multiple of 64, base 16-byte aligned, row
// coordinates must fit 32 bits).
inline bool encode_bf16_rows_map(const void* base, unsigned long long rows, int cols, int box_rows, CUtensorMap* map) {
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn || cols % 64 || (reinterpret_cast<uintptr_t>(base) & 15) || rows == 0) return false;
  if (rows > 0x7fffff00ULL || box_rows < 1 || box_rows > 256) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows}, elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace laser
