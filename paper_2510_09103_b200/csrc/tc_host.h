// Host helpers of the tensor-core path: building TMA tensor maps without linking libcuda.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adapm {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's cuTensorMapEncodeTiled, looked up through the runtime (nullptr if unavailable).
inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// Tensor map of a row-major bf16 matrix [rows, cols] with row pitch `pitch_elems`, read in boxes of
// 64 columns x box_rows rows with the 128-byte swizzle; out-of-range elements read as zero.
// Requires: base 16-byte aligned, pitch a multiple of 8 elements.  Returns false on failure.
inline bool encode_bf16_matrix(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                               uint64_t pitch_elems, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix seen as (64 columns, rows, chunks of 64 columns): one box of 64 x box_rows x chunks
// brings `box_rows` rows of 64 * chunks consecutive columns into shared memory chunk after chunk.
// 64 * chunks may exceed the row pitch: the surplus columns are the start of the next row (the last
// rows read up to 128 bytes past the matrix, which the caller's allocation must cover) and are never
// used as operand columns.  Rows out of range read as zero.
inline bool encode_bf16_chunked(CUtensorMap* out, const void* base, uint64_t rows, uint64_t pitch_elems,
                                uint32_t chunks, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {64, rows, chunks};
  const cuuint64_t strides[2] = {pitch_elems * 2, 128};
  const cuuint32_t box[3] = {64, box_rows, chunks};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of a row-major matrix [rows, cols] of 2- or 4-byte elements (row pitch = cols), moved in
// boxes of 32 columns x 128 rows: 128-byte swizzle for fp32 (128-byte box rows), 64-byte swizzle
// for bf16 (64-byte box rows).  Loads read zero out of range, stores skip what is out of range.
// Requires: base 16-byte aligned, cols * element size a multiple of 16 bytes.
inline bool encode_panel32(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, bool is_f32) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * (is_f32 ? 4u : 2u)};
  const cuuint32_t box[2] = {32, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, is_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            is_f32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace adapm
