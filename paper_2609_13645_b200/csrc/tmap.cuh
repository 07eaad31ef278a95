// Host-side helpers: TMA tensor maps for row-major bf16 matrices (encoder fetched from the driver at run time).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "common.cuh"

namespace fs {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 2-D map over a row-major matrix [rows, row_stride] of which `cols` columns are valid;
// box = 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
inline bool make_tmap_2d(CUtensorMap* tm, const bf16* base, uint64_t cols, uint64_t rows, uint64_t row_stride,
                         uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {row_stride * sizeof(bf16)};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D map with a box of 32 rows x box_cols columns (32: 64-byte rows under the 64-byte swizzle; 64: 128-byte rows under
// the 128-byte swizzle): the tiles a warp of a GEMM epilogue moves between its staging buffer and a row-major matrix.
inline bool make_tmap_2d_rows32(CUtensorMap* tm, const bf16* base, uint64_t cols, uint64_t rows, uint64_t row_stride,
                                uint32_t box_cols) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc || (box_cols != 32 && box_cols != 64)) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {row_stride * sizeof(bf16)};
  cuuint32_t box[2] = {box_cols, 32};
  cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D map over [batches][rows][row_stride] (row-major, batches contiguous): box = 64 columns x box_rows rows x 1 batch.
// Rows past the end of a batch read as zero instead of running into the next batch.
inline bool make_tmap_3d(CUtensorMap* tm, const bf16* base, uint64_t cols, uint64_t rows, uint64_t batches,
                         uint64_t row_stride, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {cols, rows, batches};
  cuuint64_t strides[2] = {row_stride * sizeof(bf16), rows * row_stride * sizeof(bf16)};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 4-D map over the chunked dS^T scratch of the attention backward, bf16 [nz][S / 32][S][32]: element (z, key j, query i)
// sits at ((z * S/32 + i / 32) * S + j) * 32 + i % 32, so that consecutive keys of one 32-query chunk are contiguous
// 64-byte rows (what the lanes of a warp of the dK/dV kernel store).  A box is 64 keys of 4 chunks (128 queries) and
// lands in shared memory as 4 blocks of [64 keys][32 queries], 64-byte rows with the 64-byte swizzle: the MN-major
// operand layout of that swizzle mode.  Strides ascend with the dimension.
inline bool make_tmap_ds_chunked(CUtensorMap* tm, const bf16* base, uint64_t S, uint64_t nz) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc || S % 128 != 0) return false;
  cuuint64_t dims[4] = {32, S, S / 32, nz};
  cuuint64_t strides[3] = {32 * sizeof(bf16), S * 32 * sizeof(bf16), S * S * sizeof(bf16)};
  cuuint32_t box[4] = {32, 64, 4, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<bf16*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace fs
