// Host-side construction of TMA tensor maps through the driver entry point (no link-time
// dependency on libcuda, so the library also loads on machines without a driver).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sol {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
  if (qres != cudaDriverEntryPointSuccess) return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// Tensor map over a bf16 tensor indexed (batch, head, row, channel) whose channels are contiguous
// and whose other strides (in elements) are free: box = 64 channels x box_rows rows of one
// (batch, head), 128-byte swizzle, out-of-range rows read as zero (ragged last block).
// Dimensions are ordered by growing stride, as the encoder wants: rows_inner = true gives
// coordinates (channel, row, head, batch), false gives (channel, head, row, batch).
inline bool make_tmap_bf16_4d(CUtensorMap* map, const void* base, int B, int H, int rows, int d, int box_rows,
                              long long row_stride, long long head_stride, long long batch_stride,
                              bool* rows_inner) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return false;
  *rows_inner = row_stride <= head_stride;
  cuuint64_t dims[4], strides[3];
  cuuint32_t box[4];
  dims[0] = (cuuint64_t)d;
  box[0] = 64;
  if (*rows_inner) {
    dims[1] = (cuuint64_t)rows; dims[2] = (cuuint64_t)H;
    strides[0] = (cuuint64_t)row_stride * 2; strides[1] = (cuuint64_t)head_stride * 2;
    box[1] = (cuuint32_t)box_rows; box[2] = 1;
  } else {
    dims[1] = (cuuint64_t)H; dims[2] = (cuuint64_t)rows;
    strides[0] = (cuuint64_t)head_stride * 2; strides[1] = (cuuint64_t)row_stride * 2;
    box[1] = 1; box[2] = (cuuint32_t)box_rows;
  }
  dims[3] = (cuuint64_t)B;
  strides[2] = (cuuint64_t)batch_stride * 2;
  box[3] = 1;
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace sol
