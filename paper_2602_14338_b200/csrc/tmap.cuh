// Host helper: build a 2-D TMA tensor map (128-byte swizzle) for a row-major matrix.
// The driver's encoder is resolved through the runtime, so the library has no link-time
// dependency on the driver library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include "common.cuh"

// rows x cols matrix, `ld_elems` elements between rows, element size `esize` bytes.
// box = box_rows x box_cols; box_cols * esize must be 128 (one swizzle row).
inline int aero_make_tmap_2d(aero_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int esize,
                             const void* base, uint64_t rows, uint64_t cols, uint64_t ld_elems,
                             uint32_t box_rows, uint32_t box_cols) {
  if (!ctx->tmap_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
      return AERO_ERR_CUDA;
    ctx->tmap_encode = fn;
  }
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ctx->tmap_encode);
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {ld_elems * (uint64_t)esize};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = encode(out, dt, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AERO_OK : AERO_ERR_CUDA;
}
