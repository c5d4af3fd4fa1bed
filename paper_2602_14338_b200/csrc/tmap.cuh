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

// Blocked 3-D view of a row-major bf16 matrix whose column count is a multiple of 64:
// dimension 0 = the 64 elements of a column block (128 bytes), dimension 1 = rows,
// dimension 2 = column blocks.  A box of (64, box_rows, n_blocks) lands in shared memory as
// n_blocks consecutive [box_rows][64] sub-tiles, which is the MN-major operand layout of
// tcgen05.mma with 128-byte swizzle -- one copy instead of one per 64-column block.
inline int aero_make_tmap_blocked(aero_ctx* ctx, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                                  uint64_t ld_elems, uint32_t box_rows, uint32_t n_blocks) {
  if (!ctx->tmap_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
      return AERO_ERR_CUDA;
    ctx->tmap_encode = fn;
  }
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ctx->tmap_encode);
  cuuint64_t gdim[3] = {64, rows, cols / 64};
  cuuint64_t gstride[2] = {ld_elems * 2, 128};
  cuuint32_t box[3] = {64, box_rows, n_blocks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AERO_OK : AERO_ERR_CUDA;
}

// The chunk's dz block is stored tiled: for each 128-row token tile and each 64-column block a
// contiguous [128][64] bf16 tile (16 KB), so that every copy of the kernels that write and read it
// -- 32 x 64 stores, 128 x 64 K-major loads, 64 x (2 x 64) MN-major loads -- moves whole contiguous
// pieces instead of 128-byte segments 300 KB apart.  Dimensions: element in block, row in tile,
// column block, tile.  A box of (64, box_rows, box_blocks, 1) lands in shared memory as
// box_blocks consecutive [box_rows][64] sub-tiles with the 128-byte swizzle.
inline int aero_make_tmap_dz(aero_ctx* ctx, CUtensorMap* out, const void* base, uint64_t n_tiles, uint64_t n_blocks,
                             uint32_t box_rows, uint32_t box_blocks) {
  if (!ctx->tmap_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
      return AERO_ERR_CUDA;
    ctx->tmap_encode = fn;
  }
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ctx->tmap_encode);
  cuuint64_t gdim[4] = {64, 128, n_blocks, n_tiles};
  cuuint64_t gstride[3] = {128, 128 * 128, n_blocks * 128 * 128};
  cuuint32_t box[4] = {64, box_rows, box_blocks, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gdim, gstride, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AERO_OK : AERO_ERR_CUDA;
}
