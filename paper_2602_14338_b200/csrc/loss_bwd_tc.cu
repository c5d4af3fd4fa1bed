// Stage (b) backward on the tensor-core path.  Token tiles are processed in chunks:
// for each chunk the lm_head kernel recomputes the logits and writes the bf16 dz block,
// then two GEMM launches produce the chunk's rows of dH and add the chunk's share of dW.
#include "gemm_bwd_kernel.cuh"
#include "lmhead_kernel.cuh"
#include "tmap.cuh"

namespace {

inline long long ldz_of(int32_t V) { return ((long long)V + 63) / 64 * 64; }

// dH rows of dropped rollouts are defined to be zero; one warp per row.
__global__ void __launch_bounds__(256) zero_dropped_rows_kernel(long long T, int d, int R,
                                                                const int64_t* __restrict__ cs,
                                                                const uint8_t* __restrict__ keep,
                                                                __nv_bfloat16* __restrict__ dH) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * 8;
  for (long long t = warp0; t < T; t += nwarps) {
    const int i = aero_owner(cs, R, t);
    if (keep[i]) continue;
    uint4* row = reinterpret_cast<uint4*>(dH + t * d);
    for (int k = lane; k < d / 8; k += 32) row[k] = make_uint4(0, 0, 0, 0);
  }
}

}  // namespace

size_t aero_bwd_ws_bytes_tc(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens) {
  (void)d;
  if (chunk_tokens < 128) chunk_tokens = 128;
  const size_t rows = (size_t)((chunk_tokens + 127) / 128 * 128);
  return aero_tiles_bytes(T, R, lmhead::BM) + 256 + aero_align_up(rows * (size_t)ldz_of(V) * 2, 256);
}

int aero_bwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                const void* H, const void* W, const int32_t* y, const int64_t* cs, const uint8_t* keep,
                const float* lse, const float* g, float grad_scale, void* dH, float* dW, int accumulate_dW,
                void* ws, size_t ws_bytes, const aero_bwd_extra& ex) {
  (void)cfg;
  if (!accumulate_dW) AERO_CUDA_TRY(cudaMemsetAsync(dW, 0, (size_t)V * d * sizeof(float), ctx->stream));
  if (T == 0 || R == 0) return AERO_OK;

  const long long ldz = ldz_of(V);
  aero_tiles tiles = aero_carve_tiles(ws, T, R, lmhead::BM);
  // tile list, then the pacing counter of the lm_head kernel, then the dz block
  const size_t tiles_bytes = aero_tiles_bytes(T, R, lmhead::BM) + 256;
  unsigned int* sync_ctr = reinterpret_cast<unsigned int*>(static_cast<char*>(ws) + tiles_bytes - 256);
  __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + tiles_bytes);
  long long tpc = (long long)((ws_bytes - tiles_bytes) / ((size_t)lmhead::BM * (size_t)ldz * 2));
  if (tpc < 1) return AERO_ERR_WORKSPACE;
  if (tpc > tiles.max_tiles) tpc = tiles.max_tiles;
  if (tpc > ctx->sm_count) tpc = tpc / ctx->sm_count * ctx->sm_count;   // whole waves of token tiles

  int rc = aero_build_tiles(ctx, T, R, cs, keep, lmhead::BM, tiles);
  if (rc) return rc;
  {
    const long long blocks = (T + 7) / 8;
    zero_dropped_rows_kernel<<<(int)(blocks < 4096 ? blocks : 4096), 256, 0, ctx->stream>>>(
        T, d, R, cs, keep, static_cast<__nv_bfloat16*>(dH));
    ctx->launches += 1;
    AERO_CUDA_TRY(cudaGetLastError());
  }

  const CUtensorMapDataType BF = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  CUtensorMap tmH_k, tmW_k, tmDZ_k, tmW_mn, tmDZ_mn, tmH_mn;
  // K-major views (inner extent 64 = one 128-byte swizzle row) for the recompute and for dz as A of dH
  if ((rc = aero_make_tmap_2d(ctx, &tmH_k, BF, 2, H, T, d, d, lmhead::BM, 64))) return rc;
  if ((rc = aero_make_tmap_2d(ctx, &tmW_k, BF, 2, W, V, d, d, lmhead::BNH, 64))) return rc;
  if ((rc = aero_make_tmap_dz(ctx, &tmDZ_k, dz, (uint64_t)tpc, (uint64_t)(ldz / 64), gemmbwd::BM, 1))) return rc;
  // MN-major operands: blocked views, one box = 64 rows x (4 or 2) column blocks of 64
  if ((rc = aero_make_tmap_blocked(ctx, &tmW_mn, W, V, d, d, 64, gemmbwd::BN / 64))) return rc;
  if ((rc = aero_make_tmap_dz(ctx, &tmDZ_mn, dz, (uint64_t)tpc, (uint64_t)(ldz / 64), 64, gemmbwd::BM / 64))) return rc;
  if ((rc = aero_make_tmap_blocked(ctx, &tmH_mn, H, T, d, d, 64, gemmbwd::BN / 64))) return rc;
  // CTA pairs: each CTA stages half of the B slab's columns
  const bool pairs = aero_gemm_pairs(ctx, d);
  CUtensorMap tmW_mn2, tmH_mn2;
  if (pairs) {
    if ((rc = aero_make_tmap_blocked(ctx, &tmW_mn2, W, V, d, d, 64, gemmbwd::PBNH / 64))) return rc;
    if ((rc = aero_make_tmap_blocked(ctx, &tmH_mn2, H, T, d, d, 64, gemmbwd::PBNH / 64))) return rc;
  }
  // store view of the dz block for the lm_head kernel's epilogue: 32 rows x 64 columns per copy
  CUtensorMap tmDZ_st;
  if ((rc = aero_make_tmap_dz(ctx, &tmDZ_st, dz, (uint64_t)tpc, (uint64_t)(ldz / 64), 32, 1))) return rc;

  const bool with_entropy = ex.entropy != nullptr && ex.ent_coef != 0.f;
  auto k_dz = with_entropy ? lmhead::lmhead_kernel<lmhead::MODE_DZ_ENT> : lmhead::lmhead_kernel<lmhead::MODE_DZ>;
  auto k_dh = gemmbwd::gemm_kernel<gemmbwd::KIND_DH>;
  auto k_dw = gemmbwd::gemm_kernel<gemmbwd::KIND_DW>;
  AERO_CUDA_TRY(cudaFuncSetAttribute(k_dz, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lmhead::SMEM_BYTES));
  AERO_CUDA_TRY(cudaFuncSetAttribute(k_dh, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::SMEM_BYTES));
  AERO_CUDA_TRY(cudaFuncSetAttribute(k_dw, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::SMEM_BYTES));
  auto k_dh2 = gemmbwd::gemm_pair_kernel<gemmbwd::KIND_DH>;
  auto k_dw2 = gemmbwd::gemm_pair_kernel<gemmbwd::KIND_DW>;
  if (pairs) {
    AERO_CUDA_TRY(cudaFuncSetAttribute(k_dh2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::PSMEM_BYTES));
    AERO_CUDA_TRY(cudaFuncSetAttribute(k_dw2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::PSMEM_BYTES));
  }

  const int n_nt = (d + gemmbwd::BN - 1) / gemmbwd::BN;
  const long long dw_units = (long long)((V + gemmbwd::BM - 1) / gemmbwd::BM) * n_nt;
  for (long long begin = 0; begin < tiles.max_tiles; begin += tpc) {
    lmhead::Params lp = {};
    lp.T = T; lp.d = d; lp.V = V; lp.R = R;
    lp.tile_row = tiles.tile_row; lp.tile_valid = tiles.tile_valid; lp.n_tiles = tiles.n_tiles;
    lp.tile_begin = (int)begin; lp.tile_end = (int)(begin + tpc);
    lp.y = y; lp.status = ctx->d_status;
    lp.lse_in = lse; lp.g_in = g; lp.logp_in = ex.logp; lp.grad_scale = grad_scale; lp.dz = dz; lp.ldz = ldz;
    lp.cs = cs; lp.w = ex.w; lp.ent_in = ex.entropy; lp.ent_coef = ex.ent_coef;
    lp.vsplit = aero_vsplit(ctx, d);
    lp.sync_ctr = sync_ctr; lp.nsync = aero_nsync(ctx); lp.w_hint = aero_w_hint(ctx, true); lp.k_zigzag = aero_k_zigzag(ctx);
    AERO_CUDA_TRY(cudaMemsetAsync(sync_ctr, 0, 256, ctx->stream));
    const long long max_pairs = ctx->sm_count / 2 > 0 ? ctx->sm_count / 2 : 1;
    const long long dz_pairs = (tpc + 1) / 2 * lp.vsplit;
    const int grid_dz = 2 * (int)(dz_pairs < max_pairs ? dz_pairs : max_pairs);
    k_dz<<<grid_dz, lmhead::THREADS, lmhead::SMEM_BYTES, ctx->stream>>>(tmH_k, tmW_k, tmDZ_st, lp);

    gemmbwd::Params gp = {};
    gp.T = T; gp.d = d; gp.V = V; gp.ldz = ldz;
    gp.tile_row = tiles.tile_row; gp.tile_valid = tiles.tile_valid; gp.n_tiles = tiles.n_tiles;
    gp.tile_begin = (int)begin; gp.tpc = (int)tpc;
    gp.dH = static_cast<__nv_bfloat16*>(dH); gp.dW = dW; gp.status = ctx->d_status;
    gp.nsync = aero_gemm_sync(ctx);
    gp.sync_ctr = sync_ctr + 4;             // (the lm_head kernel's counter comes first; all zeroed above)
    const long long dh_units = tpc * n_nt;
    if (pairs) {
      const long long dh_pu = (tpc + 1) / 2 * n_nt, dw_pu = ((long long)((V + gemmbwd::BM - 1) / gemmbwd::BM) + 1) / 2 * n_nt;
      k_dh2<<<2 * (int)(dh_pu < max_pairs ? dh_pu : max_pairs), gemmbwd::THREADS, gemmbwd::PSMEM_BYTES, ctx->stream>>>(
          tmDZ_k, tmW_mn2, gp);
      gp.sync_ctr = sync_ctr + 8;
      k_dw2<<<2 * (int)(dw_pu < max_pairs ? dw_pu : max_pairs), gemmbwd::THREADS, gemmbwd::PSMEM_BYTES, ctx->stream>>>(
          tmDZ_mn, tmH_mn2, gp);
    } else {
      k_dh<<<(int)(dh_units < ctx->sm_count ? dh_units : ctx->sm_count), gemmbwd::THREADS, gemmbwd::SMEM_BYTES,
             ctx->stream>>>(tmDZ_k, tmW_mn, gp);
      gp.sync_ctr = sync_ctr + 8;
      k_dw<<<(int)(dw_units < ctx->sm_count ? dw_units : ctx->sm_count), gemmbwd::THREADS, gemmbwd::SMEM_BYTES,
             ctx->stream>>>(tmDZ_mn, tmH_mn, gp);
    }
    ctx->launches += 3;
    AERO_CUDA_TRY(cudaGetLastError());
  }
  return AERO_OK;
}
