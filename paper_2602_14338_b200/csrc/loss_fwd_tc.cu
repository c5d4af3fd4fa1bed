// Stage (b) forward on the tensor-core path: tile list, fused lm_head kernel in
// forward mode, fixed-order reduction of the loss partials.
#include "lmhead_kernel.cuh"
#include "tmap.cuh"

namespace {

struct FwdWs {
  aero_tiles tiles;
  double* partials;
  size_t n_partials;
  float4* xstate;       // [vsplit][T] running states of the rows when the vocabulary is split
  unsigned int* sync_ctr;
};

size_t partials_bytes(int64_t T, int32_t R) {
  const size_t mt = (size_t)(T / lmhead::BM) + (size_t)R + 2;
  return aero_align_up(mt * 4 * kPartialStride * sizeof(double), 256);
}

FwdWs carve_fwd(void* ws, int64_t T, int32_t R) {
  FwdWs f;
  f.tiles = aero_carve_tiles(ws, T, R, lmhead::BM);
  char* p = static_cast<char*>(ws) + aero_tiles_bytes(T, R, lmhead::BM);
  f.partials = reinterpret_cast<double*>(p);
  f.n_partials = (size_t)f.tiles.max_tiles * 4;
  f.sync_ctr = reinterpret_cast<unsigned int*>(p + partials_bytes(T, R));
  f.xstate = reinterpret_cast<float4*>(p + partials_bytes(T, R) + 256);
  return f;
}

}  // namespace

size_t aero_fwd_ws_bytes_tc(int64_t T, int32_t d, int32_t R) {
  const int vs = aero_vsplit_cap(d);
  const size_t state = aero_align_up((size_t)vs * (size_t)(T > 0 ? T : 1) * sizeof(float4), 256);
  return aero_tiles_bytes(T, R, lmhead::BM) + partials_bytes(T, R) + 256 + state;
}

int aero_fwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                const void* H, const void* W, const int32_t* y, const float* old_logp,
                const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                float* logp, float* lse, float* g, float* loss, float* metrics, int accumulate, void* ws,
                const aero_fwd_extra& ex) {
  FwdWs f = carve_fwd(ws, T, R);
  AERO_CUDA_TRY(cudaMemsetAsync(f.partials, 0, f.n_partials * kPartialStride * sizeof(double), ctx->stream));
  AERO_CUDA_TRY(cudaMemsetAsync(f.sync_ctr, 0, 256, ctx->stream));
  if (T > 0) {
    AERO_CUDA_TRY(cudaMemsetAsync(logp, 0, (size_t)T * sizeof(float), ctx->stream));
    AERO_CUDA_TRY(cudaMemsetAsync(lse, 0, (size_t)T * sizeof(float), ctx->stream));
    if (g) AERO_CUDA_TRY(cudaMemsetAsync(g, 0, (size_t)T * sizeof(float), ctx->stream));
    if (ex.entropy) AERO_CUDA_TRY(cudaMemsetAsync(ex.entropy, 0, (size_t)T * sizeof(float), ctx->stream));
  }
  int rc = ex.logprob_only ? aero_build_dense_tiles(ctx, T, lmhead::BM, f.tiles)
                           : aero_build_tiles(ctx, T, R, cs, keep, lmhead::BM, f.tiles);
  if (rc) return rc;
  if (T > 0 && (R > 0 || ex.logprob_only)) {
    CUtensorMap tmH, tmW;
    rc = aero_make_tmap_2d(ctx, &tmH, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, H, (uint64_t)T, (uint64_t)d, (uint64_t)d,
                           lmhead::BM, lmhead::BK);
    if (rc) return rc;
    rc = aero_make_tmap_2d(ctx, &tmW, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, W, (uint64_t)V, (uint64_t)d, (uint64_t)d,
                           lmhead::BNH, lmhead::BK);
    if (rc) return rc;
    lmhead::Params p = {};
    p.T = T; p.d = d; p.V = V; p.R = R;
    p.tile_row = f.tiles.tile_row; p.tile_valid = f.tiles.tile_valid; p.n_tiles = f.tiles.n_tiles;
    p.tile_begin = 0; p.tile_end = f.tiles.max_tiles;
    p.vsplit = aero_vsplit(ctx, d); p.xstate = f.xstate;
    p.sync_ctr = f.sync_ctr; p.nsync = aero_nsync(ctx); p.w_hint = aero_w_hint(ctx, false); p.k_zigzag = aero_k_zigzag(ctx);
    p.y = y; p.status = ctx->d_status;
    p.old_logp = ex.logprob_only ? nullptr : old_logp; p.cs = cs; p.adv = adv; p.w = w;
    p.ref_logp = ex.ref_logp; p.kl_beta = ex.kl_beta; p.ent_coef = ex.ent_coef; p.ent_out = ex.entropy;
    p.clip_lo = cfg->clip_lo; p.clip_hi = cfg->clip_hi;
    p.logp = logp; p.lse_out = lse; p.g_out = g; p.partials = f.partials;
    auto kern = ex.entropy ? lmhead::lmhead_kernel<lmhead::MODE_FWD_ENT> : lmhead::lmhead_kernel<lmhead::MODE_FWD>;
    AERO_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lmhead::SMEM_BYTES));
    // one CTA pair per two token tiles, at most one pair per two SMs
    const int64_t upper_pairs = (T / lmhead::BM + R + 2) / 2 * p.vsplit;
    const int64_t max_pairs = ctx->sm_count / 2 > 0 ? ctx->sm_count / 2 : 1;
    const int grid = 2 * (int)(upper_pairs < max_pairs ? upper_pairs : max_pairs);
    kern<<<grid, lmhead::THREADS, lmhead::SMEM_BYTES, ctx->stream>>>(tmH, tmW, tmH, p);   // third map unused in forward mode
    ctx->launches += 1;
    if (p.vsplit > 1) {
      const int64_t upper_tiles = T / lmhead::BM + R + 1;
      const int mgrid = (int)(upper_tiles < 8 * ctx->sm_count ? upper_tiles : 8 * ctx->sm_count);
      lmhead::merge_kernel<<<mgrid, lmhead::BM, 0, ctx->stream>>>(p, ex.entropy ? 1 : 0);
      ctx->launches += 1;
    }
    AERO_CUDA_TRY(cudaGetLastError());
  }
  if (ex.logprob_only) return AERO_OK;
  return aero_loss_finalize(ctx, f.partials, (int)f.n_partials, kPartialStride, loss, metrics, accumulate);
}
