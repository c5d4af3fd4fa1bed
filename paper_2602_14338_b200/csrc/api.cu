// C ABI entry points: argument validation, context management and dispatch to the
// stage launchers.  Nothing here touches array data on the host.
#include "common.cuh"

#include <new>
#include <string>

#include <nvtx3/nvToolsExt.h>

namespace {

// NVTX range over one ABI call (visible in Nsight timelines; a no-op without a profiler attached)
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

int check_ctx(aero_ctx* ctx) {
  if (!ctx) return AERO_ERR_INVALID;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AERO_ERR_CUDA;
  return AERO_OK;
}

}  // namespace

extern "C" {

int aero_version(void) { return 102; }

const char* aero_error_string(int code) {
  switch (code) {
    case AERO_OK: return "ok";
    case AERO_ERR_INVALID: return "invalid argument";
    case AERO_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case AERO_ERR_WORKSPACE: return "workspace too small";
    case AERO_ERR_CUDA: return "CUDA call failed";
    case AERO_ERR_TOO_LARGE: return "problem exceeds the library-owned scratch array";
    default: return "unknown error";
  }
}

void aero_cfg_default(aero_cfg* cfg) {
  if (!cfg) return;
  cfg->uniform_policy = AERO_UNIFORM_MASK;
  cfg->rejection = 0;
  cfg->k_ratio = 1;
  cfg->rescue_S = 0;
  cfg->n_explore = 8;
  cfg->n_keep_uniform = 4;
  cfg->stats_over = AERO_STATS_KEPT;
  cfg->agg = AERO_TOKEN_MEAN;
  cfg->denom = AERO_DENOM_SURVIVING;
  cfg->alpha0 = 1.f;
  cfg->beta0 = 1.f;
  cfg->eps_std = 1e-6f;
  cfg->clip_lo = 0.2f;
  cfg->clip_hi = 0.2f;
  cfg->seed = 0;
  cfg->dtype = AERO_BF16;
  cfg->reject_high = 0;
  cfg->kl_beta = 0.f;
  cfg->ent_coef = 0.f;
}

int aero_create(aero_ctx** out, int device, void* cuda_stream) {
  if (!out) return AERO_ERR_INVALID;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return AERO_ERR_CUDA;
  AERO_CUDA_TRY(cudaSetDevice(device));
  aero_ctx* ctx = new (std::nothrow) aero_ctx();
  if (!ctx) return AERO_ERR_INVALID;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->d_status = nullptr;
  ctx->tmap_encode = nullptr;
  ctx->launches = 0;
  ctx->timing = 0;
  ctx->n_timed = 0;
  ctx->tune_vsplit = 0;
  ctx->tune_nsync = -1;
  ctx->tune_w_hint = -1;
  ctx->tune_k_zigzag = -1;
  ctx->tune_rowscale = -1;
  ctx->tune_gemm_sync = -1;
  ctx->tune_gemm_pairs = -1;
  for (int i = 0; i < 256; ++i) { ctx->ev0[i] = nullptr; ctx->ev1[i] = nullptr; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return AERO_ERR_CUDA; }
  ctx->sm_count = prop.multiProcessorCount;
  if (cudaMalloc(&ctx->d_status, sizeof(uint32_t)) != cudaSuccess) { delete ctx; return AERO_ERR_CUDA; }
  if (cudaMemset(ctx->d_status, 0, sizeof(uint32_t)) != cudaSuccess) {
    cudaFree(ctx->d_status); delete ctx; return AERO_ERR_CUDA;
  }
  *out = ctx;
  return AERO_OK;
}

int aero_destroy(aero_ctx* ctx) {
  if (!ctx) return AERO_ERR_INVALID;
  cudaSetDevice(ctx->device);
  cudaFree(ctx->d_status);
  for (int i = 0; i < 256; ++i) {
    if (ctx->ev0[i]) cudaEventDestroy(ctx->ev0[i]);
    if (ctx->ev1[i]) cudaEventDestroy(ctx->ev1[i]);
  }
  for (int i = 0; i < 16; ++i)
    if (ctx->slice_ev[i]) cudaEventDestroy(ctx->slice_ev[i]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  delete ctx;
  return AERO_OK;
}

int aero_enable_kernel_timing(aero_ctx* ctx, int on) {
  if (!ctx) return AERO_ERR_INVALID;
  ctx->timing = on ? 1 : 0;
  ctx->n_timed = 0;
  return AERO_OK;
}

int aero_kernel_timing_ms(aero_ctx* ctx, float* total_ms, int* launches) {
  if (!ctx || !total_ms || !launches) return AERO_ERR_INVALID;
  int rc = check_ctx(ctx);
  if (rc) return rc;
  AERO_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
  float sum = 0.f;
  for (int i = 0; i < ctx->n_timed; ++i) {
    float ms = 0.f;
    AERO_CUDA_TRY(cudaEventElapsedTime(&ms, ctx->ev0[i], ctx->ev1[i]));
    sum += ms;
  }
  *total_ms = sum;
  *launches = ctx->n_timed;
  ctx->n_timed = 0;
  return AERO_OK;
}

int aero_set_stream(aero_ctx* ctx, void* cuda_stream) {
  if (!ctx) return AERO_ERR_INVALID;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  return AERO_OK;
}

int aero_set_tuning(aero_ctx* ctx, const char* name, int value) {
  if (!ctx || !name) return AERO_ERR_INVALID;
  const std::string n(name);
  if (n == "vsplit") {
    if (value != 0 && value != 1 && value != 2 && value != 4) return AERO_ERR_INVALID;
    ctx->tune_vsplit = value;
  } else if (n == "nsync") {
    if (value > 4096) return AERO_ERR_INVALID;
    ctx->tune_nsync = value < 0 ? -1 : value;
  } else if (n == "rowscale") {
    ctx->tune_rowscale = value < 0 ? -1 : (value ? 1 : 0);
  } else if (n == "gemm_sync") {
    if (value > 4096) return AERO_ERR_INVALID;
    ctx->tune_gemm_sync = value < 0 ? -1 : value;
  } else if (n == "w_hint") {
    ctx->tune_w_hint = value < 0 ? -1 : (value ? 1 : 0);
  } else if (n == "k_zigzag") {
    ctx->tune_k_zigzag = value < 0 ? -1 : (value ? 1 : 0);
  } else if (n == "gemm_pairs") {
    ctx->tune_gemm_pairs = value < 0 ? -1 : (value ? 1 : 0);
  } else {
    return AERO_ERR_INVALID;
  }
  return AERO_OK;
}

int aero_last_status(aero_ctx* ctx, uint32_t* bits) {
  if (!ctx || !bits) return AERO_ERR_INVALID;
  int rc = check_ctx(ctx);
  if (rc) return rc;
  // read and clear in stream order, so that neither can overtake (or be overtaken by) kernels of
  // this context on a stream that does not synchronise with the default stream
  AERO_CUDA_TRY(cudaMemcpyAsync(bits, ctx->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, ctx->stream));
  AERO_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), ctx->stream));
  AERO_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
  return AERO_OK;
}

size_t aero_group_workspace_bytes(int32_t P, int32_t R) { return aero_group_ws_bytes_impl(P, R); }

int aero_group_stats(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                     const int32_t* go, const float* reward, const int64_t* cs,
                     const uint32_t* key, const uint8_t* keep_in,
                     const float* alpha_in, const float* beta_in,
                     float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                     float* u_tilde, float* alpha_out, float* beta_out,
                     int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                     float* metrics, void* workspace, size_t workspace_bytes) {
  Range nv("aero_group_stats");
  if (!ctx || !cfg || P < 0 || R < 0) return AERO_ERR_INVALID;
  if (!go || !cs || !kept_tok_off || !counters) return AERO_ERR_INVALID;
  if (R > 0 && (!reward || !adv || !w || !keep || !kept_ids)) return AERO_ERR_INVALID;
  if (P > 0 && (!gmask || !cat || !u_tilde || !alpha_out || !beta_out)) return AERO_ERR_INVALID;
  if ((alpha_in == nullptr) != (beta_in == nullptr)) return AERO_ERR_INVALID;
  if (cfg->k_ratio < 1 || cfg->n_explore < 1 || cfg->rescue_S < 0) return AERO_ERR_INVALID;
  if (!workspace || !aligned256(workspace)) return AERO_ERR_INVALID;
  if (workspace_bytes < aero_group_ws_bytes_impl(P, R)) return AERO_ERR_WORKSPACE;
  const int rc = check_ctx(ctx);
  if (rc) return rc;
  return aero_group_stats_launch(ctx, cfg, P, R, go, reward, cs, key, keep_in, alpha_in, beta_in,
                                 adv, w, keep, gmask, cat, u_tilde, alpha_out, beta_out,
                                 kept_ids, kept_tok_off, counters, metrics, workspace);
}

int aero_finalize_weights(aero_ctx* ctx, const aero_cfg* cfg, int32_t R, int32_t P_local, int64_t P_global,
                          float* w, const int64_t* counters_local, const int64_t* counters_global) {
  Range nv("aero_finalize_weights");
  if (!ctx || !cfg || R < 0 || P_local < 0 || P_global < P_local) return AERO_ERR_INVALID;
  if (!counters_local || !counters_global || (R > 0 && !w)) return AERO_ERR_INVALID;
  const int rc = check_ctx(ctx);
  if (rc) return rc;
  return aero_finalize_weights_launch(ctx, cfg, R, P_local, P_global, w, counters_local, counters_global);
}

size_t aero_fwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R) {
  (void)V;
  size_t a = aero_fwd_ws_bytes_fp32(T, R), b = aero_fwd_ws_bytes_tc(T, d, R);
  return a > b ? a : b;
}

static int fwd_dispatch(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                        const void* H, const void* W, const int32_t* y, const float* old_logp,
                        const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                        float* logp, float* lse, float* g, float* loss, float* metrics,
                        int accumulate, void* workspace, size_t workspace_bytes, const aero_fwd_extra& ex) {
  if (!ctx || !cfg || T < 0 || d <= 0 || V <= 0 || R < 0 || T >= (int64_t)1 << 31) return AERO_ERR_INVALID;
  if (!W) return AERO_ERR_INVALID;
  if (T > 0 && (!H || !y || !logp || !lse)) return AERO_ERR_INVALID;
  if (!ex.logprob_only) {
    if (!cs || !loss) return AERO_ERR_INVALID;
    if (T > 0 && (!old_logp || !g)) return AERO_ERR_INVALID;
    if (R > 0 && (!adv || !w || !keep)) return AERO_ERR_INVALID;
  }
  if (!workspace || !aligned256(workspace)) return AERO_ERR_INVALID;
  if (cfg->dtype != AERO_FP32 && cfg->dtype != AERO_BF16) return AERO_ERR_UNSUPPORTED;
  if (cfg->dtype == AERO_BF16 && d % 64 != 0) return AERO_ERR_UNSUPPORTED;
  if (cfg->dtype == AERO_BF16 && (!aligned16(H) || !aligned16(W))) return AERO_ERR_INVALID;
  if (workspace_bytes < aero_fwd_workspace_bytes(T, d, V, R)) return AERO_ERR_WORKSPACE;
  const int rc = check_ctx(ctx);
  if (rc) return rc;
  if (cfg->dtype == AERO_FP32) {
    return aero_fwd_fp32(ctx, cfg, T, d, V, R, static_cast<const float*>(H), static_cast<const float*>(W),
                         y, old_logp, cs, adv, w, keep, logp, lse, g, loss, metrics, accumulate, workspace, ex);
  }
  return aero_fwd_tc(ctx, cfg, T, d, V, R, H, W, y, old_logp, cs, adv, w, keep, logp, lse, g, loss,
                     metrics, accumulate, workspace, ex);
}

int aero_grpo_loss_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                       const void* H, const void* W, const int32_t* y, const float* old_logp,
                       const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                       float* logp, float* lse, float* g, float* loss, float* metrics,
                       int accumulate, void* workspace, size_t workspace_bytes) {
  Range nv("aero_grpo_loss_fwd");
  const aero_fwd_extra ex = {nullptr, 0.f, 0.f, nullptr, 0};
  return fwd_dispatch(ctx, cfg, T, d, V, R, H, W, y, old_logp, cs, adv, w, keep, logp, lse, g, loss, metrics,
                      accumulate, workspace, workspace_bytes, ex);
}

int aero_grpo_loss_reg_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y, const float* old_logp,
                           const float* ref_logp,
                           const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                           float* logp, float* lse, float* g, float* entropy, float* loss, float* metrics,
                           int accumulate, void* workspace, size_t workspace_bytes) {
  Range nv("aero_grpo_loss_reg_fwd");
  if (!cfg) return AERO_ERR_INVALID;
  const aero_fwd_extra ex = {ref_logp, ref_logp ? cfg->kl_beta : 0.f, entropy ? cfg->ent_coef : 0.f, entropy, 0};
  return fwd_dispatch(ctx, cfg, T, d, V, R, H, W, y, old_logp, cs, adv, w, keep, logp, lse, g, loss, metrics,
                      accumulate, workspace, workspace_bytes, ex);
}

int aero_logprob_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V,
                     const void* H, const void* W, const int32_t* y,
                     float* logp, float* lse, float* entropy,
                     void* workspace, size_t workspace_bytes) {
  Range nv("aero_logprob_fwd");
  const aero_fwd_extra ex = {nullptr, 0.f, 0.f, entropy, 1};
  return fwd_dispatch(ctx, cfg, T, d, V, 0, H, W, y, nullptr, nullptr, nullptr, nullptr, nullptr, logp, lse, nullptr,
                      nullptr, nullptr, 0, workspace, workspace_bytes, ex);
}

size_t aero_fwd_bwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens) {
  const size_t a = aero_fwd_bwd_ws_bytes_tc(T, d, V, R, chunk_tokens), b = aero_fwd_workspace_bytes(T, d, V, R);
  return a > b ? a : b;
}

int aero_grpo_loss_reg_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                               const void* H, const void* W, const int32_t* y, const float* old_logp,
                               const float* ref_logp,
                               const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                               float* logp, float* lse, float* g, float* entropy, float* loss, float* metrics,
                               float grad_scale, void* dH, float* dW, int accumulate_dW,
                               void* workspace, size_t workspace_bytes) {
  Range nv("aero_grpo_loss_fwd_bwd");
  if (!ctx || !cfg || T < 0 || d <= 0 || V <= 0 || R < 0 || T >= (int64_t)1 << 31) return AERO_ERR_INVALID;
  if (!W || !cs || !loss || !dW) return AERO_ERR_INVALID;
  if (T > 0 && (!H || !y || !old_logp || !logp || !lse || !g || !dH)) return AERO_ERR_INVALID;
  if (R > 0 && (!adv || !w || !keep)) return AERO_ERR_INVALID;
  if (!workspace || !aligned256(workspace)) return AERO_ERR_INVALID;
  if (cfg->dtype == AERO_FP32) {
    int rc = aero_grpo_loss_reg_fwd(ctx, cfg, T, d, V, R, H, W, y, old_logp, ref_logp, cs, adv, w, keep, logp, lse, g,
                                    entropy, loss, metrics, 0, workspace, workspace_bytes);
    if (rc) return rc;
    if (entropy)
      return aero_grpo_loss_reg_bwd(ctx, cfg, T, d, V, R, H, W, y, cs, keep, lse, g, logp, entropy, w, grad_scale, dH, dW,
                                    accumulate_dW, workspace, workspace_bytes);
    return aero_grpo_loss_bwd(ctx, cfg, T, d, V, R, H, W, y, cs, keep, lse, g, logp, grad_scale, dH, dW, accumulate_dW,
                              workspace, workspace_bytes);
  }
  if (cfg->dtype != AERO_BF16) return AERO_ERR_UNSUPPORTED;
  if (d % 64 != 0) return AERO_ERR_UNSUPPORTED;
  if (!aligned16(H) || !aligned16(W) || !aligned16(dH) || !aligned16(dW)) return AERO_ERR_INVALID;
  if (workspace_bytes < aero_fwd_bwd_ws_bytes_tc(T, d, V, R, 128)) return AERO_ERR_WORKSPACE;
  const int rc = check_ctx(ctx);
  if (rc) return rc;
  return aero_fwd_bwd_tc(ctx, cfg, T, d, V, R, H, W, y, old_logp, ref_logp, cfg->kl_beta, entropy, cfg->ent_coef, cs, adv, w,
                         keep, logp, lse, g, loss, metrics, grad_scale, dH, dW, accumulate_dW, workspace, workspace_bytes);
}

int aero_grpo_loss_kl_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                              const void* H, const void* W, const int32_t* y, const float* old_logp,
                              const float* ref_logp,
                              const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                              float* logp, float* lse, float* g, float* loss, float* metrics,
                              float grad_scale, void* dH, float* dW, int accumulate_dW,
                              void* workspace, size_t workspace_bytes) {
  return aero_grpo_loss_reg_fwd_bwd(ctx, cfg, T, d, V, R, H, W, y, old_logp, ref_logp, cs, adv, w, keep, logp, lse, g,
                                    nullptr, loss, metrics, grad_scale, dH, dW, accumulate_dW, workspace, workspace_bytes);
}

int aero_grpo_loss_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y, const float* old_logp,
                           const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                           float* logp, float* lse, float* g, float* loss, float* metrics,
                           float grad_scale, void* dH, float* dW, int accumulate_dW,
                           void* workspace, size_t workspace_bytes) {
  return aero_grpo_loss_kl_fwd_bwd(ctx, cfg, T, d, V, R, H, W, y, old_logp, nullptr, cs, adv, w, keep, logp, lse, g, loss,
                                   metrics, grad_scale, dH, dW, accumulate_dW, workspace, workspace_bytes);
}

size_t aero_bwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens) {
  return aero_bwd_ws_bytes_tc(T, d, V, R, chunk_tokens);
}

static int bwd_dispatch(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                        const void* H, const void* W, const int32_t* y,
                        const int64_t* cs, const uint8_t* keep,
                        const float* lse, const float* g, float grad_scale,
                        void* dH, float* dW, int accumulate_dW,
                        void* workspace, size_t workspace_bytes, const aero_bwd_extra& ex) {
  if (!ctx || !cfg || T < 0 || d <= 0 || V <= 0 || R < 0 || T >= (int64_t)1 << 31) return AERO_ERR_INVALID;
  if (!W || !cs || !dW) return AERO_ERR_INVALID;
  if (T > 0 && (!H || !y || !lse || !g || !dH)) return AERO_ERR_INVALID;
  if (R > 0 && !keep) return AERO_ERR_INVALID;
  if (cfg->dtype == AERO_FP32) {
    const int rc = check_ctx(ctx);
    if (rc) return rc;
    return aero_bwd_fp32(ctx, cfg, T, d, V, R, static_cast<const float*>(H), static_cast<const float*>(W),
                         y, cs, keep, lse, g, grad_scale, static_cast<float*>(dH), dW, accumulate_dW, ex);
  }
  if (cfg->dtype != AERO_BF16) return AERO_ERR_UNSUPPORTED;
  if (d % 64 != 0) return AERO_ERR_UNSUPPORTED;
  if (!aligned16(H) || !aligned16(W) || !aligned16(dH) || !aligned16(dW)) return AERO_ERR_INVALID;
  if (!workspace || !aligned256(workspace)) return AERO_ERR_INVALID;
  if (workspace_bytes < aero_bwd_ws_bytes_tc(T, d, V, R, 128)) return AERO_ERR_WORKSPACE;
  const int rc = check_ctx(ctx);
  if (rc) return rc;
  return aero_bwd_tc(ctx, cfg, T, d, V, R, H, W, y, cs, keep, lse, g, grad_scale, dH, dW, accumulate_dW,
                     workspace, workspace_bytes, ex);
}

int aero_grpo_loss_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                       const void* H, const void* W, const int32_t* y,
                       const int64_t* cs, const uint8_t* keep,
                       const float* lse, const float* g, const float* logp, float grad_scale,
                       void* dH, float* dW, int accumulate_dW,
                       void* workspace, size_t workspace_bytes) {
  Range nv("aero_grpo_loss_bwd");
  const aero_bwd_extra ex = {nullptr, nullptr, 0.f, logp};
  return bwd_dispatch(ctx, cfg, T, d, V, R, H, W, y, cs, keep, lse, g, grad_scale, dH, dW, accumulate_dW, workspace,
                      workspace_bytes, ex);
}

int aero_grpo_loss_reg_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y,
                           const int64_t* cs, const uint8_t* keep,
                           const float* lse, const float* g, const float* logp, const float* entropy, const float* w,
                           float grad_scale, void* dH, float* dW, int accumulate_dW,
                           void* workspace, size_t workspace_bytes) {
  Range nv("aero_grpo_loss_reg_bwd");
  if (!cfg) return AERO_ERR_INVALID;
  if ((entropy == nullptr) != (w == nullptr)) return AERO_ERR_INVALID;
  const aero_bwd_extra ex = {entropy, w, entropy ? cfg->ent_coef : 0.f, logp};
  return bwd_dispatch(ctx, cfg, T, d, V, R, H, W, y, cs, keep, lse, g, grad_scale, dH, dW, accumulate_dW, workspace,
                      workspace_bytes, ex);
}

}  // extern "C"
