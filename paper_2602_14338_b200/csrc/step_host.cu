// One whole step from host buffers: stage the batch on the device, run the three
// stages, return the scalars.  Only copies and calls of the public entry points.
#include "common.cuh"

namespace {

struct Carve {
  char* p;
  size_t used;
  explicit Carve(void* base) : p(static_cast<char*>(base)), used(0) {}
  template <typename T>
  T* take(size_t n) {
    T* r = reinterpret_cast<T*>(p + used);
    used += aero_align_up((n > 0 ? n : 1) * sizeof(T), 256);
    return r;
  }
};

struct StepWs {
  int32_t* go; float* reward; int64_t* cs; uint32_t* key; float* alpha; float* beta;
  char* H; int32_t* y; float* old_logp;
  float* adv; float* w; uint8_t* keep; uint8_t* gmask; uint8_t* cat;
  float* u; float* ao; float* bo; int32_t* kept_ids; int64_t* kept_tok_off;
  int64_t* counters; float* metrics; float* logp; float* lse; float* g; float* loss;
  char* sub; size_t sub_bytes;
  size_t total;
};

StepWs carve_step(void* base, int32_t P, int32_t R, int64_t T, int32_t d, int32_t V, int64_t chunk_tokens,
                  int32_t dtype) {
  const size_t esz = dtype == AERO_FP32 ? 4 : 2;
  Carve c(base);
  StepWs s;
  s.go = c.take<int32_t>((size_t)P + 1); s.reward = c.take<float>(R); s.cs = c.take<int64_t>((size_t)R + 1);
  s.key = c.take<uint32_t>(R); s.alpha = c.take<float>(P); s.beta = c.take<float>(P);
  s.H = c.take<char>((size_t)T * d * esz); s.y = c.take<int32_t>(T); s.old_logp = c.take<float>(T);
  s.adv = c.take<float>(R); s.w = c.take<float>(R); s.keep = c.take<uint8_t>(R);
  s.gmask = c.take<uint8_t>(P); s.cat = c.take<uint8_t>(P);
  s.u = c.take<float>(P); s.ao = c.take<float>(P); s.bo = c.take<float>(P);
  s.kept_ids = c.take<int32_t>(R); s.kept_tok_off = c.take<int64_t>((size_t)R + 1);
  s.counters = c.take<int64_t>(8); s.metrics = c.take<float>(8);
  s.logp = c.take<float>(T); s.lse = c.take<float>(T); s.g = c.take<float>(T); s.loss = c.take<float>(1);
  size_t sub = aero_group_workspace_bytes(P, R);
  const size_t f = aero_fwd_workspace_bytes(T, d, V, R);
  const size_t b = dtype == AERO_FP32 ? 256 : aero_fwd_bwd_workspace_bytes(T, d, V, R, chunk_tokens);
  if (f > sub) sub = f;
  if (b > sub) sub = b;
  s.sub = c.take<char>(sub);
  s.sub_bytes = sub;
  s.total = c.used;
  return s;
}

}  // namespace

extern "C" {

int64_t aero_launch_count(aero_ctx* ctx) { return ctx ? ctx->launches : -1; }

size_t aero_step_workspace_bytes(int32_t P, int32_t R, int64_t T, int32_t d, int32_t V, int64_t chunk_tokens,
                                 int32_t dtype) {
  if (P < 0 || R < 0 || T < 0 || d <= 0 || V <= 0) return 0;
  return carve_step(nullptr, P, R, T, d, V, chunk_tokens, dtype).total;
}

int aero_grpo_step_host(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R, int64_t T, int32_t d, int32_t V,
                        const int32_t* go_h, const float* reward_h, const int64_t* cs_h, const uint32_t* key_h,
                        const float* alpha_h, const float* beta_h,
                        const void* H_h, const int32_t* y_h, const float* old_logp_h,
                        const void* W, void* dH, float* dW, int accumulate_dW,
                        float* loss_h, int64_t* counters_h, float* metrics_h,
                        void* workspace, size_t workspace_bytes) {
  if (!ctx || !cfg || P < 0 || R < 0 || T < 0 || d <= 0 || V <= 0) return AERO_ERR_INVALID;
  if (!go_h || !cs_h || !W || !dW || !workspace) return AERO_ERR_INVALID;
  if (R > 0 && !reward_h) return AERO_ERR_INVALID;
  if (T > 0 && (!H_h || !y_h || !old_logp_h || !dH)) return AERO_ERR_INVALID;
  if ((alpha_h == nullptr) != (beta_h == nullptr)) return AERO_ERR_INVALID;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AERO_ERR_CUDA;
  // chunk size: whatever the given workspace affords beyond the fixed part
  const size_t fixed = carve_step(nullptr, P, R, T, d, V, 128, cfg->dtype).total;
  if (workspace_bytes < fixed) return AERO_ERR_WORKSPACE;
  const size_t per_tile = cfg->dtype == AERO_FP32 ? 1 : (size_t)128 * ((((size_t)V + 63) / 64 * 64) * 2 + (size_t)d * 2);
  int64_t chunk_tokens = 128 + (int64_t)((workspace_bytes - fixed) / per_tile) * 128;
  StepWs s = carve_step(workspace, P, R, T, d, V, chunk_tokens, cfg->dtype);
  while (s.total > workspace_bytes && chunk_tokens > 128) {     // alignment slack
    chunk_tokens -= 128;
    s = carve_step(workspace, P, R, T, d, V, chunk_tokens, cfg->dtype);
  }
  if (s.total > workspace_bytes) return AERO_ERR_WORKSPACE;
  const size_t esz = cfg->dtype == AERO_FP32 ? 4 : 2;
  cudaStream_t st = ctx->stream;
  const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
  AERO_CUDA_TRY(cudaMemcpyAsync(s.go, go_h, ((size_t)P + 1) * 4, H2D, st));
  AERO_CUDA_TRY(cudaMemcpyAsync(s.cs, cs_h, ((size_t)R + 1) * 8, H2D, st));
  if (R > 0) AERO_CUDA_TRY(cudaMemcpyAsync(s.reward, reward_h, (size_t)R * 4, H2D, st));
  if (R > 0 && key_h) AERO_CUDA_TRY(cudaMemcpyAsync(s.key, key_h, (size_t)R * 4, H2D, st));
  if (P > 0 && alpha_h) {
    AERO_CUDA_TRY(cudaMemcpyAsync(s.alpha, alpha_h, (size_t)P * 4, H2D, st));
    AERO_CUDA_TRY(cudaMemcpyAsync(s.beta, beta_h, (size_t)P * 4, H2D, st));
  }
  // H, the bulk of the bytes, goes in slices on a stream of its own (tensor-core path): the group
  // stage and the first chunks of the fused step run while the later slices arrive
  const bool sliced = T > 0 && cfg->dtype != AERO_FP32;
  if (T > 0) {
    AERO_CUDA_TRY(cudaMemcpyAsync(s.y, y_h, (size_t)T * 4, H2D, st));
    AERO_CUDA_TRY(cudaMemcpyAsync(s.old_logp, old_logp_h, (size_t)T * 4, H2D, st));
  }
  if (sliced) {
    constexpr int kSlices = 16;
    if (!ctx->copy_stream) AERO_CUDA_TRY(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < kSlices; ++i)
      if (!ctx->slice_ev[i]) AERO_CUDA_TRY(cudaEventCreateWithFlags(&ctx->slice_ev[i], cudaEventDisableTiming));
    const long long rows = ((T + kSlices - 1) / kSlices + 127) / 128 * 128;
    // whatever ran before on the caller's stream may still read the staging area
    AERO_CUDA_TRY(cudaEventRecord(ctx->slice_ev[0], st));
    AERO_CUDA_TRY(cudaStreamWaitEvent(ctx->copy_stream, ctx->slice_ev[0], 0));
    for (int i = 0; i < kSlices; ++i) {
      const long long r0 = (long long)i * rows, r1 = r0 + rows < T ? r0 + rows : T;
      if (r0 < r1)
        AERO_CUDA_TRY(cudaMemcpyAsync(s.H + (size_t)r0 * d * esz, static_cast<const char*>(H_h) + (size_t)r0 * d * esz,
                                      (size_t)(r1 - r0) * d * esz, H2D, ctx->copy_stream));
      AERO_CUDA_TRY(cudaEventRecord(ctx->slice_ev[i], ctx->copy_stream));
    }
    ctx->n_slices = kSlices;
    ctx->rows_per_slice = rows;
  } else if (T > 0) {
    AERO_CUDA_TRY(cudaMemcpyAsync(s.H, H_h, (size_t)T * d * esz, H2D, st));
  }
  int rc = aero_group_stats(ctx, cfg, P, R, s.go, s.reward, s.cs, key_h ? s.key : nullptr, nullptr,
                            alpha_h ? s.alpha : nullptr, alpha_h ? s.beta : nullptr, s.adv, s.w, s.keep, s.gmask,
                            s.cat, s.u, s.ao, s.bo, s.kept_ids, s.kept_tok_off, s.counters, s.metrics, s.sub,
                            s.sub_bytes);
  if (rc) {
    ctx->n_slices = 0;
    if (sliced) cudaStreamSynchronize(ctx->copy_stream);      // the caller may free the workspace next
    return rc;
  }
  rc = aero_grpo_loss_fwd_bwd(ctx, cfg, T, d, V, R, s.H, W, s.y, s.old_logp, s.cs, s.adv, s.w, s.keep, s.logp, s.lse,
                              s.g, s.loss, s.metrics + 4, 1.0f, dH, dW, accumulate_dW, s.sub, s.sub_bytes);
  if (sliced) {
    // the last slice may lie past the last kept row: the call still ends with all of H on the device
    ctx->n_slices = 0;
    const cudaError_t e = cudaStreamWaitEvent(st, ctx->slice_ev[15], 0);
    if (rc == AERO_OK && e != cudaSuccess) rc = AERO_ERR_CUDA;
    if (rc) cudaStreamSynchronize(ctx->copy_stream);
  }
  if (rc) return rc;
  if (loss_h) AERO_CUDA_TRY(cudaMemcpyAsync(loss_h, s.loss, 4, D2H, st));
  if (counters_h) AERO_CUDA_TRY(cudaMemcpyAsync(counters_h, s.counters, 64, D2H, st));
  if (metrics_h) AERO_CUDA_TRY(cudaMemcpyAsync(metrics_h, s.metrics, 32, D2H, st));
  AERO_CUDA_TRY(cudaStreamSynchronize(st));
  return AERO_OK;
}

}  // extern "C"
