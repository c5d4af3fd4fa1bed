// Shared declarations of the library's translation units: context, status word,
// error handling and the launch entry points each .cu file provides.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/aero.h"

struct aero_ctx {
  int device;
  cudaStream_t stream;
  uint32_t* d_status;     // device status word (OR of AERO_ST_* bits)
  int sm_count;
  void* tmap_encode;      // cuTensorMapEncodeTiled, resolved once through the runtime
  long long launches;     // kernels launched so far (host-side count)
  // optional timing of the lm_head launches of aero_grpo_loss_fwd_bwd (off by default):
  // pairs of events recorded around each launch, read back by aero_kernel_timing_ms
  int timing;
  int n_timed;
  cudaEvent_t ev0[256], ev1[256];
  // aero_grpo_step_host stages H in slices on a stream of its own; while it runs the fused
  // step, every chunk waits only for the slices its token rows lie in (n_slices > 0)
  cudaStream_t copy_stream;
  cudaEvent_t slice_ev[16];
  int n_slices;
  long long rows_per_slice;
  // tuning hooks (aero_set_tuning); the defaults mean "let the library decide"
  int tune_vsplit;        // 0: by d (aero_vsplit_auto); else 1, 2 or 4 CTA pairs per pair of token tiles
  int tune_nsync;         // < 0: the default number of meeting points; 0: no pacing; else that many
  int tune_rowscale;      // < 0 or 1: row factors in the backward GEMMs; 0: the pass that rewrites the block
  int tune_gemm_sync;     // < 0: the default number of meeting points per unit of the backward GEMMs; 0: none
  int tune_w_hint;        // < 0: by kernel mode; 1: the lm_head kernel loads W with the evict-first L2 priority; 0: plain loads
  int tune_k_zigzag;      // < 0 or 1: the lm_head kernel walks d forwards and backwards in turn (the default); 0: always forwards
  int tune_gemm_pairs;    // < 0: by d; 1: the backward GEMMs run on CTA pairs (256-row units); 0: on single CTAs
};

#define AERO_CUDA_TRY(expr)                          \
  do {                                               \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) return AERO_ERR_CUDA;    \
  } while (0)

static inline size_t aero_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ void aero_raise(uint32_t* status, uint32_t bits) {
  if (bits) atomicOr(status, bits);
}

// ---- stage (a) ---------------------------------------------------------------------
size_t aero_group_ws_bytes_impl(int32_t P, int32_t R);
int aero_group_stats_launch(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                            const int32_t* go, const float* reward, const int64_t* cs,
                            const uint32_t* key, const uint8_t* keep_in,
                            const float* alpha_in, const float* beta_in,
                            float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                            float* u_tilde, float* alpha_out, float* beta_out,
                            int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                            float* metrics, void* ws);

int aero_finalize_weights_launch(aero_ctx* ctx, const aero_cfg* cfg, int32_t R, int32_t P_local, int64_t P_global,
                                 float* w, const int64_t* counters_local, const int64_t* counters_global);

// Optional terms of the objective beyond the clipped surrogate: Eq. 2's KL to a reference
// policy and the entropy bonus of Table 9.  All-zero / NULL means the plain objective.
struct aero_fwd_extra {
  const float* ref_logp;   // [T] or NULL (no KL term)
  float kl_beta;
  float ent_coef;          // used only when `entropy` is given
  float* entropy;          // [T] out, or NULL (no entropy term)
  int logprob_only;        // all T rows, log-probs (and entropy) only: cs/adv/w/keep/old_logp unused
};
struct aero_bwd_extra {
  const float* entropy;    // [T] from the forward, or NULL
  const float* w;          // [R] rollout weights (entropy term only)
  float ent_coef;
  const float* logp;       // [T] log-probs from the forward, or NULL: the target column of dz is then
                           // formed from exp(z_y - lse) recomputed in fp32
};

// ---- stage (b): helpers shared by the fp32 and the tensor-core paths ---------------
// Row-tile work list over maximal runs of consecutive kept rollouts.
struct aero_tiles {
  int32_t* tile_row;      // [max_tiles] first token row of each tile
  int32_t* tile_valid;    // [max_tiles] leading rows of the tile that belong to its run (1..tile_rows)
  int32_t* n_tiles;       // [1]
  int32_t max_tiles;
};
aero_tiles aero_carve_tiles(void* ws, int64_t T, int32_t R, int tile_rows);
size_t aero_tiles_bytes(int64_t T, int32_t R, int tile_rows);
int aero_build_tiles(aero_ctx* ctx, int64_t T, int32_t R, const int64_t* cs, const uint8_t* keep,
                     int tile_rows, aero_tiles tiles);
// The same list over all T rows (one run): tile k starts at row k * tile_rows.
int aero_build_dense_tiles(aero_ctx* ctx, int64_t T, int tile_rows, aero_tiles tiles);

// Per-token surrogate terms and the fixed-order loss reduction.
int aero_loss_finalize(aero_ctx* ctx, const double* partials, int n_partials, int stride,
                       float* loss, float* metrics, int accumulate);

// ---- stage (b): plain fp32 path -----------------------------------------------------
size_t aero_fwd_ws_bytes_fp32(int64_t T, int32_t R);
int aero_fwd_fp32(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                  const float* H, const float* W, const int32_t* y, const float* old_logp,
                  const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                  float* logp, float* lse, float* g, float* loss, float* metrics, int accumulate, void* ws,
                  const aero_fwd_extra& ex);
int aero_bwd_fp32(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                  const float* H, const float* W, const int32_t* y, const int64_t* cs, const uint8_t* keep,
                  const float* lse, const float* g, float grad_scale, float* dH, float* dW, int accumulate_dW,
                  const aero_bwd_extra& ex);

// ---- stage (b): tcgen05 / TMEM / TMA path (bf16) -------------------------------------
// Number of CTA pairs that share a pair of token tiles and split the vocabulary between them:
// the smallest power of two that brings the H tiles all 148 CTAs keep re-reading from L2
// (148 * 128 * d * 2 bytes) under 72 MB, a bit over half of the 126 MB L2.
static inline int aero_vsplit_auto(int32_t d) {
  const double live = 148.0 * 128.0 * (double)d * 2.0;
  int s = 1;
  while (live / s > 72.0 * 1024 * 1024 && s < 8) s *= 2;
  return s;
}
// Largest split a context may be tuned to (aero_set_tuning); workspaces are sized for it.
constexpr int kAeroMaxForcedVsplit = 4;
static inline int aero_vsplit_cap(int32_t d) {
  const int a = aero_vsplit_auto(d);
  return a > kAeroMaxForcedVsplit ? a : kAeroMaxForcedVsplit;
}
static inline int aero_vsplit(const aero_ctx* ctx, int32_t d) {
  return ctx->tune_vsplit > 0 ? ctx->tune_vsplit : aero_vsplit_auto(d);
}
// Meeting points per unit of the lm_head kernel's producers (0 switches the pacing off).
static inline int aero_nsync(const aero_ctx* ctx) { return ctx->tune_nsync >= 0 ? ctx->tune_nsync : 32; }
// One-call step: the backward GEMMs take p~ as it is, with the row factors applied to the dH
// tiles and to a scaled copy of the chunk's H rows, instead of a pass that rewrites the block.
// With several vocabulary splits this needs one shift per row for all of them
// (lmhead::Params::common_shift).
static inline bool aero_rowscale(const aero_ctx* ctx) { return ctx->tune_rowscale != 0; }
// Meeting points per unit of the backward GEMMs' producers (0: none).
// Whether the backward GEMMs run on CTA pairs.  Measured: at d = 3584 the pairs make the step 7 % faster
// (a CTA stages a third fewer bytes per slab), at d = 1536 they change nothing or lose 1-2 %.
static inline bool aero_gemm_pairs(const aero_ctx* ctx, int32_t d) {
  return ctx->tune_gemm_pairs < 0 ? d > 2048 : ctx->tune_gemm_pairs != 0;
}
// The hint pays where the kernel stores nothing but per-row results (measured: forward 1.5 % faster); where it
// also streams a block of p~ or dz out with the same priority, the W lines lose against those stores (3 % slower).
static inline int aero_w_hint(const aero_ctx* ctx, bool kernel_stores_block) {
  return ctx->tune_w_hint < 0 ? (kernel_stores_block ? 0 : 1) : ctx->tune_w_hint;
}
static inline int aero_k_zigzag(const aero_ctx* ctx) { return ctx->tune_k_zigzag < 0 ? 1 : ctx->tune_k_zigzag; }
static inline int aero_gemm_sync(const aero_ctx* ctx) { return ctx->tune_gemm_sync >= 0 ? ctx->tune_gemm_sync : 1; }
size_t aero_fwd_ws_bytes_tc(int64_t T, int32_t d, int32_t R);
int aero_fwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                const void* H, const void* W, const int32_t* y, const float* old_logp,
                const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                float* logp, float* lse, float* g, float* loss, float* metrics, int accumulate, void* ws,
                const aero_fwd_extra& ex);
size_t aero_fwd_bwd_ws_bytes_tc(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens);
int aero_fwd_bwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                    const void* H, const void* W, const int32_t* y, const float* old_logp,
                    const float* ref_logp, float kl_beta, float* entropy, float ent_coef,
                    const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                    float* logp, float* lse, float* g, float* loss, float* metrics,
                    float grad_scale, void* dH, float* dW, int accumulate_dW, void* ws, size_t ws_bytes);
size_t aero_bwd_ws_bytes_tc(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens);
int aero_bwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                const void* H, const void* W, const int32_t* y, const int64_t* cs, const uint8_t* keep,
                const float* lse, const float* g, float grad_scale, void* dH, float* dW, int accumulate_dW,
                void* ws, size_t ws_bytes, const aero_bwd_extra& ex);
