/*
 * aero.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path of
 * a GRPO / AERO training step (AERO: "Adaptive Efficient Rollout Optimization",
 * arXiv 2602.14338).
 *
 * Two stages:
 *   (a) aero_group_stats     per-prompt group statistics over ragged groups:
 *                            group-relative advantage (Eq. 1), zero-advantage group
 *                            masking (Sec. 3.2), selective-rejection keep-mask
 *                            (Sec. 4.2, Strategies 2 and 3), Beta-Binomial posterior
 *                            update (Sec. 4.2 Strategy 2; Appendix C).
 *   (b) aero_grpo_loss_fwd   fused lm_head projection + online log-sum-exp + target
 *       aero_grpo_loss_bwd   gather, importance ratio, clip, weighted token mean
 *                            (Eq. 2; Appendix C "GRPO Training") and its backward to
 *                            dH and dW (Eq. 3; Appendix A).  The [T,V] logits are
 *                            never written to memory.
 *
 * Conventions
 *   - Packed ragged batch ("padding removal", Appendix C): prompt p owns rollouts
 *     go[p] .. go[p+1]-1, R = go[P]; rollout i owns token rows cs[i] .. cs[i+1]-1,
 *     T = cs[R].  Rollouts of one prompt are consecutive; rows of one rollout are
 *     consecutive.
 *   - W is the lm_head weight, [V,d] row-major; logits z_t = W h_t.  H is [T,d]
 *     row-major.  dtype is bf16 (tensor-core path, d % 64 == 0 and 16-byte aligned
 *     bases required) or fp32 (plain path for small shapes).
 *   - Unless a parameter says "host", every array pointer is a DEVICE pointer owned
 *     by the caller and must stay valid until the stream has run the call.  The
 *     library allocates no array memory: scratch is passed in as `workspace`.
 *   - Calls are asynchronous on the context's stream.  Host-side checks (null
 *     pointers, shapes, alignment, workspace size) fail with a negative return and
 *     launch nothing.  Data-dependent faults (target id outside [0,V), non-monotone
 *     offsets, non-binary reward, empty rollout, a pipeline wait that gave up) never
 *     trap: they set bits in a device status word read by aero_last_status, and the
 *     offending element is skipped or clamped.
 *   - Sign: the paper maximises J (Eq. 2); the library returns loss = -J, so dH and
 *     dW are descent directions.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with
 *     AERO_ERR_CUDA.
 *   - Every call that takes a context makes the context's device the calling thread's
 *     current CUDA device (cudaSetDevice) and leaves it so.
 *   - Argument checks come first and need no device: a call with a bad argument returns
 *     its error code whether or not the device is usable.
 *   - Each compute call is wrapped in an NVTX range named after the entry point.
 */
#ifndef AERO_H_
#define AERO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes ------------------------------------------------------------- */
#define AERO_OK               0
#define AERO_ERR_INVALID     -1   /* null pointer, negative size, misaligned base      */
#define AERO_ERR_UNSUPPORTED -2   /* shape the kernels do not cover (e.g. d % 64 != 0) */
#define AERO_ERR_WORKSPACE   -3   /* workspace smaller than aero_*_workspace_bytes     */
#define AERO_ERR_CUDA        -4   /* a CUDA runtime/driver call failed                 */
#define AERO_ERR_TOO_LARGE   -5   /* problem exceeds the library-owned scratch array   */

/* ---- device status bits (aero_last_status) ------------------------------------ */
#define AERO_ST_BAD_TARGET     1u   /* y[t] outside [0,V): row treated as dropped      */
#define AERO_ST_BAD_OFFSETS    2u   /* go[] or cs[] not non-decreasing                 */
#define AERO_ST_BAD_REWARD     4u   /* reward not exactly 0 or 1                       */
#define AERO_ST_EMPTY_ROLLOUT  8u   /* cs[i+1] == cs[i] for a present rollout          */
#define AERO_ST_TIMEOUT       16u   /* a bounded wait inside a kernel ran out          */
#define AERO_ST_RANGE         32u   /* aero_grpo_loss_fwd_bwd: more than 1024 rows of one chunk have a   */
                                    /* logit over 125 octaves above the shift taken from the row's first  */
                                    /* logits; the rows beyond the 1024 the call redoes have a saturated   */
                                    /* gradient (use aero_grpo_loss_fwd + aero_grpo_loss_bwd instead)      */

/* ---- enumerations ------------------------------------------------------------- */
#define AERO_UNIFORM_MASK   0   /* all-correct / all-incorrect groups are dropped (Sec. 3.2)      */
#define AERO_UNIFORM_BAYES  1   /* they use the posterior mean instead (Sec. 4.2 Strategy 2)      */
#define AERO_STATS_KEPT     0   /* mean/std over the curated subset (Theorem 4.1: mu = c/(c+m))   */
#define AERO_STATS_ALL      1   /* mean/std over every present rollout of the group               */
#define AERO_TOKEN_MEAN     0   /* token-level mean (Appendix C, "GRPO Training")                 */
#define AERO_SEQ_MEAN       1   /* 1/N sum_i 1/|o_i| sum_t (Eq. 2)                                */
#define AERO_DENOM_SURVIVING 0  /* normalise by surviving tokens / prompts                        */
#define AERO_DENOM_ALL      1   /* count dropped tokens / prompts too (the shrinking batch        */
                                /* gradient described in Sec. 3.1)                                */
#define AERO_BF16 0
#define AERO_FP32 1

#define AERO_CAT_ZERO    0      /* categories of Appendix C, threshold tau = 0.5, decided on      */
#define AERO_CAT_PARTIAL 1      /* integers: Partial iff 0 < c and 2c < n                         */
#define AERO_CAT_GOOD    2
#define AERO_CAT_PERFECT 3
#define AERO_CAT_EMPTY   4      /* no present rollout                                             */

/* Indices into counters[8] written by aero_group_stats. */
#define AERO_CNT_R_KEPT    0
#define AERO_CNT_T_KEPT    1
#define AERO_CNT_P_SURV    2
#define AERO_CNT_ZERO      3
#define AERO_CNT_PARTIAL   4
#define AERO_CNT_GOOD      5
#define AERO_CNT_PERFECT   6
#define AERO_CNT_T_PRESENT 7

/* Hyper-parameters (Table 9 of the paper gives the defaults noted here). */
typedef struct aero_cfg {
  int32_t uniform_policy;   /* AERO_UNIFORM_*                                   default MASK */
  int32_t rejection;        /* 1: Strategy 3 (keep all correct + k*c incorrect)  default 0   */
  int32_t k_ratio;          /* k >= 1, incorrect : correct ratio                 default 1   */
  int32_t rescue_S;         /* Strategy 1 threshold S on correct counts          default 0   */
  int32_t n_explore;        /* exploration budget the threshold refers to        default 8   */
  int32_t n_keep_uniform;   /* rollouts kept from a uniform group; <= 0: all     default 4   */
  int32_t stats_over;       /* AERO_STATS_*                                      default KEPT */
  int32_t agg;              /* AERO_TOKEN_MEAN | AERO_SEQ_MEAN                   default TOKEN_MEAN */
  int32_t denom;            /* AERO_DENOM_*                                      default SURVIVING */
  float   alpha0, beta0;    /* Beta prior used when alpha_in/beta_in are NULL    default 1, 1 */
  float   eps_std;          /* added to the standard deviation in Eq. 1          default 1e-6 */
  float   clip_lo, clip_hi; /* clip(rho, 1-clip_lo, 1+clip_hi)                   default 0.2, 0.2 */
  uint64_t seed;            /* seeds the default selection keys                  default 0   */
  int32_t dtype;            /* AERO_BF16 | AERO_FP32: type of H, W and dH        default BF16 */
  int32_t reject_high;      /* 1 (with rejection): also cut the correct rollouts of a     default 0   */
                            /* high-success mixed group to min(k*(n-c), c) (appendix ablation)       */
  float   kl_beta;          /* Eq. 2's beta (KL to a reference policy); read only by   default 0 */
                            /* the *_reg_* calls                                                 */
  float   ent_coef;         /* entropy bonus coefficient (Table 9: 1e-3); read only    default 0 */
                            /* by the *_reg_* calls                                              */
} aero_cfg;

typedef struct aero_ctx aero_ctx;   /* opaque: device id, borrowed stream, status word */

/* Library version (major*100 + minor). */
int aero_version(void);

/* Human-readable name of a return code (static string, never NULL). */
const char* aero_error_string(int code);

/* Fill *cfg with the defaults listed above. */
void aero_cfg_default(aero_cfg* cfg);

/* Create a context on CUDA device `device`.  `cuda_stream` (a cudaStream_t, may be
 * NULL for the default stream) is borrowed, not owned.  Allocates the 4-byte device
 * status word and nothing else. */
int aero_create(aero_ctx** out, int device, void* cuda_stream);
int aero_destroy(aero_ctx* ctx);
int aero_set_stream(aero_ctx* ctx, void* cuda_stream);

/* Return the OR of all status bits raised since the last call in *bits (host pointer)
 * and clear them.  The read and the clear are enqueued on the context's stream, which is
 * then synchronised, so they are ordered against the context's kernels on any stream. */
int aero_last_status(aero_ctx* ctx, uint32_t* bits);

/* Tuning hook (no passage of the paper: it only selects between equivalent schedules of
 * stage (b); results agree within rounding).  One setting per call, by name; a negative value
 * restores the library's own choice:
 *   "vsplit"     CTA pairs that share a pair of token tiles and split the vocabulary between
 *                them: 1, 2 or 4; 0 (the default) lets the library choose by d.
 *   "nsync"      meeting points per unit at which the lm_head kernel's producers wait for one
 *                another (bounded); 0 for none.
 *   "rowscale"   aero_grpo_loss_fwd_bwd: 1 applies the row factors inside the backward products
 *                (the default), 0 rewrites the chunk block in a pass of its own.
 *   "gemm_sync"  meeting points per unit of the two backward products' producers; 0 for none.
 *   "gemm_pairs" 1: the two backward products run on CTA pairs (units of 256 rows); 0: on
 *                single CTAs; by default pairs for d > 2048.
 *   "w_hint"     1: the lm_head kernel loads W with the evict-first L2 priority, 0: plain loads;
 *                by default 1 in the calls whose kernel stores per-row results only
 *                (aero_grpo_loss_fwd, aero_logprob_fwd), 0 where it also stores a chunk block.
 *   "k_zigzag"   1 (the default): the lm_head kernel walks the reduction dimension d forwards for
 *                even vocabulary tiles and backwards for odd ones (the H slabs used last are asked
 *                for first); 0: always forwards.  Changes the order of the fp32 sums of a logit.
 * The workspace sizes the *_workspace_bytes functions return cover every setting.  Returns
 * AERO_ERR_INVALID for an unknown name or a value outside the ones listed. */
int aero_set_tuning(aero_ctx* ctx, const char* name, int value);

/* ------------------------------------------------------------------------------
 * Stage (a).  Group statistics, curation and weights (Eq. 1; Sec. 3.2; Sec. 4.2
 * Strategies 2-3; Appendix C categories and posterior).
 *
 * For every prompt p, over its PRESENT rollouts (keep_in[i] != 0, or all when
 * keep_in is NULL): n = count, c = number with reward 1;
 *   category  Zero (c=0) / Partial (0<c, 2c<n) / Good (2c>=n, c<n) / Perfect (c=n);
 *   posterior alpha' = alpha + c, beta' = beta + n - c, u~ = alpha'/(alpha'+beta');
 *   keep-mask uniform group: none (MASK) or the min(n_keep_uniform, n) rollouts of
 *             smallest (key, index) (BAYES);  low-success mixed group with rejection:
 *             all correct + the min(k*c, n-c) incorrect of smallest (key, index),
 *             where low-success means Partial, or c*n_explore <= rescue_S*n when
 *             rescue_S > 0;  any other group: all present rollouts -- except that with
 *             reject_high (the appendix ablation "Effect of Discarding High-Success
 *             Rollouts") a mixed group that is not low-success keeps all incorrect + the
 *             min(k*(n-c), c) correct of smallest (key, index);
 *   advantage (r enters as the bit r > 0.5; a reward other than 0 or 1 raises
 *             AERO_ST_BAD_REWARD)
 *             mixed group: (r - mean)/(std + eps_std) with the population std over
 *             the kept subset (STATS_KEPT) or the present group (STATS_ALL);
 *             uniform group under BAYES: (r - u~)/(sqrt(u~(1-u~)) + eps_std);
 *             0 for every rollout that is not kept;
 *   weight    w_i = 1/T_kept (TOKEN_MEAN) or 1/(P_surv * n'_p * len_i) (SEQ_MEAN)
 *             for kept rollouts, 0 otherwise; with DENOM_ALL the denominators are the
 *             present tokens T_present, resp. all P prompts.
 * key == NULL selects the default key: the high 32 bits of SplitMix64 applied to
 * seed + (i+1) * 0x9E3779B97F4A7C15, i the global rollout index.
 *
 * Inputs   go [P+1] i32, reward [R] f32, cs [R+1] i64, key [R] u32 or NULL,
 *          keep_in [R] u8 or NULL, alpha_in/beta_in [P] f32 or both NULL.
 * Outputs  adv [R] f32, w [R] f32, keep [R] u8, gmask [P] u8 (1 iff any rollout
 *          kept), cat [P] u8, u_tilde/alpha_out/beta_out [P] f32, kept_ids [R] i32
 *          (first R_kept entries: kept rollout indices, ascending; rest -1),
 *          kept_tok_off [R+1] i64 (exclusive scan of kept lengths over kept_ids;
 *          entries past R_kept hold T_kept), counters [8] i64 (AERO_CNT_*),
 *          metrics [4] f32 or NULL: zero-accuracy ratio x^zero (Sec. 3.2), mean
 *          |advantage| over kept rollouts, kept rollout fraction, kept token fraction.
 *          Integer outputs are exact; alpha_out/beta_out may alias alpha_in/beta_in.
 * workspace: at least aero_group_workspace_bytes(P, R) bytes, 256-byte aligned.
 * P == 0 or R == 0 is valid (counters are zeroed).
 */
size_t aero_group_workspace_bytes(int32_t P, int32_t R);

int aero_group_stats(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                     const int32_t* go, const float* reward, const int64_t* cs,
                     const uint32_t* key, const uint8_t* keep_in,
                     const float* alpha_in, const float* beta_in,
                     float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                     float* u_tilde, float* alpha_out, float* beta_out,
                     int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                     float* metrics, void* workspace, size_t workspace_bytes);

/* Weights of a data-parallel shard (Eq. 2's normalisers 1/G and 1/|o_i|, and the token-level
 * mean of Appendix C, run over the whole batch; the paper trains with 2-4 data-parallel ranks,
 * Appendix C).  A rank that ran aero_group_stats on its own prompts only holds weights over its
 * local denominator.  Given its own counters and the element-wise sum of all ranks' counters
 * (both [8] i64 on the device, e.g. after an all-reduce), this call rescales w [R] in place by
 * local / global denominator: T_kept (TOKEN_MEAN) or P_surv (SEQ_MEAN), resp. T_present or
 * P_local / P_global under DENOM_ALL.  Advantages and the keep-mask are per prompt and need
 * nothing.  The loss and dW of the ranks then add up to those of the unsharded batch.  Nothing is
 * read back to the host. */
int aero_finalize_weights(aero_ctx* ctx, const aero_cfg* cfg, int32_t R, int32_t P_local, int64_t P_global,
                          float* w, const int64_t* counters_local, const int64_t* counters_global);

/* aero_group_stats for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this call: it computes exactly what aero_group_stats computes; only the
 * origin of the scratch memory differs.)
 *
 * Who needs it: code that is handed its input and output buffers but has no way to get a
 * workspace at the point of the call -- a plug-in inside a host program that owns all
 * device memory, or a latency-bound loop that must not call the allocator because an
 * allocation can synchronise the whole device.  Instead of a caller workspace, the scratch
 * is a fixed array in device memory that belongs to the loaded library itself:
 * AERO_STATIC_SCRATCH_BYTES (1,476,096 bytes, 1.41 MiB) per GPU that loads the library, held until the process exits, sized for at most
 * AERO_STATIC_MAX_PROMPTS prompts whatever their group sizes (R itself is not limited).
 * A batch beyond that limit returns AERO_ERR_TOO_LARGE and launches nothing.  The call,
 * and everything it calls, performs no cudaMalloc/cudaFree and uses no allocating library
 * routine.
 *
 * The first call on each device looks up the array's device address (once per device,
 * with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array: two calls whose kernels may overlap on the
 * GPU (different streams, or different contexts of this library on one device) race on
 * it -- order them on one stream or with events.  The array keeps the previous call's
 * contents; nothing in it has to start at zero: each call writes every word before reading it.
 * Arguments, outputs and status bits are those of aero_group_stats.
 */
#define AERO_STATIC_MAX_PROMPTS 65536
#define AERO_STATIC_SCRATCH_BYTES 1476096   /* size of that array */

int aero_group_stats_static(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                            const int32_t* go, const float* reward, const int64_t* cs,
                            const uint32_t* key, const uint8_t* keep_in,
                            const float* alpha_in, const float* beta_in,
                            float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                            float* u_tilde, float* alpha_out, float* beta_out,
                            int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                            float* metrics);

/* ------------------------------------------------------------------------------
 * Stage (b), forward (Eq. 2; Appendix C "GRPO Training").
 *
 * For every token row t of a kept rollout i (keep[i] != 0):
 *   z_tv = sum_k H[t,k] W[v,k]  (fp32 accumulation of bf16 products, never stored)
 *   lse_t = log sum_v exp z_tv,  logp_t = z_{t,y_t} - lse_t
 *   rho_t = exp(logp_t - old_logp_t)
 *   s_t   = min(rho_t A_i, clip(rho_t, 1-clip_lo, 1+clip_hi) A_i)
 *   loss  = - sum_t w_i s_t                       (loss = -J)
 *   g_t   = dloss/dlogp_t = - w_i A_i rho_t [rho_t A_i <= clip(rho_t) A_i]
 * (equality counts as unclipped; the two-sided form of Eq. 2 governs, so the
 * indicator is rho <= 1+clip_hi for A > 0 and rho >= 1-clip_lo for A < 0).
 * Rows of dropped rollouts get logp = lse = g = 0.
 *
 * Inputs   H [T,d], W [V,d] (cfg->dtype), y [T] i32, old_logp [T] f32, cs [R+1] i64,
 *          adv [R] f32, w [R] f32, keep [R] u8 (outputs of aero_group_stats).
 * Outputs  logp, lse, g [T] f32; loss [1] f32 (overwritten, or added to when
 *          accumulate != 0, for callers that split a batch into token ranges);
 *          metrics [4] f32 or NULL: clipped fraction of kept tokens, mean rho,
 *          mean (old_logp - logp), number of kept tokens.  The loss is reduced in a
 *          fixed order: repeated calls give identical bits.
 * workspace: at least aero_fwd_workspace_bytes(T, d, V, R) bytes, 256-byte aligned.
 */
size_t aero_fwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R);

int aero_grpo_loss_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                       const void* H, const void* W, const int32_t* y, const float* old_logp,
                       const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                       float* logp, float* lse, float* g, float* loss, float* metrics,
                       int accumulate, void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------------
 * Stage (b), backward (Eq. 3; Appendix A: grad rho = rho grad log pi, clipped tokens
 * contribute nothing).
 *
 *   dz_tv = grad_scale * g_t * (1[v == y_t] - exp(z_tv - lse_t))     (recomputed)
 *   dH[t,:] = sum_v dz_tv W[v,:]          dW[v,:] (+)= sum_t dz_tv H[t,:]
 * dz is rounded to bf16 before the two products (fp32 accumulation).  Token rows
 * are processed in chunks whose dz block lives in `workspace`; a larger workspace
 * means fewer passes over dW.  Rows of dropped rollouts get dH = 0.
 * The target column is formed as -grad_scale g_t expm1(logp_t): for a confident token
 * (p close to 1, where Eq. 3's factor 1 - p is tiny) this keeps the relative accuracy of
 * the log-prob, which 1 - exp(z - lse_t) loses to the rounding of lse_t.  logp is the
 * forward's output; NULL falls back to z_{t,y_t} - lse_t recomputed in fp32 (relative error
 * of that entry about 4e-6 / (1 - p)).
 *
 * Inputs   as the forward, plus lse, g and (optionally) logp from it.
 * Outputs  dH [T,d] (cfg->dtype); dW [V,d] f32, overwritten or, when
 *          accumulate_dW != 0, added to.
 * workspace: at least aero_bwd_workspace_bytes(T, d, V, R, chunk_tokens); chunk_tokens
 *          (a multiple of 128, >= 128) is the number of token rows per chunk the
 *          caller is prepared to pay for; the call uses as many as the given
 *          workspace_bytes allows.
 */
size_t aero_bwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens);

int aero_grpo_loss_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                       const void* H, const void* W, const int32_t* y,
                       const int64_t* cs, const uint8_t* keep,
                       const float* lse, const float* g, const float* logp, float grad_scale,
                       void* dH, float* dW, int accumulate_dW,
                       void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------------
 * Stage (b), forward and backward in one call (Eq. 2, Eq. 3; same results as
 * aero_grpo_loss_fwd followed by aero_grpo_loss_bwd, same arguments).
 *
 * The two separate calls must recompute the logits in the backward (8 d V FLOP per token).
 * Called together, the forward of each chunk of token rows also leaves
 * p~_tv = exp(z_tv - c_t) in bf16 in the chunk's scratch block, c_t being a per-row shift taken
 * from the row's first logits; when lse_t and g_t are known the block stands for
 * dz_tv = grad_scale (g_t 1[v == y_t] - g_t exp(c_t - lse_t) p~_tv) (the row factor is applied inside
 * the backward products, or by a pass that rewrites the block), and dH, dW follow as in
 * aero_grpo_loss_bwd: 6 d V FLOP per token.  bf16 shares fp32's exponent range, so p~ carries the
 * same 2^-9 relative rounding dz has in the two-call path; the target column is written from the
 * fp32 log-prob as -grad_scale g_t expm1(logp_t), never by subtracting from the rounded p~.  A row
 * with a logit too far above its shift for bf16 to hold (about 87 above the largest of the row's
 * first 32 logits) is redone from H and W by a kernel of its own, up to 1024 such rows per chunk
 * (beyond: AERO_ST_RANGE).  Neither the logits nor anything of size [T,V] is stored: the scratch
 * block is one chunk of rows of unnormalised probabilities, where the backward's holds dz.
 *
 * workspace: at least aero_fwd_bwd_workspace_bytes(T, d, V, R, chunk_tokens), 256-byte aligned.
 * fp32 inputs run the two plain calls one after the other.
 */
size_t aero_fwd_bwd_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens);

int aero_grpo_loss_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y, const float* old_logp,
                           const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                           float* logp, float* lse, float* g, float* loss, float* metrics,
                           float grad_scale, void* dH, float* dW, int accumulate_dW,
                           void* workspace, size_t workspace_bytes);

/* aero_grpo_loss_fwd_bwd with Eq. 2's KL term: ref_logp [T] f32 (NULL: no KL term, the call is
 * aero_grpo_loss_fwd_bwd) and cfg->kl_beta, defined as for aero_grpo_loss_reg_fwd below.  The term
 * only changes loss and g_t, so it costs nothing in the backward. */
int aero_grpo_loss_kl_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                              const void* H, const void* W, const int32_t* y, const float* old_logp,
                              const float* ref_logp,
                              const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                              float* logp, float* lse, float* g, float* loss, float* metrics,
                              float grad_scale, void* dH, float* dW, int accumulate_dW,
                              void* workspace, size_t workspace_bytes);

/* aero_grpo_loss_fwd_bwd with both regularisers of Eq. 2 and Table 9 (defined with
 * aero_grpo_loss_reg_fwd below): ref_logp [T] f32 or NULL as above, entropy [T] f32 out or NULL (NULL:
 * no entropy term; with both NULL the call is aero_grpo_loss_fwd_bwd).  The entropy term of dz needs
 * log p_tv per entry; the step takes it back from the stored block, log p_tv = log p~_tv + c_t - lse_t,
 * in the pass that rewrites the block to dz (the row-factor form does not apply: the term is no
 * multiple of p~ along a row).  The bf16 rounding of p~ moves that logarithm by at most 2^-9
 * absolute; the target column uses the fp32 log-prob.  An entry whose p~ underflowed to 0 gets 0
 * (p log p -> 0).  6 d V FLOP per token plus one pass over the chunk block, against 8 d V through
 * aero_grpo_loss_reg_fwd + aero_grpo_loss_reg_bwd. */
int aero_grpo_loss_reg_fwd_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                               const void* H, const void* W, const int32_t* y, const float* old_logp,
                               const float* ref_logp,
                               const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                               float* logp, float* lse, float* g, float* entropy, float* loss, float* metrics,
                               float grad_scale, void* dH, float* dW, int accumulate_dW,
                               void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------------
 * Stage (b) with the regularisers of Eq. 2 and Table 9.
 *
 * Per kept token of rollout i, with D_t = exp(q_t) - q_t - 1, q_t = ref_logp_t - logp_t
 * (a non-negative per-token estimate of Eq. 2's D_KL[pi_theta || pi_ref]; the paper does
 * not print the estimator, this is the one GRPO uses) and H_t = -sum_v p_tv log p_tv the
 * entropy of the token's distribution (Table 9 "entropy coefficient"):
 *   loss  = sum_t w_i ( -s_t + kl_beta D_t - ent_coef H_t )
 *   g_t   = -w_i A_i rho_t [unclipped] + kl_beta w_i (1 - exp(q_t))
 *   dz_tv = grad_scale ( g_t (1[v == y_t] - p_tv) + ent_coef w_i p_tv (log p_tv + H_t) )
 * The entropy is carried through the same online pass as the log-sum-exp
 * (H_t = lse_t - sum_v p_tv z_tv); nothing of size [T,V] is stored.
 *
 * aero_grpo_loss_reg_fwd: arguments of aero_grpo_loss_fwd plus ref_logp [T] f32 (NULL:
 *   no KL term, kl_beta ignored) and entropy [T] f32 out (NULL: no entropy term,
 *   ent_coef ignored).  With both NULL it is aero_grpo_loss_fwd.
 * aero_grpo_loss_reg_bwd: arguments of aero_grpo_loss_bwd (logp included, may be NULL) plus
 *   entropy [T] from the forward and w [R] (both NULL: no entropy term).
 * aero_logprob_fwd: the log-prob pass alone over all T rows (what produces old_logp and
 *   ref_logp, Appendix C "Rollout"/"GRPO Training"): logp, lse [T] f32 and, if not NULL,
 *   entropy [T] f32.  Workspace: aero_fwd_workspace_bytes(T, d, V, 0).
 */
int aero_grpo_loss_reg_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y, const float* old_logp,
                           const float* ref_logp,
                           const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                           float* logp, float* lse, float* g, float* entropy, float* loss, float* metrics,
                           int accumulate, void* workspace, size_t workspace_bytes);

int aero_grpo_loss_reg_bwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                           const void* H, const void* W, const int32_t* y,
                           const int64_t* cs, const uint8_t* keep,
                           const float* lse, const float* g, const float* logp,
                           const float* entropy, const float* w,
                           float grad_scale, void* dH, float* dW, int accumulate_dW,
                           void* workspace, size_t workspace_bytes);

int aero_logprob_fwd(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V,
                     const void* H, const void* W, const int32_t* y,
                     float* logp, float* lse, float* entropy,
                     void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------------
 * One whole step of the path from HOST buffers: stage (a), forward and backward
 * (the same operations and citations as the three calls above), for callers whose
 * rollout batch lives in host memory.  The call copies the batch to the device,
 * runs aero_group_stats and aero_grpo_loss_fwd_bwd on the context's
 * stream, copies the scalars back and synchronises the stream before returning.
 * H, the bulk of the bytes, is copied in 16 slices on a second stream that the context
 * owns; each chunk of the forward waits only for the slices its token rows lie in (the
 * call reads the chunks' row ranges back once, after the group stage), so with pinned
 * host memory most of the transfer runs under the first chunks' kernels.
 *
 * HOST inputs (pinned memory makes the copies asynchronous): go_h [P+1] i32,
 *   reward_h [R] f32, cs_h [R+1] i64, key_h [R] u32 or NULL, alpha_h/beta_h [P] f32 or
 *   both NULL, H_h [T,d] (cfg->dtype), y_h [T] i32, old_logp_h [T] f32.
 * DEVICE arrays: W [V,d] (the resident weight), dH [T,d] and dW [V,d] f32 (outputs, as in
 *   aero_grpo_loss_bwd), workspace of at least aero_step_workspace_bytes(...) bytes,
 *   256-byte aligned; it holds the staged inputs and every intermediate array.
 * HOST outputs: loss_h [1] f32, counters_h [8] i64 (AERO_CNT_*), metrics_h [8] f32 (the
 *   four group metrics followed by the four token metrics); any may be NULL.
 * Errors as above; the status word is read with aero_last_status.
 */
size_t aero_step_workspace_bytes(int32_t P, int32_t R, int64_t T, int32_t d, int32_t V, int64_t chunk_tokens,
                                 int32_t dtype);

int aero_grpo_step_host(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R, int64_t T, int32_t d, int32_t V,
                        const int32_t* go_h, const float* reward_h, const int64_t* cs_h, const uint32_t* key_h,
                        const float* alpha_h, const float* beta_h,
                        const void* H_h, const int32_t* y_h, const float* old_logp_h,
                        const void* W, void* dH, float* dW, int accumulate_dW,
                        float* loss_h, int64_t* counters_h, float* metrics_h,
                        void* workspace, size_t workspace_bytes);

/* ------------------------------------------------------------------------------
 * Rollout allocation controller of one training step, simulated on P prompts with hidden
 * success rates (Algorithm 1; Sec. 4.2 Strategy 1; Appendix C "AERO": categorisation,
 * iterative rejection sampling with increment 2 for at most 10 iterations, n_p <= 32,
 * sum_p n_p <= 16 |P|).  No language model is involved: rollout j (in generation order) of
 * prompt p is correct iff the draw -- the high 32 bits of SplitMix64 applied to
 * cfg->seed + (p * n_max + j + 1) * 0x9E3779B97F4A7C15 -- is below thr[p]
 * (thr[p] = floor(u_p * 2^32) for success rate u_p).
 *   1. exploration: cfg->n_explore rollouts per prompt, c_p of them correct;
 *   2. rescue set: c_p <= cfg->rescue_S.  In each of up to k_max iterations every prompt
 *      still in the set asks for min(n_extra, n_max - n_p) more rollouts (asking for none
 *      leaves the set); requests are granted in prompt order while their running sum stays
 *      within what is left of n_budget * P (the paper does not say how a short budget is
 *      shared); a granted prompt draws its rollouts and leaves the set as soon as one is
 *      correct;
 *   3. n_train[p]: the number of rollouts the curation rule of aero_group_stats keeps from
 *      a group with n_p rollouts of which c_p are correct.
 * Inputs   thr [P] u32.   Outputs  n_gen, c, n_train [P] i32; counters [8] i64: rollouts
 *          generated, rollouts kept for training, zero-accuracy prompts after exploration,
 *          zero-accuracy prompts at the end, prompts rescued, iterations that granted
 *          anything, budget left, P.  All outputs are integers and exact.
 * workspace: at least aero_allocate_workspace_bytes(P) bytes, 256-byte aligned.
 */
typedef struct aero_alloc_cfg {
  int32_t n_extra;    /* rescue increment (Strategy 1 "n_extra, e.g., 2")        default 2  */
  int32_t k_max;      /* iterations (Appendix C)                                  default 10 */
  int32_t n_max;      /* per-prompt cap (Appendix C)                              default 32 */
  int32_t n_budget;   /* mean rollouts per prompt the step may spend (Appendix C) default 16 */
} aero_alloc_cfg;

void aero_alloc_cfg_default(aero_alloc_cfg* ac);
size_t aero_allocate_workspace_bytes(int32_t P);
int aero_allocate_sim(aero_ctx* ctx, const aero_cfg* cfg, const aero_alloc_cfg* ac, int32_t P, const uint32_t* thr,
                      int32_t* n_gen, int32_t* c, int32_t* n_train, int64_t* counters,
                      void* workspace, size_t workspace_bytes);

/* Optional timing of the dominant kernel.  With timing on, aero_grpo_loss_fwd_bwd records a pair of
 * CUDA events on the context's stream around each launch of its lm_head kernel (up to 256 launches
 * between read-outs; the events are created on first use).  aero_kernel_timing_ms synchronises the
 * stream, returns the summed duration and the number of launches since the last read-out (host
 * pointers) and starts over.  Off by default; meant for benchmarks. */
int aero_enable_kernel_timing(aero_ctx* ctx, int on);
int aero_kernel_timing_ms(aero_ctx* ctx, float* total_ms, int* launches);

/* Self-test of the bounded waits (no passage of the paper).  Every wait inside the tensor-core
 * kernels gives up after a time limit, raises AERO_ST_TIMEOUT and lets the kernel end normally.
 * This call launches a one-warp kernel of its own that waits, for at most limit_us microseconds
 * (1 .. 1000000), on a barrier nobody arrives at: afterwards aero_last_status must report
 * AERO_ST_TIMEOUT and the context must be usable as before.  Nothing else is touched. */
int aero_selftest_bounded_wait(aero_ctx* ctx, uint32_t limit_us);

/* Number of kernels the library has launched through this context since it was created
 * (copies and memsets are not counted).  Host-side counter, no synchronisation. */
int64_t aero_launch_count(aero_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif  /* AERO_H_ */
