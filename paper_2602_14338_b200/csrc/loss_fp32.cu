// Stage (b) in plain fp32 for small shapes (the tiny reference workload): one warp
// per token row (forward, dH) or per vocabulary row (dW).  Logits are recomputed on
// the fly and never stored.  This path exists for inputs given in fp32; the bf16
// tensor-core path is the fast one.
#include "loss_common.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kChunk = 128;             // output columns a warp accumulates at a time (4 per lane)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float dot_row(const float* __restrict__ a, const float* __restrict__ b, int d) {
  float acc = 0.f;
  for (int k = 0; k < d; ++k) acc = fmaf(a[k], b[k], acc);
  return acc;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
fwd_fp32_kernel(aero_cfg cfg, long long T, int d, int V, int R,
                const float* __restrict__ H, const float* __restrict__ W, const int32_t* __restrict__ y,
                const float* __restrict__ old_logp, const int64_t* __restrict__ cs,
                const float* __restrict__ adv, const float* __restrict__ wgt, const uint8_t* __restrict__ keep,
                float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ g,
                double* __restrict__ partials, uint32_t* status, aero_fwd_extra ex) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * kWarpsPerBlock;
  for (long long t = warp0; t < T; t += nwarps) {
    double* pr = partials + (size_t)t * kPartialStride;
    const int i = ex.logprob_only ? 0 : aero_owner(cs, R, t);
    const bool kp = ex.logprob_only ? true : keep[i] != 0;
    const int yt = y[t];
    const bool bad = yt < 0 || yt >= V;
    if (bad && kp && lane == 0) aero_raise(status, AERO_ST_BAD_TARGET);
    if (!kp || bad) {
      if (lane == 0) {
        logp[t] = 0.f; lse[t] = 0.f;
        if (g) g[t] = 0.f;
        if (ex.entropy) ex.entropy[t] = 0.f;
        for (int k = 0; k < kPartialStride; ++k) pr[k] = 0.0;
      }
      continue;
    }
    const float* h = H + (size_t)t * d;
    // running sums over every column but the target's own: with a = z_y - m the log-prob is
    // -log(1 + l e^-a), which keeps the relative accuracy of 1 - p_y for a confident token
    float m = -INFINITY, l = 0.f, sz = 0.f;       // sz = sum_{v != y} exp(z_v - m) z_v, for the entropy
    for (int v = lane; v < V; v += 32) {
      if (v == yt) continue;
      const float z = dot_row(h, W + (size_t)v * d, d);
      const float mn = fmaxf(m, z);
      const float sc = __expf(m - mn), e = __expf(z - mn);
      l = l * sc + e;
      sz = sz * sc + e * z;
      m = mn;
    }
    const float M = warp_max(m);
    const float sc = m > -INFINITY ? __expf(m - M) : 0.f;
    l = warp_sum(l * sc);
    sz = warp_sum(sz * sc);
    if (lane == 0) {
      const float zy = dot_row(h, W + (size_t)yt * d, d);
      float ls = zy, lp = 0.f, ent = 0.f;         // (a vocabulary of one: p_y = 1)
      if (l > 0.f) {
        const float a = zy - M, big = fmaxf(a, 0.f);
        const float ey = expf(a - big), lr = l * expf(-big);
        ls = M + big + logf(lr + ey);
        lp = a > -30.f ? -log1pf(l * expf(-a)) : a - logf(l + expf(a));
        ent = ls - (sz * expf(-big) + ey * zy) / (lr + ey);      // H = lse - E_p[z]
      }
      logp[t] = lp; lse[t] = ls;
      if (ex.entropy) ex.entropy[t] = ent;
      for (int k = 0; k < kPartialStride; ++k) pr[k] = 0.0;
      if (!ex.logprob_only) {
        const SurrogateOut so = aero_surrogate(lp, old_logp[t], adv[i], wgt[i], cfg.clip_lo, cfg.clip_hi);
        float gt = so.g, obj = so.s;              // per-token objective: s - beta D + c_H H
        if (ex.ref_logp) {
          const float q = ex.ref_logp[t] - lp;
          const float eq = __expf(q);
          obj -= ex.kl_beta * (eq - q - 1.f);
          gt += ex.kl_beta * wgt[i] * (1.f - eq);
        }
        if (ex.entropy) obj += ex.ent_coef * ent;
        g[t] = gt;
        pr[0] = (double)wgt[i] * (double)obj;
        pr[1] = so.clipped;
        pr[2] = so.rho;
        pr[3] = (double)old_logp[t] - (double)lp;
        pr[4] = 1.0;
      }
    }
  }
}

// Per-row constants of dz = gs * (g (1[v=y] - p) + e p (z - lse + H)) = 1[v=y] coef + p (c0 + et z).
struct RowDz { float coef, c0, et; };
// One entry of a dz row.  The target column is coef (1 - p_y) + et p_y (log p_y + H) with
// 1 - p_y = -expm1(log p_y), log p_y being the forward's log-prob when it is given.
__device__ __forceinline__ float dz_entry(const RowDz& rd, float z, float ls, bool is_target, const float* logp, long long t) {
  const float base = __expf(z - ls) * fmaf(rd.et, z, rd.c0);
  if (!is_target) return base;
  const float lp = logp ? logp[t] : z - ls;
  return -rd.coef * expm1f(lp) + __expf(lp) * (fmaf(rd.et, z, rd.c0) + rd.coef);
}
__device__ __forceinline__ RowDz row_dz(long long t, float gs, const float* __restrict__ g, const float* __restrict__ lse,
                                        const int64_t* __restrict__ cs, int R, const uint8_t* __restrict__ keep,
                                        const aero_bwd_extra& ex) {
  RowDz r;
  r.coef = g[t] * gs;
  r.c0 = -r.coef;
  r.et = 0.f;
  if (ex.entropy && ex.ent_coef != 0.f) {
    const int i = aero_owner(cs, R, t);
    if (keep[i]) {
      r.et = ex.ent_coef * ex.w[i] * gs;
      r.c0 += r.et * (ex.entropy[t] - lse[t]);
    }
  }
  return r;
}

// dH[t, :] = g_t * gs * (W[y_t, :] - sum_v p_tv W[v, :]), one warp per token row.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_dh_fp32_kernel(long long T, int d, int V, const float* __restrict__ H, const float* __restrict__ W,
                   const int32_t* __restrict__ y, const float* __restrict__ lse, const float* __restrict__ g,
                   float gs, float* __restrict__ dH, const int64_t* __restrict__ cs, int R,
                   const uint8_t* __restrict__ keep, aero_bwd_extra ex) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * kWarpsPerBlock;
  for (long long t = warp0; t < T; t += nwarps) {
    const RowDz rd = row_dz(t, gs, g, lse, cs, R, keep, ex);
    float* out = dH + (size_t)t * d;
    if (rd.coef == 0.f && rd.et == 0.f) {
      for (int k = lane; k < d; k += 32) out[k] = 0.f;
      continue;
    }
    const float* h = H + (size_t)t * d;
    const float ls = lse[t];
    const int yt = y[t];
    for (int c0 = 0; c0 < d; c0 += kChunk) {
      float acc[kChunk / 32];
#pragma unroll
      for (int q = 0; q < kChunk / 32; ++q) acc[q] = 0.f;
      for (int v = 0; v < V; ++v) {
        const float* wv = W + (size_t)v * d;
        float part = 0.f;
        for (int k = lane; k < d; k += 32) part = fmaf(h[k], wv[k], part);
        const float z = warp_sum(part);
        const float dz = dz_entry(rd, z, ls, v == yt, ex.logp, t);
#pragma unroll
        for (int q = 0; q < kChunk / 32; ++q) {
          const int k = c0 + q * 32 + lane;
          if (k < d) acc[q] = fmaf(dz, wv[k], acc[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < kChunk / 32; ++q) {
        const int k = c0 + q * 32 + lane;
        if (k < d) out[k] = acc[q];
      }
    }
  }
}

// dW[v, :] (+)= sum_t dz_tv H[t, :], one warp per vocabulary row, tokens in order.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_dw_fp32_kernel(long long T, int d, int V, const float* __restrict__ H, const float* __restrict__ W,
                   const int32_t* __restrict__ y, const float* __restrict__ lse, const float* __restrict__ g,
                   float gs, float* __restrict__ dW, int accumulate, const int64_t* __restrict__ cs, int R,
                   const uint8_t* __restrict__ keep, aero_bwd_extra ex) {
  const int lane = threadIdx.x & 31;
  const int warp0 = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * kWarpsPerBlock;
  for (int v = warp0; v < V; v += nwarps) {
    const float* wv = W + (size_t)v * d;
    float* out = dW + (size_t)v * d;
    for (int c0 = 0; c0 < d; c0 += kChunk) {
      float acc[kChunk / 32];
#pragma unroll
      for (int q = 0; q < kChunk / 32; ++q) acc[q] = 0.f;
      for (long long t = 0; t < T; ++t) {
        const RowDz rd = row_dz(t, gs, g, lse, cs, R, keep, ex);
        if (rd.coef == 0.f && rd.et == 0.f) continue;
        const float* h = H + (size_t)t * d;
        float part = 0.f;
        for (int k = lane; k < d; k += 32) part = fmaf(h[k], wv[k], part);
        const float z = warp_sum(part);
        const float dz = dz_entry(rd, z, lse[t], v == y[t], ex.logp, t);
#pragma unroll
        for (int q = 0; q < kChunk / 32; ++q) {
          const int k = c0 + q * 32 + lane;
          if (k < d) acc[q] = fmaf(dz, h[k], acc[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < kChunk / 32; ++q) {
        const int k = c0 + q * 32 + lane;
        if (k < d) out[k] = accumulate ? out[k] + acc[q] : acc[q];
      }
    }
  }
}

}  // namespace

size_t aero_fwd_ws_bytes_fp32(int64_t T, int32_t R) {
  (void)R;
  return aero_align_up((size_t)(T > 0 ? T : 1) * kPartialStride * sizeof(double), 256);
}

int aero_fwd_fp32(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                  const float* H, const float* W, const int32_t* y, const float* old_logp,
                  const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                  float* logp, float* lse, float* g, float* loss, float* metrics, int accumulate, void* ws,
                  const aero_fwd_extra& ex) {
  double* partials = static_cast<double*>(ws);
  if (T > 0 && (R > 0 || ex.logprob_only)) {
    const long long blocks = (T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int grid = (int)(blocks < 65535 ? blocks : 65535);
    fwd_fp32_kernel<<<grid, kWarpsPerBlock * 32, 0, ctx->stream>>>(*cfg, T, d, V, R, H, W, y, old_logp, cs, adv, w,
                                                                   keep, logp, lse, g, partials, ctx->d_status, ex);
    ctx->launches += 1;
    AERO_CUDA_TRY(cudaGetLastError());
  }
  if (ex.logprob_only) return AERO_OK;
  return aero_loss_finalize(ctx, partials, (T > 0 && R > 0) ? (int)T : 0, kPartialStride, loss, metrics, accumulate);
}

int aero_bwd_fp32(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                  const float* H, const float* W, const int32_t* y, const int64_t* cs, const uint8_t* keep,
                  const float* lse, const float* g, float grad_scale, float* dH, float* dW, int accumulate_dW,
                  const aero_bwd_extra& ex) {
  (void)cfg;
  if (T > 0) {
    const long long blocks = (T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int grid = (int)(blocks < 65535 ? blocks : 65535);
    bwd_dh_fp32_kernel<<<grid, kWarpsPerBlock * 32, 0, ctx->stream>>>(T, d, V, H, W, y, lse, g, grad_scale, dH, cs, R,
                                                                      keep, ex);
    ctx->launches += 1;
    AERO_CUDA_TRY(cudaGetLastError());
  }
  const int vblocks = (V + kWarpsPerBlock - 1) / kWarpsPerBlock;
  bwd_dw_fp32_kernel<<<vblocks < 65535 ? vblocks : 65535, kWarpsPerBlock * 32, 0, ctx->stream>>>(
      T, d, V, H, W, y, lse, g, grad_scale, dW, accumulate_dW, cs, R, keep, ex);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}
