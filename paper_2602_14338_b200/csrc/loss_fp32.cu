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
                double* __restrict__ partials, uint32_t* status) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * kWarpsPerBlock;
  for (long long t = warp0; t < T; t += nwarps) {
    double* pr = partials + (size_t)t * kPartialStride;
    const int i = aero_owner(cs, R, t);
    const int yt = y[t];
    const bool bad = yt < 0 || yt >= V;
    if (bad && keep[i] && lane == 0) aero_raise(status, AERO_ST_BAD_TARGET);
    if (!keep[i] || bad) {
      if (lane == 0) {
        logp[t] = 0.f; lse[t] = 0.f; g[t] = 0.f;
        for (int k = 0; k < kPartialStride; ++k) pr[k] = 0.0;
      }
      continue;
    }
    const float* h = H + (size_t)t * d;
    float m = -INFINITY, l = 0.f;
    for (int v = lane; v < V; v += 32) {
      const float z = dot_row(h, W + (size_t)v * d, d);
      const float mn = fmaxf(m, z);
      l = l * __expf(m - mn) + __expf(z - mn);
      m = mn;
    }
    const float M = warp_max(m);
    l = warp_sum(l * __expf(m - M));
    const float ls = M + __logf(l);
    if (lane == 0) {
      const float zy = dot_row(h, W + (size_t)yt * d, d);
      const float lp = zy - ls;
      const SurrogateOut so = aero_surrogate(lp, old_logp[t], adv[i], wgt[i], cfg.clip_lo, cfg.clip_hi);
      logp[t] = lp; lse[t] = ls; g[t] = so.g;
      pr[0] = (double)wgt[i] * (double)so.s;
      pr[1] = so.clipped;
      pr[2] = so.rho;
      pr[3] = (double)old_logp[t] - (double)lp;
      pr[4] = 1.0;
    }
  }
}

// dH[t, :] = g_t * gs * (W[y_t, :] - sum_v p_tv W[v, :]), one warp per token row.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
bwd_dh_fp32_kernel(long long T, int d, int V, const float* __restrict__ H, const float* __restrict__ W,
                   const int32_t* __restrict__ y, const float* __restrict__ lse, const float* __restrict__ g,
                   float gs, float* __restrict__ dH) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * kWarpsPerBlock;
  for (long long t = warp0; t < T; t += nwarps) {
    const float gt = g[t] * gs;
    float* out = dH + (size_t)t * d;
    if (gt == 0.f) {
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
        const float dz = gt * ((v == yt ? 1.f : 0.f) - __expf(z - ls));
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
                   float gs, float* __restrict__ dW, int accumulate) {
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
        const float gt = g[t] * gs;
        if (gt == 0.f) continue;
        const float* h = H + (size_t)t * d;
        float part = 0.f;
        for (int k = lane; k < d; k += 32) part = fmaf(h[k], wv[k], part);
        const float z = warp_sum(part);
        const float dz = gt * ((v == y[t] ? 1.f : 0.f) - __expf(z - lse[t]));
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
                  float* logp, float* lse, float* g, float* loss, float* metrics, int accumulate, void* ws) {
  double* partials = static_cast<double*>(ws);
  if (T > 0 && R > 0) {
    const long long blocks = (T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int grid = (int)(blocks < 65535 ? blocks : 65535);
    fwd_fp32_kernel<<<grid, kWarpsPerBlock * 32, 0, ctx->stream>>>(*cfg, T, d, V, R, H, W, y, old_logp, cs, adv, w,
                                                                   keep, logp, lse, g, partials, ctx->d_status);
    ctx->launches += 1;
    AERO_CUDA_TRY(cudaGetLastError());
  }
  return aero_loss_finalize(ctx, partials, (T > 0 && R > 0) ? (int)T : 0, kPartialStride, loss, metrics, accumulate);
}

int aero_bwd_fp32(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                  const float* H, const float* W, const int32_t* y, const int64_t* cs, const uint8_t* keep,
                  const float* lse, const float* g, float grad_scale, float* dH, float* dW, int accumulate_dW) {
  (void)cfg; (void)cs; (void)keep; (void)R;
  if (T > 0) {
    const long long blocks = (T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int grid = (int)(blocks < 65535 ? blocks : 65535);
    bwd_dh_fp32_kernel<<<grid, kWarpsPerBlock * 32, 0, ctx->stream>>>(T, d, V, H, W, y, lse, g, grad_scale, dH);
    ctx->launches += 1;
    AERO_CUDA_TRY(cudaGetLastError());
  }
  const int vblocks = (V + kWarpsPerBlock - 1) / kWarpsPerBlock;
  bwd_dw_fp32_kernel<<<vblocks < 65535 ? vblocks : 65535, kWarpsPerBlock * 32, 0, ctx->stream>>>(
      T, d, V, H, W, y, lse, g, grad_scale, dW, accumulate_dW);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}
