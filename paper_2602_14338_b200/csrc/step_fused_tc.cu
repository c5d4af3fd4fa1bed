// Stage (b), forward and backward in one call on the tensor-core path.  Token tiles are processed
// in chunks; per chunk:
//   lmhead_kernel<MODE_FWD_P>  logits, online log-sum-exp, Eq. 2, and p~ = exp(z - c_t) in bf16 into
//                              the chunk's tiled block (instead of recomputing the logits later)
//   merge_kernel               (large d only) merges the running states of the vocabulary splits
//   scale_dz_kernel            dz = gs (g_t 1[v = y_t] - g_t exp(c_t - lse_t) p~), in place (the target's entry
//                              as -gs g_t expm1(logp_t), not by subtraction from the rounded p~)
//   gemm_kernel<DH>, <DW>      dH rows of the chunk, dW += dz^T H
// When every row has one shift c_t (one vocabulary split, or several that share the shift) it has
// one factor s_t = -gs g_t exp(c_t - lse_t), and the rewriting pass is replaced by
//   row_factors_kernel         p~[t, y_t] = expm1(logp_t) exp(lse_t - c_t), i.e. lowered by the row's sum of p~
//                              (so that dz = s_t p~), s_t, and the chunk's rows of H times s_t
//   gemm_kernel<DH>, <DW>      dH = s_t (p~ W) with the factor applied to the finished tile,
//                              dW += p~^T (s H)
//   range_fix_kernel           rows in which bf16 could not hold exp(z - c_t) (a logit more than ~87 above the
//                              shift; the forward lists them) get their dz row recomputed from H and W
// and once at the end the fixed-order reduction of the loss partials.
#include "gemm_bwd_kernel.cuh"
#include "lmhead_kernel.cuh"
#include "tmap.cuh"

#include <vector>

namespace {

inline long long ldz_of(int32_t V) { return ((long long)V + 63) / 64 * 64; }
// bytes of one token tile in the chunk's blocks: 128 rows of p~ / dz, and of the scaled H rows if used
inline size_t chunk_tile_bytes(int32_t d, int32_t V) {
  return (size_t)128 * ((size_t)ldz_of(V) * 2 + (size_t)d * 2);
}
constexpr int kRangeCap = 1024;      // rows per chunk the step can redo after a saturated exp(z - c_t)

struct ScaleArgs {
  __nv_bfloat16* dz;        // tiled: [tile - tile_begin][ldz / 64][128][64]
  int nblk;                 // ldz / 64
  const int32_t* tile_row;
  const int32_t* tile_valid;
  const int32_t* n_tiles;
  int tile_begin, tile_end;
  long long T;
  int V, vsplit, nvt;
  const int32_t* y;
  const float* lse;
  const float* g;
  const float* logp;
  const float* shift;       // [vsplit][T], log2 domain
  float grad_scale;
  const float* ent;         // entropy term: H_t per row,
  const float* row_et;      // ... ent_coef * w_i per row,
  const float* zmax;        // ... and the row's largest logit outside the target's column (all NULL without the term)
};

constexpr int kBlocksPerCta = 8;     // 64-column blocks one CTA rescales for its token tile

// One CTA: one token tile x kBlocksPerCta column blocks of the chunk's block, 16 bytes per thread
// and step.  Rows past the tile's run, or whose g is 0, come out as zeros (p~ is 0 or g is).
// With the entropy term (Table 9's bonus) an entry gets e_t p (log p + H_t) more, e_t = ent_coef w_i
// grad_scale, where log p comes back from the stored value: log p = log p~ + c_t - lse_t.  The
// rounding of p~ to bf16 moves that logarithm by up to 2^-8 absolute, which is nothing for the many
// small entries (the error of the entry is that times p) but would be all of the entry where one
// column holds nearly the whole probability (log p + H_t close to 0).  The two columns that can do
// so take exact logarithms: the target's from the fp32 log-prob, the largest other logit's from
// its fp32 value, kept by the forward; an entry is taken for the latter when its stored value is
// within bf16 rounding of it.
template <bool ENT>
__global__ void __launch_bounds__(256) scale_dz_kernel(ScaleArgs a) {
  const int n_tiles = min(*a.n_tiles, a.tile_end);
  const int tile = a.tile_begin + blockIdx.y;
  if (tile >= n_tiles) return;
  const int row0 = a.tile_row[tile], valid = a.tile_valid[tile];
  const int b0 = blockIdx.x * kBlocksPerCta;
  const int nb = min(kBlocksPerCta, a.nblk - b0);
  constexpr float kLog2e = 1.4426950408889634f;
  for (int e = threadIdx.x; e < nb * 128 * 8; e += 256) {
    const int blk = e / (128 * 8), r = (e / 8) % 128, seg = e % 8;
    const int b = b0 + blk;
    const long long row = (long long)row0 + r;
    uint4* ptr = reinterpret_cast<uint4*>(a.dz + (((size_t)blockIdx.y * a.nblk + b) * 128 + r) * 64 + seg * 8);
    float coef = 0.f, sc = 0.f, tgt = 0.f;
    float et = 0.f, e2 = 0.f, pe = 0.f, hent = 0.f;   // entropy term: e_t, log2 of p / p~, p / p~, H_t
    float lpm = 0.f, ptm_lo = INFINITY, ptm_hi = -INFINITY;   // ... log p of the largest other column, its p~ +- rounding
    int yt = -1;
    if (r < valid && row < a.T) {
      coef = a.g[row] * a.grad_scale;
      yt = a.y[row];
      if (ENT) et = a.row_et[row] * a.grad_scale;
      if (coef != 0.f || et != 0.f) {
        const float lp = a.logp[row];
        tgt = -coef * expm1f(lp);                   // coef (1 - p_y), exact for p_y close to 1
        // the vocabulary split that produced this column block, and its shift
        const int j = b / (lmhead::BN / 64);
        int s = 0;
        while (s + 1 < a.vsplit && j >= (int)((long long)(s + 1) * a.nvt / a.vsplit)) ++s;
        e2 = a.shift[(size_t)s * a.T + row] - a.lse[row] * kLog2e;
        pe = exp2f(e2);
        sc = -coef * pe;
        if (ENT) {
          hent = a.ent[row];
          tgt = fmaf(et * __expf(lp), lp + hent, tgt);
          lpm = a.zmax[row] - a.lse[row];
          const float ptm = exp2f(lpm * kLog2e - e2);          // what the forward stored for that column, before rounding
          ptm_lo = ptm * (1.f - 0.0059f);                      // 1.5 bf16 steps either way
          ptm_hi = ptm * (1.f + 0.0059f);
        }
      }
    }
    uint4 v = *ptr;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
    const int col0 = b * 64 + seg * 8;
    constexpr float kLn2 = 0.6931471805599453f;
    // dz = p (-coef + e_t (log p + H_t)) with p = p~ pe; an entry that underflowed to 0 stays 0
    auto entry = [&](float pt) {
      if (!ENT) return sc * pt;
      if (pt <= 0.f) return 0.f;
      const float lpv = (pt >= ptm_lo && pt <= ptm_hi) ? lpm : (__log2f(pt) + e2) * kLn2;
      return pt * fmaf(et * pe, lpv + hent, sc);
    };
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float2 f = __bfloat1622float2(h[q]);
      f.x = col0 + 2 * q == yt ? tgt : entry(f.x);
      f.y = col0 + 2 * q + 1 == yt ? tgt : entry(f.y);
      h[q] = __floats2bfloat162_rn(f.x, f.y);
    }
    *ptr = v;
  }
}

struct RowArgs {
  __nv_bfloat16* dz;        // tiled as above
  int nblk;
  const int32_t* tile_row;
  const int32_t* tile_valid;
  const int32_t* n_tiles;
  int tile_begin, tile_end;
  long long T;
  int d;
  const int32_t* y;
  const float* lse;
  const float* g;
  const float* logp;
  const float* shift;       // [T], log2 domain
  float grad_scale;
  const __nv_bfloat16* H;   // [T, d]
  __nv_bfloat16* Hs;        // [tile - tile_begin][128][d]: s_t H[t, :], zero rows where there is no token
  float* row_scale;         // [T]: s_t
};

// One warp per row of the chunk's token tiles.  dz_tv = gs g_t (1[v = y_t] - p_tv) with
// p_tv = p~_tv exp(c_t - lse_t), so with s_t = -gs g_t exp(c_t - lse_t) and the target's entry
// lowered by exp(lse_t - c_t) (the sum of the row's p~), dz = s_t p~ everywhere.  The lowered
// entry is (p_y - 1) exp(lse_t - c_t); it is written as expm1(logp_t) exp(lse_t - c_t) from the
// fp32 log-prob, because subtracting from the bf16-rounded p~_y would leave an error of
// 2^-9 p_y / (1 - p_y) relative, which is everything for a confident token.
__global__ void __launch_bounds__(256) row_factors_kernel(RowArgs a) {
  const int n_tiles = min(*a.n_tiles, a.tile_end);
  const int lt = blockIdx.x / 16;                       // 16 blocks of 8 rows per tile
  const int tile = a.tile_begin + lt;
  const int r = (blockIdx.x % 16) * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  constexpr float kLog2e = 1.4426950408889634f;
  uint4* dst = reinterpret_cast<uint4*>(a.Hs + ((size_t)lt * 128 + r) * a.d);
  float sc = 0.f;
  long long row = -1;
  if (tile < n_tiles && r < a.tile_valid[tile]) {
    row = (long long)a.tile_row[tile] + r;
    if (row >= a.T) row = -1;
  }
  if (row >= 0) {
    const float coef = a.g[row] * a.grad_scale;
    if (coef != 0.f) {
      const float e = a.shift[row] - a.lse[row] * kLog2e;
      sc = -coef * exp2f(e);
      if (lane == 0) {
        const int yt = a.y[row];
        __nv_bfloat16* pt = a.dz + (((size_t)lt * a.nblk + yt / 64) * 128 + r) * 64 + yt % 64;
        // (lse_t far above c_t: the factor s_t underflows with exp2(e) and the row's dz is zero to rounding;
        // the clamp only keeps this entry finite, so that 0 * entry stays 0)
        *pt = __float2bfloat16_rn(expm1f(a.logp[row]) * exp2f(fminf(-e, 126.f)));
      }
    }
    if (lane == 0) a.row_scale[row] = sc;
  }
  if (sc == 0.f) {
    for (int k = lane; k < a.d / 8; k += 32) dst[k] = make_uint4(0, 0, 0, 0);
  } else {
    const uint4* src = reinterpret_cast<const uint4*>(a.H + row * a.d);
    for (int k = lane; k < a.d / 8; k += 32) {
      uint4 v = src[k];
      __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __bfloat1622float2(h[q]);
        h[q] = __floats2bfloat162_rn(sc * f.x, sc * f.y);
      }
      dst[k] = v;
    }
  }
}

struct RangeArgs {
  const int* rows;          // chunk-local rows (tile in chunk * 128 + row in tile) listed by the forward
  const int* count;
  int cap;
  __nv_bfloat16* dz;        // tiled as above
  int nblk;
  const int32_t* tile_row;
  int tile_begin;
  long long T;
  int d, V;
  const int32_t* y;
  const float* lse;
  const float* g;
  const float* logp;
  float grad_scale;
  const __nv_bfloat16* H;   // [T, d]
  const __nv_bfloat16* W;   // [V, d]
  __nv_bfloat16* Hs;        // row-factor form: the row's copy of H (unscaled here); NULL otherwise
  float* row_scale;         // row-factor form: set to 1 for a redone row
  const float* ent;         // entropy term: H_t and ent_coef * w_i per row; both NULL without the term
  const float* row_et;
};

// The forward could not hold exp(z - c_t) of these rows in bf16: write their dz rows from the
// definition, one warp per (row, vocabulary column), logits as fp32 dot products of the bf16
// operands.  Rare by construction (a logit ~87 above the row's first ones), so speed is no concern;
// without listed rows the kernel reads one word and returns.
__global__ void __launch_bounds__(256) range_fix_kernel(RangeArgs a) {
  const int n = min(*a.count, a.cap);
  if (n == 0) return;
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * 8;
  const long long ldz = (long long)a.nblk * 64;
  for (long long u = warp0; u < (long long)n * ldz; u += nwarps) {
    const int e = (int)(u / ldz), v = (int)(u % ldz);
    const int local = a.rows[e], lt = local / 128, r = local % 128;
    const long long row = (long long)a.tile_row[a.tile_begin + lt] + r;
    if (row >= a.T) continue;
    const float coef = a.g[row] * a.grad_scale;
    const float et = a.row_et != nullptr ? a.row_et[row] * a.grad_scale : 0.f;
    float val = 0.f;
    if (v < a.V && (coef != 0.f || et != 0.f)) {
      const uint4* h = reinterpret_cast<const uint4*>(a.H + row * a.d);
      const uint4* w = reinterpret_cast<const uint4*>(a.W + (long long)v * a.d);
      float acc = 0.f;
      for (int k = lane; k < a.d / 8; k += 32) {
        const uint4 hv = h[k], wv = w[k];
        const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
        const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 x = __bfloat1622float2(hp[q]), yv = __bfloat1622float2(wp[q]);
          acc = fmaf(x.x, yv.x, acc);
          acc = fmaf(x.y, yv.y, acc);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      const float lpv = v == a.y[row] ? a.logp[row] : acc - a.lse[row];
      val = v == a.y[row] ? -coef * expm1f(lpv) : -coef * __expf(lpv);
      if (et != 0.f) val = fmaf(et * __expf(lpv), lpv + a.ent[row], val);
    }
    if (lane == 0) a.dz[(((size_t)lt * a.nblk + v / 64) * 128 + r) * 64 + v % 64] = __float2bfloat16_rn(val);
    if (a.Hs != nullptr && v == 0) {
      // the row's factor is already in its dz entries: unit factor, plain copy of the H row
      if (lane == 0) a.row_scale[row] = 1.f;
      const uint4* src = reinterpret_cast<const uint4*>(a.H + row * a.d);
      uint4* dst = reinterpret_cast<uint4*>(a.Hs + ((size_t)lt * 128 + r) * a.d);
      for (int k = lane; k < a.d / 8; k += 32) dst[k] = src[k];
    }
  }
}

// Entropy term: ent_coef * w_i for every token row of a kept rollout (one warp per rollout), so
// that the per-row kernels need no search for the row's owner.
__global__ void __launch_bounds__(256) row_entropy_weights_kernel(int R, const int64_t* __restrict__ cs,
                                                                  const uint8_t* __restrict__ keep,
                                                                  const float* __restrict__ w, float ent_coef,
                                                                  long long T, float* __restrict__ row_et) {
  const int lane = threadIdx.x & 31;
  const int warp0 = blockIdx.x * 8 + (threadIdx.x >> 5), nwarps = gridDim.x * 8;
  for (int i = warp0; i < R; i += nwarps) {
    const float v = keep[i] ? ent_coef * w[i] : 0.f;
    long long t1 = cs[i + 1];
    if (t1 > T) t1 = T;
    for (long long t = cs[i] + lane; t < t1; t += 32)
      if (t >= 0) row_et[t] = v;
  }
}

// dH rows of dropped rollouts are defined to be zero; one warp per row.
__global__ void __launch_bounds__(256) zero_dropped_rows_fused(long long T, int d, int R, const int64_t* __restrict__ cs,
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

struct FusedWs {
  aero_tiles tiles;
  double* partials;
  size_t n_partials;
  unsigned int* sync_ctr;
  float4* xstate;
  float* shift;
  float* row_scale;
  float* zmax;
  int* range_count;
  int* range_rows;
  __nv_bfloat16* dz;
  size_t head_bytes;
};

size_t partials_bytes(int64_t T, int32_t R) {
  const size_t mt = (size_t)(T / lmhead::BM) + (size_t)R + 2;
  return aero_align_up(mt * 4 * kPartialStride * sizeof(double), 256);
}

FusedWs carve(void* ws, int64_t T, int32_t d, int32_t R) {
  FusedWs f;
  const int vs = aero_vsplit_cap(d);
  const size_t Tn = (size_t)(T > 0 ? T : 1);
  char* p = static_cast<char*>(ws);
  f.tiles = aero_carve_tiles(ws, T, R, lmhead::BM);
  size_t off = aero_tiles_bytes(T, R, lmhead::BM);
  f.partials = reinterpret_cast<double*>(p + off);             off += partials_bytes(T, R);
  f.n_partials = (size_t)f.tiles.max_tiles * 4;
  f.sync_ctr = reinterpret_cast<unsigned int*>(p + off);       off += 256;
  f.range_count = reinterpret_cast<int*>(p + off);             off += 256;
  f.range_rows = reinterpret_cast<int*>(p + off);              off += aero_align_up(kRangeCap * sizeof(int), 256);
  f.xstate = reinterpret_cast<float4*>(p + off);               off += aero_align_up(vs * Tn * sizeof(float4), 256);
  f.shift = reinterpret_cast<float*>(p + off);                 off += aero_align_up(vs * Tn * sizeof(float), 256);
  f.row_scale = reinterpret_cast<float*>(p + off);             off += aero_align_up(Tn * sizeof(float), 256);
  f.zmax = reinterpret_cast<float*>(p + off);                  off += aero_align_up(Tn * sizeof(float), 256);
  f.dz = reinterpret_cast<__nv_bfloat16*>(p + off);
  f.head_bytes = off;
  return f;
}

}  // namespace

size_t aero_fwd_bwd_ws_bytes_tc(int64_t T, int32_t d, int32_t V, int32_t R, int64_t chunk_tokens) {
  if (chunk_tokens < 128) chunk_tokens = 128;
  const size_t tiles = (size_t)((chunk_tokens + 127) / 128);
  return carve(nullptr, T, d, R).head_bytes + aero_align_up(tiles * chunk_tile_bytes(d, V), 256);
}

int aero_fwd_bwd_tc(aero_ctx* ctx, const aero_cfg* cfg, int64_t T, int32_t d, int32_t V, int32_t R,
                    const void* H, const void* W, const int32_t* y, const float* old_logp,
                    const float* ref_logp, float kl_beta, float* entropy, float ent_coef,
                    const int64_t* cs, const float* adv, const float* w, const uint8_t* keep,
                    float* logp, float* lse, float* g, float* loss, float* metrics,
                    float grad_scale, void* dH, float* dW, int accumulate_dW, void* ws, size_t ws_bytes) {
  FusedWs f = carve(ws, T, d, R);
  const bool with_ent = entropy != nullptr;
  AERO_CUDA_TRY(cudaMemsetAsync(f.partials, 0, f.n_partials * kPartialStride * sizeof(double), ctx->stream));
  if (T > 0) {
    AERO_CUDA_TRY(cudaMemsetAsync(logp, 0, (size_t)T * sizeof(float), ctx->stream));
    AERO_CUDA_TRY(cudaMemsetAsync(lse, 0, (size_t)T * sizeof(float), ctx->stream));
    AERO_CUDA_TRY(cudaMemsetAsync(g, 0, (size_t)T * sizeof(float), ctx->stream));
    if (with_ent) AERO_CUDA_TRY(cudaMemsetAsync(entropy, 0, (size_t)T * sizeof(float), ctx->stream));
  }
  if (!accumulate_dW) AERO_CUDA_TRY(cudaMemsetAsync(dW, 0, (size_t)V * d * sizeof(float), ctx->stream));
  int rc = aero_build_tiles(ctx, T, R, cs, keep, lmhead::BM, f.tiles);
  if (rc) return rc;
  // H still arriving in slices (aero_grpo_step_host): the tile list comes to the host once, so
  // that each chunk can wait for just the slices its rows lie in
  std::vector<int32_t> tile_row_h;
  int32_t n_tiles_h = 0;
  if (ctx->n_slices > 0 && T > 0 && R > 0) {
    tile_row_h.resize((size_t)f.tiles.max_tiles);
    AERO_CUDA_TRY(cudaMemcpyAsync(tile_row_h.data(), f.tiles.tile_row, sizeof(int32_t) * (size_t)f.tiles.max_tiles,
                                  cudaMemcpyDeviceToHost, ctx->stream));
    AERO_CUDA_TRY(cudaMemcpyAsync(&n_tiles_h, f.tiles.n_tiles, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    AERO_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
  }
  if (T > 0 && R > 0) {
    const long long ldz = ldz_of(V);
    long long tpc = (long long)((ws_bytes - f.head_bytes) / chunk_tile_bytes(d, V));
    if (tpc < 1) return AERO_ERR_WORKSPACE;
    if (tpc > f.tiles.max_tiles) tpc = f.tiles.max_tiles;
    if (tpc > 32768) tpc = 32768;                                          // grid.y of the rescaling kernel
    if (tpc > ctx->sm_count) tpc = tpc / ctx->sm_count * ctx->sm_count;   // whole waves of token tiles
    {
      const long long blocks = (T + 7) / 8;
      zero_dropped_rows_fused<<<(int)(blocks < 4096 ? blocks : 4096), 256, 0, ctx->stream>>>(
          T, d, R, cs, keep, static_cast<__nv_bfloat16*>(dH));
      ctx->launches += 1;
    }
    const CUtensorMapDataType BF = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUtensorMap tmH_k, tmW_k, tmDZ_st, tmDZ_k, tmDZ_mn, tmW_mn, tmH_mn;
    const uint64_t nblk = (uint64_t)(ldz / 64);
    if ((rc = aero_make_tmap_2d(ctx, &tmH_k, BF, 2, H, T, d, d, lmhead::BM, 64))) return rc;
    if ((rc = aero_make_tmap_2d(ctx, &tmW_k, BF, 2, W, V, d, d, lmhead::BNH, 64))) return rc;
    if ((rc = aero_make_tmap_dz(ctx, &tmDZ_st, f.dz, (uint64_t)tpc, nblk, 32, 1))) return rc;
    if ((rc = aero_make_tmap_dz(ctx, &tmDZ_k, f.dz, (uint64_t)tpc, nblk, gemmbwd::BM, 1))) return rc;
    if ((rc = aero_make_tmap_dz(ctx, &tmDZ_mn, f.dz, (uint64_t)tpc, nblk, 64, gemmbwd::BM / 64))) return rc;
    if ((rc = aero_make_tmap_blocked(ctx, &tmW_mn, W, V, d, d, 64, gemmbwd::BN / 64))) return rc;
    if ((rc = aero_make_tmap_blocked(ctx, &tmH_mn, H, T, d, d, 64, gemmbwd::BN / 64))) return rc;
    // the entropy term is no multiple of p~ along a row: it takes the pass that rewrites the block, and
    // the array of row factors then holds ent_coef * w_i per row
    const bool rowscale = aero_rowscale(ctx) && !with_ent;
    if (with_ent) {
      const int blocks = (R + 7) / 8;
      row_entropy_weights_kernel<<<blocks < 4096 ? (blocks > 0 ? blocks : 1) : 4096, 256, 0, ctx->stream>>>(
          R, cs, keep, w, ent_coef, T, f.row_scale);
      ctx->launches += 1;
    }
    __nv_bfloat16* Hs = f.dz + (size_t)tpc * lmhead::BM * (size_t)ldz;      // after the chunk's p~ block
    CUtensorMap tmHs_mn;
    if (rowscale && (rc = aero_make_tmap_blocked(ctx, &tmHs_mn, Hs, tpc * lmhead::BM, d, d, 64, gemmbwd::BN / 64))) return rc;
    // CTA pairs: each CTA stages half of the B slab's columns
    const bool gemm_pairs = aero_gemm_pairs(ctx, d);
    CUtensorMap tmW_mn2, tmB_dw2;
    if (gemm_pairs) {
      if ((rc = aero_make_tmap_blocked(ctx, &tmW_mn2, W, V, d, d, 64, gemmbwd::PBNH / 64))) return rc;
      if (rowscale) rc = aero_make_tmap_blocked(ctx, &tmB_dw2, Hs, tpc * lmhead::BM, d, d, 64, gemmbwd::PBNH / 64);
      else rc = aero_make_tmap_blocked(ctx, &tmB_dw2, H, T, d, d, 64, gemmbwd::PBNH / 64);
      if (rc) return rc;
    }

    auto k_fwd = with_ent ? lmhead::lmhead_kernel<lmhead::MODE_FWD_P_ENT> : lmhead::lmhead_kernel<lmhead::MODE_FWD_P>;
    auto k_dh = gemmbwd::gemm_kernel<gemmbwd::KIND_DH>;
    auto k_dw = gemmbwd::gemm_kernel<gemmbwd::KIND_DW>;
    AERO_CUDA_TRY(cudaFuncSetAttribute(k_fwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lmhead::SMEM_BYTES));
    AERO_CUDA_TRY(cudaFuncSetAttribute(k_dh, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::SMEM_BYTES));
    AERO_CUDA_TRY(cudaFuncSetAttribute(k_dw, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::SMEM_BYTES));
    auto k_dh2 = gemmbwd::gemm_pair_kernel<gemmbwd::KIND_DH>;
    auto k_dw2 = gemmbwd::gemm_pair_kernel<gemmbwd::KIND_DW>;
    if (gemm_pairs) {
      AERO_CUDA_TRY(cudaFuncSetAttribute(k_dh2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::PSMEM_BYTES));
      AERO_CUDA_TRY(cudaFuncSetAttribute(k_dw2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemmbwd::PSMEM_BYTES));
    }

    const int vs = aero_vsplit(ctx, d);
    const int nvt = (V + lmhead::BN - 1) / lmhead::BN;
    const int n_nt = (d + gemmbwd::BN - 1) / gemmbwd::BN;
    const long long dw_units = (long long)((V + gemmbwd::BM - 1) / gemmbwd::BM) * n_nt;
    const long long max_pairs = ctx->sm_count / 2 > 0 ? ctx->sm_count / 2 : 1;
    for (long long begin = 0; begin < f.tiles.max_tiles; begin += tpc) {
      if (ctx->n_slices > 0) {
        if (begin >= n_tiles_h) break;                        // the tile list is known: no empty chunks
        const long long last_tile = (begin + tpc < n_tiles_h ? begin + tpc : (long long)n_tiles_h) - 1;
        const long long last_row = (long long)tile_row_h[(size_t)last_tile] + lmhead::BM - 1;
        long long slice = last_row / ctx->rows_per_slice;
        if (slice > ctx->n_slices - 1) slice = ctx->n_slices - 1;
        AERO_CUDA_TRY(cudaStreamWaitEvent(ctx->stream, ctx->slice_ev[slice], 0));
      }
      lmhead::Params p = {};
      p.T = T; p.d = d; p.V = V; p.R = R;
      p.tile_row = f.tiles.tile_row; p.tile_valid = f.tiles.tile_valid; p.n_tiles = f.tiles.n_tiles;
      p.tile_begin = (int)begin; p.tile_end = (int)(begin + tpc);
      p.y = y; p.status = ctx->d_status;
      p.vsplit = vs; p.xstate = f.xstate; p.sync_ctr = f.sync_ctr; p.nsync = aero_nsync(ctx); p.w_hint = aero_w_hint(ctx, true); p.k_zigzag = aero_k_zigzag(ctx);
      p.old_logp = old_logp; p.cs = cs; p.adv = adv; p.w = w;
      p.ref_logp = ref_logp; p.kl_beta = ref_logp ? kl_beta : 0.f;
      p.ent_out = entropy; p.ent_coef = with_ent ? ent_coef : 0.f; p.zmax_out = with_ent ? f.zmax : nullptr;
      p.clip_lo = cfg->clip_lo; p.clip_hi = cfg->clip_hi;
      p.logp = logp; p.lse_out = lse; p.g_out = g; p.partials = f.partials;
      p.shift_out = f.shift; p.dz = f.dz; p.ldz = ldz;
      p.common_shift = rowscale && vs > 1 ? 1 : 0;
      p.range_rows = f.range_rows; p.range_count = f.range_count; p.range_cap = kRangeCap;
      AERO_CUDA_TRY(cudaMemsetAsync(f.sync_ctr, 0, 512, ctx->stream));      // pacing counter and the range list's count
      const long long pairs = (tpc + 1) / 2 * vs;
      const int grid = 2 * (int)(pairs < max_pairs ? pairs : max_pairs);
      const bool timed = ctx->timing && ctx->n_timed < 256;
      if (timed) {
        if (!ctx->ev0[ctx->n_timed]) {
          AERO_CUDA_TRY(cudaEventCreate(&ctx->ev0[ctx->n_timed]));
          AERO_CUDA_TRY(cudaEventCreate(&ctx->ev1[ctx->n_timed]));
        }
        AERO_CUDA_TRY(cudaEventRecord(ctx->ev0[ctx->n_timed], ctx->stream));
      }
      k_fwd<<<grid, lmhead::THREADS, lmhead::SMEM_BYTES, ctx->stream>>>(tmH_k, tmW_k, tmDZ_st, p);
      if (timed) {
        AERO_CUDA_TRY(cudaEventRecord(ctx->ev1[ctx->n_timed], ctx->stream));
        ctx->n_timed += 1;
      }
      ctx->launches += 1;
      if (vs > 1) {
        lmhead::merge_kernel<<<(int)(tpc < 8 * ctx->sm_count ? tpc : 8 * ctx->sm_count), lmhead::BM, 0, ctx->stream>>>(p, with_ent ? 1 : 0);
        ctx->launches += 1;
      }
      if (rowscale) {
        RowArgs ra;
        ra.dz = f.dz; ra.nblk = (int)nblk; ra.tile_row = f.tiles.tile_row; ra.tile_valid = f.tiles.tile_valid;
        ra.n_tiles = f.tiles.n_tiles; ra.tile_begin = (int)begin; ra.tile_end = (int)(begin + tpc);
        ra.T = T; ra.d = d; ra.y = y; ra.lse = lse; ra.g = g; ra.logp = logp; ra.shift = f.shift; ra.grad_scale = grad_scale;
        ra.H = static_cast<const __nv_bfloat16*>(H); ra.Hs = Hs; ra.row_scale = f.row_scale;
        row_factors_kernel<<<(unsigned)(tpc * 16), 256, 0, ctx->stream>>>(ra);
      } else {
        ScaleArgs sa;
        sa.dz = f.dz; sa.nblk = (int)nblk; sa.tile_row = f.tiles.tile_row; sa.tile_valid = f.tiles.tile_valid;
        sa.n_tiles = f.tiles.n_tiles; sa.tile_begin = (int)begin; sa.tile_end = (int)(begin + tpc);
        sa.T = T; sa.V = V; sa.vsplit = vs; sa.nvt = nvt; sa.y = y; sa.lse = lse; sa.g = g; sa.logp = logp; sa.shift = f.shift;
        sa.grad_scale = grad_scale;
        sa.ent = entropy; sa.row_et = with_ent ? f.row_scale : nullptr; sa.zmax = with_ent ? f.zmax : nullptr;
        const dim3 sgrid((unsigned)((nblk + kBlocksPerCta - 1) / kBlocksPerCta), (unsigned)tpc);
        if (with_ent) scale_dz_kernel<true><<<sgrid, 256, 0, ctx->stream>>>(sa);
        else scale_dz_kernel<false><<<sgrid, 256, 0, ctx->stream>>>(sa);
      }
      {
        RangeArgs fa;
        fa.rows = f.range_rows; fa.count = f.range_count; fa.cap = kRangeCap; fa.dz = f.dz; fa.nblk = (int)nblk;
        fa.tile_row = f.tiles.tile_row; fa.tile_begin = (int)begin; fa.T = T; fa.d = d; fa.V = V; fa.y = y;
        fa.lse = lse; fa.g = g; fa.logp = logp; fa.grad_scale = grad_scale;
        fa.H = static_cast<const __nv_bfloat16*>(H); fa.W = static_cast<const __nv_bfloat16*>(W);
        fa.Hs = rowscale ? Hs : nullptr; fa.row_scale = rowscale ? f.row_scale : nullptr;
        fa.ent = entropy; fa.row_et = with_ent ? f.row_scale : nullptr;
        range_fix_kernel<<<2 * ctx->sm_count, 256, 0, ctx->stream>>>(fa);
      }

      gemmbwd::Params gp = {};
      gp.T = T; gp.d = d; gp.V = V; gp.ldz = ldz;
      gp.tile_row = f.tiles.tile_row; gp.tile_valid = f.tiles.tile_valid; gp.n_tiles = f.tiles.n_tiles;
      gp.tile_begin = (int)begin; gp.tpc = (int)tpc;
      gp.dH = static_cast<__nv_bfloat16*>(dH); gp.dW = dW; gp.status = ctx->d_status;
      gp.row_scale = rowscale ? f.row_scale : nullptr;
      gp.h_local = rowscale ? 1 : 0;
      gp.nsync = aero_gemm_sync(ctx);
      gp.sync_ctr = f.sync_ctr + 4;           // (the lm_head kernel's counter comes first; all zeroed above)
      const long long dh_units = tpc * n_nt;
      if (gemm_pairs) {
        const long long dh_pu = (tpc + 1) / 2 * n_nt, dw_pu = ((long long)((V + gemmbwd::BM - 1) / gemmbwd::BM) + 1) / 2 * n_nt;
        k_dh2<<<2 * (int)(dh_pu < max_pairs ? dh_pu : max_pairs), gemmbwd::THREADS, gemmbwd::PSMEM_BYTES, ctx->stream>>>(
            tmDZ_k, tmW_mn2, gp);
        gp.sync_ctr = f.sync_ctr + 8;
        k_dw2<<<2 * (int)(dw_pu < max_pairs ? dw_pu : max_pairs), gemmbwd::THREADS, gemmbwd::PSMEM_BYTES, ctx->stream>>>(
            tmDZ_mn, tmB_dw2, gp);
      } else {
        k_dh<<<(int)(dh_units < ctx->sm_count ? dh_units : ctx->sm_count), gemmbwd::THREADS, gemmbwd::SMEM_BYTES,
               ctx->stream>>>(tmDZ_k, tmW_mn, gp);
        gp.sync_ctr = f.sync_ctr + 8;
        k_dw<<<(int)(dw_units < ctx->sm_count ? dw_units : ctx->sm_count), gemmbwd::THREADS, gemmbwd::SMEM_BYTES,
               ctx->stream>>>(tmDZ_mn, rowscale ? tmHs_mn : tmH_mn, gp);
      }
      ctx->launches += 4;
      AERO_CUDA_TRY(cudaGetLastError());
    }
  }
  return aero_loss_finalize(ctx, f.partials, (int)f.n_partials, kPartialStride, loss, metrics, 0);
}
