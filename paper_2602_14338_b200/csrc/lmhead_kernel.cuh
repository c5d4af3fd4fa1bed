// Token-stationary lm_head kernel: for each 128-row token tile, walk all vocabulary
// tiles of 256 columns; logits z = H W^T are accumulated in TMEM by tcgen05.mma from
// bf16 operands staged by TMA, and consumed straight from TMEM by the epilogue warps.
// The logits never reach shared or global memory.
//
//   MODE_FWD : online log-sum-exp over vocabulary tiles + target pick, then the clipped
//              surrogate of Eq. 2 per token (logp, lse, g, per-tile loss partials), with the
//              KL-to-reference term when a reference log-prob is given; or, without old
//              log-probs, the log-probs alone.
//   MODE_DZ  : dz = coef_t * (1[v == y_t] - exp(z - lse_t)) rounded to bf16 and stored to
//              the chunk's scratch block (Eq. 3 through the softmax).
//   MODE_FWD_P : the forward of a fused step.  Besides the log-probs it stores, for its chunk of
//              token tiles, p~ = exp(z - c_t) in bf16 into the block the dz mode would write,
//              with one shift c_t per row and vocabulary split (the row's first logits plus a
//              margin: bf16 has fp32's exponent range, so any c_t within ~85 of the row's
//              log-sum-exp loses nothing but the usual 2^-9 relative rounding).  Once lse_t and
//              g_t are known, dz = g_t 1[v=y_t] - g_t exp(c_t - lse_t) p~ is an element-wise
//              rescale of that block (scale_dz_kernel), which replaces the recompute of the
//              logits in the backward: 6 d V instead of 8 d V FLOP per token.
//   The _ENT variants add the entropy bonus (Table 9): the forward also carries
//   sum_v exp(z - m) z, giving H_t = lse_t - E_p[z]; the backward adds
//   e_t p_tv (z_tv - lse_t + H_t) to dz, e_t = ent_coef * w_i.
//
// CTAs work in pairs (a cluster of two, tcgen05 cta_group::2): the pair takes two token tiles,
// one per CTA, and one MMA covers both (M = 256).  Each CTA stages its own 128 rows of H and
// only half of the 256 W rows of the vocabulary tile; the tensor cores of the pair share the
// two halves, so a CTA moves 32 KB per 64-deep slab instead of 48 KB.  Each CTA's TMEM holds
// the 128 x 256 logits of its own token tile.
//
// Warp roles (192 threads, one CTA per SM): warps 0-3 epilogue (warp q reads TMEM lanes
// 32q..32q+31, one token row per thread), warp 4 TMA producer, warp 5 TMEM owner and, in the
// CTA of cluster rank 0, MMA issuer for the pair.  Two 256-column TMEM accumulators let the
// MMA of vocabulary tile j+1 overlap the epilogue of tile j.
//
// Barriers: full[s] lives in the rank-0 CTA and collects the bytes of both CTAs' loads;
// empty[s] and tfull[b] exist in both CTAs and are signalled for both by the issuer's commits;
// tempty[b] lives in the rank-0 CTA and counts the eight epilogue warps of the pair.
#pragma once

#include "loss_common.cuh"
#include "tc_ptx.cuh"

namespace lmhead {

#ifndef AERO_TC_STAGES
#define AERO_TC_STAGES 6          // depth of the TMA -> MMA shared-memory ring
#endif
// BM rows of H per CTA, BN vocabulary columns per accumulator, BNH of them staged by each CTA
constexpr int BM = 128, BN = 256, BNH = BN / 2, BK = 64, STAGES = AERO_TC_STAGES, UMMA_K = 16;
constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BNH * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 192;
// bit 0: dz mode, bit 1: entropy term, bit 2: the forward also stores exp(z - c_t) of the chunk (see MODE_FWD_P)
constexpr int MODE_FWD = 0, MODE_DZ = 1, MODE_FWD_ENT = 2, MODE_DZ_ENT = 3, MODE_FWD_P = 4, MODE_FWD_P_ENT = 6;
constexpr float kShiftMargin = 40.f;   // c_t = (largest logit of the row's first 32 columns) + this margin
constexpr float kMasked = -1e30f;   // stands for -inf in columns past V (finite, so that 0 * z stays 0)
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

struct Ctl {
  uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};
// dz staging for the TMA stores of MODE_DZ: per epilogue warp two buffers of 32 rows x 64 bf16
constexpr uint32_t STG_BUF_BYTES = 32 * 64 * 2, STG_BYTES = 4 * 2 * STG_BUF_BYTES;
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES + STG_BYTES + sizeof(Ctl);

struct Params {
  long long T;
  int d, V, R;
  const int32_t* tile_row;
  const int32_t* tile_valid;
  const int32_t* n_tiles;
  int tile_begin, tile_end;     // this launch covers tiles [tile_begin, min(tile_end, *n_tiles))
  const int32_t* y;
  uint32_t* status;
  // Vocabulary split: `vsplit` CTA pairs share a pair of token tiles and walk 1/vsplit of the
  // vocabulary tiles each, so that the H tiles all CTAs re-read from L2 (148 * 128 * d * 2 bytes,
  // 136 MB at d = 3584) shrink to what L2 holds.  Forward modes then leave the per-row running
  // state in xstate [vsplit][T] for merge_kernel instead of finishing the row.
  int vsplit;
  float4* xstate;
  // Pacing: all CTAs re-read the same W tiles from L2, which only works while they walk the
  // vocabulary in step; small rate differences between SMs add up over a long launch.  The
  // producers therefore meet at `nsync` points per unit on a counter in global memory
  // (zeroed before the launch).  The wait is short and bounded: a CTA that is not there in time
  // is simply not waited for.
  unsigned int* sync_ctr;
  int nsync;
  // W tiles are needed by all their sharers within microseconds of one another (pacing) and not
  // again before the next wave of token tiles; a CTA's own H tile is needed again for every
  // vocabulary tile.  With w_hint the W loads carry the evict-first priority, so that the stream
  // of W lines is what L2 gives up first and the H tiles stay.
  int w_hint;
  // With k_zigzag the producer walks the reduction dimension forwards for even vocabulary tiles and
  // backwards for odd ones, so that the slabs of the CTA's own H tile it used last are the ones it
  // asks for first: a cyclic walk is the worst case for a cache that gives up the oldest lines.  The
  // order depends on the tile index alone, so a tile's sums are the same whichever CTA computes it.
  int k_zigzag;
  const int64_t* cs;
  const float* w;
  float ent_coef;
  // forward modes
  const float* old_logp;        // NULL: log-probs only, no objective
  const float* ref_logp;        // NULL: no KL term
  const float* adv;
  float clip_lo, clip_hi, kl_beta;
  float* logp;
  float* lse_out;
  float* g_out;
  float* ent_out;               // entropy per row (entropy modes)
  float* zmax_out;              // largest logit of the row outside the target's column, or NULL (-inf if there is none)
  float* shift_out;             // MODE_FWD_P: c_t * log2(e) per split and row, [vsplit][T]
  int common_shift;             // MODE_FWD_P with vsplit > 1: every split takes c_t from the row's first 32 logits
                                // of the whole vocabulary (the later splits compute that tile once more for it)
  // MODE_FWD_P: rows with a logit too far above c_t for bf16 to hold exp(z - c_t) are listed here (row index
  // inside the chunk) so that the step can redo them; AERO_ST_RANGE is raised only if the list overflows
  int* range_rows;
  int* range_count;
  int range_cap;
  double* partials;             // [tile][4 epilogue warps][kPartialStride]
  // dz modes
  const float* lse_in;
  const float* g_in;
  const float* logp_in;         // NULL, or the forward's log-probs: the target column is then -coef expm1(logp_t)
  const float* ent_in;
  float grad_scale;
  __nv_bfloat16* dz;            // tiled: [tile - tile_begin][ldz / 64][128 rows][64 columns]
  long long ldz;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// End of a token row in the forward modes: log-sum-exp, log-prob, entropy, then Eq. 2 (with the
// KL term when a reference is given) and the warp's record of loss partials.  Called by the four
// epilogue warps of a tile (warp = 0..3), with the merged running state of the row.
// The running state leaves the target's own column out: m2 is the largest of the other logits
// (log2 domain), l = sum_{v != y} 2^(z_v log2e - m2), sz = sum_{v != y} 2^(..) z_v.  With
// a = z_y log2e - m2 the log-prob is -log(1 + l 2^-a): for a confident token (l 2^-a tiny) this
// keeps the relative accuracy of 1 - p_y = l / (l + 2^a), which z_y - lse loses to the rounding
// of lse at the magnitude of the logits and to the rounding of a sum that sits next to 1.
__device__ __forceinline__ void finish_rows(const Params& p, bool ent_mode, bool live, long long row, int tile, int warp,
                                            int lane, float m2, float l, float zy, float sz) {
  double part[kPartialStride] = {0.0, 0.0, 0.0, 0.0, 0.0};
  if (live) {
    float ls, lp, ent = 0.f;
    if (l > 0.f) {
      const float a = fmaf(zy, kLog2e, -m2);               // the target's exponent relative to m2
      const float big = fmaxf(a, 0.f);                     // everything below is scaled by 2^-big: no overflow
      const float ey = exp2f(a - big), lr = l * exp2f(-big);
      ls = (m2 + big + log2f(lr + ey)) * kLn2;
      lp = a > -40.f ? -log1pf(l * exp2f(-a)) : (a - log2f(l + exp2f(a))) * kLn2;
      if (ent_mode) ent = ls - (sz * exp2f(-big) + ey * zy) / (lr + ey);       // H = lse - E_p[z]
    } else {                                               // no other column carries weight: p_y = 1
      ls = zy;
      lp = 0.f;
    }
    p.logp[row] = lp;
    p.lse_out[row] = ls;
    if (ent_mode) p.ent_out[row] = ent;
    if (p.zmax_out != nullptr) p.zmax_out[row] = l > 0.f ? m2 * kLn2 : -INFINITY;
    if (p.old_logp != nullptr) {
      const int i = aero_owner(p.cs, p.R, row);
      const float old = p.old_logp[row];
      const float wi = p.w[i];
      const SurrogateOut so = aero_surrogate(lp, old, p.adv[i], wi, p.clip_lo, p.clip_hi);
      float g = so.g;
      float obj = so.s;                              // per-token objective: s - beta D + c_H H
      if (p.ref_logp != nullptr) {
        const float q = p.ref_logp[row] - lp;
        const float eq = __expf(q);
        obj -= p.kl_beta * (eq - q - 1.f);
        g += p.kl_beta * wi * (1.f - eq);
      }
      if (ent_mode) obj += p.ent_coef * ent;
      p.g_out[row] = g;
      part[0] = (double)wi * (double)obj;
      part[1] = so.clipped;
      part[2] = so.rho;
      part[3] = (double)old - (double)lp;
      part[4] = 1.0;
    }
  }
  // fixed-shape reduction: a shuffle tree per warp; the four warps' records are
  // added later by the finalising kernel in a fixed order
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int k = 0; k < kPartialStride; ++k) part[k] += __shfl_xor_sync(0xffffffffu, part[k], o);
  if (lane == 0)
    for (int k = 0; k < kPartialStride; ++k) p.partials[((size_t)tile * 4 + warp) * kPartialStride + k] = part[k];
}

// Forward modes with a vocabulary split: one block of 128 threads per token tile merges the
// vsplit running states of each row and finishes it.
static __global__ void __launch_bounds__(BM) merge_kernel(const Params p, int ent_mode) {
  const int n_tiles = min(*p.n_tiles, p.tile_end);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int tile = p.tile_begin + blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long row = (long long)p.tile_row[tile] + threadIdx.x;
    const bool valid_row = (int)threadIdx.x < p.tile_valid[tile] && row < p.T;
    int yt = -1;
    if (valid_row) yt = p.y[row];
    const bool live = valid_row && yt >= 0 && yt < p.V;      // a bad target was reported by the lm_head kernel
    float m2 = -INFINITY, l = 0.f, zy = 0.f, sz = 0.f;
    if (live) {
      for (int s = 0; s < p.vsplit; ++s) {
        const float4 o = p.xstate[(size_t)s * p.T + row];
        const float mm = fmaxf(m2, o.x);
        const float sa = ex2(m2 - mm), sb = ex2(o.x - mm);
        l = l * sa + o.y * sb;
        sz = sz * sa + o.w * sb;
        zy += o.z;
        m2 = mm;
      }
    }
    finish_rows(p, ent_mode != 0, live, row, tile, warp, lane, m2, l, zy, sz);
  }
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
lmhead_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW,
              const __grid_constant__ CUtensorMap tmDZ, const Params p) {
  constexpr bool IS_DZ = (MODE & 1) != 0, ENT = (MODE & 2) != 0, STORE_P = (MODE & 4) != 0;
  constexpr bool STORES = IS_DZ || STORE_P;       // the epilogue writes a tile of the chunk's block
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stg_all = smem + (size_t)STAGES * STAGE_BYTES;
  Ctl* ctl = reinterpret_cast<Ctl*>(stg_all + STG_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t rank = tc::cluster_ctarank();        // 0 issues the MMAs of the pair
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&ctl->full[s], 1); tc::mbar_init(&ctl->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&ctl->tfull[b], 1); tc::mbar_init(&ctl->tempty[b], 8); }
    ctl->abort = 0;
    tc::fence_barrier_init();
  }
  if (warp == 4 && lane == 0) { tc::prefetch_tmap(&tmH); tc::prefetch_tmap(&tmW); }
  if (warp == 5) { tc::tmem_alloc_pair(&ctl->tmem_base, 512); tc::tmem_relinquish_pair(); }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();        // the peer's barriers exist before anything signals them
  tc::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort;

  const int n_tiles = min(*p.n_tiles, p.tile_end);
  const int nkb = p.d / BK;
  const int nvt = (p.V + BN - 1) / BN;
  // The pair's k-th unit is token tiles first, first + 1 (the second may not exist: its CTA
  // then stages the first tile's rows again and discards the result) and one of the vsplit
  // ranges of vocabulary tiles; the pairs that share tiles are neighbours.
  const int vsplit = p.vsplit;
  auto unit_first = [&](int k) { return p.tile_begin + 2 * ((pair + k * npairs) / vsplit); };
  auto unit_j0 = [&](int k) { return (int)((long long)((pair + k * npairs) % vsplit) * nvt / vsplit); };
  auto unit_j1 = [&](int k) { return (int)((long long)((pair + k * npairs) % vsplit + 1) * nvt / vsplit); };
  // with a common shift, a unit of a later split starts with vocabulary tile 0, used for the shift alone
  auto unit_pre = [&](int k) { return (STORE_P && p.common_shift && (pair + k * npairs) % vsplit != 0) ? 1 : 0; };

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      unsigned int meetings = 0;
      const uint64_t pol_w = tc::l2_policy_evict_first();
      // every CTA takes part in the same number of meetings: units of the longest schedule x nsync
      const int total_units = ((n_tiles - p.tile_begin + 1) / 2) * vsplit;
      const int max_units = total_units > 0 ? (total_units + npairs - 1) / npairs : 0;
      for (int k = 0; ok && unit_first(k) < n_tiles; ++k) {
        const int mine = unit_first(k) + (int)rank;
        const int row0 = p.tile_row[mine < n_tiles ? mine : unit_first(k)];
        int next_meet = 0;
        for (int j0 = unit_j0(k), jj = j0 - unit_pre(k), j1 = unit_j1(k); ok && jj < j1; ++jj) {
          const int j = jj < j0 ? 0 : jj;
          if (p.nsync > 0 && next_meet < p.nsync && jj - j0 >= (int)((long long)next_meet * (j1 - j0) / p.nsync)) {
            ++next_meet;
            ++meetings;
            atomicAdd(p.sync_ctr, 1u);
            const unsigned int target = meetings * gridDim.x;
            const unsigned long long t0 = tc::globaltimer_ns();
            while (*reinterpret_cast<volatile unsigned int*>(p.sync_ctr) < target) {
              if (tc::globaltimer_ns() - t0 > 200000ull) break;       // 0.2 ms: go on alone
              __nanosleep(200);
            }
          }
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            if (!tc::mbar_wait(&ctl->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
            uint8_t* a_s = smem + (size_t)s * STAGE_BYTES;
            const uint32_t full0 = tc::mapa_shared(tc::smem_u32(&ctl->full[s]), 0);
            if (rank == 0) tc::mbar_arrive_expect_tx(&ctl->full[s], 2 * STAGE_BYTES);
            const int kx = (p.k_zigzag && (j & 1) ? nkb - 1 - kb : kb) * BK;
            tc::tma_load_2d_pair(a_s, &tmH, kx, row0, full0);
            if (p.w_hint) tc::tma_load_2d_pair_hint(a_s + A_BYTES, &tmW, kx, j * BN + (int)rank * BNH, full0, pol_w);
            else tc::tma_load_2d_pair(a_s + A_BYTES, &tmW, kx, j * BN + (int)rank * BNH, full0);
          }
        }
        // a unit whose range has fewer vocabulary tiles than meeting points still counts them all
        if (p.nsync > 0 && next_meet < p.nsync) {
          atomicAdd(p.sync_ctr, (unsigned)(p.nsync - next_meet));
          meetings += (unsigned)(p.nsync - next_meet);
        }
      }
      // out of units: stand in for the meetings the longest schedule still has
      if (p.nsync > 0 && meetings < (unsigned)(max_units * p.nsync))
        atomicAdd(p.sync_ctr, (unsigned)(max_units * p.nsync) - meetings);
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = tc::make_idesc_bf16(2 * BM, BN, 0, 0);
      uint32_t it = 0, at = 0;
      bool ok = true;
      for (int k = 0; ok && unit_first(k) < n_tiles; ++k) {
        for (int j = unit_j0(k) - unit_pre(k), j1 = unit_j1(k); ok && j < j1; ++j, ++at) {
          const uint32_t buf = at & 1u, aph = (at >> 1) & 1u;
          if (!tc::mbar_wait(&ctl->tempty[buf], aph ^ 1u, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t tmem_d = tmem_base + buf * BN;
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            if (!tc::mbar_wait(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const uint32_t a_addr = tc::smem_u32(smem + (size_t)s * STAGE_BYTES);
            const uint64_t adesc = tc::make_smem_desc(a_addr, 16, 1024);
            const uint64_t bdesc = tc::make_smem_desc(a_addr + A_BYTES, 16, 1024);
#pragma unroll
            for (int kk = 0; kk < BK / UMMA_K; ++kk) {
              // advance 32 bytes (16 bf16) inside the 128-byte swizzle row: +2 in 16-byte units
              tc::umma_bf16_pair(tmem_d, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
            }
            tc::umma_commit_pair(&ctl->empty[s], 3);     // frees the stage in both CTAs when these MMAs retire
          }
          if (ok) tc::umma_commit_pair(&ctl->tfull[buf], 3);
        }
      }
    }
  } else {
    // ---------------- epilogue warps 0..3 ----------------
    uint32_t at = 0, nstore = 0;
    bool ok = true;
    const int r_in_tile = warp * 32 + lane;
    uint8_t* stg_warp = stg_all + warp * 2 * STG_BUF_BYTES;
    const uint64_t pol_store = tc::l2_policy_evict_first();
    for (int k = 0; ok && unit_first(k) < n_tiles; ++k) {
      const int tile = unit_first(k) + (int)rank;
      const bool have_tile = tile < n_tiles;
      const long long row = have_tile ? (long long)p.tile_row[tile] + r_in_tile : 0;
      const bool valid_row = have_tile && r_in_tile < p.tile_valid[tile] && row < p.T;
      int yt = -1;
      if (valid_row) yt = p.y[row];
      const bool bad_y = valid_row && (yt < 0 || yt >= p.V);
      if (bad_y) { aero_raise(p.status, AERO_ST_BAD_TARGET); yt = -1; }
      const bool live = valid_row && !bad_y;

      float m2 = -INFINITY, l = 0.f, zy = 0.f, sz = 0.f;   // forward running state (log2 domain); sz = sum e^(z-m) z
      float c2 = 0.f;                                      // MODE_FWD_P: shift of the stored exponentials, log2 domain
      bool c2_set = false;                                 // ... taken from vocabulary tile 0 by a later split
      float lse2 = 0.f, coef = 0.f, et = 0.f, c0 = 0.f;     // dz per-row constants: dz = 1[y] coef + p (c0 + et z)
      float ls_nat = 0.f, lp_row = 0.f, ent_row = 0.f;      // ... and what the target column needs besides
      bool have_lp = false;
      if (IS_DZ) {
        if (live) {
          const float ls = p.lse_in[row];
          ls_nat = ls;
          lse2 = ls * kLog2e;
          coef = p.g_in[row] * p.grad_scale;
          c0 = -coef;
          if (p.logp_in != nullptr) { lp_row = p.logp_in[row]; have_lp = true; }
          if (ENT) {
            et = p.ent_coef * p.w[aero_owner(p.cs, p.R, row)] * p.grad_scale;
            ent_row = p.ent_in[row];
            c0 += et * (ent_row - ls);
          }
        }
      }
      // Target column of a dz row: coef (1 - p_y) + et p_y (log p_y + H_t), with 1 - p_y = -expm1(log p_y)
      // so that a confident token (p_y close to 1) keeps the relative accuracy of its log-prob.
      auto dz_target = [&](float z) {
        const float lpy = have_lp ? lp_row : z - ls_nat;
        float v = -coef * expm1f(lpy);
        if (ENT) v = fmaf(et * __expf(lpy), lpy + ent_row, v);
        return v;
      };
      bool range_hit = false;                              // MODE_FWD_P: exp(z - c_t) saturated somewhere in this row

      for (int j0 = unit_j0(k), jj = j0 - unit_pre(k), j1 = unit_j1(k); ok && jj < j1; ++jj, ++at) {
        const int j = jj < j0 ? 0 : jj;
        const uint32_t buf = at & 1u, aph = (at >> 1) & 1u;
        // the TMEM loads below are warp-collective: take the decision for the whole warp
        if (!__all_sync(0xffffffffu, tc::mbar_wait(&ctl->tfull[buf], aph, abort_flag))) { ok = false; break; }
        tc::tc_fence_after();
        if (!have_tile) {
          // nothing to read: hand the accumulator straight back
          tc::tc_fence_before();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive_cluster(tc::mapa_shared(tc::smem_u32(&ctl->tempty[buf]), 0));
          continue;
        }
        if (jj < j0) {
          // vocabulary tile 0 again, for the shift alone: the row's first 32 logits
          uint32_t r0[32];
          __syncwarp();
          tc::tmem_ld_32x32(tmem_base + ((uint32_t)(warp * 32) << 16) + buf * BN, r0);
          tc::tmem_ld_wait();
          // (the same 32 logits the first split sees: columns past V and the target's own masked)
          float cmax = yt == 0 ? kMasked : __uint_as_float(r0[0]);
#pragma unroll
          for (int q = 1; q < 32; ++q) cmax = fmaxf(cmax, (q < p.V && q != yt) ? __uint_as_float(r0[q]) : kMasked);
          c2 = fmaf(cmax + kShiftMargin, kLog2e, 0.f);
          c2_set = true;
          tc::tc_fence_before();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive_cluster(tc::mapa_shared(tc::smem_u32(&ctl->tempty[buf]), 0));
          continue;
        }
        const int col_base = j * BN;
        const int ncol = min(BN, (STORES ? (int)p.ldz : p.V) - col_base);
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + buf * BN;
        // 32 columns of this thread's row as 16 packed words -> half of the row's 128-byte line in the
        // staging buffer (16-byte chunks XOR-swizzled with the row, matching the store's tensor map);
        // every second call sends the 32 x 64 buffer to the chunk's block.
        auto stage_store = [&](const uint32_t (&pk)[16], int c, int col0) {
          const int half = c & 1;
          if (half == 0) {
            // the buffer is free once the store issued two blocks ago has read it
            if (lane == 0) tc::tma_store_wait_read<1>();
            __syncwarp();
          }
          uint8_t* stg = stg_warp + (nstore & 1u) * STG_BUF_BYTES;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int chunk = (half * 4 + q) ^ (lane & 7);
            *reinterpret_cast<uint4*>(stg + lane * 128 + chunk * 16) =
                make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
          }
          if (half == 1) {
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              // p~ is read back only by the rescaling pass, long after it has left L2: do not let it
              // push the H and W tiles out on its way
              if (STORE_P) tc::tma_store_4d_hint(&tmDZ, stg, 0, warp * 32, (col0 - 32) / 64, tile - p.tile_begin, pol_store);
              else tc::tma_store_4d(&tmDZ, stg, 0, warp * 32, (col0 - 32) / 64, tile - p.tile_begin);
              tc::tma_store_commit();
            }
            ++nstore;
          }
        };
        // One 32-column chunk of this thread's row, already in registers.
        auto process = [&](const uint32_t (&r)[32], int c) {
          const int col0 = col_base + c * 32;
          if (!IS_DZ) {
            float z[32];
#pragma unroll
            for (int q = 0; q < 32; ++q) z[q] = __uint_as_float(r[q]);
            if (col0 + 32 > p.V) {
#pragma unroll
              for (int q = 0; q < 32; ++q) if (col0 + q >= p.V) z[q] = kMasked;
            }
            if ((unsigned)(yt - col0) < 32u) {
              // the target's column is kept out of the running sums (see finish_rows)
              const int sel = yt - col0;
#pragma unroll
              for (int q = 0; q < 32; ++q) if (q == sel) { zy = z[q]; z[q] = kMasked; }
            }
            float cmax = z[0];
#pragma unroll
            for (int q = 1; q < 32; ++q) cmax = fmaxf(cmax, z[q]);
            const float m2n = fmaxf(m2, cmax * kLog2e);
            if (STORE_P && !c2_set && m2 == -INFINITY) c2 = fmaf(cmax + kShiftMargin, kLog2e, 0.f);   // first chunk of the row
            float acc = 0.f, accz = 0.f;
            if (STORE_P) {
              // e^(z - c) = e^(z - m) * 2^(m2 - c2): one extra multiply per logit
              const float d2 = m2n - c2;
              range_hit |= live && d2 > 126.f;
              const float sc = live ? ex2(fminf(d2, 126.f)) : 0.f;
              uint32_t pk[16];
#pragma unroll
              for (int q = 0; q < 32; q += 2) {
                const float e0 = ex2(fmaf(z[q], kLog2e, -m2n)), e1 = ex2(fmaf(z[q + 1], kLog2e, -m2n));
                acc += e0 + e1;
                if (ENT) accz = fmaf(e0, z[q], fmaf(e1, z[q + 1], accz));
                pk[q >> 1] = pack_bf16(e0 * sc, e1 * sc);
              }
              stage_store(pk, c, col0);
            } else {
#pragma unroll
              for (int q = 0; q < 32; ++q) {
                const float e = ex2(fmaf(z[q], kLog2e, -m2n));
                acc += e;
                if (ENT) accz = fmaf(e, z[q], accz);
              }
            }
            const float scale = ex2(m2 - m2n);
            l = fmaf(l, scale, acc);
            if (ENT) sz = fmaf(sz, scale, accz);
            m2 = m2n;
          } else {
            // 32 columns -> 16 packed words -> half of this row's 128-byte line in the staging
            // buffer (16-byte chunks XOR-swizzled with the row, matching the store's tensor map)
            uint32_t pk[16];
            if (live && col0 + 32 <= p.V) {
              float v[32];
#pragma unroll
              for (int q = 0; q < 32; ++q) {
                const float z = __uint_as_float(r[q]);
                const float pr = ex2(fmaf(z, kLog2e, -lse2));
                v[q] = ENT ? pr * fmaf(et, z, c0) : c0 * pr;
              }
              if ((unsigned)(yt - col0) < 32u) {
                // (the target's logit is picked out first, so that its formula is instantiated once, not per column)
                const int sel = yt - col0;
                float zs = 0.f;
#pragma unroll
                for (int q = 0; q < 32; ++q) if (q == sel) zs = __uint_as_float(r[q]);
                const float tv = dz_target(zs);
#pragma unroll
                for (int q = 0; q < 32; ++q) if (q == sel) v[q] = tv;
              }
#pragma unroll
              for (int q = 0; q < 32; q += 2) pk[q >> 1] = pack_bf16(v[q], v[q + 1]);
            } else {
              float tv = 0.f;
              if (live && (unsigned)(yt - col0) < 32u) {
                const int sel = yt - col0;
                float zs = 0.f;
#pragma unroll
                for (int q = 0; q < 32; ++q) if (q == sel) zs = __uint_as_float(r[q]);
                tv = dz_target(zs);
              }
#pragma unroll
              for (int q = 0; q < 32; q += 2) {
                const float z0 = __uint_as_float(r[q]), z1 = __uint_as_float(r[q + 1]);
                float v0 = ex2(fmaf(z0, kLog2e, -lse2)) * (ENT ? fmaf(et, z0, c0) : c0);
                float v1 = ex2(fmaf(z1, kLog2e, -lse2)) * (ENT ? fmaf(et, z1, c0) : c0);
                if (col0 + q == yt) v0 = tv;
                if (col0 + q + 1 == yt) v1 = tv;
                if (!live || col0 + q >= p.V) v0 = 0.f;
                if (!live || col0 + q + 1 >= p.V) v1 = 0.f;
                pk[q >> 1] = pack_bf16(v0, v1);
              }
            }
            stage_store(pk, c, col0);
          }
        };
        // TMEM loads are software-pipelined: the load of chunk c+1 is in flight while chunk c
        // is processed (every load is warp-collective, hence the __syncwarp before each)
        const int nch = (ncol + 31) / 32;
        uint32_t ra[32], rb[32];
        __syncwarp();
        tc::tmem_ld_32x32(taddr, ra);
        for (int c = 0; c < nch; c += 2) {
          tc::tmem_ld_wait();
          if (c + 1 < nch) { __syncwarp(); tc::tmem_ld_32x32(taddr + (c + 1) * 32, rb); }
          process(ra, c);
          if (c + 1 < nch) {
            tc::tmem_ld_wait();
            if (c + 2 < nch) { __syncwarp(); tc::tmem_ld_32x32(taddr + (c + 2) * 32, ra); }
            process(rb, c + 1);
          }
        }
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive_cluster(tc::mapa_shared(tc::smem_u32(&ctl->tempty[buf]), 0));
      }

      if (STORE_P && ok && have_tile && live) p.shift_out[(size_t)((pair + k * npairs) % vsplit) * p.T + row] = c2;
      if (STORE_P && range_hit) {
        const int slot = atomicAdd(p.range_count, 1);
        if (slot < p.range_cap) p.range_rows[slot] = (tile - p.tile_begin) * BM + r_in_tile;
        else aero_raise(p.status, AERO_ST_RANGE);
      }
      if (!IS_DZ && ok && have_tile) {
        if (vsplit > 1) {
          if (live) p.xstate[(size_t)((pair + k * npairs) % vsplit) * p.T + row] = make_float4(m2, l, zy, sz);
        } else {
          finish_rows(p, ENT, live, row, tile, warp, lane, m2, l, zy, sz);
        }
      }
    }
  }

  // ---------------- teardown ----------------
  if (STORES && warp < 4 && lane == 0) tc::tma_store_wait_all<0>();   // own stores have landed
  __syncwarp();
  if (*abort_flag) {
    // a wait gave up: let copies and MMAs already in flight land before shared memory and
    // TMEM are released
    const unsigned long long t0 = tc::globaltimer_ns();
    while (tc::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc::tc_fence_before();
  __syncthreads();
  // neither CTA may leave, or free its TMEM, while the other can still signal its barriers,
  // read its shared memory or write its accumulators
  tc::cluster_sync_all();
  if (threadIdx.x == 0 && *abort_flag) aero_raise(p.status, AERO_ST_TIMEOUT);
  if (warp == 5) {
    tc::tc_fence_after();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace lmhead
