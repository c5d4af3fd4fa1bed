// The two products of the backward pass over one chunk of token tiles, on tcgen05/TMEM
// with TMA-fed bf16 operands and fp32 accumulation:
//
//   KIND_DH : dH[rows of the chunk, :]  = dz[rows, V] * W[V, d]       (reduce over vocabulary)
//   KIND_DW : dW[V, d]                 += dz[rows, V]^T * H[rows, d]  (reduce over the chunk's rows)
//
// dz is the chunk's scratch block written by the lm_head kernel in dz mode, stored as contiguous
// [128 rows][64 columns] tiles (tile-major, then column block).  W and H are
// used as stored (row-major, d contiguous), i.e. as MN-major B operands; dz is a K-major
// A operand for dH and an MN-major A operand for dW, so nothing is transposed in memory.
// Output tiles are 128 x 256; a unit is one output tile, units are numbered row-tile-major
// so that CTAs running at the same time share operand tiles through L2.
// Warp roles as in the lm_head kernel: warps 0-3 epilogue, warp 4 TMA, warp 5 MMA.
#pragma once

#include "loss_common.cuh"
#include "tc_ptx.cuh"

namespace gemmbwd {

#ifndef AERO_TC_STAGES
#define AERO_TC_STAGES 4          // depth of the TMA -> MMA shared-memory ring
#endif
constexpr int BM = 128, BN = 256, BK = 64, STAGES = AERO_TC_STAGES, UMMA_K = 16;
constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr uint32_t BOX_BYTES = 64 * 64 * 2;     // one 64 x 64 bf16 box of an MN-major operand
constexpr int THREADS = 192;
constexpr int KIND_DH = 0, KIND_DW = 1;

struct Ctl {
  uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES + sizeof(Ctl);

struct Params {
  long long T;
  int d, V;
  long long ldz;
  const int32_t* tile_row;
  const int32_t* tile_valid;
  const int32_t* n_tiles;
  int tile_begin, tpc;          // the chunk covers tiles [tile_begin, tile_begin + tpc) below *n_tiles
  __nv_bfloat16* dH;
  float* dW;
  uint32_t* status;
  const float* row_scale;       // dH: factor of each token row, applied to the finished tile (NULL: none)
  int h_local;                  // dW: operand B holds the chunk's rows tile after tile, not all T rows
  // Pacing: CTAs that run at the same time share operand tiles through L2 (the units of one row tile read the
  // same dz tiles, the units of one column tile the same W or H slab), which works only while they walk the
  // reduction dimension in step; small rate differences between SMs add up over the dozens of units a CTA
  // processes.  The producers therefore meet `nsync` times per unit on a counter in global memory (zeroed
  // before the launch).  The wait is short and bounded: a CTA that is not there in time is not waited for.
  unsigned int* sync_ctr;
  int nsync;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int KIND>
__global__ void __launch_bounds__(THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + (size_t)STAGES * STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&ctl->full[s], 1); tc::mbar_init(&ctl->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&ctl->tfull[b], 1); tc::mbar_init(&ctl->tempty[b], 4); }
    ctl->abort = 0;
    tc::fence_barrier_init();
  }
  if (warp == 4 && lane == 0) { tc::prefetch_tmap(&tmA); tc::prefetch_tmap(&tmB); }
  if (warp == 5) { tc::tmem_alloc(&ctl->tmem_base, 512); tc::tmem_relinquish(); }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort;

  int chunk_tiles = *p.n_tiles - p.tile_begin;
  chunk_tiles = chunk_tiles < 0 ? 0 : (chunk_tiles > p.tpc ? p.tpc : chunk_tiles);
  const int n_nt = (p.d + BN - 1) / BN;
  const int n_mt = KIND == KIND_DH ? chunk_tiles : (p.V + BM - 1) / BM;
  const int nkb = KIND == KIND_DH ? (int)(p.ldz / BK) : chunk_tiles * (BM / BK);
  const int n_units = nkb > 0 ? n_mt * n_nt : 0;

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int row_cur = 0, row_next = 0;
      unsigned int meetings = 0;
      const int max_units = (n_units + (int)gridDim.x - 1) / (int)gridDim.x;     // of the longest schedule
      for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
        const int mt = u / n_nt, nt = u % n_nt;
        int next_meet = 0;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          if (p.nsync > 0 && next_meet < p.nsync && kb >= (int)((long long)next_meet * nkb / p.nsync)) {
            ++next_meet;
            ++meetings;
            atomicAdd(p.sync_ctr, 1u);
            const unsigned int target = meetings * gridDim.x;
            const unsigned long long t0 = tc::globaltimer_ns();
            while (*reinterpret_cast<volatile unsigned int*>(p.sync_ctr) < target) {
              if (tc::globaltimer_ns() - t0 > 50000ull) break;        // 50 us: go on alone
              __nanosleep(100);
            }
          }
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!tc::mbar_wait(&ctl->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* a_s = smem + (size_t)s * STAGE_BYTES;
          uint8_t* b_s = a_s + A_BYTES;
          tc::mbar_arrive_expect_tx(&ctl->full[s], STAGE_BYTES);
          if (KIND == KIND_DH) {
            // A: dz rows of the tile (K-major, K = vocabulary); B: W rows kb*64.. as four
            // 64-column blocks (MN-major, blocked view)
            tc::tma_load_4d(a_s, &tmA, 0, 0, kb, mt, &ctl->full[s]);
            tc::tma_load_3d(b_s, &tmB, 0, kb * BK, nt * (BN / 64), &ctl->full[s]);
          } else {
            // A: two 64-column blocks of dz over 64 chunk rows (MN-major);
            // B: the 64 rows of H those chunk rows stand for, four 64-column blocks (MN-major)
            if ((kb % (BM / BK)) == 0) {
              // the row of the tile after this one is fetched now and used two slabs later
              row_cur = kb == 0 ? __ldg(p.tile_row + p.tile_begin) : row_next;
              const int nxt = kb / (BM / BK) + 1;
              row_next = nxt < chunk_tiles ? __ldg(p.tile_row + p.tile_begin + nxt) : 0;
            }
            const int hrow = p.h_local ? kb * BK : row_cur + (kb % (BM / BK)) * BK;
            tc::tma_load_4d(a_s, &tmA, 0, (kb % (BM / BK)) * BK, mt * (BM / 64), kb / (BM / BK), &ctl->full[s]);
            tc::tma_load_3d(b_s, &tmB, 0, hrow, nt * (BN / 64), &ctl->full[s]);
          }
        }
        // a unit with fewer slabs than meeting points still counts them all
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
    if (lane == 0) {
      constexpr uint32_t idesc = tc::make_idesc_bf16(BM, BN, KIND == KIND_DW ? 1 : 0, 1);
      uint32_t it = 0, at = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x, ++at) {
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
          // K-major: 128-byte rows, 8-row groups 1024 B apart; one UMMA_K step = 32 B.
          // MN-major: 64-wide blocks BOX_BYTES apart, 8 k-rows = 1024 B; one UMMA_K step = 2048 B.
          const uint64_t adesc = KIND == KIND_DW ? tc::make_smem_desc(a_addr, BOX_BYTES, 1024)
                                                 : tc::make_smem_desc(a_addr, 16, 1024);
          const uint64_t bdesc = tc::make_smem_desc(a_addr + A_BYTES, BOX_BYTES, 1024);
          constexpr uint32_t a_step = KIND == KIND_DW ? (2048u >> 4) : (32u >> 4);
          constexpr uint32_t b_step = 2048u >> 4;
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk)
            tc::umma_bf16(tmem_d, adesc + a_step * kk, bdesc + b_step * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          tc::umma_commit(&ctl->empty[s]);
        }
        if (ok) tc::umma_commit(&ctl->tfull[buf]);
      }
    }
  } else {
    // ---------------- epilogue warps 0..3 ----------------
    uint32_t at = 0;
    bool ok = true;
    const int r_in_tile = warp * 32 + lane;
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x, ++at) {
      const int mt = u / n_nt, nt = u % n_nt;
      const uint32_t buf = at & 1u, aph = (at >> 1) & 1u;
      if (!__all_sync(0xffffffffu, tc::mbar_wait(&ctl->tfull[buf], aph, abort_flag))) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + buf * BN;
      long long out_row;
      bool row_ok;
      if (KIND == KIND_DH) {
        const int tile = p.tile_begin + mt;
        out_row = (long long)p.tile_row[tile] + r_in_tile;
        row_ok = r_in_tile < p.tile_valid[tile] && out_row < p.T;
      } else {
        out_row = (long long)mt * BM + r_in_tile;
        row_ok = out_row < p.V;
      }
      const int ncol = min(BN, p.d - nt * BN);
      for (int c = 0; c * 32 < ncol; ++c) {
        uint32_t r[32];
        __syncwarp();                       // the TMEM load is warp-collective
        tc::tmem_ld_32x32(taddr + c * 32, r);
        tc::tmem_ld_wait();
        const int col0 = nt * BN + c * 32;
        if (!row_ok) {
          // rows outside the tile's run, past T or past V: nothing to write
        } else if (KIND == KIND_DH) {
          uint4* dst = reinterpret_cast<uint4*>(p.dH + out_row * p.d + col0);
          if (p.row_scale) {
            const float sc = p.row_scale[out_row];
#pragma unroll
            for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(sc * __uint_as_float(r[q]));
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            dst[q] = make_uint4(pack_bf16(__uint_as_float(r[8 * q]), __uint_as_float(r[8 * q + 1])),
                                pack_bf16(__uint_as_float(r[8 * q + 2]), __uint_as_float(r[8 * q + 3])),
                                pack_bf16(__uint_as_float(r[8 * q + 4]), __uint_as_float(r[8 * q + 5])),
                                pack_bf16(__uint_as_float(r[8 * q + 6]), __uint_as_float(r[8 * q + 7])));
          }
        } else {
          float4* dst = reinterpret_cast<float4*>(p.dW + out_row * p.d + col0);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 v = dst[q];
            v.x += __uint_as_float(r[4 * q]);
            v.y += __uint_as_float(r[4 * q + 1]);
            v.z += __uint_as_float(r[4 * q + 2]);
            v.w += __uint_as_float(r[4 * q + 3]);
            dst[q] = v;
          }
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl->tempty[buf]);
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    const unsigned long long t0 = tc::globaltimer_ns();
    while (tc::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) aero_raise(p.status, AERO_ST_TIMEOUT);
  if (warp == 5) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

// ---- the same two products on CTA pairs (a cluster of two, tcgen05 cta_group::2) -------------------
// A unit is 256 x 256: the pair takes two row tiles (dH: two token tiles; dW: two blocks of 128
// vocabulary rows), one per CTA, and one MMA covers both.  Each CTA stages its own 128-row A tile and
// only half of the 256 columns of the B slab; the tensor cores of the pair share the two halves, so a
// CTA moves 32 KB per 64-deep slab instead of 48 KB and the ring holds six slabs.  Barriers as in the
// lm_head kernel: full[s] lives in the rank-0 CTA and collects the bytes of both CTAs' loads; empty[s]
// and tfull[b] exist in both CTAs and are signalled for both by the issuer's commits; tempty[b] lives
// in the rank-0 CTA and counts the eight epilogue warps of the pair.
constexpr int PSTAGES = 6, PBNH = BN / 2;
constexpr uint32_t PB_BYTES = PBNH * BK * 2, PSTAGE_BYTES = A_BYTES + PB_BYTES;

struct PCtl {
  uint64_t full[PSTAGES], empty[PSTAGES], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};
constexpr size_t PSMEM_BYTES = 1024 + (size_t)PSTAGES * PSTAGE_BYTES + sizeof(PCtl);

template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  PCtl* ctl = reinterpret_cast<PCtl*>(smem + (size_t)PSTAGES * PSTAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();        // 0 issues the MMAs of the pair
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) { tc::mbar_init(&ctl->full[s], 1); tc::mbar_init(&ctl->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&ctl->tfull[b], 1); tc::mbar_init(&ctl->tempty[b], 8); }
    ctl->abort = 0;
    tc::fence_barrier_init();
  }
  if (warp == 4 && lane == 0) { tc::prefetch_tmap(&tmA); tc::prefetch_tmap(&tmB); }
  if (warp == 5) { tc::tmem_alloc_pair(&ctl->tmem_base, 512); tc::tmem_relinquish_pair(); }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();        // the peer's barriers exist before anything signals them
  tc::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort;

  int chunk_tiles = *p.n_tiles - p.tile_begin;
  chunk_tiles = chunk_tiles < 0 ? 0 : (chunk_tiles > p.tpc ? p.tpc : chunk_tiles);
  const int n_nt = (p.d + BN - 1) / BN;
  const int n_mt = KIND == KIND_DH ? chunk_tiles : (p.V + BM - 1) / BM;      // row tiles of 128
  const int n_mp = (n_mt + 1) / 2;                                           // ... in pairs
  const int nkb = KIND == KIND_DH ? (int)(p.ldz / BK) : chunk_tiles * (BM / BK);
  const int n_units = nkb > 0 ? n_mp * n_nt : 0;

  if (warp == 4) {
    // ---------------- TMA producer (one per CTA) ----------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int row_cur = 0, row_next = 0;
      unsigned int meetings = 0;
      const int max_units = (n_units + npairs - 1) / npairs;     // of the longest schedule
      for (int u = pair; ok && u < n_units; u += npairs) {
        const int mp = u / n_nt, nt = u % n_nt;
        // the pair's second row tile may not exist: its CTA then stages the first one again (dH) or rows
        // past V, which the copy fills with zeros (dW), and discards the result
        const int mt = (KIND == KIND_DH && 2 * mp + (int)rank >= n_mt) ? 2 * mp : 2 * mp + (int)rank;
        int next_meet = 0;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          if (p.nsync > 0 && next_meet < p.nsync && kb >= (int)((long long)next_meet * nkb / p.nsync)) {
            ++next_meet;
            ++meetings;
            atomicAdd(p.sync_ctr, 1u);
            const unsigned int target = meetings * gridDim.x;
            const unsigned long long t0 = tc::globaltimer_ns();
            while (*reinterpret_cast<volatile unsigned int*>(p.sync_ctr) < target) {
              if (tc::globaltimer_ns() - t0 > 50000ull) break;        // 50 us: go on alone
              __nanosleep(100);
            }
          }
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!tc::mbar_wait(&ctl->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* a_s = smem + (size_t)s * PSTAGE_BYTES;
          uint8_t* b_s = a_s + A_BYTES;
          const uint32_t full0 = tc::mapa_shared(tc::smem_u32(&ctl->full[s]), 0);
          if (rank == 0) tc::mbar_arrive_expect_tx(&ctl->full[s], 2 * PSTAGE_BYTES);
          if (KIND == KIND_DH) {
            tc::tma_load_4d_pair(a_s, &tmA, 0, 0, kb, mt, full0);
            tc::tma_load_3d_pair(b_s, &tmB, 0, kb * BK, nt * (BN / 64) + (int)rank * (PBNH / 64), full0);
          } else {
            if ((kb % (BM / BK)) == 0) {
              row_cur = kb == 0 ? __ldg(p.tile_row + p.tile_begin) : row_next;
              const int nxt = kb / (BM / BK) + 1;
              row_next = nxt < chunk_tiles ? __ldg(p.tile_row + p.tile_begin + nxt) : 0;
            }
            const int hrow = p.h_local ? kb * BK : row_cur + (kb % (BM / BK)) * BK;
            tc::tma_load_4d_pair(a_s, &tmA, 0, (kb % (BM / BK)) * BK, mt * (BM / 64), kb / (BM / BK), full0);
            tc::tma_load_3d_pair(b_s, &tmB, 0, hrow, nt * (BN / 64) + (int)rank * (PBNH / 64), full0);
          }
        }
        if (p.nsync > 0 && next_meet < p.nsync) {
          atomicAdd(p.sync_ctr, (unsigned)(p.nsync - next_meet));
          meetings += (unsigned)(p.nsync - next_meet);
        }
      }
      if (p.nsync > 0 && meetings < (unsigned)(max_units * p.nsync))
        atomicAdd(p.sync_ctr, (unsigned)(max_units * p.nsync) - meetings);
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer (rank 0, for the pair) ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = tc::make_idesc_bf16(2 * BM, BN, KIND == KIND_DW ? 1 : 0, 1);
      uint32_t it = 0, at = 0;
      bool ok = true;
      for (int u = pair; ok && u < n_units; u += npairs, ++at) {
        const uint32_t buf = at & 1u, aph = (at >> 1) & 1u;
        if (!tc::mbar_wait(&ctl->tempty[buf], aph ^ 1u, abort_flag)) { ok = false; break; }
        tc::tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!tc::mbar_wait(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t a_addr = tc::smem_u32(smem + (size_t)s * PSTAGE_BYTES);
          const uint64_t adesc = KIND == KIND_DW ? tc::make_smem_desc(a_addr, BOX_BYTES, 1024)
                                                 : tc::make_smem_desc(a_addr, 16, 1024);
          const uint64_t bdesc = tc::make_smem_desc(a_addr + A_BYTES, BOX_BYTES, 1024);
          constexpr uint32_t a_step = KIND == KIND_DW ? (2048u >> 4) : (32u >> 4);
          constexpr uint32_t b_step = 2048u >> 4;
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk)
            tc::umma_bf16_pair(tmem_d, adesc + a_step * kk, bdesc + b_step * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          tc::umma_commit_pair(&ctl->empty[s], 3);     // frees the stage in both CTAs when these MMAs retire
        }
        if (ok) tc::umma_commit_pair(&ctl->tfull[buf], 3);
      }
    }
  } else {
    // ---------------- epilogue warps 0..3 (each CTA its own row tile) ----------------
    uint32_t at = 0;
    bool ok = true;
    const int r_in_tile = warp * 32 + lane;
    for (int u = pair; ok && u < n_units; u += npairs, ++at) {
      const int mp = u / n_nt, nt = u % n_nt;
      const int mt = 2 * mp + (int)rank;
      const uint32_t buf = at & 1u, aph = (at >> 1) & 1u;
      if (!__all_sync(0xffffffffu, tc::mbar_wait(&ctl->tfull[buf], aph, abort_flag))) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + buf * BN;
      long long out_row = 0;
      bool row_ok = false;
      if (mt < n_mt) {
        if (KIND == KIND_DH) {
          const int tile = p.tile_begin + mt;
          out_row = (long long)p.tile_row[tile] + r_in_tile;
          row_ok = r_in_tile < p.tile_valid[tile] && out_row < p.T;
        } else {
          out_row = (long long)mt * BM + r_in_tile;
          row_ok = out_row < p.V;
        }
      }
      const int ncol = min(BN, p.d - nt * BN);
      if (mt < n_mt) {
        for (int c = 0; c * 32 < ncol; ++c) {
          uint32_t r[32];
          __syncwarp();                       // the TMEM load is warp-collective
          tc::tmem_ld_32x32(taddr + c * 32, r);
          tc::tmem_ld_wait();
          const int col0 = nt * BN + c * 32;
          if (!row_ok) {
            // rows outside the tile's run, past T or past V: nothing to write
          } else if (KIND == KIND_DH) {
            uint4* dst = reinterpret_cast<uint4*>(p.dH + out_row * p.d + col0);
            if (p.row_scale) {
              const float sc = p.row_scale[out_row];
#pragma unroll
              for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(sc * __uint_as_float(r[q]));
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              dst[q] = make_uint4(pack_bf16(__uint_as_float(r[8 * q]), __uint_as_float(r[8 * q + 1])),
                                  pack_bf16(__uint_as_float(r[8 * q + 2]), __uint_as_float(r[8 * q + 3])),
                                  pack_bf16(__uint_as_float(r[8 * q + 4]), __uint_as_float(r[8 * q + 5])),
                                  pack_bf16(__uint_as_float(r[8 * q + 6]), __uint_as_float(r[8 * q + 7])));
            }
          } else {
            float4* dst = reinterpret_cast<float4*>(p.dW + out_row * p.d + col0);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float4 v = dst[q];
              v.x += __uint_as_float(r[4 * q]);
              v.y += __uint_as_float(r[4 * q + 1]);
              v.z += __uint_as_float(r[4 * q + 2]);
              v.w += __uint_as_float(r[4 * q + 3]);
              dst[q] = v;
            }
          }
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(tc::mapa_shared(tc::smem_u32(&ctl->tempty[buf]), 0));
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
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

}  // namespace gemmbwd
