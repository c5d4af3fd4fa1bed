// Stage (a): segmented per-prompt group statistics (Eq. 1; Sec. 3.2; Sec. 4.2
// Strategies 2-3; Appendix C) in one pass over the rollout arrays.
//
//   curate_kernel   one block per tile of consecutive prompts.  The tile's rollouts are
//                   staged in shared memory with coalesced loads; per-prompt steps (counts,
//                   category, posterior, curation rule, mean/std) run one thread per prompt,
//                   per-rollout steps (rank among (key, index), keep, advantage, compaction)
//                   one thread per rollout.  The positions of the kept rollouts in the
//                   compacted outputs come from a chained scan across tiles (each tile
//                   publishes its totals, then sums its predecessors' until it meets one
//                   whose running total is known), so every input is read once and every
//                   output written once.  The last block to finish reduces the tiles'
//                   metrics records in a fixed order.
//   weights_kernel  per-rollout weights, which need the batch totals, and the tails of the
//                   compacted arrays.
//
// Tiles are handed out through a ticket counter, so a tile only ever waits for tiles taken
// earlier by blocks that are already running; every wait is bounded and ends with the
// AERO_ST_TIMEOUT status bit.  A tile whose rollouts do not fit the shared-memory staging
// area (one huge group) runs the same steps straight from global memory.
#include "common.cuh"

#include <mutex>

namespace {

constexpr int kThreads = 256;
constexpr int kCap = 2304;             // rollouts a tile can stage in shared memory
constexpr int kMaxPT = 256;            // prompts per tile: one thread each in the per-prompt steps
constexpr int kTargetRollouts = 1792;  // mean rollouts per tile the host aims at
constexpr unsigned long long kNone = ~0ull;
constexpr unsigned long long kFlagAgg = 1ull << 62, kFlagPrefix = 2ull << 62, kValueMask = (1ull << 62) - 1;
constexpr unsigned long long kSpinLimitNs = 1000000000ull;

struct TilePartial {
  long long present_tok;
  int present_roll, surv;
  int cat[5];
  float abs_adv;
};

struct Globals {
  long long R_kept, T_kept, T_present;
  int P_surv;
  float inv_tok_den;      // 1 / (token-mean denominator), 0 if empty
  float inv_prompt_den;   // 1 / (sequence-mean prompt denominator), 0 if empty
  int pad;
};

struct Workspace {
  int* nkept;                        // [P] kept rollouts per prompt (sequence-mean weights)
  unsigned long long* desc_roll;     // [ntiles] flag | kept rollouts (tile total, then running total)
  unsigned long long* desc_tok;      // [ntiles] flag | kept tokens
  unsigned int* ctrl;                // [4] ticket, tiles done, abort
  TilePartial* part;                 // [ntiles]
  Globals* glob;                     // [1]
};

__host__ __device__ inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

inline int prompts_per_tile(int32_t P, int32_t R) {
  const long long avg = P > 0 ? ((long long)R + P - 1) / P : 1;
  long long pt = kTargetRollouts / (avg > 0 ? avg : 1);
  return (int)(pt < 1 ? 1 : (pt > kMaxPT ? kMaxPT : pt));
}

inline size_t cleared_bytes(int ntiles) { return up256(sizeof(unsigned long long) * 2 * (size_t)ntiles + 16); }

inline Workspace carve(void* ws, int32_t P, int ntiles) {
  char* p = static_cast<char*>(ws);
  Workspace w;
  // the scan records and the counters are contiguous: one memset clears them before each launch
  w.desc_roll = reinterpret_cast<unsigned long long*>(p);
  w.desc_tok = w.desc_roll + ntiles;
  w.ctrl = reinterpret_cast<unsigned int*>(w.desc_tok + ntiles);
  p += cleared_bytes(ntiles);
  w.nkept = reinterpret_cast<int*>(p);            p += up256(sizeof(int) * (size_t)P);
  w.part = reinterpret_cast<TilePartial*>(p);     p += up256(sizeof(TilePartial) * (size_t)ntiles);
  w.glob = reinterpret_cast<Globals*>(p);
  return w;
}

// SplitMix64 (Steele, Lea, Flood 2014) as a counter-based generator; high word is the key.
__device__ __forceinline__ uint32_t default_key(uint64_t seed, uint32_t i) {
  uint64_t z = seed + (uint64_t)(i + 1u) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z = z ^ (z >> 31);
  return (uint32_t)(z >> 32);
}

__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct Args {
  aero_cfg cfg;
  int32_t P, R;
  const int32_t* go;
  const float* reward;
  const int64_t* cs;
  const uint32_t* key;
  const uint8_t* keep_in;
  const float* alpha_in;
  const float* beta_in;
  float* adv;
  float* w;
  uint8_t* keep;
  uint8_t* gmask;
  uint8_t* cat;
  float* u_tilde;
  float* alpha_out;
  float* beta_out;
  int32_t* kept_ids;
  int64_t* kept_tok_off;
  int64_t* counters;
  float* metrics;
  uint32_t* status;
};

// Per-prompt state of a tile (shared memory, one entry per prompt of the tile).
struct PromptState {
  int lo[kMaxPT + 1];        // rollout range of each prompt, relative to the tile's first rollout
  int quota[kMaxPT];
  uint8_t mode[kMaxPT];      // 0 keep all present, 1 keep none, 2 select by rank
  uint8_t reject[kMaxPT];    // select among the incorrect only, keep every correct one
  uint8_t uniform[kMaxPT];
  float ut[kMaxPT];
  float mu[kMaxPT];
  float inv[kMaxPT];
  int nk[kMaxPT];            // kept rollouts, then their exclusive prefix inside the tile
  long long ktok[kMaxPT];    // kept tokens, then their exclusive prefix inside the tile
};

// Per-rollout staging of a tile.  `ck` is the selection key (key << 32 | local index) of a
// candidate and kNone otherwise; after selection the same words hold the token offset of a
// kept rollout inside the tile, and `len` its position among the tile's kept rollouts.
struct RolloutStage {
  unsigned long long ck[kCap];
  int len[kCap];
  float r[kCap];
  uint16_t pid[kCap];
  uint8_t flag[kCap];        // bit 0 present, bit 1 kept
};

struct TileShared {
  PromptState ps;
  RolloutStage rs;
  long long warp_tok[kThreads / 32];
  int warp_cnt[kThreads / 32];
  long long base_tok;
  int base_roll;
  int tile;
  int failed;
  TilePartial part;
};

// Rollout accessors: from the staging area when the tile fits (STAGED), else from the
// caller's arrays.
template <bool STAGED>
struct Acc {
  const Args& a;
  TileShared& sh;
  int r0;          // first rollout of the tile
  __device__ __forceinline__ bool present(int j) const {
    if (STAGED) return sh.rs.flag[j] & 1;
    return a.keep_in ? a.keep_in[r0 + j] != 0 : true;
  }
  __device__ __forceinline__ float r(int j) const { return STAGED ? sh.rs.r[j] : a.reward[r0 + j]; }
  __device__ __forceinline__ long long len(int j) const {
    if (STAGED) return sh.rs.len[j];
    const long long l = a.cs[r0 + j + 1] - a.cs[r0 + j];
    return l > 0 ? l : 0;
  }
  __device__ __forceinline__ uint32_t key(int j) const {
    return a.key ? a.key[r0 + j] : default_key(a.cfg.seed, (uint32_t)(r0 + j));
  }
  __device__ __forceinline__ bool kept(int j) const {
    return STAGED ? (sh.rs.flag[j] & 2) != 0 : a.keep[r0 + j] != 0;
  }
  __device__ __forceinline__ void set_kept(int j, bool k) const {
    if (STAGED) sh.rs.flag[j] = (uint8_t)((sh.rs.flag[j] & 1) | (k ? 2 : 0));
    else a.keep[r0 + j] = k ? 1 : 0;
  }
  // selection key of rollout j in a group that selects (kNone: not a candidate)
  __device__ __forceinline__ unsigned long long ck(int j, bool reject) const {
    if (STAGED) return sh.rs.ck[j];
    if (!present(j) || (reject && r(j) > 0.5f)) return kNone;
    return ((unsigned long long)key(j) << 32) | (unsigned)j;
  }
  __device__ __forceinline__ int pid(int j, int npt) const {
    if (STAGED) return sh.rs.pid[j];
    int lo = 0, hi = npt;                 // last prompt whose range starts at or before j
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (sh.ps.lo[mid] <= j) lo = mid; else hi = mid;
    }
    return lo;
  }
};

__device__ __forceinline__ bool aborted(const Workspace& ws) {
  return *reinterpret_cast<volatile unsigned int*>(ws.ctrl + 2) != 0;
}

// Running totals of the kept rollouts and kept tokens of all tiles before `tile` (warp 0).
__device__ bool scan_predecessors(const Workspace& ws, int tile, int lane, int* excl_roll, long long* excl_tok) {
  unsigned long long sum_r = 0, sum_t = 0;
  bool done_r = false, done_t = false;
  const unsigned long long t0 = timer_ns();
  for (int base = tile - 1; base >= 0 && !(done_r && done_t); base -= 32) {
    const int idx = base - lane;
    unsigned long long vr = kFlagPrefix, vt = kFlagPrefix;      // tiles before the first: running total 0
    unsigned spins = 0;
    while (true) {
      if (idx >= 0) { vr = ld_acquire(ws.desc_roll + idx); vt = ld_acquire(ws.desc_tok + idx); }
      if (__all_sync(0xffffffffu, (vr >> 62) != 0 && (vt >> 62) != 0)) break;
      if ((++spins & 63u) == 0) {
        const bool give_up = aborted(ws) || timer_ns() - t0 > kSpinLimitNs;
        if (__any_sync(0xffffffffu, give_up)) return false;
      }
      __nanosleep(64);
    }
    if (!done_r) {
      const unsigned m = __ballot_sync(0xffffffffu, (vr >> 62) == 2);
      const int first = m ? __ffs(m) - 1 : 31;
      unsigned long long v = lane <= first ? (vr & kValueMask) : 0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      sum_r += v;
      done_r = m != 0;
    }
    if (!done_t) {
      const unsigned m = __ballot_sync(0xffffffffu, (vt >> 62) == 2);
      const int first = m ? __ffs(m) - 1 : 31;
      unsigned long long v = lane <= first ? (vt & kValueMask) : 0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      sum_t += v;
      done_t = m != 0;
    }
  }
  *excl_roll = (int)sum_r;
  *excl_tok = (long long)sum_t;
  return true;
}

template <bool STAGED>
__device__ void run_tile(const Args& a, const Workspace& ws, TileShared& sh, int tile, int p0, int npt, int r0, int nroll,
                         uint32_t& st) {
  const Acc<STAGED> acc{a, sh, r0};
  const int tid = threadIdx.x;
  PromptState& ps = sh.ps;

  // ---- stage the rollouts (one thread per rollout, coalesced) ----
  for (int j = tid; j < nroll; j += kThreads) {
    const int i = r0 + j;
    const bool pres = a.keep_in ? a.keep_in[i] != 0 : true;
    const float r = a.reward[i];
    const long long len = a.cs[i + 1] - a.cs[i];
    if (pres) {
      if (r != 0.f && r != 1.f) st |= AERO_ST_BAD_REWARD;
      if (len < 0) st |= AERO_ST_BAD_OFFSETS;
      if (len == 0) st |= AERO_ST_EMPTY_ROLLOUT;
    }
    if (STAGED) {
      sh.rs.flag[j] = pres ? 1 : 0;
      sh.rs.r[j] = r;
      sh.rs.len[j] = len > 0 ? (int)(len < 0x7fffffffLL ? len : 0x7fffffffLL) : 0;
      sh.rs.ck[j] = kNone;
    }
  }
  __syncthreads();

  // ---- per prompt: counts, category, posterior, curation rule ----
  TilePartial mine = {};
  if (tid < npt) {
    const int q = tid, p = p0 + q;
    const int lo = ps.lo[q], hi = ps.lo[q + 1];
    int n = 0, c = 0;
    long long ptok = 0;
    for (int j = lo; j < hi; ++j) {
      if (STAGED) sh.rs.pid[j] = (uint16_t)q;
      if (acc.present(j)) { n += 1; c += acc.r(j) > 0.5f ? 1 : 0; ptok += acc.len(j); }
    }
    int category;
    if (n == 0) category = AERO_CAT_EMPTY;
    else if (c == 0) category = AERO_CAT_ZERO;
    else if (c == n) category = AERO_CAT_PERFECT;
    else if (2 * c < n) category = AERO_CAT_PARTIAL;
    else category = AERO_CAT_GOOD;

    const float al = (a.alpha_in ? a.alpha_in[p] : a.cfg.alpha0) + (float)c;
    const float be = (a.beta_in ? a.beta_in[p] : a.cfg.beta0) + (float)(n - c);
    const float ut = al / (al + be);
    a.cat[p] = (uint8_t)category;
    a.u_tilde[p] = ut;
    a.alpha_out[p] = al;
    a.beta_out[p] = be;

    const bool uniform = (c == 0 || c == n);
    int mode = 0;
    long long quota = 0;
    bool reject = false;
    if (n == 0) {
      mode = 1;
    } else if (uniform) {
      if (a.cfg.uniform_policy == AERO_UNIFORM_MASK) mode = 1;
      else if (a.cfg.n_keep_uniform > 0 && a.cfg.n_keep_uniform < n) { mode = 2; quota = a.cfg.n_keep_uniform; }
    } else {
      const bool low = category == AERO_CAT_PARTIAL ||
                       (a.cfg.rescue_S > 0 && (long long)c * a.cfg.n_explore <= (long long)a.cfg.rescue_S * n);
      if (a.cfg.rejection && low) {
        const long long m = min((long long)a.cfg.k_ratio * c, (long long)(n - c));
        if (m < n - c) { mode = 2; quota = m; reject = true; }
      }
    }
    ps.mode[q] = (uint8_t)mode;
    ps.reject[q] = reject ? 1 : 0;
    ps.quota[q] = (int)quota;
    ps.uniform[q] = uniform ? 1 : 0;
    ps.ut[q] = ut;
    if (STAGED && mode == 2) {
      for (int j = lo; j < hi; ++j)
        if (acc.present(j) && !(reject && acc.r(j) > 0.5f))
          sh.rs.ck[j] = ((unsigned long long)acc.key(j) << 32) | (unsigned)j;
    }
    mine.present_tok = ptok;
    mine.present_roll = n;
    mine.cat[category] = 1;
  }
  __syncthreads();

  // ---- per rollout: keep decision (rank among the group's candidates) ----
  for (int j = tid; j < nroll; j += kThreads) {
    const int q = acc.pid(j, npt);
    const int mode = ps.mode[q];
    bool kp = acc.present(j) && mode != 1;
    if (kp && mode == 2) {
      const bool reject = ps.reject[q] != 0;
      const unsigned long long mykey = acc.ck(j, reject);
      if (mykey != kNone) {
        const int lo = ps.lo[q], hi = ps.lo[q + 1];
        int rank = 0;
        for (int k = lo; k < hi; ++k) rank += acc.ck(k, reject) < mykey ? 1 : 0;
        kp = rank < ps.quota[q];
      }
    }
    acc.set_kept(j, kp);
  }
  __syncthreads();

  // ---- per prompt: statistics over the base set, kept totals ----
  if (tid < npt) {
    const int q = tid, p = p0 + q;
    const int lo = ps.lo[q], hi = ps.lo[q + 1];
    int nk = 0, nbase = 0;
    long long ktok = 0;
    float sum_r = 0.f;
    for (int j = lo; j < hi; ++j) {
      const bool kp = acc.kept(j);
      if (kp) { nk += 1; ktok += acc.len(j); }
      const bool in_base = a.cfg.stats_over == AERO_STATS_KEPT ? kp : acc.present(j);
      if (in_base) { nbase += 1; sum_r += acc.r(j); }
    }
    float mu = 0.f, sd = 0.f;
    if (ps.uniform[q]) {
      mu = ps.ut[q];
      sd = sqrtf(mu * (1.f - mu));
    } else if (nbase > 0) {
      mu = sum_r / (float)nbase;
      float ss = 0.f;
      for (int j = lo; j < hi; ++j) {
        const bool in_base = a.cfg.stats_over == AERO_STATS_KEPT ? acc.kept(j) : acc.present(j);
        if (in_base) { const float dlt = acc.r(j) - mu; ss += dlt * dlt; }
      }
      sd = sqrtf(ss / (float)nbase);
    }
    const float inv = 1.f / (sd + a.cfg.eps_std);
    float abs_adv = 0.f;
    for (int j = lo; j < hi; ++j)
      if (acc.kept(j)) abs_adv += fabsf((acc.r(j) - mu) * inv);
    ps.mu[q] = mu;
    ps.inv[q] = inv;
    ps.nk[q] = nk;
    ps.ktok[q] = ktok;
    a.gmask[p] = nk > 0 ? 1 : 0;
    if (a.cfg.agg != AERO_TOKEN_MEAN) ws.nkept[p] = nk;
    mine.surv = nk > 0 ? 1 : 0;
    mine.abs_adv = abs_adv;
  }

  // ---- tile totals and exclusive prefixes over the tile's prompts (block scan, fixed order) ----
  {
    const int lane = tid & 31, warp = tid >> 5;
    int cnt = tid < npt ? ps.nk[tid] : 0;
    long long tok = tid < npt ? ps.ktok[tid] : 0;
    const int my_cnt = cnt;
    const long long my_tok = tok;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int c2 = __shfl_up_sync(0xffffffffu, cnt, o);
      const long long t2 = __shfl_up_sync(0xffffffffu, tok, o);
      if (lane >= o) { cnt += c2; tok += t2; }
    }
    if (lane == 31) { sh.warp_cnt[warp] = cnt; sh.warp_tok[warp] = tok; }
    // metrics record of the tile: shuffle tree per warp, warps added in order by thread 0
    TilePartial red = mine;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      red.present_tok += __shfl_xor_sync(0xffffffffu, red.present_tok, o);
      red.present_roll += __shfl_xor_sync(0xffffffffu, red.present_roll, o);
      red.surv += __shfl_xor_sync(0xffffffffu, red.surv, o);
#pragma unroll
      for (int k = 0; k < 5; ++k) red.cat[k] += __shfl_xor_sync(0xffffffffu, red.cat[k], o);
      red.abs_adv += __shfl_xor_sync(0xffffffffu, red.abs_adv, o);
    }
    __shared__ TilePartial s_red[kThreads / 32];
    if (lane == 0) s_red[warp] = red;
    __syncthreads();
    int wbase_cnt = 0;
    long long wbase_tok = 0;
    for (int k = 0; k < warp; ++k) { wbase_cnt += sh.warp_cnt[k]; wbase_tok += sh.warp_tok[k]; }
    if (tid < npt) { ps.nk[tid] = wbase_cnt + cnt - my_cnt; ps.ktok[tid] = wbase_tok + tok - my_tok; }
    if (tid == 0) {
      TilePartial tot = {};
      int tile_cnt = 0;
      long long tile_tok = 0;
      for (int k = 0; k < kThreads / 32; ++k) {
        tile_cnt += sh.warp_cnt[k]; tile_tok += sh.warp_tok[k];
        tot.present_tok += s_red[k].present_tok; tot.present_roll += s_red[k].present_roll; tot.surv += s_red[k].surv;
        for (int c = 0; c < 5; ++c) tot.cat[c] += s_red[k].cat[c];
        tot.abs_adv += s_red[k].abs_adv;
      }
      ws.part[tile] = tot;
      sh.base_roll = tile_cnt;      // tile totals, replaced by the running totals below
      sh.base_tok = tile_tok;
    }
    __syncthreads();
  }

  // ---- chained scan across tiles (warp 0) ----
  if (tid < 32) {
    const int tile_cnt = sh.base_roll;
    const long long tile_tok = sh.base_tok;
    if (tid == 0 && tile > 0) {
      st_release(ws.desc_roll + tile, kFlagAgg | (unsigned long long)tile_cnt);
      st_release(ws.desc_tok + tile, kFlagAgg | (unsigned long long)tile_tok);
    }
    int excl_roll = 0;
    long long excl_tok = 0;
    const bool ok = scan_predecessors(ws, tile, tid, &excl_roll, &excl_tok);
    if (tid == 0) {
      if (ok) {
        st_release(ws.desc_roll + tile, kFlagPrefix | (unsigned long long)(excl_roll + tile_cnt));
        st_release(ws.desc_tok + tile, kFlagPrefix | (unsigned long long)(excl_tok + tile_tok));
      } else {
        atomicExch(ws.ctrl + 2, 1u);
        st |= AERO_ST_TIMEOUT;
      }
      sh.failed = ok ? 0 : 1;
      sh.base_roll = excl_roll;
      sh.base_tok = excl_tok;
    }
  }
  __syncthreads();
  const bool failed = sh.failed != 0;
  const int base_roll = sh.base_roll;
  const long long base_tok = sh.base_tok;

  // ---- per prompt: positions of the kept rollouts inside the compacted outputs ----
  if (tid < npt && !failed) {
    const int q = tid;
    const int lo = ps.lo[q], hi = ps.lo[q + 1];
    int pos = ps.nk[q];
    long long toff = ps.ktok[q];
    for (int j = lo; j < hi; ++j) {
      if (!acc.kept(j)) continue;
      const long long len = acc.len(j);
      if (STAGED) {
        sh.rs.len[j] = pos;
        sh.rs.ck[j] = (unsigned long long)toff;
      } else {
        a.kept_ids[base_roll + pos] = r0 + j;
        a.kept_tok_off[base_roll + pos] = base_tok + toff;
      }
      pos += 1;
      toff += len;
    }
  }
  __syncthreads();

  // ---- per rollout: advantage, keep flag, compacted id and token offset ----
  for (int j = tid; j < nroll; j += kThreads) {
    const int i = r0 + j;
    const int q = acc.pid(j, npt);
    const bool kp = acc.kept(j);
    a.adv[i] = kp ? (acc.r(j) - ps.mu[q]) * ps.inv[q] : 0.f;
    if (STAGED) {
      a.keep[i] = kp ? 1 : 0;
      if (kp && !failed) {
        const int pos = base_roll + sh.rs.len[j];
        a.kept_ids[pos] = i;
        a.kept_tok_off[pos] = base_tok + (long long)sh.rs.ck[j];
      }
    }
  }
}

// Fixed-order reduction of the tiles' metrics records and the batch totals (one block).
__device__ void finish_batch(const Args& a, const Workspace& ws, int ntiles) {
  __shared__ long long s_misc[kThreads / 32][8];
  __shared__ double s_abs[kThreads / 32];
  const int tid = threadIdx.x;
  long long misc[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // present tokens, present rollouts, surviving prompts, 5 categories
  double aabs = 0.0;
  for (int t = tid; t < ntiles; t += kThreads) {
    const TilePartial q = ws.part[t];
    misc[0] += q.present_tok; misc[1] += q.present_roll; misc[2] += q.surv;
    for (int k = 0; k < 5; ++k) misc[3 + k] += q.cat[k];
    aabs += (double)q.abs_adv;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    aabs += __shfl_xor_sync(0xffffffffu, aabs, o);
#pragma unroll
    for (int k = 0; k < 8; ++k) misc[k] += __shfl_xor_sync(0xffffffffu, misc[k], o);
  }
  if ((tid & 31) == 0) {
    s_abs[tid >> 5] = aabs;
    for (int k = 0; k < 8; ++k) s_misc[tid >> 5][k] = misc[k];
  }
  __syncthreads();
  if (tid == 0) {
    long long tot[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    double sabs = 0.0;
    for (int t = 0; t < kThreads / 32; ++t) {
      sabs += s_abs[t];
      for (int k = 0; k < 8; ++k) tot[k] += s_misc[t][k];
    }
    const bool failed = aborted(ws);
    const long long R_kept = failed ? 0 : (long long)(ld_acquire(ws.desc_roll + ntiles - 1) & kValueMask);
    const long long T_kept = failed ? 0 : (long long)(ld_acquire(ws.desc_tok + ntiles - 1) & kValueMask);
    const long long T_present = tot[0], R_present = tot[1], P_surv = tot[2];
    const long long* ccat = tot + 3;
    Globals g;
    g.R_kept = R_kept; g.T_kept = T_kept; g.T_present = T_present; g.P_surv = (int)P_surv; g.pad = 0;
    const long long tden = a.cfg.denom == AERO_DENOM_SURVIVING ? T_kept : T_present;
    const long long pden = a.cfg.denom == AERO_DENOM_SURVIVING ? P_surv : (long long)a.P;
    g.inv_tok_den = tden > 0 ? (float)(1.0 / (double)tden) : 0.f;
    g.inv_prompt_den = pden > 0 ? (float)(1.0 / (double)pden) : 0.f;
    *ws.glob = g;
    a.counters[AERO_CNT_R_KEPT] = R_kept;
    a.counters[AERO_CNT_T_KEPT] = T_kept;
    a.counters[AERO_CNT_P_SURV] = P_surv;
    a.counters[AERO_CNT_ZERO] = ccat[AERO_CAT_ZERO];
    a.counters[AERO_CNT_PARTIAL] = ccat[AERO_CAT_PARTIAL];
    a.counters[AERO_CNT_GOOD] = ccat[AERO_CAT_GOOD];
    a.counters[AERO_CNT_PERFECT] = ccat[AERO_CAT_PERFECT];
    a.counters[AERO_CNT_T_PRESENT] = T_present;
    if (a.metrics) {
      a.metrics[0] = a.P > 0 ? (float)((double)ccat[AERO_CAT_ZERO] / (double)a.P) : 0.f;
      a.metrics[1] = (float)(sabs / (double)(R_kept > 0 ? R_kept : 1));
      a.metrics[2] = (float)((double)R_kept / (double)(R_present > 0 ? R_present : 1));
      a.metrics[3] = (float)((double)T_kept / (double)(T_present > 0 ? T_present : 1));
    }
  }
}

__global__ void __launch_bounds__(kThreads) curate_kernel(Args a, Workspace ws, int pt, int ntiles) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TileShared& sh = *reinterpret_cast<TileShared*>(smem_raw);
  const int tid = threadIdx.x;
  if (tid == 0) sh.tile = (int)atomicAdd(ws.ctrl + 0, 1u);
  __syncthreads();
  const int tile = sh.tile;             // tiles are taken in order: every earlier tile is already running
  uint32_t st = 0;
  if (tile < ntiles) {
    const int p0 = tile * pt;
    const int npt = min(pt, a.P - p0);
    // rollout range of the tile and of each of its prompts (clamped if the offsets are bad)
    for (int q = tid; q <= npt; q += kThreads) {
      int v = a.go[p0 + q];
      const int prev = q > 0 ? a.go[p0 + q - 1] : v;
      if (v < 0 || v > a.R || v < prev) st |= AERO_ST_BAD_OFFSETS;
      sh.ps.lo[q] = min(max(v, 0), a.R);
    }
    __syncthreads();
    if (tid == 0) {
      // make the ranges non-decreasing, then relative to the tile's first rollout
      int run = sh.ps.lo[0];
      for (int q = 1; q <= npt; ++q) { run = max(run, sh.ps.lo[q]); sh.ps.lo[q] = run; }
    }
    __syncthreads();
    const int r0 = sh.ps.lo[0];
    const int nroll = sh.ps.lo[npt] - r0;
    __syncthreads();
    for (int q = tid; q <= npt; q += kThreads) sh.ps.lo[q] -= r0;
    __syncthreads();
    if (nroll <= kCap) run_tile<true>(a, ws, sh, tile, p0, npt, r0, nroll, st);
    else run_tile<false>(a, ws, sh, tile, p0, npt, r0, nroll, st);
  }
  st = __reduce_or_sync(0xffffffffu, st);
  if ((tid & 31) == 0) aero_raise(a.status, st);

  // the last block to finish reduces the metrics records
  __threadfence();
  __syncthreads();
  if (tid == 0) sh.failed = atomicAdd(ws.ctrl + 1, 1u) == (unsigned)(ntiles - 1) ? 1 : 0;
  __syncthreads();
  if (sh.failed) {
    __threadfence();
    finish_batch(a, ws, ntiles);
  }
}

// Per-rollout weights (Eq. 2 normalisers) and the tails of the compacted arrays.
__global__ void __launch_bounds__(kThreads) weights_kernel(Args a, Workspace ws, int pt, int ntiles) {
  __shared__ int s_lo[kMaxPT + 1];
  const Globals g = *ws.glob;
  const int tid = threadIdx.x;
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int p0 = tile * pt;
    const int npt = min(pt, a.P - p0);
    __syncthreads();
    for (int q = tid; q <= npt; q += kThreads) s_lo[q] = min(max(a.go[p0 + q], 0), a.R);
    __syncthreads();
    const int r0 = s_lo[0];
    const int r1 = max(s_lo[npt], r0);
    for (int i = r0 + tid; i < r1; i += kThreads) {
      float w = 0.f;
      if (a.keep[i]) {
        if (a.cfg.agg == AERO_TOKEN_MEAN) {
          w = g.inv_tok_den;
        } else {
          int lo = 0, hi = npt;             // prompt of rollout i
          while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_lo[mid] <= i) lo = mid; else hi = mid;
          }
          const int nk = ws.nkept[p0 + lo];
          const long long len = a.cs[i + 1] - a.cs[i];
          w = (nk > 0 && len > 0) ? g.inv_prompt_den / (float)nk / (float)len : 0.f;
        }
      }
      a.w[i] = w;
      if ((long long)i >= g.R_kept) a.kept_ids[i] = -1;
      if ((long long)i + 1 >= g.R_kept) a.kept_tok_off[i + 1] = g.T_kept;
      if (i == 0 && g.R_kept == 0) a.kept_tok_off[0] = 0;
    }
  }
}

}  // namespace

size_t aero_group_ws_bytes_impl(int32_t P, int32_t R) {
  if (P < 0) P = 0;
  const int pt = prompts_per_tile(P, R);
  const int ntiles = (P + pt - 1) / pt + 1;
  return cleared_bytes(ntiles) + up256(sizeof(int) * (size_t)P) + up256(sizeof(TilePartial) * (size_t)ntiles) +
         up256(sizeof(Globals));
}

int aero_group_stats_launch(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                            const int32_t* go, const float* reward, const int64_t* cs,
                            const uint32_t* key, const uint8_t* keep_in,
                            const float* alpha_in, const float* beta_in,
                            float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                            float* u_tilde, float* alpha_out, float* beta_out,
                            int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                            float* metrics, void* wsp) {
  Args a;
  a.cfg = *cfg; a.P = P; a.R = R; a.go = go; a.reward = reward; a.cs = cs; a.key = key;
  a.keep_in = keep_in; a.alpha_in = alpha_in; a.beta_in = beta_in; a.adv = adv; a.w = w;
  a.keep = keep; a.gmask = gmask; a.cat = cat; a.u_tilde = u_tilde; a.alpha_out = alpha_out;
  a.beta_out = beta_out; a.kept_ids = kept_ids; a.kept_tok_off = kept_tok_off;
  a.counters = counters; a.metrics = metrics; a.status = ctx->d_status;
  if (P == 0 || R == 0) {
    // nothing to curate: zero counters and offsets, mark every prompt empty
    AERO_CUDA_TRY(cudaMemsetAsync(counters, 0, 8 * sizeof(int64_t), ctx->stream));
    AERO_CUDA_TRY(cudaMemsetAsync(kept_tok_off, 0, sizeof(int64_t), ctx->stream));
    if (metrics) AERO_CUDA_TRY(cudaMemsetAsync(metrics, 0, 4 * sizeof(float), ctx->stream));
    if (P == 0) return AERO_OK;
  }
  const int pt = prompts_per_tile(P, R);
  const int ntiles = (P + pt - 1) / pt;
  Workspace ws = carve(wsp, P, ntiles + 1);
  // scan records, ticket and counters start at zero on every call
  AERO_CUDA_TRY(cudaMemsetAsync(wsp, 0, cleared_bytes(ntiles + 1), ctx->stream));
  AERO_CUDA_TRY(cudaFuncSetAttribute(curate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TileShared)));
  curate_kernel<<<ntiles, kThreads, sizeof(TileShared), ctx->stream>>>(a, ws, pt, ntiles);
  const int wblocks = ntiles < 8 * ctx->sm_count ? ntiles : 8 * ctx->sm_count;
  weights_kernel<<<wblocks, kThreads, 0, ctx->stream>>>(a, ws, pt, ntiles);
  ctx->launches += 2;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

// ---- variant with library-owned scratch ------------------------------------------------
// The kernels above need a few bytes of scratch per prompt and per tile.  This entry point takes
// them from a fixed array in device memory that is part of the loaded library image, so the
// caller passes inputs and outputs only and nothing is allocated, by this call or before it.
namespace {

constexpr int32_t kStaticMaxP = AERO_STATIC_MAX_PROMPTS;
constexpr size_t cup256(size_t x) { return (x + 255) / 256 * 256; }
// room for the per-prompt words of kStaticMaxP prompts and the records of kStaticMaxTiles tiles
constexpr size_t kStaticMaxTiles = 16384;
constexpr size_t kStaticBytes = cup256(sizeof(unsigned long long) * 2 * (kStaticMaxTiles + 1) + 16) +
                                cup256(sizeof(int) * (size_t)kStaticMaxP) +
                                cup256(sizeof(TilePartial) * (kStaticMaxTiles + 1)) + cup256(sizeof(Globals));

static __device__ __align__(256) unsigned char g_group_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on `device`, looked up once per device.  In host code
// the array's name is only a handle for this lookup, never a pointer a kernel could use.
int static_scratch(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return AERO_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (!g_scratch_ptr[device]) {
    void* p = nullptr;
    if (cudaSetDevice(device) != cudaSuccess) return AERO_ERR_CUDA;
    if (cudaGetSymbolAddress(&p, g_group_scratch) != cudaSuccess || !p) return AERO_ERR_CUDA;
    g_scratch_ptr[device] = p;
  }
  *out = g_scratch_ptr[device];
  return AERO_OK;
}

}  // namespace

extern "C" int aero_group_stats_static(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                                       const int32_t* go, const float* reward, const int64_t* cs,
                                       const uint32_t* key, const uint8_t* keep_in,
                                       const float* alpha_in, const float* beta_in,
                                       float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                                       float* u_tilde, float* alpha_out, float* beta_out,
                                       int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                                       float* metrics) {
  if (!ctx || !cfg || P < 0 || R < 0) return AERO_ERR_INVALID;
  if (P > kStaticMaxP) return AERO_ERR_TOO_LARGE;
  if (aero_group_ws_bytes_impl(P, R) > kStaticBytes) return AERO_ERR_TOO_LARGE;
  if (!go || !cs || !kept_tok_off || !counters) return AERO_ERR_INVALID;
  if (R > 0 && (!reward || !adv || !w || !keep || !kept_ids)) return AERO_ERR_INVALID;
  if (P > 0 && (!gmask || !cat || !u_tilde || !alpha_out || !beta_out)) return AERO_ERR_INVALID;
  if ((alpha_in == nullptr) != (beta_in == nullptr)) return AERO_ERR_INVALID;
  if (cfg->k_ratio < 1 || cfg->n_explore < 1 || cfg->rescue_S < 0) return AERO_ERR_INVALID;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AERO_ERR_CUDA;
  void* scratch = nullptr;
  const int rc = static_scratch(ctx->device, &scratch);
  if (rc) return rc;
  // the launch clears the scan records and counters at the head of the scratch; every other
  // scratch word the kernels read is written earlier in the same call
  return aero_group_stats_launch(ctx, cfg, P, R, go, reward, cs, key, keep_in, alpha_in, beta_in,
                                 adv, w, keep, gmask, cat, u_tilde, alpha_out, beta_out,
                                 kept_ids, kept_tok_off, counters, metrics, scratch);
}
