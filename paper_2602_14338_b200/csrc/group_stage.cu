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
  unsigned nc[kMaxPT];       // present rollouts | correct ones << 16   (staged path)
  unsigned kb[kMaxPT];       // kept rollouts | kept correct ones << 16 (staged path)
  int quota[kMaxPT];
  uint8_t mode[kMaxPT];      // 0 keep all present, 1 keep none, 2 select by rank
  uint8_t reject[kMaxPT];    // 1: select among the incorrect only; 2: among the correct only; 0: among all
  uint8_t uniform[kMaxPT];
  float ut[kMaxPT];
  float mu[kMaxPT];
  float inv[kMaxPT];
  int nk[kMaxPT];            // global path: kept rollouts, then their exclusive prefix inside the tile
  long long ktok[kMaxPT];    // global path: kept tokens, then their exclusive prefix inside the tile
};

// Per-rollout staging of a tile.  `ck` orders the candidates of a selection:
// correct << 63 | key << 16 | local index for a present rollout, all ones for an absent one, so
// that in a group that selects among its incorrect rollouts no correct one ever compares
// smaller.  After the selection the same words hold a kept rollout's token offset inside its
// 32-rollout chunk, and `len` its position among the chunk's kept rollouts.
constexpr int kChunks = kCap / 32;
struct RolloutStage {
  unsigned long long ck[kCap];
  int len[kCap];
  uint16_t pid[kCap];
  uint8_t flag[kCap];        // bit 0 present, bit 1 correct, bit 2 kept
  long long chunk_tok[kChunks];   // kept tokens per chunk, then their exclusive prefix inside the tile
  int chunk_cnt[kChunks];
};

struct TileShared {
  PromptState ps;
  RolloutStage rs;
  TilePartial red[kThreads / 32];
  long long warp_tok[kThreads / 32];
  int warp_cnt[kThreads / 32];
  long long base_tok;
  int base_roll;
  int tile;
  int failed;
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
      __nanosleep(200);
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

// Publish the tile's totals, sum the predecessors', publish the running totals (warp 0).
// Leaves the totals of all earlier tiles in sh.base_roll / sh.base_tok.
__device__ void chain_tile(const Workspace& ws, TileShared& sh, int tile, int tile_cnt, long long tile_tok, uint32_t& st) {
  const int lane = threadIdx.x;
  if (lane == 0 && tile > 0) {
    st_release(ws.desc_roll + tile, kFlagAgg | (unsigned long long)tile_cnt);
    st_release(ws.desc_tok + tile, kFlagAgg | (unsigned long long)tile_tok);
  }
  int excl_roll = 0;
  long long excl_tok = 0;
  const bool ok = scan_predecessors(ws, tile, lane, &excl_roll, &excl_tok);
  if (lane == 0) {
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

// Category, posterior and curation rule of one prompt from its counts (Appendix C; Sec. 4.2).
struct Rule {
  int category, mode;
  long long quota;
  int reject;          // 0: every present rollout is a candidate; 1: the incorrect ones (all correct kept);
                       // 2: the correct ones (all incorrect kept)
  bool uniform;
  float al, be, ut;
};
__device__ __forceinline__ Rule decide(const Args& a, int p, int n, int c) {
  Rule r;
  if (n == 0) r.category = AERO_CAT_EMPTY;
  else if (c == 0) r.category = AERO_CAT_ZERO;
  else if (c == n) r.category = AERO_CAT_PERFECT;
  else if (2 * c < n) r.category = AERO_CAT_PARTIAL;
  else r.category = AERO_CAT_GOOD;
  r.al = (a.alpha_in ? a.alpha_in[p] : a.cfg.alpha0) + (float)c;
  r.be = (a.beta_in ? a.beta_in[p] : a.cfg.beta0) + (float)(n - c);
  r.ut = r.al / (r.al + r.be);
  r.uniform = (c == 0 || c == n);
  r.mode = 0;
  r.quota = 0;
  r.reject = 0;
  if (n == 0) {
    r.mode = 1;
  } else if (r.uniform) {
    if (a.cfg.uniform_policy == AERO_UNIFORM_MASK) r.mode = 1;
    else if (a.cfg.n_keep_uniform > 0 && a.cfg.n_keep_uniform < n) { r.mode = 2; r.quota = a.cfg.n_keep_uniform; }
  } else {
    const bool low = r.category == AERO_CAT_PARTIAL ||
                     (a.cfg.rescue_S > 0 && (long long)c * a.cfg.n_explore <= (long long)a.cfg.rescue_S * n);
    if (a.cfg.rejection && low) {
      const long long m = min((long long)a.cfg.k_ratio * c, (long long)(n - c));
      if (m < n - c) { r.mode = 2; r.quota = m; r.reject = 1; }
    } else if (a.cfg.rejection && a.cfg.reject_high) {
      const long long m = min((long long)a.cfg.k_ratio * (n - c), (long long)c);
      if (m < c) { r.mode = 2; r.quota = m; r.reject = 2; }
    }
  }
  return r;
}

// Metrics record of the tile: shuffle tree per warp, warps added in order by thread 0.
__device__ __forceinline__ void reduce_partial(TileShared& sh, TilePartial mine) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine.present_tok += __shfl_xor_sync(0xffffffffu, mine.present_tok, o);
    mine.present_roll += __shfl_xor_sync(0xffffffffu, mine.present_roll, o);
    mine.surv += __shfl_xor_sync(0xffffffffu, mine.surv, o);
#pragma unroll
    for (int k = 0; k < 5; ++k) mine.cat[k] += __shfl_xor_sync(0xffffffffu, mine.cat[k], o);
    mine.abs_adv += __shfl_xor_sync(0xffffffffu, mine.abs_adv, o);
  }
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = mine;
}
__device__ __forceinline__ TilePartial sum_partials(const TileShared& sh) {
  TilePartial tot = {};
  for (int k = 0; k < kThreads / 32; ++k) {
    tot.present_tok += sh.red[k].present_tok; tot.present_roll += sh.red[k].present_roll; tot.surv += sh.red[k].surv;
    for (int c = 0; c < 5; ++c) tot.cat[c] += sh.red[k].cat[c];
    tot.abs_adv += sh.red[k].abs_adv;
  }
  return tot;
}

// A tile whose rollouts fit the staging area.  Rewards enter as the bit r > 0.5 (they must be
// exactly 0 or 1; anything else raises AERO_ST_BAD_REWARD), so per-prompt sums are counts,
// gathered with shared-memory atomics, and mean and deviation are closed forms of the counts.
__device__ void run_tile_staged(const Args& a, const Workspace& ws, TileShared& sh, int tile, int p0, int npt, int r0,
                                int nroll, uint32_t& st) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  PromptState& ps = sh.ps;
  RolloutStage& rs = sh.rs;

  // ---- which prompt owns which rollout ----
  if (tid < npt) {
    for (int j = ps.lo[tid]; j < ps.lo[tid + 1]; ++j) rs.pid[j] = (uint16_t)tid;
    ps.nc[tid] = 0;
    ps.kb[tid] = 0;
  }
  __syncthreads();

  // ---- stage the rollouts (coalesced) and count per prompt ----
  TilePartial mine = {};
  for (int j = tid; j < nroll; j += kThreads) {
    const int i = r0 + j;
    const bool pres = a.keep_in ? a.keep_in[i] != 0 : true;
    const float r = a.reward[i];
    const long long len = a.cs[i + 1] - a.cs[i];
    const bool corr = r > 0.5f;
    unsigned long long ck = kNone;
    if (pres) {
      if (r != 0.f && r != 1.f) st |= AERO_ST_BAD_REWARD;
      if (len < 0) st |= AERO_ST_BAD_OFFSETS;
      if (len == 0) st |= AERO_ST_EMPTY_ROLLOUT;
      const uint32_t key = a.key ? a.key[i] : default_key(a.cfg.seed, (uint32_t)i);
      ck = (corr ? 1ull << 63 : 0ull) | ((unsigned long long)key << 16) | (unsigned)j;
      atomicAdd(&ps.nc[rs.pid[j]], corr ? 0x10001u : 1u);
      mine.present_tok += len > 0 ? len : 0;
      mine.present_roll += 1;
    }
    rs.ck[j] = ck;
    rs.len[j] = len > 0 ? (int)(len < 0x7fffffffLL ? len : 0x7fffffffLL) : 0;
    rs.flag[j] = (uint8_t)((pres ? 1 : 0) | (corr ? 2 : 0));
  }
  __syncthreads();

  // ---- per prompt: category, posterior, curation rule ----
  if (tid < npt) {
    const int p = p0 + tid;
    const int n = (int)(ps.nc[tid] & 0xffffu), c = (int)(ps.nc[tid] >> 16);
    const Rule ru = decide(a, p, n, c);
    a.cat[p] = (uint8_t)ru.category;
    a.u_tilde[p] = ru.ut;
    a.alpha_out[p] = ru.al;
    a.beta_out[p] = ru.be;
    ps.mode[tid] = (uint8_t)ru.mode;
    ps.reject[tid] = (uint8_t)ru.reject;
    // every incorrect rollout orders before every correct one: when the correct ones are the
    // candidates, the n - c incorrect ones are counted by each rank and the quota allows for them
    ps.quota[tid] = (int)ru.quota + (ru.reject == 2 ? n - c : 0);
    ps.uniform[tid] = ru.uniform ? 1 : 0;
    ps.ut[tid] = ru.ut;
    mine.cat[ru.category] = 1;
  }
  __syncthreads();

  // ---- per rollout: keep decision (rank among the group's candidates) ----
  for (int j = tid; j < nroll; j += kThreads) {
    const int q = rs.pid[j];
    const int mode = ps.mode[q];
    const uint8_t f = rs.flag[j];
    bool kp = (f & 1) && mode != 1;
    const int rej = ps.reject[q];
    if (kp && mode == 2 && !(rej == 1 && (f & 2)) && !(rej == 2 && !(f & 2))) {
      const unsigned long long mykey = rs.ck[j];
      const int lo = ps.lo[q], hi = ps.lo[q + 1];
      int rank = 0;
#pragma unroll 4
      for (int k = lo; k < hi; ++k) rank += rs.ck[k] < mykey ? 1 : 0;
      kp = rank < ps.quota[q];
    }
    if (kp) {
      rs.flag[j] = f | 4;
      atomicAdd(&ps.kb[q], (f & 2) ? 0x10001u : 1u);
    }
  }
  __syncthreads();

  // ---- per prompt: mean and deviation of the base set; per chunk of 32 rollouts: kept counts and tokens ----
  if (tid < npt) {
    const int p = p0 + tid;
    const int nk = (int)(ps.kb[tid] & 0xffffu), ck = (int)(ps.kb[tid] >> 16);
    const bool over_kept = a.cfg.stats_over == AERO_STATS_KEPT;
    const int nb = over_kept ? nk : (int)(ps.nc[tid] & 0xffffu);
    const int cb = over_kept ? ck : (int)(ps.nc[tid] >> 16);
    float mu = 0.f, sd = 0.f;
    if (ps.uniform[tid]) {
      mu = ps.ut[tid];
      sd = sqrtf(mu * (1.f - mu));
    } else if (nb > 0) {
      mu = (float)cb / (float)nb;
      const float d1 = 1.f - mu;
      sd = sqrtf(((float)cb * d1 * d1 + (float)(nb - cb) * mu * mu) / (float)nb);
    }
    const float inv = 1.f / (sd + a.cfg.eps_std);
    ps.mu[tid] = mu;
    ps.inv[tid] = inv;
    a.gmask[p] = nk > 0 ? 1 : 0;
    if (a.cfg.agg != AERO_TOKEN_MEAN) ws.nkept[p] = nk;
    mine.surv = nk > 0 ? 1 : 0;
    mine.abs_adv = ((float)ck * fabsf(1.f - mu) + (float)(nk - ck) * fabsf(mu)) * inv;
  }
  for (int j0 = warp * 32; j0 < nroll; j0 += kThreads) {     // whole warps: the scan is warp-wide
    const int j = j0 + lane;
    const bool kp = j < nroll && (rs.flag[j] & 4);
    const unsigned kept_mask = __ballot_sync(0xffffffffu, kp);
    long long tok = kp ? rs.len[j] : 0;
    if (__reduce_max_sync(0xffffffffu, (unsigned)tok) < (1u << 26)) {      // 32 lengths below 2^26: a 32-bit scan
      unsigned t32 = (unsigned)tok;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned t2 = __shfl_up_sync(0xffffffffu, t32, o);
        if (lane >= o) t32 += t2;
      }
      tok = t32;
    } else {
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const long long t2 = __shfl_up_sync(0xffffffffu, tok, o);
        if (lane >= o) tok += t2;
      }
    }
    if (kp) {
      rs.ck[j] = (unsigned long long)(tok - rs.len[j]);
      rs.len[j] = __popc(kept_mask & ((1u << lane) - 1u));
    }
    if (lane == 31) { rs.chunk_cnt[j0 >> 5] = __popc(kept_mask); rs.chunk_tok[j0 >> 5] = tok; }
  }
  reduce_partial(sh, mine);
  __syncthreads();

  // ---- warp 0: exclusive prefixes over the chunks, then the chained scan across tiles; meanwhile
  // the other warps write what does not depend on it: advantage and keep flag per rollout ----
  if (tid >= 32) {
    for (int j = tid - 32; j < nroll; j += kThreads - 32) {
      const int q = rs.pid[j];
      const uint8_t f = rs.flag[j];
      const bool kp = (f & 4) != 0;
      a.adv[r0 + j] = kp ? (((f & 2) ? 1.f : 0.f) - ps.mu[q]) * ps.inv[q] : 0.f;
      a.keep[r0 + j] = kp ? 1 : 0;
    }
  } else {
    const int nchunks = (nroll + 31) >> 5;
    int run_cnt = 0;
    long long run_tok = 0;
    for (int c0 = 0; c0 < nchunks; c0 += 32) {
      const int c = c0 + lane;
      int cnt = c < nchunks ? rs.chunk_cnt[c] : 0;
      long long tok = c < nchunks ? rs.chunk_tok[c] : 0;
      const int my_cnt = cnt;
      const long long my_tok = tok;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int c2 = __shfl_up_sync(0xffffffffu, cnt, o);
        const long long t2 = __shfl_up_sync(0xffffffffu, tok, o);
        if (lane >= o) { cnt += c2; tok += t2; }
      }
      if (c < nchunks) { rs.chunk_cnt[c] = run_cnt + cnt - my_cnt; rs.chunk_tok[c] = run_tok + tok - my_tok; }
      run_cnt += __shfl_sync(0xffffffffu, cnt, 31);
      run_tok += __shfl_sync(0xffffffffu, tok, 31);
    }
    if (tid == 0) ws.part[tile] = sum_partials(sh);
    chain_tile(ws, sh, tile, run_cnt, run_tok, st);
  }
  __syncthreads();
  const bool failed = sh.failed != 0;
  const int base_roll = sh.base_roll;
  const long long base_tok = sh.base_tok;

  // ---- per kept rollout: compacted id and token offset ----
  if (!failed) {
    for (int j = tid; j < nroll; j += kThreads) {
      if (!(rs.flag[j] & 4)) continue;
      const int pos = base_roll + rs.chunk_cnt[j >> 5] + rs.len[j];
      a.kept_ids[pos] = r0 + j;
      a.kept_tok_off[pos] = base_tok + rs.chunk_tok[j >> 5] + (long long)rs.ck[j];
    }
  }
}

// A tile whose rollouts exceed the staging area (a very large group): the same steps with
// one thread per prompt walking the caller's arrays.
__device__ void run_tile_global(const Args& a, const Workspace& ws, TileShared& sh, int tile, int p0, int npt, int r0,
                                uint32_t& st) {
  const int tid = threadIdx.x;
  PromptState& ps = sh.ps;
  auto present = [&](int j) { return a.keep_in ? a.keep_in[r0 + j] != 0 : true; };
  auto length = [&](int j) { const long long l = a.cs[r0 + j + 1] - a.cs[r0 + j]; return l > 0 ? l : 0; };
  auto order_key = [&](int j) {
    if (!present(j)) return kNone;
    const uint32_t key = a.key ? a.key[r0 + j] : default_key(a.cfg.seed, (uint32_t)(r0 + j));
    return ((unsigned long long)key << 32) | (unsigned)j;
  };
  TilePartial mine = {};
  if (tid < npt) {
    const int p = p0 + tid;
    const int lo = ps.lo[tid], hi = ps.lo[tid + 1];
    int n = 0, c = 0;
    for (int j = lo; j < hi; ++j) {
      if (!present(j)) continue;
      const float r = a.reward[r0 + j];
      const long long len = a.cs[r0 + j + 1] - a.cs[r0 + j];
      if (r != 0.f && r != 1.f) st |= AERO_ST_BAD_REWARD;
      if (len < 0) st |= AERO_ST_BAD_OFFSETS;
      if (len == 0) st |= AERO_ST_EMPTY_ROLLOUT;
      n += 1; c += r > 0.5f ? 1 : 0;
      mine.present_tok += len > 0 ? len : 0;
    }
    mine.present_roll = n;
    const Rule ru = decide(a, p, n, c);
    a.cat[p] = (uint8_t)ru.category;
    a.u_tilde[p] = ru.ut;
    a.alpha_out[p] = ru.al;
    a.beta_out[p] = ru.be;
    mine.cat[ru.category] = 1;

    int nk = 0, ck = 0;
    long long ktok = 0;
    for (int j = lo; j < hi; ++j) {
      const bool corr = a.reward[r0 + j] > 0.5f;
      bool kp = present(j) && ru.mode != 1;
      if (kp && ru.mode == 2 && !(ru.reject == 1 && corr) && !(ru.reject == 2 && !corr)) {
        const unsigned long long mykey = order_key(j);
        long long rank = 0;
        for (int k = lo; k < hi; ++k) {
          const bool ck = a.reward[r0 + k] > 0.5f;
          if ((ru.reject == 1 && ck) || (ru.reject == 2 && !ck)) continue;
          rank += order_key(k) < mykey ? 1 : 0;
        }
        kp = rank < ru.quota;
      }
      a.keep[r0 + j] = kp ? 1 : 0;
      if (kp) { nk += 1; ck += corr ? 1 : 0; ktok += length(j); }
    }
    const bool over_kept = a.cfg.stats_over == AERO_STATS_KEPT;
    const int nb = over_kept ? nk : n, cb = over_kept ? ck : c;
    float mu = 0.f, sd = 0.f;
    if (ru.uniform) {
      mu = ru.ut;
      sd = sqrtf(mu * (1.f - mu));
    } else if (nb > 0) {
      mu = (float)cb / (float)nb;
      const float d1 = 1.f - mu;
      sd = sqrtf(((float)cb * d1 * d1 + (float)(nb - cb) * mu * mu) / (float)nb);
    }
    const float inv = 1.f / (sd + a.cfg.eps_std);
    for (int j = lo; j < hi; ++j)
      a.adv[r0 + j] = a.keep[r0 + j] ? ((a.reward[r0 + j] > 0.5f ? 1.f : 0.f) - mu) * inv : 0.f;
    ps.nk[tid] = nk;
    ps.ktok[tid] = ktok;
    a.gmask[p] = nk > 0 ? 1 : 0;
    if (a.cfg.agg != AERO_TOKEN_MEAN) ws.nkept[p] = nk;
    mine.surv = nk > 0 ? 1 : 0;
    mine.abs_adv = ((float)ck * fabsf(1.f - mu) + (float)(nk - ck) * fabsf(mu)) * inv;
  }

  // tile totals and exclusive prefixes over the tile's prompts (block scan, fixed order)
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
  reduce_partial(sh, mine);
  __syncthreads();
  int wbase_cnt = 0;
  long long wbase_tok = 0;
  for (int k = 0; k < warp; ++k) { wbase_cnt += sh.warp_cnt[k]; wbase_tok += sh.warp_tok[k]; }
  const int excl_cnt = wbase_cnt + cnt - my_cnt;
  const long long excl_tok = wbase_tok + tok - my_tok;
  if (tid < 32) {
    int tile_cnt = 0;
    long long tile_tok = 0;
    for (int k = 0; k < kThreads / 32; ++k) { tile_cnt += sh.warp_cnt[k]; tile_tok += sh.warp_tok[k]; }
    if (tid == 0) ws.part[tile] = sum_partials(sh);
    chain_tile(ws, sh, tile, tile_cnt, tile_tok, st);
  }
  __syncthreads();
  if (tid < npt && !sh.failed) {
    int pos = sh.base_roll + excl_cnt;
    long long toff = sh.base_tok + excl_tok;
    for (int j = ps.lo[tid]; j < ps.lo[tid + 1]; ++j) {
      if (!a.keep[r0 + j]) continue;
      a.kept_ids[pos] = r0 + j;
      a.kept_tok_off[pos] = toff;
      pos += 1;
      toff += length(j);
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

__global__ void __launch_bounds__(kThreads, 4) curate_kernel(Args a, Workspace ws, int pt, int ntiles) {
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
    // rollout range of the tile and of each of its prompts (clamped if the offsets are bad), later made
    // relative to the tile's first rollout
    for (int q = tid; q <= npt; q += kThreads) {
      int v = a.go[p0 + q];
      const int prev = q > 0 ? a.go[p0 + q - 1] : v;
      if (v < 0 || v > a.R || v < prev) st |= AERO_ST_BAD_OFFSETS;
      sh.ps.lo[q] = min(max(v, 0), a.R);
    }
    // bad offsets only: make the ranges non-decreasing (serial, so kept off the normal path)
    if (__syncthreads_or((st & AERO_ST_BAD_OFFSETS) != 0)) {
      if (tid == 0) {
        int run = sh.ps.lo[0];
        for (int q = 1; q <= npt; ++q) { run = max(run, sh.ps.lo[q]); sh.ps.lo[q] = run; }
      }
      __syncthreads();
    }
    const int r0 = sh.ps.lo[0];
    const int nroll = sh.ps.lo[npt] - r0;
    __syncthreads();
    for (int q = tid; q <= npt; q += kThreads) sh.ps.lo[q] -= r0;
    __syncthreads();
    if (nroll <= kCap) run_tile_staged(a, ws, sh, tile, p0, npt, r0, nroll, st);
    else run_tile_global(a, ws, sh, tile, p0, npt, r0, st);
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
