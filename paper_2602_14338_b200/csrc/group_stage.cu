// Stage (a): segmented per-prompt group statistics (Eq. 1; Sec. 3.2; Sec. 4.2
// Strategies 2-3; Appendix C) in four launches.
//
//   curate_kernel   one warp per share of up to 32 consecutive prompts, eight shares to a tile.
//                   A warp stages its share's rollouts with coalesced loads (sort words with
//                   the lengths in shared memory, presence and correctness as bit masks) and
//                   runs the per-prompt steps (counts, category, posterior, curation rule,
//                   mean/std, and for a selection in a group of at most 16 its threshold from
//                   a sorting network on registers) one lane per prompt and the per-rollout
//                   steps (keep by threshold or by rank among (key, index), advantage) one
//                   lane per rollout.  Warps never wait for one another; each leaves its
//                   totals of kept rollouts and tokens, each tile its sums of them and its
//                   metrics record.
//   run_prefix_kernel, totals_kernel
//                   exclusive prefixes of the tiles' totals in two levels (runs of 1024 tiles,
//                   then the runs), the batch totals, counters and metrics (fixed order).
//   emit_kernel     the same shares again: compacted ids and token offsets of the kept rollouts
//                   from the first pass's kept bits and lengths and the prefixes, per-rollout weights (which need the
//                   batch totals), and the tails of the compacted arrays.
//
// Splitting where the batch-wide prefix is needed costs the second pass a read of 4 bytes per
// rollout (the first pass leaves kept bit | length where the weight will go) and saves every wait
// between blocks: no launch depends on the order in which its blocks run.  A share whose rollouts do not fit the warp's staging area
// (a huge group, or a rollout of 2^22 tokens or more) runs the first launch's steps straight from
// global memory, one lane per prompt.
#include "common.cuh"

#include <mutex>

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kBlocksPerSM = 6;
constexpr int kWCap = 416;             // rollouts a warp can stage
constexpr int kWChunks = kWCap / 32;
constexpr int kLenBits = 22;           // staged rollouts are shorter than 2^22 tokens
constexpr unsigned kLenMask = (1u << kLenBits) - 1u;
constexpr unsigned kKeptBit = 1u << 31;    // first pass -> second pass, in w: kept bit | length (at most 2^31 - 1)
constexpr int kMaxPW = 32;             // prompts per warp: one lane each in the per-prompt steps
constexpr int kWTarget = 300;          // mean rollouts per warp the host aims at
constexpr int kRunThreads = 256;
constexpr int kRunTiles = kRunThreads * 4;   // tiles per run of the batch-wide prefix
constexpr unsigned long long kNone = ~0ull;

struct TilePartial {
  long long present_tok;
  int present_roll, surv;
  int cat[5];
  float abs_adv;
};

struct RunPartial {
  long long misc[8];      // present tokens, present rollouts, surviving prompts, 5 categories
  double abs_adv;
};

struct Globals {
  long long R_kept, T_kept, T_present;
  int P_surv;
  float inv_tok_den;      // 1 / (token-mean denominator), 0 if empty
  float inv_prompt_den;   // 1 / (sequence-mean prompt denominator), 0 if empty
  int pad;
};

struct Workspace {
  int* nkept;              // [P] kept rollouts per prompt (sequence-mean weights)
  int* share_cnt;          // [ntiles * kWarps] kept rollouts per share
  long long* share_tok;    // [ntiles * kWarps] kept tokens per share
  int* tile_cnt;           // [ntiles] kept rollouts per tile, then of the earlier tiles of its run
  long long* tile_tok;     // [ntiles] kept tokens per tile, then of the earlier tiles of its run
  TilePartial* part;       // [ntiles]
  int* run_cnt;            // [nruns] kept rollouts per run of kRunTiles tiles, then of all earlier runs
  long long* run_tok;      // [nruns] likewise for kept tokens
  RunPartial* run_part;    // [nruns]
  Globals* glob;           // [1]
};

__host__ __device__ constexpr size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// Prompts per warp: as many as keep the mean share near kWTarget rollouts, which leaves the
// staging area a margin of more than three standard deviations for group sizes spread
// uniformly around their mean.
inline int prompts_per_warp(int32_t P, int32_t R) {
  if (P <= 0 || R <= 0) return kMaxPW;
  const long long pw = (long long)kWTarget * P / R;
  return (int)(pw < 1 ? 1 : (pw > kMaxPW ? kMaxPW : pw));
}

constexpr size_t runs_of(size_t ntiles) { return (ntiles + kRunTiles - 1) / kRunTiles; }

constexpr size_t workspace_bytes(size_t P, size_t ntiles) {
  return up256(sizeof(int) * P) + up256(sizeof(int) * ntiles * kWarps) + up256(sizeof(long long) * ntiles * kWarps) +
         up256(sizeof(int) * ntiles) + up256(sizeof(long long) * ntiles) + up256(sizeof(TilePartial) * ntiles) +
         up256(sizeof(int) * runs_of(ntiles)) + up256(sizeof(long long) * runs_of(ntiles)) +
         up256(sizeof(RunPartial) * runs_of(ntiles)) + up256(sizeof(Globals));
}

inline Workspace carve(void* ws, int32_t P, int ntiles) {
  char* p = static_cast<char*>(ws);
  Workspace w;
  w.nkept = reinterpret_cast<int*>(p);              p += up256(sizeof(int) * (size_t)P);
  w.share_cnt = reinterpret_cast<int*>(p);          p += up256(sizeof(int) * (size_t)ntiles * kWarps);
  w.share_tok = reinterpret_cast<long long*>(p);    p += up256(sizeof(long long) * (size_t)ntiles * kWarps);
  w.tile_cnt = reinterpret_cast<int*>(p);           p += up256(sizeof(int) * (size_t)ntiles);
  w.tile_tok = reinterpret_cast<long long*>(p);     p += up256(sizeof(long long) * (size_t)ntiles);
  w.part = reinterpret_cast<TilePartial*>(p);       p += up256(sizeof(TilePartial) * (size_t)ntiles);
  const size_t nruns = runs_of((size_t)ntiles);
  w.run_cnt = reinterpret_cast<int*>(p);            p += up256(sizeof(int) * nruns);
  w.run_tok = reinterpret_cast<long long*>(p);      p += up256(sizeof(long long) * nruns);
  w.run_part = reinterpret_cast<RunPartial*>(p);    p += up256(sizeof(RunPartial) * nruns);
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

// Token count of rollout i as the stage uses it: negative lengths (bad offsets) count as 0 and
// a length is capped at 2^31 - 1.
__device__ __forceinline__ int clamped_len(long long len) {
  return len > 0 ? (int)(len < 0x7fffffffLL ? len : 0x7fffffffLL) : 0;
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

// What the rollouts of one prompt need to know about it (shared memory, one entry per prompt of
// a warp's share).
struct PromptRule {
  float adv_correct, adv_incorrect;   // advantage of a kept rollout by its reward bit
  unsigned range;      // first rollout | one past the last << 16, relative to the share's first rollout; or, with
                       // bit 3 of sel, the high word of the largest sort word a selection keeps
  unsigned sel;        // bit 0: keep none; bit 1: the incorrect rollouts are ranked; bit 2: the correct ones are;
                       // bit 3: a ranked rollout is kept iff its sort word's high half is at most `range`; quota << 4
};

// Staging of one warp's share.  `ck` orders the candidates of a selection and carries the
// rollout's length: correct << 63 | key << 31 | local index << 22 | length for a present rollout,
// all ones for an absent one, so that in a group that selects among its incorrect rollouts no
// correct one ever compares smaller.  One bit per rollout in `pmask` (present) and `cmask` (present and correct), one word
// per chunk of 32 rollouts.
struct WarpStage {          // a warp's view of the block's staging arrays
  unsigned long long* ck;   // [kWCap]
  PromptRule* rule;         // [kMaxPW]
  unsigned* pmask;          // [kWChunks]
  unsigned* cmask;          // [kWChunks]
  uint8_t* pid;             // [kWCap] which prompt of the share owns the rollout
};

// The sort words of all warps come first and the other arrays (more than kWCap words together)
// after them, so that a read up to kWCap entries past the end of any warp's sort words stays
// inside the block's shared memory: the rank loop reads past a short group without clamping
// and discards what it read.
struct BlockShared {
  unsigned long long ck[kWarps][kWCap];
  PromptRule rule[kWarps][kMaxPW];
  uint8_t pid[kWarps][kWCap];
  unsigned pmask[kWarps][kWChunks], cmask[kWarps][kWChunks];
  TilePartial red[kWarps];
  long long share_tok[kWarps];
  int share_cnt[kWarps];
};
static_assert(sizeof(BlockShared) - sizeof(unsigned long long) * kWarps * kWCap >= sizeof(unsigned long long) * kWCap,
              "the arrays after the sort words must cover the longest read past them");

// A warp's share of a tile: prompts [p0, p0 + np), their rollouts [r0, r0 + nroll); lane q holds
// the rollout range [lo, hi) of prompt p0 + q, relative to r0 (empty for q >= np).
struct Share {
  int p0, np;
  int r0, nroll;
  int lo, hi;
};

// Reads the share's group offsets, clamping them into [0, R] and into non-decreasing order if
// they are bad (which also raises AERO_ST_BAD_OFFSETS).
__device__ __forceinline__ Share load_share(const Args& a, int share, int pw, uint32_t& st) {
  const int lane = threadIdx.x & 31;
  Share sh;
  sh.p0 = share * pw;
  sh.np = max(0, min(pw, a.P - sh.p0));
  sh.r0 = sh.nroll = sh.lo = sh.hi = 0;
  if (sh.np == 0) return sh;
  const int v = lane < sh.np ? a.go[sh.p0 + lane] : 0;
  const int end = a.go[sh.p0 + sh.np];
  int prev = __shfl_up_sync(0xffffffffu, v, 1);
  if (lane == 0) prev = sh.p0 > 0 ? a.go[sh.p0 - 1] : v;
  bool bad = lane < sh.np && (v < 0 || v > a.R || v < prev);
  if (lane == sh.np - 1) bad = bad || end < v || end > a.R || end < 0;
  int lo = min(max(v, 0), a.R);
  int last = min(max(end, 0), a.R);
  if (__any_sync(0xffffffffu, bad)) {
    st |= AERO_ST_BAD_OFFSETS;
    if (lane >= sh.np) lo = 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, lo, o);
      if (lane >= o) lo = max(lo, u);
    }
    last = max(last, __shfl_sync(0xffffffffu, lo, sh.np - 1));
  }
  int hi = __shfl_down_sync(0xffffffffu, lo, 1);
  if (lane >= sh.np - 1) hi = last;
  if (lane >= sh.np) lo = last;
  sh.r0 = __shfl_sync(0xffffffffu, lo, 0);
  sh.nroll = last - sh.r0;
  sh.lo = lo - sh.r0;
  sh.hi = hi - sh.r0;
  return sh;
}

// Metrics record of a warp's share: integer fields by warp reduction, the float by a shuffle tree
// (fixed order).
__device__ __forceinline__ TilePartial warp_partial(TilePartial mine) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine.present_tok += __shfl_xor_sync(0xffffffffu, mine.present_tok, o);
    mine.abs_adv += __shfl_xor_sync(0xffffffffu, mine.abs_adv, o);
  }
  mine.present_roll = __reduce_add_sync(0xffffffffu, mine.present_roll);
  mine.surv = __reduce_add_sync(0xffffffffu, mine.surv);
#pragma unroll
  for (int k = 0; k < 5; ++k) mine.cat[k] = __reduce_add_sync(0xffffffffu, mine.cat[k]);
  return mine;
}

// Set bits of a chunked bit mask inside the rollout range [lo, hi).
__device__ __forceinline__ int range_popc(const unsigned* mask, int lo, int hi) {
  int cnt = 0;
  if (hi > lo) {
    const int w0 = lo >> 5, w1 = (hi - 1) >> 5;
    for (int w = w0; w <= w1; ++w) {
      unsigned m = mask[w];
      if (w == w0) m &= 0xffffffffu << (lo & 31);
      if (w == w1) m &= 0xffffffffu >> (31 - ((hi - 1) & 31));
      cnt += __popc(m);
    }
  }
  return cnt;
}

// Mean and reciprocal deviation of a group's base set from its counts (Eq. 1 with binary
// rewards; posterior mean and Bernoulli deviation for a uniform group).
__device__ __forceinline__ void group_moments(const Args& a, const Rule& ru, int nb, int cb, float* mu_out, float* inv_out) {
  float mu = 0.f, sd = 0.f;
  if (ru.uniform) {
    mu = ru.ut;
    sd = sqrtf(mu * (1.f - mu));
  } else if (nb > 0) {
    mu = (float)cb / (float)nb;
    const float d1 = 1.f - mu;
    sd = sqrtf(((float)cb * d1 * d1 + (float)(nb - cb) * mu * mu) / (float)nb);
  }
  *mu_out = mu;
  *inv_out = 1.f / (sd + a.cfg.eps_std);
}

// Selection in a group of at most N rollouts by threshold: the high halves of the group's sort
// words (correct << 31 | key >> 1; all ones for an absent rollout and past the group's end) go
// through Batcher's odd-even merge sort as a fixed network of min/max on registers, every index a
// compile-time constant.  With v the sorted halves, a rollout of rank below `idx + 1` has a half
// at most v[idx]; the converse holds when v[idx + 1] > v[idx].  Returns whether it does (else
// the group is ranked by the loop, which compares whole words) and v[idx] in *thr.
template <int N>
__device__ __forceinline__ bool threshold_half(const unsigned long long* grp, int n, int idx, unsigned* thr) {
  unsigned v[N];
  const unsigned* half = reinterpret_cast<const unsigned*>(grp) + 1;
#pragma unroll
  for (int t = 0; t < N; ++t) v[t] = t < n ? half[2 * t] : 0xffffffffu;
  // pass (p, k) compares a with a + k for every a whose offset from k % p, taken modulo 2k, is
  // below k, when both lie in the same block of 2p
#pragma unroll
  for (int p = 1; p < N; p <<= 1) {
#pragma unroll
    for (int k = p; k >= 1; k >>= 1) {
#pragma unroll
      for (int a = 0; a < N; ++a) {
        const int r = k % p, b = a + k;
        if (a >= r && (a - r) % (2 * k) < k && b < N && a / (2 * p) == b / (2 * p)) {
          const unsigned x = v[a], y = v[b];
          v[a] = min(x, y);
          v[b] = max(x, y);
        }
      }
    }
  }
  unsigned lo = v[0], up = v[1];
#pragma unroll
  for (int t = 1; t + 1 < N; ++t) {
    lo = idx == t ? v[t] : lo;
    up = idx == t ? v[t + 1] : up;
  }
  *thr = lo;
  return up > lo;
}

// A share whose rollouts fit the warp's staging area, have between 1 and 2^22 - 1 tokens each
// and rewards of exactly 0 or 1.  Rewards enter as the bit r > 0.5, so per-prompt sums are bit counts and mean and deviation are closed
// forms of the counts; the number of rollouts a selection keeps is known from the rule alone,
// so the per-prompt outputs are written before any rollout is ranked.  Returns false, with
// nothing written, if a rollout does not qualify; else the share's kept rollouts and tokens.
template <bool HAS_KEEP_IN, bool HAS_KEY>
__device__ __forceinline__ bool curate_staged(const Args& a, const Workspace& ws, const WarpStage& S, const Share& sh,
                                              TilePartial& mine, uint32_t& st, int* cnt_out, long long* tok_out) {
  const int lane = threadIdx.x & 31;
  const int r0 = sh.r0, nroll = sh.nroll;

  // ---- which prompt owns which rollout ----
  if (lane < sh.np)
    for (int j = sh.lo; j < sh.hi; ++j) S.pid[j] = (uint8_t)lane;

  // ---- stage the rollouts (coalesced), one bit each for present and correct ----
  // (lanes past the share's end read its last rollout again and count as absent)
  // A reward other than 0 or 1, or a length outside [1, 2^22), sends the whole share to the
  // path that walks global memory, which also raises the status bits.
  bool irregular = false;
  unsigned ptok = 0;       // at most kWChunks lengths below 2^22 per lane
#pragma unroll 2
  for (int c = 0; c * 32 < nroll; ++c) {
    const int j = c * 32 + lane;
    const int i = r0 + min(j, nroll - 1);
    const float r = a.reward[i];
    const long long len = a.cs[i + 1] - a.cs[i];
    bool pres = j < nroll;
    if (HAS_KEEP_IN) pres = pres && a.keep_in[i] != 0;
    const bool corr = r > 0.5f;
    const uint32_t key = HAS_KEY ? a.key[i] : default_key(a.cfg.seed, (uint32_t)i);
    irregular |= pres && ((r != 0.f && r != 1.f) || (unsigned long long)(len - 1) >= (unsigned long long)kLenMask);
    const unsigned l = (unsigned)len & kLenMask;
    const unsigned long long ck =
        (corr ? 1ull << 63 : 0ull) | ((unsigned long long)key << 31) | ((unsigned long long)(unsigned)j << kLenBits) | l;
    S.ck[min(j, kWCap - 1)] = pres ? ck : kNone;
    ptok += pres ? l : 0u;
    const unsigned pm = __ballot_sync(0xffffffffu, pres);
    const unsigned cm = __ballot_sync(0xffffffffu, pres && corr);
    if (lane == 0) { S.pmask[c] = pm; S.cmask[c] = cm; }
  }
  if (__any_sync(0xffffffffu, irregular)) return false;
  mine.present_tok = ptok;
  __syncwarp();

  // ---- per prompt: counts, category, posterior, curation rule, moments of the base set ----
  int sort_n = 0, sort_idx = 0;      // a selection in a group of at most 16: its size and the place of its threshold
  if (lane < sh.np) {
    const int p = sh.p0 + lane;
    const int n = HAS_KEEP_IN ? range_popc(S.pmask, sh.lo, sh.hi) : sh.hi - sh.lo;
    const int c = range_popc(S.cmask, sh.lo, sh.hi);
    const Rule ru = decide(a, p, n, c);
    a.cat[p] = (uint8_t)ru.category;
    a.u_tilde[p] = ru.ut;
    a.alpha_out[p] = ru.al;
    a.beta_out[p] = ru.be;
    // keys with the index appended are distinct, so a selection keeps exactly its quota
    int nk = n, ck = c;
    if (ru.mode == 1) { nk = 0; ck = 0; }
    else if (ru.mode == 2) {
      const int q = (int)ru.quota;
      if (ru.reject == 0) { nk = q; ck = c > 0 ? q : 0; }
      else if (ru.reject == 1) { nk = c + q; ck = c; }
      else { nk = (n - c) + q; ck = q; }
    }
    const bool over_kept = a.cfg.stats_over == AERO_STATS_KEPT;
    float mu, inv;
    group_moments(a, ru, over_kept ? nk : n, over_kept ? ck : c, &mu, &inv);
    a.gmask[p] = nk > 0 ? 1 : 0;
    if (a.cfg.agg != AERO_TOKEN_MEAN) ws.nkept[p] = nk;
    PromptRule pr;
    pr.adv_correct = (1.f - mu) * inv;
    pr.adv_incorrect = (0.f - mu) * inv;
    pr.range = (unsigned)sh.lo | ((unsigned)sh.hi << 16);
    // every incorrect rollout orders before every correct one: when the correct ones are the
    // candidates, the n - c incorrect ones are counted by each rank and the quota allows for them
    const bool sel = ru.mode == 2;
    const int quota = (int)ru.quota + (ru.reject == 2 ? n - c : 0);
    if (sel && sh.hi - sh.lo <= 16 && quota > 0 && quota < sh.hi - sh.lo) { sort_n = sh.hi - sh.lo; sort_idx = quota - 1; }
    pr.sel = (ru.mode == 1 ? 1u : 0u) | (sel && ru.reject != 2 ? 2u : 0u) | (sel && ru.reject != 1 ? 4u : 0u) |
             ((unsigned)quota << 4);
    S.rule[lane] = pr;
    mine.present_roll = n;
#pragma unroll
    for (int k = 0; k < 5; ++k) mine.cat[k] = ru.category == k ? 1 : 0;
    mine.surv = nk > 0 ? 1 : 0;
    mine.abs_adv = ((float)ck * fabsf(1.f - mu) + (float)(nk - ck) * fabsf(mu)) * inv;
  }
  // ---- per prompt with a selection in a small group: its threshold, where that decides exactly ----
  const int widest = (int)__reduce_max_sync(0xffffffffu, (unsigned)sort_n);
  if (widest > 0) {
    unsigned thr = 0;
    const bool exact = widest > 8 ? threshold_half<16>(S.ck + sh.lo, sort_n, sort_idx, &thr)
                                  : threshold_half<8>(S.ck + sh.lo, sort_n, sort_idx, &thr);
    if (sort_n > 0 && exact) {
      S.rule[lane].range = thr;
      S.rule[lane].sel |= 8u;
    }
  }
  __syncwarp();

  // ---- per rollout: keep decision (threshold, or rank among the group's candidates), advantage ----
  int cnt = 0;
  unsigned ktok = 0;       // at most kWChunks lengths below 2^22 per lane
  for (int c = 0; c * 32 < nroll; ++c) {
    const int j = c * 32 + lane;
    const bool valid = j < nroll;
    const PromptRule pr = S.rule[valid ? S.pid[j] : 0];
    const unsigned long long mykey = S.ck[min(j, kWCap - 1)];
    const bool pres = (S.pmask[c] >> lane) & 1u;
    const bool corr = (S.cmask[c] >> lane) & 1u;
    bool kp = pres && !(pr.sel & 1u);
    const bool ranked = pres && (pr.sel & (corr ? 4u : 2u));
    const bool by_half = (pr.sel & 8u) != 0;
    if (ranked && by_half) kp = (unsigned)(mykey >> 32) <= pr.range;
    // the others: the loop runs as long as the longest group among the chunk's rollouts ranked by it, the
    // same for all lanes
    const int lo = by_half ? 0 : (int)(pr.range & 0xffffu);
    const int span = ranked && !by_half ? (int)(pr.range >> 16) - lo : 0;
    const int longest = (int)__reduce_max_sync(0xffffffffu, (unsigned)span);
    if (longest > 0) {
      // (reads past the lane's own group stay inside the block's shared memory and are not counted)
      const unsigned long long* grp = S.ck + lo;
      int rank = 0;
#pragma unroll 4
      for (int d = 0; d < longest; ++d) {
        const unsigned long long other = grp[d];
        rank += (d < span && other < mykey) ? 1 : 0;
      }
      if (span > 0) kp = rank < (int)(pr.sel >> 4);
    }
    const unsigned km = __ballot_sync(0xffffffffu, kp);
    if (valid) {
      a.adv[r0 + j] = kp ? (corr ? pr.adv_correct : pr.adv_incorrect) : 0.f;
      a.keep[r0 + j] = kp ? 1 : 0;
      a.w[r0 + j] = __uint_as_float(kp ? kKeptBit | ((unsigned)mykey & kLenMask) : 0u);     // for the second pass
    }
    cnt += __popc(km);
    ktok += kp ? (unsigned)mykey & kLenMask : 0u;
  }
  long long tok = ktok;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tok += __shfl_xor_sync(0xffffffffu, tok, o);
  *cnt_out = cnt;
  *tok_out = tok;
  return true;
}

// A share whose rollouts exceed the staging area (a very large group): the same steps with one
// lane per prompt walking the caller's arrays.
__device__ void curate_global(const Args& a, const Workspace& ws, const Share& sh, TilePartial& mine, uint32_t& st,
                              int* cnt_out, long long* tok_out) {
  const int lane = threadIdx.x & 31;
  const int r0 = sh.r0;
  auto present = [&](int j) { return a.keep_in ? a.keep_in[r0 + j] != 0 : true; };
  auto order_key = [&](int j) {
    if (!present(j)) return kNone;
    const uint32_t key = a.key ? a.key[r0 + j] : default_key(a.cfg.seed, (uint32_t)(r0 + j));
    return ((unsigned long long)key << 32) | (unsigned)j;
  };
  int nk = 0;
  long long ktok = 0;
  if (lane < sh.np) {
    const int p = sh.p0 + lane;
    const int lo = sh.lo, hi = sh.hi;
    int n = 0, c = 0;
    for (int j = lo; j < hi; ++j) {
      if (!present(j)) continue;
      const float r = a.reward[r0 + j];
      const long long len = a.cs[r0 + j + 1] - a.cs[r0 + j];
      if (r != 0.f && r != 1.f) st |= AERO_ST_BAD_REWARD;
      if (len < 0) st |= AERO_ST_BAD_OFFSETS;
      if (len == 0) st |= AERO_ST_EMPTY_ROLLOUT;
      n += 1; c += r > 0.5f ? 1 : 0;
      mine.present_tok += clamped_len(len);
    }
    mine.present_roll = n;
    const Rule ru = decide(a, p, n, c);
    a.cat[p] = (uint8_t)ru.category;
    a.u_tilde[p] = ru.ut;
    a.alpha_out[p] = ru.al;
    a.beta_out[p] = ru.be;
#pragma unroll
    for (int k = 0; k < 5; ++k) mine.cat[k] = ru.category == k ? 1 : 0;

    int ck = 0;
    for (int j = lo; j < hi; ++j) {
      const bool corr = a.reward[r0 + j] > 0.5f;
      bool kp = present(j) && ru.mode != 1;
      if (kp && ru.mode == 2 && !(ru.reject == 1 && corr) && !(ru.reject == 2 && !corr)) {
        const unsigned long long mykey = order_key(j);
        long long rank = 0;
        for (int k = lo; k < hi; ++k) {
          const bool other = a.reward[r0 + k] > 0.5f;
          if ((ru.reject == 1 && other) || (ru.reject == 2 && !other)) continue;
          rank += order_key(k) < mykey ? 1 : 0;
        }
        kp = rank < ru.quota;
      }
      const int len = clamped_len(a.cs[r0 + j + 1] - a.cs[r0 + j]);
      a.keep[r0 + j] = kp ? 1 : 0;
      a.w[r0 + j] = __uint_as_float(kp ? kKeptBit | (unsigned)len : 0u);                    // for the second pass
      if (kp) { nk += 1; ck += corr ? 1 : 0; ktok += len; }
    }
    const bool over_kept = a.cfg.stats_over == AERO_STATS_KEPT;
    float mu, inv;
    group_moments(a, ru, over_kept ? nk : n, over_kept ? ck : c, &mu, &inv);
    for (int j = lo; j < hi; ++j)
      a.adv[r0 + j] = a.keep[r0 + j] ? ((a.reward[r0 + j] > 0.5f ? 1.f : 0.f) - mu) * inv : 0.f;
    a.gmask[p] = nk > 0 ? 1 : 0;
    if (a.cfg.agg != AERO_TOKEN_MEAN) ws.nkept[p] = nk;
    mine.surv = nk > 0 ? 1 : 0;
    mine.abs_adv = ((float)ck * fabsf(1.f - mu) + (float)(nk - ck) * fabsf(mu)) * inv;
  }
  *cnt_out = __reduce_add_sync(0xffffffffu, nk);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ktok += __shfl_xor_sync(0xffffffffu, ktok, o);
  *tok_out = ktok;
}

template <bool HAS_KEEP_IN, bool HAS_KEY>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM) curate_kernel(Args a, Workspace ws, int pw) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  BlockShared& bs = *reinterpret_cast<BlockShared*>(smem_raw);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile = blockIdx.x;
  uint32_t st = 0;
  const Share sh = load_share(a, tile * kWarps + warp, pw, st);
  TilePartial mine = {};
  int cnt = 0;
  long long tok = 0;
  if (sh.np > 0) {
    const WarpStage S = {bs.ck[warp], bs.rule[warp], bs.pmask[warp], bs.cmask[warp], bs.pid[warp]};
    const bool done = sh.nroll <= kWCap && curate_staged<HAS_KEEP_IN, HAS_KEY>(a, ws, S, sh, mine, st, &cnt, &tok);
    if (!done) curate_global(a, ws, sh, mine, st, &cnt, &tok);
  }
  mine = warp_partial(mine);
  if (lane == 0) {
    bs.red[warp] = mine;
    bs.share_cnt[warp] = cnt;
    bs.share_tok[warp] = tok;
    ws.share_cnt[tile * kWarps + warp] = cnt;
    ws.share_tok[tile * kWarps + warp] = tok;
  }
  st = __reduce_or_sync(0xffffffffu, st);
  if (lane == 0) aero_raise(a.status, st);
  __syncthreads();
  // the tile's record: its warps added in order
  if (threadIdx.x == 0) {
    TilePartial tot = {};
    int tcnt = 0;
    long long ttok = 0;
    for (int k = 0; k < kWarps; ++k) {
      tot.present_tok += bs.red[k].present_tok; tot.present_roll += bs.red[k].present_roll; tot.surv += bs.red[k].surv;
      for (int c = 0; c < 5; ++c) tot.cat[c] += bs.red[k].cat[c];
      tot.abs_adv += bs.red[k].abs_adv;
      tcnt += bs.share_cnt[k];
      ttok += bs.share_tok[k];
    }
    ws.part[tile] = tot;
    ws.tile_cnt[tile] = tcnt;
    ws.tile_tok[tile] = ttok;
  }
}

// Level 1 of the batch-wide prefix: one block per run of kRunTiles consecutive tiles (each
// thread owns four of them) turns the run's tile totals into exclusive prefixes inside the run
// and leaves the run's totals and the sum of its metrics records, all sums in a fixed order.
__global__ void __launch_bounds__(kRunThreads) run_prefix_kernel(Workspace ws, int ntiles) {
  __shared__ long long s_tok[kRunThreads / 32];
  __shared__ int s_cnt[kRunThreads / 32];
  __shared__ RunPartial s_part[kRunThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = min(blockIdx.x * kRunTiles + tid * 4, ntiles), t1 = min(t0 + 4, ntiles);
  int c[4];
  long long k[4];
  int cnt = 0;
  long long tok = 0;
  RunPartial mine = {};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    c[e] = 0; k[e] = 0;
    if (t0 + e < t1) {
      c[e] = ws.tile_cnt[t0 + e];
      k[e] = ws.tile_tok[t0 + e];
      const TilePartial q = ws.part[t0 + e];
      mine.misc[0] += q.present_tok; mine.misc[1] += q.present_roll; mine.misc[2] += q.surv;
#pragma unroll
      for (int m = 0; m < 5; ++m) mine.misc[3 + m] += q.cat[m];
      mine.abs_adv += (double)q.abs_adv;
    }
    cnt += c[e];
    tok += k[e];
  }
  int icnt = cnt;
  long long itok = tok;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int c2 = __shfl_up_sync(0xffffffffu, icnt, o);
    const long long t2 = __shfl_up_sync(0xffffffffu, itok, o);
    if (lane >= o) { icnt += c2; itok += t2; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine.abs_adv += __shfl_xor_sync(0xffffffffu, mine.abs_adv, o);
#pragma unroll
    for (int m = 0; m < 8; ++m) mine.misc[m] += __shfl_xor_sync(0xffffffffu, mine.misc[m], o);
  }
  if (lane == 31) { s_cnt[warp] = icnt; s_tok[warp] = itok; }
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  int run_cnt = icnt - cnt;
  long long run_tok = itok - tok;
  for (int w = 0; w < warp; ++w) { run_cnt += s_cnt[w]; run_tok += s_tok[w]; }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (t0 + e < t1) {
      ws.tile_cnt[t0 + e] = run_cnt;
      ws.tile_tok[t0 + e] = run_tok;
    }
    run_cnt += c[e];
    run_tok += k[e];
  }
  if (tid == 0) {
    RunPartial tot = {};
    int rc = 0;
    long long rt = 0;
    for (int w = 0; w < kRunThreads / 32; ++w) {
      tot.abs_adv += s_part[w].abs_adv;
      for (int m = 0; m < 8; ++m) tot.misc[m] += s_part[w].misc[m];
      rc += s_cnt[w];
      rt += s_tok[w];
    }
    ws.run_part[blockIdx.x] = tot;
    ws.run_cnt[blockIdx.x] = rc;
    ws.run_tok[blockIdx.x] = rt;
  }
}

// Level 2, one block: exclusive prefixes of the runs' totals (each thread owns consecutive
// runs), then the batch totals, counters and metrics, all sums in a fixed order.
__global__ void __launch_bounds__(kRunThreads) totals_kernel(Args a, Workspace ws, int nruns) {
  __shared__ long long s_tok[kRunThreads / 32];
  __shared__ long long s_cnt[kRunThreads / 32];
  __shared__ RunPartial s_part[kRunThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (nruns + kRunThreads - 1) / kRunThreads;
  const int t0 = min(tid * per, nruns), t1 = min(t0 + per, nruns);
  long long cnt = 0, tok = 0;
  RunPartial mine = {};
  for (int t = t0; t < t1; ++t) {
    cnt += ws.run_cnt[t];
    tok += ws.run_tok[t];
    const RunPartial q = ws.run_part[t];
    mine.abs_adv += q.abs_adv;
#pragma unroll
    for (int m = 0; m < 8; ++m) mine.misc[m] += q.misc[m];
  }
  long long icnt = cnt, itok = tok;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long c2 = __shfl_up_sync(0xffffffffu, icnt, o);
    const long long t2 = __shfl_up_sync(0xffffffffu, itok, o);
    if (lane >= o) { icnt += c2; itok += t2; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine.abs_adv += __shfl_xor_sync(0xffffffffu, mine.abs_adv, o);
#pragma unroll
    for (int m = 0; m < 8; ++m) mine.misc[m] += __shfl_xor_sync(0xffffffffu, mine.misc[m], o);
  }
  if (lane == 31) { s_cnt[warp] = icnt; s_tok[warp] = itok; }
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  long long run_cnt = icnt - cnt, run_tok = itok - tok;
  for (int w = 0; w < warp; ++w) { run_cnt += s_cnt[w]; run_tok += s_tok[w]; }
  for (int t = t0; t < t1; ++t) {
    const int c = ws.run_cnt[t];
    const long long k = ws.run_tok[t];
    ws.run_cnt[t] = (int)run_cnt;
    ws.run_tok[t] = run_tok;
    run_cnt += c;
    run_tok += k;
  }
  if (tid == 0) {
    long long tot[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    double sabs = 0.0;
    long long R_kept = 0, T_kept = 0;
    for (int w = 0; w < kRunThreads / 32; ++w) {
      sabs += s_part[w].abs_adv;
      for (int m = 0; m < 8; ++m) tot[m] += s_part[w].misc[m];
      R_kept += s_cnt[w];
      T_kept += s_tok[w];
    }
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

// Compacted ids and token offsets of the kept rollouts, per-rollout weights (Eq. 2 normalisers)
// and the tails of the compacted arrays; one warp per share, one lane per rollout.
template <bool SEQ_MEAN>
__global__ void __launch_bounds__(kThreads) emit_kernel(Args a, Workspace ws, int pw) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile = blockIdx.x;
  uint32_t st = 0;      // bad offsets were reported by the first launch
  // kept rollouts and tokens before this share: earlier runs, earlier tiles of the run, earlier warps of
  // the tile (these loads do not depend on the share's offsets and are issued ahead of them)
  const Globals g = *ws.glob;
  int pos0 = lane < warp ? ws.share_cnt[tile * kWarps + lane] : 0;
  long long tok0 = lane < warp ? ws.share_tok[tile * kWarps + lane] : 0;
  const int before_cnt = ws.run_cnt[tile / kRunTiles] + ws.tile_cnt[tile];
  const long long before_tok = ws.run_tok[tile / kRunTiles] + ws.tile_tok[tile];
  const Share sh = load_share(a, tile * kWarps + warp, pw, st);
  if (sh.np == 0 || sh.nroll == 0) return;
  pos0 = __reduce_add_sync(0xffffffffu, pos0);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tok0 += __shfl_xor_sync(0xffffffffu, tok0, o);
  pos0 += before_cnt;
  tok0 += before_tok;
  const unsigned below = (1u << lane) - 1u;
  // one chunk of 32 rollouts, its keep flags and lengths already loaded
  auto emit_chunk = [&](int c0, int i, bool valid, bool kp, int len) {
    const unsigned km = __ballot_sync(0xffffffffu, kp);
    if (km) {
      long long incl;
      if (__reduce_max_sync(0xffffffffu, kp ? (unsigned)len : 0u) < (1u << 26)) {   // the chunk's sum fits 32 bits
        unsigned t32 = kp ? (unsigned)len : 0u;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned t2 = __shfl_up_sync(0xffffffffu, t32, o);
          if (lane >= o) t32 += t2;
        }
        incl = t32;
      } else {
        incl = kp ? len : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const long long t2 = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t2;
        }
      }
      // (with offsets that are not a partition of the rollouts the shares may overlap and the
      // counts exceed R: such entries are dropped, the status bit has been raised)
      const int pos = pos0 + __popc(km & below);
      if (kp && pos < a.R) {
        a.kept_ids[pos] = i;
        a.kept_tok_off[pos] = tok0 + incl - len;
      }
      pos0 += __popc(km);
      tok0 += __shfl_sync(0xffffffffu, incl, 31);
    }
    float w = kp ? g.inv_tok_den : 0.f;
    if (SEQ_MEAN) {
      // the rollout's prompt is the last one of the share that starts at or before it
      const int j = c0 + lane;
      int q = 0;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        const int cand = q + s;
        const int start = __shfl_sync(0xffffffffu, sh.lo, cand & 31);
        if (cand < sh.np && start <= j) q = cand;
      }
      const int nk = kp ? ws.nkept[sh.p0 + q] : 0;
      w = (nk > 0 && len > 0) ? g.inv_prompt_den / (float)nk / (float)len : 0.f;
    }
    if (valid) a.w[i] = w;
    // tails of the compacted arrays, only where the chunk reaches them
    if ((long long)sh.r0 + c0 + 32 >= g.R_kept && valid) {
      if ((long long)i >= g.R_kept) a.kept_ids[i] = -1;
      if ((long long)i + 1 >= g.R_kept) a.kept_tok_off[i + 1] = g.T_kept;
      if (i == 0 && g.R_kept == 0) a.kept_tok_off[0] = 0;
    }
  };
  // two chunks per turn, the loads of both issued before either is processed; lanes past the
  // share's end read its last rollout again and count as not kept
  for (int c0 = 0; c0 < sh.nroll; c0 += 64) {
    const int j0 = c0 + lane, j1 = j0 + 32;
    const bool v0 = j0 < sh.nroll, v1 = j1 < sh.nroll;
    const int i0 = sh.r0 + min(j0, sh.nroll - 1), i1 = sh.r0 + min(j1, sh.nroll - 1);
    // what the first pass left in w: the kept bit and the rollout's length
    const unsigned k0 = __float_as_uint(a.w[i0]), k1 = __float_as_uint(a.w[i1]);
    emit_chunk(c0, i0, v0, v0 && (k0 & kKeptBit), (int)(k0 & ~kKeptBit));
    if (c0 + 32 < sh.nroll) emit_chunk(c0 + 32, i1, v1, v1 && (k1 & kKeptBit), (int)(k1 & ~kKeptBit));
  }
}

}  // namespace

size_t aero_group_ws_bytes_impl(int32_t P, int32_t R) {
  if (P < 0) P = 0;
  const int pt = prompts_per_warp(P, R) * kWarps;
  const int ntiles = (P + pt - 1) / pt;
  return workspace_bytes((size_t)P, (size_t)ntiles);
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
  const int pw = prompts_per_warp(P, R);
  const int pt = pw * kWarps;
  const int ntiles = (P + pt - 1) / pt;
  Workspace ws = carve(wsp, P, ntiles);
  auto curate = keep_in ? (key ? curate_kernel<true, true> : curate_kernel<true, false>)
                        : (key ? curate_kernel<false, true> : curate_kernel<false, false>);
  AERO_CUDA_TRY(cudaFuncSetAttribute(curate, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BlockShared)));
  curate<<<ntiles, kThreads, sizeof(BlockShared), ctx->stream>>>(a, ws, pw);
  const int nruns = (int)runs_of((size_t)ntiles);
  run_prefix_kernel<<<nruns, kRunThreads, 0, ctx->stream>>>(ws, ntiles);
  totals_kernel<<<1, kRunThreads, 0, ctx->stream>>>(a, ws, nruns);
  if (cfg->agg != AERO_TOKEN_MEAN) emit_kernel<true><<<ntiles, kThreads, 0, ctx->stream>>>(a, ws, pw);
  else emit_kernel<false><<<ntiles, kThreads, 0, ctx->stream>>>(a, ws, pw);
  ctx->launches += 4;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

// ---- weights of a data-parallel shard -----------------------------------------------------
namespace {

// Eq. 2's normalisers are batch-wide.  A rank that ran the group stage on its own prompts holds
// weights over its local denominator; multiplying by local / global denominator (both read from
// the counters on the device, so the host never waits) gives the weights of the whole batch.
__global__ void __launch_bounds__(256) finalize_weights_kernel(aero_cfg cfg, int R, long long P_local, long long P_global,
                                                               float* __restrict__ w,
                                                               const int64_t* __restrict__ cl, const int64_t* __restrict__ cg) {
  long long num, den;
  if (cfg.agg == AERO_TOKEN_MEAN) {
    const int k = cfg.denom == AERO_DENOM_SURVIVING ? AERO_CNT_T_KEPT : AERO_CNT_T_PRESENT;
    num = cl[k]; den = cg[k];
  } else if (cfg.denom == AERO_DENOM_SURVIVING) {
    num = cl[AERO_CNT_P_SURV]; den = cg[AERO_CNT_P_SURV];
  } else {
    num = P_local; den = P_global;
  }
  const double f = den > 0 ? (double)num / (double)den : 0.0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < R; i += gridDim.x * blockDim.x)
    w[i] = (float)((double)w[i] * f);
}

}  // namespace

int aero_finalize_weights_launch(aero_ctx* ctx, const aero_cfg* cfg, int32_t R, int32_t P_local, int64_t P_global,
                                 float* w, const int64_t* counters_local, const int64_t* counters_global) {
  if (R == 0) return AERO_OK;
  const int blocks = (R + 255) / 256 < 4 * ctx->sm_count ? (R + 255) / 256 : 4 * ctx->sm_count;
  finalize_weights_kernel<<<blocks, 256, 0, ctx->stream>>>(*cfg, R, P_local, P_global, w, counters_local, counters_global);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

// ---- variant with library-owned scratch ------------------------------------------------
// The kernels above need a few bytes of scratch per prompt and per tile.  This entry point takes
// them from a fixed array in device memory that is part of the loaded library image, so the
// caller passes inputs and outputs only and nothing is allocated, by this call or before it.
namespace {

constexpr int32_t kStaticMaxP = AERO_STATIC_MAX_PROMPTS;
// room for kStaticMaxP prompts in the smallest tiles there are (one prompt per warp)
constexpr size_t kStaticBytes = workspace_bytes((size_t)kStaticMaxP, ((size_t)kStaticMaxP + kWarps - 1) / kWarps);
static_assert(kStaticBytes == AERO_STATIC_SCRATCH_BYTES, "the header states the size of the array");

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
  // every scratch word the kernels read is written earlier in the same call
  return aero_group_stats_launch(ctx, cfg, P, R, go, reward, cs, key, keep_in, alpha_in, beta_in,
                                 adv, w, keep, gmask, cat, u_tilde, alpha_out, beta_out,
                                 kept_ids, kept_tok_off, counters, metrics, scratch);
}

