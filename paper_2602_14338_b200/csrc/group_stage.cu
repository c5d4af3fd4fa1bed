// Stage (a): segmented per-prompt group statistics (Eq. 1; Sec. 3.2; Sec. 4.2
// Strategies 2-3; Appendix C).  Three launches:
//   group_kernel    a team of L lanes per prompt: counts, category, posterior,
//                   keep-mask by rank among (key, index), advantages; per-block totals
//   scan_kernel     one block: exclusive scan of the per-block totals, global counters
//   compact_kernel  same team layout: compact ids, kept-token offsets and weights
// Reductions inside a team are warp shuffles; a block covers consecutive prompts, so
// its loads and stores touch one contiguous range of the rollout arrays.
#include "common.cuh"

#include <mutex>

namespace {

constexpr int kThreads = 256;

struct BlockPartial {
  long long kept_tok, present_tok;
  int kept_roll, present_roll, surv;
  int cat[5];
  float abs_adv;
  int pad;
};

struct Globals {
  long long R_kept, T_kept, T_present;
  int P_surv;
  float inv_tok_den;      // 1 / (token-mean denominator), 0 if empty
  float inv_prompt_den;   // 1 / (sequence-mean prompt denominator), 0 if empty
  int pad;
};

struct BlockOffset {
  long long tok;
  int roll;
  int pad;
};

struct Workspace {
  int* nkept;             // [P]
  long long* tkept;       // [P]
  BlockPartial* part;     // [nb]
  BlockOffset* off;       // [nb]
  Globals* glob;          // [1]
};

__host__ __device__ inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

inline int team_lanes(int32_t P, int32_t R) {
  long long avg = P > 0 ? ((long long)R + P - 1) / P : 1;
  return avg <= 8 ? 8 : (avg <= 16 ? 16 : 32);
}

inline Workspace carve(void* ws, int32_t P, int nb) {
  char* p = static_cast<char*>(ws);
  Workspace w;
  w.nkept = reinterpret_cast<int*>(p);            p += up256(sizeof(int) * (size_t)P);
  w.tkept = reinterpret_cast<long long*>(p);      p += up256(sizeof(long long) * (size_t)P);
  w.part = reinterpret_cast<BlockPartial*>(p);    p += up256(sizeof(BlockPartial) * (size_t)nb);
  w.off = reinterpret_cast<BlockOffset*>(p);      p += up256(sizeof(BlockOffset) * (size_t)nb);
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

template <int L, typename T>
__device__ __forceinline__ T team_sum(T v, unsigned mask) {
#pragma unroll
  for (int o = L / 2; o > 0; o >>= 1) v += __shfl_xor_sync(mask, v, o, L);
  return v;
}

template <int L>
__device__ __forceinline__ unsigned team_mask() {
  const unsigned lane = threadIdx.x & 31u;
  if (L == 32) return 0xffffffffu;
  return ((1u << (L & 31)) - 1u) << (lane / L * L);
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

template <int L>
__global__ void __launch_bounds__(kThreads) group_kernel(Args a, Workspace ws) {
  constexpr int PPB = kThreads / L;
  __shared__ BlockPartial s_part[PPB];
  const int team = threadIdx.x / L;
  const int lane = threadIdx.x % L;
  const unsigned mask = team_mask<L>();
  const int p = blockIdx.x * PPB + team;
  BlockPartial mine = {};
  uint32_t st = 0;

  if (p < a.P) {
    int lo = a.go[p], hi = a.go[p + 1];
    if (lo < 0 || hi < lo || hi > a.R) {
      st |= AERO_ST_BAD_OFFSETS;
      lo = min(max(lo, 0), a.R);
      hi = min(max(hi, lo), a.R);
    }
    // counts over present rollouts
    int n = 0, c = 0;
    long long ptok = 0;
    for (int base = lo; base < hi; base += L) {
      const int i = base + lane;
      if (i < hi) {
        const bool pres = a.keep_in ? a.keep_in[i] != 0 : true;
        if (pres) {
          const float r = a.reward[i];
          const long long len = a.cs[i + 1] - a.cs[i];
          if (r != 0.f && r != 1.f) st |= AERO_ST_BAD_REWARD;
          if (len < 0) st |= AERO_ST_BAD_OFFSETS;
          if (len == 0) st |= AERO_ST_EMPTY_ROLLOUT;
          n += 1;
          c += r > 0.5f ? 1 : 0;
          ptok += len > 0 ? len : 0;
        }
      }
    }
    n = team_sum<L>(n, mask);
    c = team_sum<L>(c, mask);
    ptok = team_sum<L>(ptok, mask);

    int category;
    if (n == 0) category = AERO_CAT_EMPTY;
    else if (c == 0) category = AERO_CAT_ZERO;
    else if (c == n) category = AERO_CAT_PERFECT;
    else if (2 * c < n) category = AERO_CAT_PARTIAL;
    else category = AERO_CAT_GOOD;

    const float al = (a.alpha_in ? a.alpha_in[p] : a.cfg.alpha0) + (float)c;
    const float be = (a.beta_in ? a.beta_in[p] : a.cfg.beta0) + (float)(n - c);
    const float ut = al / (al + be);

    // curation rule: 0 keep all present, 1 keep none, 2 select by rank
    const bool uniform = (c == 0 || c == n);
    int mode = 0;
    long long quota = 0;
    bool reject = false;     // select among the incorrect, keep every correct one
    if (n == 0) {
      mode = 1;
    } else if (uniform) {
      if (a.cfg.uniform_policy == AERO_UNIFORM_MASK) mode = 1;
      else if (a.cfg.n_keep_uniform > 0 && a.cfg.n_keep_uniform < n) { mode = 2; quota = a.cfg.n_keep_uniform; }
    } else {
      const bool low = category == AERO_CAT_PARTIAL ||
                       (a.cfg.rescue_S > 0 &&
                        (long long)c * a.cfg.n_explore <= (long long)a.cfg.rescue_S * n);
      if (a.cfg.rejection && low) {
        const long long m = min((long long)a.cfg.k_ratio * c, (long long)(n - c));
        if (m < n - c) { mode = 2; quota = m; reject = true; }
      }
    }

    // keep-mask and sums over the statistics base
    int nk = 0, nbase = 0;
    long long ktok = 0;
    float sum_r = 0.f;
    for (int base = lo; base < hi; base += L) {
      const int i = base + lane;
      if (i < hi) {
        const bool pres = a.keep_in ? a.keep_in[i] != 0 : true;
        const float r = a.reward[i];
        const bool corr = r > 0.5f;
        bool kp = pres && mode != 1;
        if (kp && mode == 2 && !(reject && corr)) {
          const uint32_t ki = a.key ? a.key[i] : default_key(a.cfg.seed, (uint32_t)i);
          long long rank = 0;
          for (int j = lo; j < hi; ++j) {
            const bool pj = a.keep_in ? a.keep_in[j] != 0 : true;
            if (!pj) continue;
            if (reject && a.reward[j] > 0.5f) continue;
            const uint32_t kj = a.key ? a.key[j] : default_key(a.cfg.seed, (uint32_t)j);
            rank += (kj < ki || (kj == ki && j < i)) ? 1 : 0;
          }
          kp = rank < quota;
        }
        a.keep[i] = kp ? 1 : 0;
        if (kp) {
          const long long len = a.cs[i + 1] - a.cs[i];
          nk += 1;
          ktok += len > 0 ? len : 0;
        }
        const bool in_base = a.cfg.stats_over == AERO_STATS_KEPT ? kp : pres;
        if (in_base) { nbase += 1; sum_r += r; }
      }
    }
    nk = team_sum<L>(nk, mask);
    nbase = team_sum<L>(nbase, mask);
    ktok = team_sum<L>(ktok, mask);
    sum_r = team_sum<L>(sum_r, mask);

    float mu = 0.f, sd = 0.f;
    if (uniform) {
      mu = ut;
      sd = sqrtf(ut * (1.f - ut));
    } else if (nbase > 0) {
      mu = sum_r / (float)nbase;
      float ss = 0.f;
      for (int base = lo; base < hi; base += L) {
        const int i = base + lane;
        if (i < hi) {
          const bool pres = a.keep_in ? a.keep_in[i] != 0 : true;
          const bool in_base = a.cfg.stats_over == AERO_STATS_KEPT ? a.keep[i] != 0 : pres;
          if (in_base) { const float dlt = a.reward[i] - mu; ss += dlt * dlt; }
        }
      }
      ss = team_sum<L>(ss, mask);
      sd = sqrtf(ss / (float)nbase);
    }
    const float inv = 1.f / (sd + a.cfg.eps_std);
    float abs_adv = 0.f;
    for (int base = lo; base < hi; base += L) {
      const int i = base + lane;
      if (i < hi) {
        float av = 0.f;
        if (a.keep[i]) av = (a.reward[i] - mu) * inv;
        a.adv[i] = av;
        abs_adv += fabsf(av);
      }
    }
    abs_adv = team_sum<L>(abs_adv, mask);

    if (lane == 0) {
      a.cat[p] = (uint8_t)category;
      a.gmask[p] = nk > 0 ? 1 : 0;
      a.u_tilde[p] = ut;
      a.alpha_out[p] = al;
      a.beta_out[p] = be;
      ws.nkept[p] = nk;
      ws.tkept[p] = ktok;
      mine.kept_tok = ktok;
      mine.present_tok = ptok;
      mine.kept_roll = nk;
      mine.present_roll = n;
      mine.surv = nk > 0 ? 1 : 0;
      mine.cat[category] = 1;
      mine.abs_adv = abs_adv;
    }
  }
  st = __reduce_or_sync(0xffffffffu, st);
  if ((threadIdx.x & 31) == 0) aero_raise(a.status, st);
  if (lane == 0) s_part[team] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    BlockPartial tot = {};
    for (int t = 0; t < PPB; ++t) {      // fixed order: the float sum is reproducible
      tot.kept_tok += s_part[t].kept_tok;
      tot.present_tok += s_part[t].present_tok;
      tot.kept_roll += s_part[t].kept_roll;
      tot.present_roll += s_part[t].present_roll;
      tot.surv += s_part[t].surv;
      for (int k = 0; k < 5; ++k) tot.cat[k] += s_part[t].cat[k];
      tot.abs_adv += s_part[t].abs_adv;
    }
    ws.part[blockIdx.x] = tot;
  }
}

// One block of 1024 threads: exclusive scan of the per-block totals in block order.
__global__ void __launch_bounds__(1024) scan_kernel(Args a, Workspace ws, int nb) {
  __shared__ long long s_tok[1024];
  __shared__ int s_roll[1024];
  __shared__ double s_abs[32];
  __shared__ long long s_misc[32][8];   // present tokens, present rollouts, surviving prompts, 5 categories
  const int tid = threadIdx.x;
  const int per = (nb + 1023) / 1024;
  const int b0 = min(tid * per, nb), b1 = min(b0 + per, nb);
  long long tok = 0;
  long long misc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int roll = 0;
  double aabs = 0.0;
  for (int b = b0; b < b1; ++b) {
    const BlockPartial q = ws.part[b];
    tok += q.kept_tok; roll += q.kept_roll;
    misc[0] += q.present_tok; misc[1] += q.present_roll; misc[2] += q.surv;
    for (int k = 0; k < 5; ++k) misc[3 + k] += q.cat[k];
    aabs += (double)q.abs_adv;
  }
  // totals that are not scanned: shuffle tree per warp (fixed shape, so the
  // floating-point sum is reproducible), then 32 partial sums in order
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
  s_tok[tid] = tok; s_roll[tid] = roll;
  __syncthreads();
  // Hillis-Steele inclusive scan on the two scanned quantities
  for (int o = 1; o < 1024; o <<= 1) {
    long long t2 = 0; int r2 = 0;
    if (tid >= o) { t2 = s_tok[tid - o]; r2 = s_roll[tid - o]; }
    __syncthreads();
    s_tok[tid] += t2; s_roll[tid] += r2;
    __syncthreads();
  }
  long long run_tok = s_tok[tid] - tok;
  int run_roll = s_roll[tid] - roll;
  for (int b = b0; b < b1; ++b) {
    BlockOffset o; o.tok = run_tok; o.roll = run_roll; o.pad = 0;
    ws.off[b] = o;
    run_tok += ws.part[b].kept_tok;
    run_roll += ws.part[b].kept_roll;
  }
  if (tid == 0) {
    const long long T_kept = s_tok[1023], R_kept = s_roll[1023];
    long long tot[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    double sabs = 0.0;
    for (int t = 0; t < 32; ++t) {
      sabs += s_abs[t];
      for (int k = 0; k < 8; ++k) tot[k] += s_misc[t][k];
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

template <int L>
__global__ void __launch_bounds__(kThreads) compact_kernel(Args a, Workspace ws) {
  constexpr int PPB = kThreads / L;
  __shared__ int s_roll[PPB];
  __shared__ long long s_tok[PPB];
  const int team = threadIdx.x / L;
  const int lane = threadIdx.x % L;
  const unsigned mask = team_mask<L>();
  const int p = blockIdx.x * PPB + team;
  const Globals g = *ws.glob;
  int nk = 0;
  long long tk = 0;
  if (p < a.P) { nk = ws.nkept[p]; tk = ws.tkept[p]; }
  if (lane == 0) { s_roll[team] = nk; s_tok[team] = tk; }
  __syncthreads();
  const BlockOffset bo = ws.off[blockIdx.x];
  int roll_base = bo.roll;
  long long tok_base = bo.tok;
  for (int t = 0; t < team; ++t) { roll_base += s_roll[t]; tok_base += s_tok[t]; }
  if (p >= a.P) return;

  int lo = a.go[p], hi = a.go[p + 1];
  lo = min(max(lo, 0), a.R);
  hi = min(max(hi, lo), a.R);
  const float seq_scale = nk > 0 ? g.inv_prompt_den / (float)nk : 0.f;
  for (int base = lo; base < hi; base += L) {
    const int i = base + lane;
    int flag = 0;
    long long len = 0;
    if (i < hi) {
      flag = a.keep[i] ? 1 : 0;
      len = a.cs[i + 1] - a.cs[i];
      if (len < 0) len = 0;
    }
    // inclusive scan across the team
    int fsum = flag;
    long long tsum = flag ? len : 0;
#pragma unroll
    for (int o = 1; o < L; o <<= 1) {
      const int f2 = __shfl_up_sync(mask, fsum, o, L);
      const long long t2 = __shfl_up_sync(mask, tsum, o, L);
      if (lane >= o) { fsum += f2; tsum += t2; }
    }
    if (i < hi) {
      if (flag) {
        const int pos = roll_base + fsum - 1;
        a.kept_ids[pos] = i;
        a.kept_tok_off[pos] = tok_base + tsum - len;
        a.w[i] = a.cfg.agg == AERO_TOKEN_MEAN ? g.inv_tok_den
                                              : (len > 0 ? seq_scale / (float)len : 0.f);
      } else {
        a.w[i] = 0.f;
      }
      if ((long long)i >= g.R_kept) a.kept_ids[i] = -1;
      if ((long long)i + 1 >= g.R_kept) a.kept_tok_off[i + 1] = g.T_kept;
      if (i == 0 && g.R_kept == 0) a.kept_tok_off[0] = 0;
    }
    roll_base += __shfl_sync(mask, fsum, L - 1, L);
    tok_base += __shfl_sync(mask, tsum, L - 1, L);
  }
}

template <int L>
int launch_all(aero_ctx* ctx, const Args& a, void* wsp) {
  constexpr int PPB = kThreads / L;
  const int nb = (a.P + PPB - 1) / PPB;
  Workspace ws = carve(wsp, a.P, nb);
  group_kernel<L><<<nb, kThreads, 0, ctx->stream>>>(a, ws);
  scan_kernel<<<1, 1024, 0, ctx->stream>>>(a, ws, nb);
  compact_kernel<L><<<nb, kThreads, 0, ctx->stream>>>(a, ws);
  ctx->launches += 3;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

}  // namespace

size_t aero_group_ws_bytes_impl(int32_t P, int32_t R) {
  if (P < 0) P = 0;
  const int nb = (P + 7) / 8 + 1;    // the smallest team (8 lanes) gives the most blocks
  return up256(sizeof(int) * (size_t)P) + up256(sizeof(long long) * (size_t)P) +
         up256(sizeof(BlockPartial) * (size_t)nb) + up256(sizeof(BlockOffset) * (size_t)nb) +
         up256(sizeof(Globals));
}

int aero_group_stats_launch(aero_ctx* ctx, const aero_cfg* cfg, int32_t P, int32_t R,
                            const int32_t* go, const float* reward, const int64_t* cs,
                            const uint32_t* key, const uint8_t* keep_in,
                            const float* alpha_in, const float* beta_in,
                            float* adv, float* w, uint8_t* keep, uint8_t* gmask, uint8_t* cat,
                            float* u_tilde, float* alpha_out, float* beta_out,
                            int32_t* kept_ids, int64_t* kept_tok_off, int64_t* counters,
                            float* metrics, void* ws) {
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
  switch (team_lanes(P, R)) {
    case 8: return launch_all<8>(ctx, a, ws);
    case 16: return launch_all<16>(ctx, a, ws);
    default: return launch_all<32>(ctx, a, ws);
  }
}

// ---- variant with library-owned scratch ------------------------------------------------
// The three kernels above need a few bytes of scratch per prompt.  This entry point takes
// them from a fixed array in device memory that is part of the loaded library image, so the
// caller passes inputs and outputs only and nothing is allocated, by this call or before it.
namespace {

constexpr int32_t kStaticMaxP = AERO_STATIC_MAX_PROMPTS;
constexpr size_t cup256(size_t x) { return (x + 255) / 256 * 256; }
constexpr size_t kStaticNb = (size_t)(kStaticMaxP + 7) / 8 + 1;
constexpr size_t kStaticBytes = cup256(sizeof(int) * (size_t)kStaticMaxP) + cup256(sizeof(long long) * (size_t)kStaticMaxP) +
                                cup256(sizeof(BlockPartial) * kStaticNb) + cup256(sizeof(BlockOffset) * kStaticNb) +
                                cup256(sizeof(Globals));

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
  // every scratch word the kernels read is written earlier in the same call, so nothing
  // has to be cleared between calls
  return aero_group_stats_launch(ctx, cfg, P, R, go, reward, cs, key, keep_in, alpha_in, beta_in,
                                 adv, w, keep, gmask, cat, u_tilde, alpha_out, beta_out,
                                 kept_ids, kept_tok_off, counters, metrics, scratch);
}
