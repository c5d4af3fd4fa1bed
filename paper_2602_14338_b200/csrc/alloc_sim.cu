// Rollout allocation controller of one training step, simulated on prompts with hidden
// success rates (Algorithm 1; Sec. 4.2 Strategy 1 "iterative rescue"; Appendix C "AERO":
// increment 2, at most 10 iterations, n_p <= 32, sum n_p <= 16 |P|).
//
//   explore_kernel  n_explore draws per prompt, rescue-set membership, first requests
//   budget_kernel   one block: budget left, exclusive scan of the per-block request totals
//   step_kernel     one rescue iteration: requests are granted in prompt order while their running
//                   sum fits the budget; granted prompts draw, and leave the set on a success
//   finish_kernel   curated training size per prompt (the group stage's rule), counters
//
// A draw is the high word of SplitMix64 on (seed, prompt * n_max + rollout); a rollout is
// correct iff its draw is below the prompt's threshold, so every decision is an integer compare.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;

struct SimState {
  int32_t* n;            // [P] rollouts generated so far
  int32_t* c;            // [P] correct ones
  uint8_t* flags;        // [P] bit 0: in the rescue set, bit 1: left it by a success
  int32_t* incl;         // [P] inclusive sum of the current requests inside the prompt's block
  long long* block_tot;  // [nb] requests per block
  long long* block_off;  // [nb] requests of all earlier blocks
  long long* scal;       // [0] budget left, [1] largest granted running sum of the last iteration,
                         // [2] iterations that granted something
};

__host__ __device__ inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

SimState carve(void* ws, int32_t P, int nb) {
  char* p = static_cast<char*>(ws);
  SimState s;
  s.scal = reinterpret_cast<long long*>(p);       p += 256;
  s.n = reinterpret_cast<int32_t*>(p);            p += up256(sizeof(int32_t) * (size_t)P);
  s.c = reinterpret_cast<int32_t*>(p);            p += up256(sizeof(int32_t) * (size_t)P);
  s.incl = reinterpret_cast<int32_t*>(p);         p += up256(sizeof(int32_t) * (size_t)P);
  s.flags = reinterpret_cast<uint8_t*>(p);        p += up256((size_t)P);
  s.block_tot = reinterpret_cast<long long*>(p);  p += up256(sizeof(long long) * (size_t)nb);
  s.block_off = reinterpret_cast<long long*>(p);
  return s;
}

// SplitMix64 (Steele, Lea, Flood 2014) as a counter-based generator; the draw is the high word.
__device__ __forceinline__ uint32_t draw(uint64_t seed, uint64_t i) {
  uint64_t z = seed + (i + 1ull) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z = z ^ (z >> 31);
  return (uint32_t)(z >> 32);
}

__device__ __forceinline__ int count_correct(uint64_t seed, long long p, int n_max, int j0, int j1, uint32_t thr) {
  int c = 0;
  for (int j = j0; j < j1; ++j) c += draw(seed, (uint64_t)p * (uint64_t)n_max + (uint64_t)j) < thr ? 1 : 0;
  return c;
}

struct SimArgs {
  aero_cfg cfg;
  aero_alloc_cfg ac;
  int32_t P;
  const uint32_t* thr;
  int32_t* n_gen;
  int32_t* c_out;
  int32_t* n_train;
  int64_t* counters;
};

// Request of a prompt in the rescue set; a prompt that can ask for nothing leaves the set.
__device__ __forceinline__ int request_of(const SimArgs& a, int n, uint8_t& flags) {
  if (!(flags & 1)) return 0;
  const int req = min(a.ac.n_extra, a.ac.n_max - n);
  if (req <= 0) { flags &= (uint8_t)~1u; return 0; }
  return req;
}

// Inclusive sum of `req` over the block in thread order; the block total goes to block_tot.
__device__ __forceinline__ void scan_requests(int req, int p, int P, SimState s) {
  __shared__ int s_warp[kThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int v = req;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += u;
  }
  if (lane == 31) s_warp[warp] = v;
  __syncthreads();
  int base = 0;
  for (int k = 0; k < warp; ++k) base += s_warp[k];
  if (p < P) s.incl[p] = base + v;
  if (threadIdx.x == kThreads - 1) s.block_tot[blockIdx.x] = base + v;
  __syncthreads();
}

__global__ void __launch_bounds__(kThreads) explore_kernel(SimArgs a, SimState s) {
  const int p = blockIdx.x * kThreads + threadIdx.x;
  int req = 0;
  if (p < a.P) {
    const int n = a.cfg.n_explore;
    const int c = count_correct(a.cfg.seed, p, a.ac.n_max, 0, n, a.thr[p]);
    uint8_t flags = c <= a.cfg.rescue_S ? 1 : 0;
    flags |= c == 0 ? 4 : 0;                  // bit 2: zero accuracy after exploration
    req = request_of(a, n, flags);
    s.n[p] = n; s.c[p] = c; s.flags[p] = flags;
  }
  scan_requests(req, p, a.P, s);
}

__global__ void __launch_bounds__(1024) budget_kernel(SimState s, int nb, long long initial_budget, int first) {
  __shared__ long long s_warp[32];
  __shared__ long long s_carry;
  if (threadIdx.x == 0) {
    if (first) { s.scal[0] = initial_budget; s.scal[2] = 0; }
    else {
      s.scal[0] -= s.scal[1];
      if (s.scal[1] > 0) s.scal[2] += 1;
    }
    s.scal[1] = 0;
    s_carry = 0;
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b0 = 0; b0 < nb; b0 += 1024) {
    const int b = b0 + threadIdx.x;
    const long long mine = b < nb ? s.block_tot[b] : 0;
    long long v = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    if (lane == 31) s_warp[warp] = v;
    __syncthreads();
    long long base = s_carry;
    for (int k = 0; k < warp; ++k) base += s_warp[k];
    if (b < nb) s.block_off[b] = base + v - mine;
    __syncthreads();
    if (threadIdx.x == 1023) s_carry = base + v;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kThreads) step_kernel(SimArgs a, SimState s) {
  const int p = blockIdx.x * kThreads + threadIdx.x;
  int next_req = 0;
  if (p < a.P) {
    int n = s.n[p];
    uint8_t flags = s.flags[p];
    const int req = request_of(a, n, flags);       // the request whose prefix sum is in s.incl
    if (req > 0) {
      const long long running = s.block_off[blockIdx.x] + s.incl[p];
      if (running <= s.scal[0]) {
        const int new_c = count_correct(a.cfg.seed, p, a.ac.n_max, n, n + req, a.thr[p]);
        n += req;
        s.n[p] = n;
        s.c[p] += new_c;
        if (new_c > 0) flags = (uint8_t)((flags & ~1u) | 2u);      // early exit on the first success
        atomicMax(reinterpret_cast<unsigned long long*>(s.scal + 1), (unsigned long long)running);
      }
    }
    next_req = request_of(a, n, flags);
    s.flags[p] = flags;
  }
  scan_requests(next_req, p, a.P, s);
}

// Rollouts the curation rule of the group stage keeps from a group of n rollouts with c correct.
__device__ __forceinline__ int curated_size(const aero_cfg& cfg, int n, int c) {
  if (n == 0) return 0;
  if (c == 0 || c == n) {
    if (cfg.uniform_policy == AERO_UNIFORM_MASK) return 0;
    return cfg.n_keep_uniform <= 0 ? n : min(cfg.n_keep_uniform, n);
  }
  const bool low = 2 * c < n || (cfg.rescue_S > 0 && (long long)c * cfg.n_explore <= (long long)cfg.rescue_S * n);
  if (cfg.rejection && low) return c + (int)min((long long)cfg.k_ratio * c, (long long)(n - c));
  if (cfg.rejection && cfg.reject_high) return (n - c) + (int)min((long long)cfg.k_ratio * (n - c), (long long)c);
  return n;
}

__global__ void __launch_bounds__(kThreads) finish_kernel(SimArgs a, SimState s) {
  __shared__ long long s_red[kThreads / 32][5];
  const int p = blockIdx.x * kThreads + threadIdx.x;
  long long v[5] = {0, 0, 0, 0, 0};       // generated, kept for training, zero before, zero after, rescued
  if (p < a.P) {
    const int n = s.n[p], c = s.c[p];
    const uint8_t flags = s.flags[p];
    const int nt = curated_size(a.cfg, n, c);
    a.n_gen[p] = n; a.c_out[p] = c; a.n_train[p] = nt;
    v[0] = n; v[1] = nt; v[2] = (flags & 4) ? 1 : 0; v[3] = c == 0 ? 1 : 0; v[4] = (flags & 2) ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int k = 0; k < 5; ++k) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
  if ((threadIdx.x & 31) == 0)
    for (int k = 0; k < 5; ++k) s_red[threadIdx.x >> 5][k] = v[k];
  __syncthreads();
  if (threadIdx.x < 5) {
    long long t = 0;
    for (int w = 0; w < kThreads / 32; ++w) t += s_red[w][threadIdx.x];
    atomicAdd(reinterpret_cast<unsigned long long*>(a.counters + threadIdx.x), (unsigned long long)t);   // integers: order-free
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    // the last iteration's grants have not been folded into the scalars yet
    const long long granted_last = s.scal[1];
    a.counters[5] = s.scal[2] + (granted_last > 0 ? 1 : 0);
    a.counters[7] = a.P;
  }
}

// budget left = n_budget * P - rollouts generated (after all blocks have added their counts)
__global__ void budget_left_kernel(SimArgs a) { a.counters[6] = (long long)a.ac.n_budget * a.P - a.counters[0]; }

}  // namespace

extern "C" {

void aero_alloc_cfg_default(aero_alloc_cfg* ac) {
  if (!ac) return;
  ac->n_extra = 2;
  ac->k_max = 10;
  ac->n_max = 32;
  ac->n_budget = 16;
}

size_t aero_allocate_workspace_bytes(int32_t P) {
  if (P < 0) P = 0;
  const size_t nb = ((size_t)P + kThreads - 1) / kThreads + 1;
  return 256 + 3 * up256(sizeof(int32_t) * (size_t)P) + up256((size_t)P) + 2 * up256(sizeof(long long) * nb);
}

int aero_allocate_sim(aero_ctx* ctx, const aero_cfg* cfg, const aero_alloc_cfg* ac, int32_t P, const uint32_t* thr,
                      int32_t* n_gen, int32_t* c, int32_t* n_train, int64_t* counters,
                      void* workspace, size_t workspace_bytes) {
  if (!ctx || !cfg || !ac || P < 0 || !counters) return AERO_ERR_INVALID;
  if (P > 0 && (!thr || !n_gen || !c || !n_train)) return AERO_ERR_INVALID;
  if (ac->n_extra < 1 || ac->k_max < 0 || ac->n_max < 1 || ac->n_budget < 0 || cfg->n_explore < 0 ||
      cfg->n_explore > ac->n_max || cfg->k_ratio < 1)
    return AERO_ERR_INVALID;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return AERO_ERR_INVALID;
  if (workspace_bytes < aero_allocate_workspace_bytes(P)) return AERO_ERR_WORKSPACE;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AERO_ERR_CUDA;
  AERO_CUDA_TRY(cudaMemsetAsync(counters, 0, 8 * sizeof(int64_t), ctx->stream));
  if (P == 0) return AERO_OK;
  const int nb = (P + kThreads - 1) / kThreads;
  SimState s = carve(workspace, P, nb + 1);
  SimArgs a;
  a.cfg = *cfg; a.ac = *ac; a.P = P; a.thr = thr; a.n_gen = n_gen; a.c_out = c; a.n_train = n_train; a.counters = counters;
  long long budget = (long long)ac->n_budget * P - (long long)cfg->n_explore * P;
  if (budget < 0) budget = 0;
  explore_kernel<<<nb, kThreads, 0, ctx->stream>>>(a, s);
  for (int it = 0; it < ac->k_max; ++it) {
    budget_kernel<<<1, 1024, 0, ctx->stream>>>(s, nb, budget, it == 0 ? 1 : 0);
    step_kernel<<<nb, kThreads, 0, ctx->stream>>>(a, s);
  }
  if (ac->k_max == 0) budget_kernel<<<1, 1024, 0, ctx->stream>>>(s, nb, budget, 1);
  finish_kernel<<<nb, kThreads, 0, ctx->stream>>>(a, s);
  budget_left_kernel<<<1, 1, 0, ctx->stream>>>(a);
  ctx->launches += 3 + 2 * ac->k_max;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

}  // extern "C"
