// Device helpers shared by the fp32 and the tensor-core versions of stage (b).
#pragma once
#include "common.cuh"

constexpr int kPartialStride = 5;   // doubles per partial: sum w*s, clipped count, sum rho, sum(old-logp), kept count

// Rollout that owns packed token row t: the last i with cs[i] <= t (cs is non-decreasing).
__device__ __forceinline__ int aero_owner(const int64_t* __restrict__ cs, int R, long long t) {
  int lo = 0, hi = R;            // invariant: cs[lo] <= t < cs[hi] for valid input
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cs[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

struct SurrogateOut {
  float s;       // min(rho A, clip(rho) A)
  float g;       // d(loss)/d(logp) = -w A rho [unclipped]
  float rho;
  float clipped; // 1 if the token is clipped and A != 0
};

// Eq. 2 for one token (two-sided clip; equality counts as unclipped).
__device__ __forceinline__ SurrogateOut aero_surrogate(float logp, float old_logp, float A, float w,
                                                       float clip_lo, float clip_hi) {
  SurrogateOut o;
  o.rho = __expf(logp - old_logp);
  const float cl = fminf(fmaxf(o.rho, 1.f - clip_lo), 1.f + clip_hi);
  const float a = o.rho * A, b = cl * A;
  o.s = fminf(a, b);
  const bool unclipped = a <= b;
  o.g = unclipped ? -w * A * o.rho : 0.f;
  o.clipped = (!unclipped && A != 0.f) ? 1.f : 0.f;
  return o;
}
