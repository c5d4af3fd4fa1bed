"""Seeded synthetic rollout batches (inputs only; none of the method's arithmetic).

The paper trains on rollouts of Qwen2.5 models over math/code prompts; those
datasets and weights are not used here.  These generators reproduce only the
shapes and distributions of such batches: ragged groups of rollouts per prompt,
lognormal response lengths, binary rewards drawn per prompt, Gaussian hidden
states and lm_head weights.  Everything is a pure function of the seed.
"""
from __future__ import annotations

import dataclasses

import numpy as np


@dataclasses.dataclass
class Workload:
    name: str
    P: int                    # prompts
    n_lo: int                 # group size range (inclusive)
    n_hi: int
    len_median: float         # lognormal median of response length (tokens)
    len_cap: int
    len_sigma: float          # lognormal sigma; 0 -> uniform in [len_lo, len_cap]
    len_lo: int
    d: int
    V: int
    dtype: str                # "bf16" | "fp32"
    beta_a: float             # per-prompt success rate ~ Beta(beta_a, beta_b)
    beta_b: float
    old_noise: float          # std of old_logp - logp
    aero: bool                # rejection + Bayesian uniform groups, Gamma(2,1) priors
    force_uniform: bool       # group 0 all-correct, group 1 all-incorrect
    seed: int


# The five benchmark workloads: a tiny fp32 case, Qwen2.5-Math-1.5B and Qwen2.5-7B
# shaped GRPO batches, an AERO-curated ragged batch and a long-response stress case.
WORKLOADS = {
    0: Workload("tiny", 4, 4, 4, 0.0, 64, 0.0, 16, 64, 512, "fp32", 1.0, 1.0, 0.05, False, True, 1000),
    1: Workload("qwen2.5-math-1.5b", 64, 8, 8, 512.0, 3072, 0.4, 1, 1536, 151936, "bf16", 0.5, 0.5, 0.05, False, False, 1001),
    2: Workload("qwen2.5-7b", 128, 8, 8, 768.0, 4096, 0.4, 1, 3584, 152064, "bf16", 0.5, 0.5, 0.05, False, False, 1002),
    3: Workload("aero-adaptive-7b", 256, 2, 16, 512.0, 4096, 0.4, 1, 3584, 152064, "bf16", 0.5, 0.5, 0.05, True, False, 1003),
    4: Workload("stress-7b", 256, 16, 16, 1024.0, 8192, 0.4, 1, 3584, 152064, "bf16", 0.3, 0.3, 0.1, False, False, 1004),
}


def scaled(wl: Workload, **over) -> Workload:
    """A copy of a workload with some fields replaced (used for reduced test sizes)."""
    return dataclasses.replace(wl, **over)


@dataclasses.dataclass
class Structure:
    go: np.ndarray        # int32 [P+1] group offsets
    cs: np.ndarray        # int64 [R+1] token offsets
    reward: np.ndarray    # float32 [R] in {0,1}
    key: np.ndarray       # uint32 [R] selection keys
    alpha: np.ndarray     # float32 [P] prior pseudo-counts (or None)
    beta: np.ndarray
    y: np.ndarray         # int32 [T] target tokens
    noise: np.ndarray     # float32 [T] perturbation added to the log-probs to make old_logp


def make_structure(wl: Workload) -> Structure:
    rng = np.random.default_rng(wl.seed)
    n = rng.integers(wl.n_lo, wl.n_hi + 1, size=wl.P)
    go = np.zeros(wl.P + 1, dtype=np.int32)
    go[1:] = np.cumsum(n)
    R = int(go[-1])
    if wl.len_sigma > 0:
        ln = np.rint(np.exp(np.log(wl.len_median) + wl.len_sigma * rng.standard_normal(R)))
        ln = np.clip(ln, wl.len_lo, wl.len_cap).astype(np.int64)
    else:
        ln = rng.integers(wl.len_lo, wl.len_cap + 1, size=R).astype(np.int64)
    cs = np.zeros(R + 1, dtype=np.int64)
    cs[1:] = np.cumsum(ln)
    T = int(cs[-1])
    p_succ = rng.beta(wl.beta_a, wl.beta_b, size=wl.P)
    reward = (rng.random(R) < np.repeat(p_succ, n)).astype(np.float32)
    if wl.force_uniform and wl.P >= 2:
        reward[go[0]:go[1]] = 1.0
        reward[go[1]:go[2]] = 0.0
    key = rng.integers(0, 2 ** 32, size=R, dtype=np.uint64).astype(np.uint32)
    if wl.aero:
        alpha = rng.gamma(2.0, 1.0, size=wl.P).astype(np.float32)
        beta = rng.gamma(2.0, 1.0, size=wl.P).astype(np.float32)
    else:
        alpha = beta = None
    y = rng.integers(0, wl.V, size=T, dtype=np.int64).astype(np.int32)
    noise = (wl.old_noise * rng.standard_normal(T)).astype(np.float32)
    return Structure(go, cs, reward, key, alpha, beta, y, noise)


def make_tensors(wl: Workload, T: int, device="cpu"):
    """H [T,d] ~ N(0,1) and W [V,d] ~ N(0,0.02) as torch tensors of the workload's dtype."""
    import torch

    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.seed)
    W = torch.empty((wl.V, wl.d), dtype=torch.float32, device=device)
    W.normal_(0.0, 0.02, generator=gen)
    W = W.to(dt)
    H = torch.empty((T, wl.d), dtype=dt, device=device)
    step = max(1, (1 << 28) // wl.d)       # bound the fp32 staging buffer
    for a in range(0, T, step):
        b = min(T, a + step)
        tmp = torch.empty((b - a, wl.d), dtype=torch.float32, device=device)
        tmp.normal_(0.0, 1.0, generator=gen)
        H[a:b] = tmp.to(dt)
    return H, W


def peak_hidden(H, W, y, strength):
    """Overwrite H so that logits are peaked at the target: H_t = strength_t * W[y_t]/|W[y_t]| + 0.25 * H_t
    (strength a number, or one value per row).  Used for parity cases in which the softmax part of the
    gradient is not negligible, and for rows whose target probability is close to 1."""
    import torch

    Wy = W[torch.as_tensor(y, device=W.device).long()].float()
    Wy = Wy / Wy.norm(dim=1, keepdim=True).clamp_min(1e-12)
    s = torch.as_tensor(strength, dtype=torch.float32, device=W.device)
    if s.ndim == 1:
        s = s[:, None]
    return (s * Wy + 0.25 * H.float()).to(H.dtype)


def success_thresholds(P: int, beta_a: float, beta_b: float, seed: int) -> np.ndarray:
    """Hidden per-prompt success rates u ~ Beta(beta_a, beta_b) as 32-bit thresholds floor(u * 2^32)
    (inputs of the allocation-controller simulation; a draw below the threshold is a correct rollout)."""
    rng = np.random.default_rng(seed)
    u = rng.beta(beta_a, beta_b, size=P)
    return np.minimum(np.floor(u * 2.0 ** 32), 2.0 ** 32 - 1).astype(np.uint32)
