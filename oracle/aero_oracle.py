"""CPU oracle for the GRPO/AERO hot path (test infrastructure, not a product path).

This module is the slow, plain, fp64 statement of what the CUDA library
computes.  It exists so that tests, the smoke check and the benchmark's CPU
baseline can compare against something written directly from the paper.  It
shares no code with the CUDA path and nothing in the library may call it.

Every function cites the passage of the paper (AERO, arXiv 2602.14338) that
defines what it computes.  Where the paper leaves a choice open, the reading
taken is stated in the docstring.

Parity unpinned (no passage of the paper fixes the value; pinned only by
brute force inside the tests):
  * the per-token estimator of Eq. 2's KL term (the paper prints D_KL[pi || pi_ref]
    and nothing more; here the non-negative estimator exp(q) - q - 1 with
    q = ref_logp - logp, the one GRPO uses);
  * which individual incorrect rollouts the rejection step keeps (the paper
    says "top-m most informative" without defining it; here: smallest key);
  * the denominator of the Bayesian advantage for uniform groups (the paper
    only says the mean is replaced by the posterior mean; here the Bernoulli
    standard deviation at the posterior mean is used).

Notation (packed ragged batch, as in the paper's "padding removal"):
  P prompts; prompt p owns rollouts go[p]..go[p+1]-1; R = go[P]
  rollout i owns token rows cs[i]..cs[i+1]-1 of the packed arrays; T = cs[R]
  r_i in {0,1} reward of rollout i; y_t target token of row t
  W [V,d] lm_head weight, logits z_t = W h_t.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

# ----------------------------------------------------------------------------
# configuration (mirrors the hyper-parameter table of the paper, Table 9)
# ----------------------------------------------------------------------------
UNIFORM_MASK = 0    # uniform-outcome groups are dropped (plain GRPO/DAPO behaviour, Sec. 3.2)
UNIFORM_BAYES = 1   # uniform-outcome groups use the posterior mean (Sec. 4.2, Strategy 2)
STATS_KEPT = 0      # mean/std over the curated subset (Theorem 4.1 uses mu = c/(c+m))
STATS_ALL = 1       # mean/std over every present rollout of the group
AGG_TOKEN_MEAN = 0  # token-level expectation (Appendix C, "GRPO Training")
AGG_SEQ_MEAN = 1    # 1/N sum_i 1/|o_i| sum_t (Eq. 2)
DENOM_SURVIVING = 0
DENOM_ALL = 1

CAT_ZERO, CAT_PARTIAL, CAT_GOOD, CAT_PERFECT, CAT_EMPTY = 0, 1, 2, 3, 4


@dataclasses.dataclass
class Cfg:
    uniform_policy: int = UNIFORM_MASK
    rejection: int = 0
    k_ratio: int = 1            # Sec. 4.2 Strategy 3, m = k*c; paper uses k=1
    reject_high: int = 0        # ablation "Effect of Discarding High-Success Rollouts": 1 = also
                                # down-sample the correct rollouts of mixed groups with u >= 0.5
    rescue_S: int = 0           # Sec. 4.2 Strategy 1; paper uses S=0
    n_explore: int = 8
    n_keep_uniform: int = 4     # "typically 4 rollouts from n" (Strategy 2); <=0 keeps all
    stats_over: int = STATS_KEPT
    agg: int = AGG_TOKEN_MEAN
    denom: int = DENOM_SURVIVING
    alpha0: float = 1.0
    beta0: float = 1.0
    eps_std: float = 1e-6
    clip_lo: float = 0.2        # Table 9: clip ratio 0.2
    clip_hi: float = 0.2
    seed: int = 0
    kl_beta: float = 0.0        # Eq. 2's beta (the paper never gives a value; Theorem 4.1 sets 0)
    ent_coef: float = 0.0       # Table 9: entropy coefficient 1e-3


# ----------------------------------------------------------------------------
# default selection key: SplitMix64 (Steele, Lea, Flood 2014) used as a
# counter-based generator on (seed, rollout index); the key is the high word.
# ----------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def default_key(seed: int, i: int) -> int:
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    z = z ^ (z >> 31)
    return z >> 32


# ----------------------------------------------------------------------------
# stage (a): segmented group stage
# ----------------------------------------------------------------------------
def group_stats(cfg: Cfg, go, reward, cs, key=None, keep_in=None,
                alpha_in=None, beta_in=None):
    """Per-prompt group statistics, curation mask, advantages and weights.

    Steps, in the paper's order:
      1. counts n_p (present rollouts) and c_p (correct ones)      [Sec. 3.2]
      2. category Zero / Partial / Good / Perfect with tau = 0.5,
         decided on integers (2c < n)                    [Appendix C, item 1]
      3. Beta-Binomial posterior alpha' = alpha + c, beta' = beta + n - c,
         u~ = alpha' / (alpha' + beta'), for every prompt, with n counted
         before any subsampling            [Sec. 4.2 Strategy 2; Appendix C]
      4. keep-mask: uniform groups are dropped (MASK) or cut to
         n_keep_uniform rollouts chosen by smallest key (BAYES); with
         rejection on, low-success mixed groups keep all c correct rollouts
         and the m = min(k*c, n-c) incorrect ones of smallest (key, index);
         every other group keeps all        [Sec. 4.2 Strategies 2 and 3];
         with reject_high also on, a mixed group that is not low-success keeps
         all n-c incorrect rollouts and the min(k*(n-c), c) correct ones of
         smallest (key, index) (the appendix ablation: 5 correct / 3 incorrect
         under 1:1 keeps 3 and 3)
      5. advantage (r - mean)/std over the kept subset with population std
         (the proof of Theorem 4.1 uses sigma^2 = mu(1-mu)); uniform groups:
         0 under MASK, (r - u~)/sqrt(u~(1-u~)) under BAYES   [Eq. 1; Sec. 3.2]
      6. weights of the token sum: 1/T_kept (token mean) or
         1/(P_den * n'_p * len_i) (Eq. 2); offsets by exclusive scan.
    """
    go = np.asarray(go, dtype=np.int64)
    cs = np.asarray(cs, dtype=np.int64)
    reward = np.asarray(reward, dtype=np.float64)
    P = len(go) - 1
    R = int(go[P])
    present = np.ones(R, dtype=bool) if keep_in is None else (np.asarray(keep_in) != 0)
    if key is None:
        key = np.array([default_key(cfg.seed, i) for i in range(R)], dtype=np.uint64)
    key = np.asarray(key, dtype=np.uint64)
    a_in = np.full(P, cfg.alpha0, dtype=np.float64) if alpha_in is None else np.asarray(alpha_in, np.float64)
    b_in = np.full(P, cfg.beta0, dtype=np.float64) if beta_in is None else np.asarray(beta_in, np.float64)

    keep = np.zeros(R, dtype=np.uint8)
    gmask = np.zeros(P, dtype=np.uint8)
    cat = np.zeros(P, dtype=np.uint8)
    adv = np.zeros(R, dtype=np.float64)
    u_tilde = np.zeros(P, dtype=np.float64)
    alpha_out = np.zeros(P, dtype=np.float64)
    beta_out = np.zeros(P, dtype=np.float64)
    n_kept_group = np.zeros(P, dtype=np.int64)
    cat_count = [0, 0, 0, 0, 0]

    for p in range(P):
        members = [i for i in range(int(go[p]), int(go[p + 1])) if present[i]]
        n = len(members)
        correct = [i for i in members if reward[i] > 0.5]
        wrong = [i for i in members if not reward[i] > 0.5]
        c = len(correct)
        # step 2
        if n == 0:
            category = CAT_EMPTY
        elif c == 0:
            category = CAT_ZERO
        elif c == n:
            category = CAT_PERFECT
        elif 2 * c < n:
            category = CAT_PARTIAL
        else:
            category = CAT_GOOD
        cat[p] = category
        cat_count[category] += 1
        # step 3
        alpha_out[p] = a_in[p] + c
        beta_out[p] = b_in[p] + (n - c)
        u_tilde[p] = alpha_out[p] / (alpha_out[p] + beta_out[p])
        if n == 0:
            continue
        uniform = (c == 0 or c == n)
        # step 4
        if uniform:
            if cfg.uniform_policy == UNIFORM_MASK:
                kept = []
            else:
                order = sorted(members, key=lambda i: (int(key[i]), i))
                q = n if cfg.n_keep_uniform <= 0 else min(cfg.n_keep_uniform, n)
                kept = order[:q]
        else:
            low = (category == CAT_PARTIAL) or (
                cfg.rescue_S > 0 and c * cfg.n_explore <= cfg.rescue_S * n)
            if cfg.rejection and low:
                m = min(cfg.k_ratio * c, n - c)
                order = sorted(wrong, key=lambda i: (int(key[i]), i))
                kept = correct + order[:m]
            elif cfg.rejection and cfg.reject_high:
                m = min(cfg.k_ratio * (n - c), c)
                order = sorted(correct, key=lambda i: (int(key[i]), i))
                kept = sorted(order[:m] + wrong)
            else:
                kept = members
        for i in kept:
            keep[i] = 1
        n_kept_group[p] = len(kept)
        gmask[p] = 1 if kept else 0
        if not kept:
            continue
        # step 5
        if uniform:
            ut = u_tilde[p]
            sd = math.sqrt(ut * (1.0 - ut))
            for i in kept:
                adv[i] = (reward[i] - ut) / (sd + cfg.eps_std)
        else:
            base = kept if cfg.stats_over == STATS_KEPT else members
            mu = sum(reward[i] for i in base) / len(base)
            var = sum((reward[i] - mu) ** 2 for i in base) / len(base)
            sd = math.sqrt(var)
            for i in kept:
                adv[i] = (reward[i] - mu) / (sd + cfg.eps_std)

    # step 6
    lens = cs[1:] - cs[:-1]
    kept_ids = np.nonzero(keep)[0].astype(np.int32)
    kept_tok_off = np.zeros(R + 1, dtype=np.int64)
    kept_tok_off[1:len(kept_ids) + 1] = np.cumsum(lens[kept_ids])
    T_kept = int(kept_tok_off[len(kept_ids)])
    kept_tok_off[len(kept_ids) + 1:] = T_kept
    T_present = int(lens[present].sum())
    P_surv = int(gmask.sum())
    w = np.zeros(R, dtype=np.float64)
    if cfg.agg == AGG_TOKEN_MEAN:
        den = T_kept if cfg.denom == DENOM_SURVIVING else T_present
        if den > 0:
            w[keep != 0] = 1.0 / den
    else:
        den = P_surv if cfg.denom == DENOM_SURVIVING else P
        for p in range(P):
            for i in range(int(go[p]), int(go[p + 1])):
                if keep[i] and den > 0:
                    w[i] = 1.0 / (den * n_kept_group[p] * lens[i])
    counters = np.array([len(kept_ids), T_kept, P_surv, cat_count[CAT_ZERO],
                         cat_count[CAT_PARTIAL], cat_count[CAT_GOOD],
                         cat_count[CAT_PERFECT], T_present], dtype=np.int64)
    n_kept = max(len(kept_ids), 1)
    metrics = np.array([
        cat_count[CAT_ZERO] / max(P, 1),            # zero-accuracy ratio x^zero (Sec. 3.2)
        float(np.abs(adv[keep != 0]).sum()) / n_kept,   # mean |advantage| over kept rollouts
        len(kept_ids) / max(int(present.sum()), 1),     # kept rollout fraction
        T_kept / max(T_present, 1),                     # kept token fraction
    ], dtype=np.float64)
    return dict(adv=adv, w=w, keep=keep, gmask=gmask, cat=cat, u_tilde=u_tilde,
                alpha_out=alpha_out, beta_out=beta_out, kept_ids=kept_ids,
                kept_tok_off=kept_tok_off, counters=counters, metrics=metrics)


# ----------------------------------------------------------------------------
# stage (b): log-prob, clipped surrogate, backward
# ----------------------------------------------------------------------------
def token_rollout(cs, T):
    """Row t -> index of the rollout that owns it (packed layout)."""
    cs = np.asarray(cs, dtype=np.int64)
    owner = np.zeros(T, dtype=np.int64)
    for i in range(len(cs) - 1):
        owner[cs[i]:cs[i + 1]] = i
    return owner


def logits(H, W):
    """z = H W^T, every entry, in fp64 (Appendix C: pi = softmax(f_theta(s)))."""
    return np.asarray(H, np.float64) @ np.asarray(W, np.float64).T


def log_softmax_pick(z, y):
    """lse_t = log sum_v exp z_tv (max subtracted) and logp_t = z_{t,y_t} - lse_t."""
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    zy = z[np.arange(z.shape[0]), np.asarray(y, np.int64)]
    return zy - lse, lse


def surrogate(cfg: Cfg, logp, old_logp, adv_t, w_t):
    """Per-token clipped surrogate of Eq. 2 and its derivative w.r.t. logp.

    rho = exp(logp - old); s = min(rho*A, clip(rho, 1-eps_lo, 1+eps_hi)*A).
    Eq. 2 is two-sided, so the indicator of the gradient is
    I = [rho*A <= clip(rho)*A]: rho <= 1+eps for A>0 (Eq. 3 / Appendix A),
    rho >= 1-eps for A<0; equality counts as unclipped.  The library returns
    loss = -J, so  loss = -sum_t w_t s_t  and  g_t = dloss/dlogp_t = -w_t A rho I.
    """
    logp = np.asarray(logp, np.float64)
    rho = np.exp(logp - np.asarray(old_logp, np.float64))
    clipped = np.clip(rho, 1.0 - cfg.clip_lo, 1.0 + cfg.clip_hi)
    a = rho * adv_t
    b = clipped * adv_t
    s = np.minimum(a, b)
    ind = (a <= b).astype(np.float64)
    g = -w_t * adv_t * rho * ind
    return s, g, rho, ind


def grpo_loss_fwd(cfg: Cfg, H, W, y, old_logp, cs, adv, w, keep):
    """Forward of stage (b) by the plain definition: all V logits per kept
    token, softmax, target log-prob, then Eq. 2.  Rows of dropped rollouts
    carry logp = lse = g = 0."""
    H = np.asarray(H, np.float64)
    T = H.shape[0]
    owner = token_rollout(cs, T)
    kept_t = np.asarray(keep)[owner] != 0
    idx = np.nonzero(kept_t)[0]
    logp = np.zeros(T)
    lse = np.zeros(T)
    g = np.zeros(T)
    s = np.zeros(T)
    rho = np.zeros(T)
    ind = np.zeros(T)
    if len(idx):
        z = logits(H[idx], W)
        lp, ls = log_softmax_pick(z, np.asarray(y)[idx])
        adv_t = np.asarray(adv, np.float64)[owner[idx]]
        w_t = np.asarray(w, np.float64)[owner[idx]]
        s_k, g_k, rho_k, ind_k = surrogate(cfg, lp, np.asarray(old_logp, np.float64)[idx], adv_t, w_t)
        logp[idx], lse[idx], g[idx], s[idx], rho[idx], ind[idx] = lp, ls, g_k, s_k, rho_k, ind_k
    w_full = np.asarray(w, np.float64)[owner]
    loss = -float(np.sum(w_full * s))
    nk = max(len(idx), 1)
    active = kept_t & (np.asarray(adv, np.float64)[owner] != 0)
    metrics = np.array([
        float(np.sum((ind == 0) & active)) / nk,                       # clip fraction
        float(rho[idx].sum()) / nk,                                    # mean ratio
        float((np.asarray(old_logp, np.float64)[idx] - logp[idx]).sum()) / nk,  # mean(old - new)
        float(len(idx)),
    ])
    return dict(logp=logp, lse=lse, g=g, loss=loss, rho=rho, ind=ind, metrics=metrics)


def grpo_loss_bwd(H, W, y, cs, keep, lse, g, grad_scale=1.0, dw_rows=None):
    """Backward of stage (b): dz_tv = g_t (1[v = y_t] - exp(z_tv - lse_t)),
    dH_t = sum_v dz_tv W_v, dW_v = sum_t dz_tv H_t  (softmax cross-entropy chain
    rule applied to Eq. 3's rho * grad log pi).  `dw_rows` restricts the dW
    output to the listed vocabulary rows (same definition, fewer outputs)."""
    H = np.asarray(H, np.float64)
    W = np.asarray(W, np.float64)
    T, d = H.shape
    V = W.shape[0]
    owner = token_rollout(cs, T)
    idx = np.nonzero(np.asarray(keep)[owner] != 0)[0]
    dH = np.zeros((T, d))
    rows = np.arange(V) if dw_rows is None else np.asarray(dw_rows, np.int64)
    dW = np.zeros((len(rows), d))
    if len(idx):
        z = logits(H[idx], W)
        dz = -np.exp(z - np.asarray(lse, np.float64)[idx][:, None])
        dz[np.arange(len(idx)), np.asarray(y, np.int64)[idx]] += 1.0
        dz *= (grad_scale * np.asarray(g, np.float64)[idx])[:, None]
        dH[idx] = dz @ W
        dW = dz[:, rows].T @ H[idx]
    return dH, dW


# ----------------------------------------------------------------------------
# stage (b) with the regularisers of Eq. 2 and Table 9: KL to a reference policy
# and an entropy bonus
# ----------------------------------------------------------------------------
def entropy_rows(z):
    """Entropy of softmax(z_t) per row, H_t = -sum_v p_tv log p_tv, from the definition."""
    m = z.max(axis=1, keepdims=True)
    e = np.exp(z - m)
    p = e / e.sum(axis=1, keepdims=True)
    logp = (z - m) - np.log(e.sum(axis=1, keepdims=True))
    return -(p * logp).sum(axis=1)


def kl_to_reference(logp, ref_logp):
    """Per-token estimate of Eq. 2's D_KL[pi_theta || pi_ref] on the sampled token:
    D = exp(q) - q - 1 with q = ref_logp - logp (non-negative, zero iff q = 0), and its
    derivative dD/dlogp = 1 - exp(q).  The paper does not print the estimator: this is a
    reading (parity unpinned)."""
    q = np.asarray(ref_logp, np.float64) - np.asarray(logp, np.float64)
    return np.exp(q) - q - 1.0, 1.0 - np.exp(q)


def grpo_loss_reg_fwd(cfg: Cfg, H, W, y, old_logp, ref_logp, cs, adv, w, keep):
    """Forward with the regularisers.  Per kept token of rollout i:
        loss_t = w_i * ( -s_t + kl_beta * D_t - ent_coef * H_t )        (loss = -J, Eq. 2)
        g_t    = dloss/dlogp_t = -w_i A_i rho_t I_t + kl_beta w_i (1 - exp(ref_t - logp_t))
    The entropy acts on every logit, not only through logp_t, so it is returned per row
    (`entropy`) for the backward.  ref_logp may be None when kl_beta == 0."""
    base = grpo_loss_fwd(cfg, H, W, y, old_logp, cs, adv, w, keep)
    H = np.asarray(H, np.float64)
    T = H.shape[0]
    owner = token_rollout(cs, T)
    kept_t = np.asarray(keep)[owner] != 0
    idx = np.nonzero(kept_t)[0]
    w_t = np.asarray(w, np.float64)[owner]
    ent = np.zeros(T)
    kl = np.zeros(T)
    g = base["g"].copy()
    if len(idx):
        ent[idx] = entropy_rows(logits(H[idx], W))
        if cfg.kl_beta != 0.0:
            D, dD = kl_to_reference(base["logp"][idx], np.asarray(ref_logp, np.float64)[idx])
            kl[idx] = D
            g[idx] += cfg.kl_beta * w_t[idx] * dD
    loss = base["loss"] + float(np.sum(w_t * (cfg.kl_beta * kl - cfg.ent_coef * ent)))
    out = dict(base)
    out.update(g=g, loss=loss, entropy=ent, kl=kl)
    return out


def grpo_loss_reg_bwd(cfg: Cfg, H, W, y, cs, keep, lse, g, entropy, w, grad_scale=1.0, dw_rows=None):
    """Backward with the entropy bonus: with p = softmax(z_t) and e_t = ent_coef * w_i,
        dz_tv = grad_scale * ( g_t (1[v = y_t] - p_tv) + e_t p_tv (log p_tv + H_t) ),
    the second term being d(-e_t H_t)/dz_tv; then dH = dz W and dW = dz^T H as before."""
    H = np.asarray(H, np.float64)
    W = np.asarray(W, np.float64)
    T, d = H.shape
    V = W.shape[0]
    owner = token_rollout(cs, T)
    idx = np.nonzero(np.asarray(keep)[owner] != 0)[0]
    dH = np.zeros((T, d))
    rows = np.arange(V) if dw_rows is None else np.asarray(dw_rows, np.int64)
    dW = np.zeros((len(rows), d))
    if len(idx):
        z = logits(H[idx], W)
        logp_all = z - np.asarray(lse, np.float64)[idx][:, None]
        p = np.exp(logp_all)
        dz = -p * np.asarray(g, np.float64)[idx][:, None]
        dz[np.arange(len(idx)), np.asarray(y, np.int64)[idx]] += np.asarray(g, np.float64)[idx]
        e_t = cfg.ent_coef * np.asarray(w, np.float64)[owner[idx]]
        dz += e_t[:, None] * p * (logp_all + np.asarray(entropy, np.float64)[idx][:, None])
        dz *= grad_scale
        dH[idx] = dz @ W
        dW = dz[:, rows].T @ H[idx]
    return dH, dW


# ----------------------------------------------------------------------------
# rollout allocation controller of one training step, simulated on prompts with
# hidden success rates (Algorithm 1; Sec. 4.2 Strategy 1; Appendix C "AERO")
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class AllocCfg:
    n_extra: int = 2       # rescue increment Delta n (Strategy 1: "n_extra, e.g., 2"; Appendix C: Delta n = 2)
    k_max: int = 10        # Appendix C: up to K_max = 10 iterations
    n_max: int = 32        # Appendix C: n_p <= n_max = 32
    n_budget: int = 16     # Appendix C: sum_p n_p <= n_budget * |P|


def curated_size(cfg: Cfg, n: int, c: int) -> int:
    """Number of rollouts the curation rule of group_stats keeps from a group with n rollouts, c correct."""
    if n == 0:
        return 0
    if c == 0 or c == n:
        if cfg.uniform_policy == UNIFORM_MASK:
            return 0
        return n if cfg.n_keep_uniform <= 0 else min(cfg.n_keep_uniform, n)
    low = (2 * c < n) or (cfg.rescue_S > 0 and c * cfg.n_explore <= cfg.rescue_S * n)
    if cfg.rejection and low:
        return c + min(cfg.k_ratio * c, n - c)
    if cfg.rejection and cfg.reject_high:
        return (n - c) + min(cfg.k_ratio * (n - c), c)
    return n


def allocate_sim(cfg: Cfg, acfg: AllocCfg, thr):
    """One step of the allocation controller over P simulated prompts.

    Rollout j (in generation order) of prompt p is correct iff the draw
    default_key(cfg.seed, p * n_max + j) < thr[p]; thr[p] = floor(u_p * 2^32) encodes the
    hidden success rate u_p.  Steps:
      1. exploration: n_explore rollouts per prompt, c_p correct        [Algorithm 1, Stage 1]
      2. rescue set: c_p <= rescue_S.  For up to k_max iterations every prompt still in the
         set asks for min(n_extra, n_max - n_p) more rollouts (asking for none leaves the
         set); requests are granted in prompt order while their running sum stays within the
         budget left of n_budget * P; a granted prompt draws its rollouts and leaves the set
         as soon as one of them is correct ("early exit upon first success")
                                                [Sec. 4.2 Strategy 1; Appendix C items 2-3]
      3. curated training size per prompt by the rule of group_stats        [Sec. 4.4]
    The paper does not say how a short budget is shared: prompt order is a reading.
    Returns n_gen, c, n_train per prompt and counters
    [rollouts generated, rollouts kept for training, zero-accuracy prompts after exploration,
     zero-accuracy prompts at the end, prompts rescued, iterations run, budget left, P]."""
    thr = np.asarray(thr, dtype=np.uint64)
    P = len(thr)
    n = np.full(P, cfg.n_explore, dtype=np.int64)
    c = np.zeros(P, dtype=np.int64)
    for p in range(P):
        for j in range(cfg.n_explore):
            c[p] += 1 if default_key(cfg.seed, p * acfg.n_max + j) < int(thr[p]) else 0
    zero_before = int((c == 0).sum())
    rescue = c <= cfg.rescue_S
    rescued = np.zeros(P, dtype=bool)          # left the rescue set by drawing a correct rollout
    remaining = max(acfg.n_budget * P - cfg.n_explore * P, 0)
    iters = 0
    for _ in range(acfg.k_max):
        running = 0
        granted_any = False
        for p in range(P):
            if not rescue[p]:
                continue
            req = min(acfg.n_extra, acfg.n_max - int(n[p]))
            if req <= 0:
                rescue[p] = False
                continue
            running += req
            if running > remaining:
                continue                      # not granted this iteration; stays in the set
            granted_any = True
            new_c = 0
            for j in range(int(n[p]), int(n[p]) + req):
                new_c += 1 if default_key(cfg.seed, p * acfg.n_max + j) < int(thr[p]) else 0
            n[p] += req
            c[p] += new_c
            if new_c > 0:
                rescue[p] = False
                rescued[p] = True
        if not granted_any:
            break
        iters += 1
        remaining = acfg.n_budget * P - int(n.sum())
    n_train = np.array([curated_size(cfg, int(n[p]), int(c[p])) for p in range(P)], dtype=np.int64)
    counters = np.array([int(n.sum()), int(n_train.sum()), zero_before, int((c == 0).sum()), int(rescued.sum()), iters,
                         acfg.n_budget * P - int(n.sum()), P], dtype=np.int64)
    return dict(n_gen=n.astype(np.int32), c=c.astype(np.int32), n_train=n_train.astype(np.int32), counters=counters)
