"""Helpers shared by the GPU parity tests: build a seeded batch, run the oracle and the
CUDA library on the same inputs, compare."""
import numpy as np
import torch

from oracle import aero_oracle as O
from paper_2602_14338_b200 import binding as B
from paper_2602_14338_b200 import synth


def oracle_cfg(**kw):
    return O.Cfg(**kw)


def lib_cfg(ocfg, dtype):
    return B.cfg_default(uniform_policy=ocfg.uniform_policy, rejection=ocfg.rejection, k_ratio=ocfg.k_ratio, reject_high=ocfg.reject_high,
                         rescue_S=ocfg.rescue_S, n_explore=ocfg.n_explore, n_keep_uniform=ocfg.n_keep_uniform,
                         stats_over=ocfg.stats_over, agg=ocfg.agg, denom=ocfg.denom, alpha0=ocfg.alpha0,
                         beta0=ocfg.beta0, eps_std=ocfg.eps_std, clip_lo=ocfg.clip_lo, clip_hi=ocfg.clip_hi,
                         seed=ocfg.seed, dtype=B.AERO_BF16 if dtype == "bf16" else B.AERO_FP32,
                         kl_beta=ocfg.kl_beta, ent_coef=ocfg.ent_coef)


def cfg_for(wl, **over):
    kw = dict(seed=wl.seed)
    if wl.aero:
        kw.update(uniform_policy=O.UNIFORM_BAYES, rejection=1, k_ratio=1)
    kw.update(over)
    return O.Cfg(**kw)


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def group_inputs_device(st):
    d = dict(go=dev(st.go), reward=dev(st.reward), cs=dev(st.cs), key=dev(st.key.view(np.int32)))
    d["alpha"] = dev(st.alpha) if st.alpha is not None else None
    d["beta"] = dev(st.beta) if st.beta is not None else None
    return d


def run_group_gpu(ctx, cfg, st, use_key=True, keep_in=None):
    gi = group_inputs_device(st)
    out = ctx.group_stats(cfg, gi["go"], gi["reward"], gi["cs"], key=gi["key"] if use_key else None,
                          keep_in=keep_in, alpha_in=gi["alpha"], beta_in=gi["beta"])
    return gi, out


def check_group(out, ref, R, P):
    """Integer outputs bit-exact, floats to fp32 rounding."""
    g = {k: v.cpu().numpy() for k, v in out.items()}
    assert np.array_equal(g["keep"][:R], ref["keep"])
    assert np.array_equal(g["gmask"][:P], ref["gmask"])
    assert np.array_equal(g["cat"][:P], ref["cat"])
    assert np.array_equal(g["counters"], ref["counters"])
    nk = int(ref["counters"][0])
    assert np.array_equal(g["kept_ids"][:nk], ref["kept_ids"])
    assert (g["kept_ids"][nk:R] == -1).all()
    assert np.array_equal(g["kept_tok_off"][:R + 1], ref["kept_tok_off"])
    np.testing.assert_allclose(g["adv"][:R], ref["adv"], rtol=2e-5, atol=1e-6)
    np.testing.assert_allclose(g["w"][:R], ref["w"], rtol=2e-6, atol=0)
    np.testing.assert_allclose(g["u_tilde"][:P], ref["u_tilde"], rtol=1e-6)
    np.testing.assert_allclose(g["alpha_out"][:P], ref["alpha_out"], rtol=1e-6)
    np.testing.assert_allclose(g["beta_out"][:P], ref["beta_out"], rtol=1e-6)
    np.testing.assert_allclose(g["metrics"], ref["metrics"], rtol=1e-5, atol=1e-7)


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a)


class Batch:
    """A full stage-(b) problem on host (fp64 views of the exact low-precision inputs) and device."""

    def __init__(self, wl, ocfg, peak=0.0, st=None, keep_rollouts=None):
        self.wl, self.ocfg = wl, ocfg
        st = st or synth.make_structure(wl)
        if keep_rollouts is not None:       # first whole rollouts only (subsample of a large workload)
            R = keep_rollouts
            P = int(np.searchsorted(st.go, R, side="left"))
            assert st.go[P] == R, "subsample must end on a group boundary"
            T = int(st.cs[R])
            st = synth.Structure(st.go[:P + 1], st.cs[:R + 1], st.reward[:R], st.key[:R],
                                 None if st.alpha is None else st.alpha[:P],
                                 None if st.beta is None else st.beta[:P], st.y[:T], st.noise[:T])
        self.st = st
        self.P, self.R, self.T = len(st.go) - 1, len(st.reward), int(st.cs[-1])
        H, W = synth.make_tensors(wl, self.T, device="cpu")
        if np.ndim(peak) > 0 or peak > 0:          # a number, or one strength per token row
            H = synth.peak_hidden(H, W, st.y, peak)
        self.H_t, self.W_t = H, W
        self.H = H.double().numpy()
        self.W = W.double().numpy()
        self.ref_g = O.group_stats(ocfg, st.go, st.reward, st.cs, key=st.key, alpha_in=st.alpha, beta_in=st.beta)
        z = O.logits(self.H, self.W)
        lp, _ = O.log_softmax_pick(z, st.y)
        del z
        self.old = (lp + st.noise.astype(np.float64)).astype(np.float32)

    def oracle_fwd(self):
        rg = self.ref_g
        # the library receives fp32 advantages and weights: give the oracle the same rounded values
        adv32 = rg["adv"].astype(np.float32).astype(np.float64)
        w32 = rg["w"].astype(np.float32).astype(np.float64)
        return O.grpo_loss_fwd(self.ocfg, self.H, self.W, self.st.y, self.old, self.st.cs, adv32, w32, rg["keep"])

    def oracle_bwd(self, f, grad_scale=1.0, dw_rows=None):
        return O.grpo_loss_bwd(self.H, self.W, self.st.y, self.st.cs, self.ref_g["keep"], f["lse"], f["g"],
                               grad_scale, dw_rows=dw_rows)

    def to_device(self):
        st, rg = self.st, self.ref_g
        return dict(H=self.H_t.cuda(), W=self.W_t.cuda(), y=dev(st.y), old=dev(self.old), cs=dev(st.cs),
                    adv=dev(rg["adv"], torch.float32), w=dev(rg["w"], torch.float32), keep=dev(rg["keep"]))
