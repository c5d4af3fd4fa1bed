"""Pins for the oracle's log-prob / clipped-surrogate stage: brute force with
scalar loops, library softmax / autograd, finite differences and the closed
forms the paper states.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import aero_oracle as O


def _batch(seed=0, P=3, n=4, d=8, V=13, noise=0.3):
    rng = np.random.default_rng(seed)
    go = np.arange(P + 1, dtype=np.int32) * n
    R = P * n
    lens = rng.integers(1, 6, R)
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    T = int(cs[-1])
    reward = rng.integers(0, 2, R).astype(np.float32)
    reward[0:n] = [1, 0, 0, 1][:n] + [0] * max(0, n - 4)
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d)) * 0.7
    y = rng.integers(0, V, T).astype(np.int32)
    return go, cs, reward, H, W, y, rng


def _with_old(cfg, go, cs, reward, H, W, y, rng, noise):
    gs = O.group_stats(cfg, go, reward, cs)
    z = O.logits(H, W)
    logp, _ = O.log_softmax_pick(z, y)
    old = logp + noise * rng.standard_normal(len(logp))
    return gs, old


def test_logits_and_logp_brute_force_scalar_loops():
    go, cs, reward, H, W, y, rng = _batch(1)
    T, d = H.shape
    V = W.shape[0]
    z = O.logits(H, W)
    logp, lse = O.log_softmax_pick(z, y)
    for t in range(T):
        zt = [sum(H[t, k] * W[v, k] for k in range(d)) for v in range(V)]
        for v in range(V):
            assert z[t, v] == pytest.approx(zt[v], rel=1e-12, abs=1e-12)
        tot = sum(math.exp(a) for a in zt)            # no max subtraction: plain definition
        assert lse[t] == pytest.approx(math.log(tot), rel=1e-12)
        assert logp[t] == pytest.approx(math.log(math.exp(zt[y[t]]) / tot), rel=1e-11)
        assert logp[t] <= 0.0


def test_logp_equals_negative_library_cross_entropy():
    go, cs, reward, H, W, y, rng = _batch(2, d=16, V=50)
    z = O.logits(H, W)
    logp, lse = O.log_softmax_pick(z, y)
    zt = torch.tensor(H) @ torch.tensor(W).T
    ce = torch.nn.functional.cross_entropy(zt, torch.tensor(y).long(), reduction="none")
    assert np.allclose(logp, -ce.numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(lse, torch.logsumexp(zt, dim=1).numpy(), rtol=1e-12)


def test_logsumexp_is_shift_safe():
    # huge logits must not overflow (max-subtracted form)
    z = np.array([[1000.0, 999.0, 0.0], [-1000.0, -1001.0, -5000.0]])
    logp, lse = O.log_softmax_pick(z, np.array([0, 1]))
    assert lse[0] == pytest.approx(1000.0 + math.log(1 + math.exp(-1)))
    assert logp[1] == pytest.approx(-1.0 - math.log(1 + math.exp(-1)))


@pytest.mark.parametrize("agg", [O.AGG_TOKEN_MEAN, O.AGG_SEQ_MEAN])
def test_old_equals_new_gives_ratio_one_and_unclipped_surrogate(agg):
    # rho = 1 -> s = A, loss = -sum_i w_i len_i A_i, g = -w_i A_i
    cfg = O.Cfg(agg=agg)
    go, cs, reward, H, W, y, rng = _batch(3)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.0)
    f = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
    owner = O.token_rollout(cs, H.shape[0])
    kept = gs["keep"][owner] != 0
    assert np.allclose(f["rho"][kept], 1.0)
    lens = cs[1:] - cs[:-1]
    assert f["loss"] == pytest.approx(-float((gs["w"] * lens * gs["adv"]).sum()), rel=1e-12, abs=1e-15)
    assert np.allclose(f["g"], -(gs["w"] * gs["adv"])[owner] * kept, rtol=1e-12)
    assert f["metrics"][0] == 0.0 and f["metrics"][1] == pytest.approx(1.0)
    if agg == O.AGG_SEQ_MEAN:
        # within each surviving group advantages sum to zero, so Eq. 2 at rho = 1 vanishes
        assert abs(f["loss"]) < 1e-12


def test_clip_cases_by_hand():
    # Eq. 2 with eps = 0.2: boundary, inside and outside, both advantage signs (Appendix A case analysis).
    cfg = O.Cfg(clip_lo=0.2, clip_hi=0.2)
    rho = np.array([1.2, 1.2 + 1e-9, 1.1, 0.8, 0.8 - 1e-9, 0.5, 1.5, 1.0])
    logp = np.log(rho)
    old = np.zeros_like(rho)
    for A in (2.0, -2.0, 0.0):
        s, g, r, ind = O.surrogate(cfg, logp, old, np.full_like(rho, A), np.full_like(rho, 0.5))
        if A > 0:
            want_s = A * np.minimum(rho, 1.2)
            want_I = (rho <= 1.2)
        elif A < 0:
            want_s = A * np.maximum(rho, 0.8)
            want_I = (rho >= 0.8)
        else:
            want_s = np.zeros_like(rho)
            want_I = np.ones_like(rho, bool)
        assert np.allclose(s, want_s, rtol=1e-13, atol=1e-15)
        assert np.allclose(g, -0.5 * A * rho * want_I, rtol=1e-13, atol=0)
        if A != 0:
            assert np.array_equal(ind.astype(bool), want_I)


def _torch_loss(cfg, H, W, y, old, owner, adv, w, kept):
    """Independent statement of Eq. 2 with library log_softmax; autograd differentiates it."""
    z = H @ W.T
    lp = torch.log_softmax(z, dim=1).gather(1, y[:, None])[:, 0]
    rho = torch.exp(lp - old)
    A = adv[owner]
    s = torch.minimum(rho * A, torch.clamp(rho, 1 - cfg.clip_lo, 1 + cfg.clip_hi) * A)
    return -(w[owner] * s * kept).sum()


@pytest.mark.parametrize("seed,noise,aero", [(4, 0.05, False), (5, 0.4, False), (6, 0.4, True)])
def test_backward_equals_autograd_of_library_statement(seed, noise, aero):
    cfg = O.Cfg(rejection=1, uniform_policy=O.UNIFORM_BAYES) if aero else O.Cfg()
    go, cs, reward, H, W, y, rng = _batch(seed, P=4, n=5, d=6, V=11)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, noise)
    f = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
    dH, dW = O.grpo_loss_bwd(H, W, y, cs, gs["keep"], f["lse"], f["g"], 1.0)
    owner = O.token_rollout(cs, H.shape[0])
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    loss = _torch_loss(cfg, Ht, Wt, torch.tensor(y).long(), torch.tensor(old), torch.tensor(owner),
                       torch.tensor(gs["adv"]), torch.tensor(gs["w"]),
                       torch.tensor((gs["keep"][owner] != 0).astype(np.float64)))
    loss.backward()
    assert f["loss"] == pytest.approx(loss.item(), rel=1e-12, abs=1e-14)
    assert np.allclose(dH, Ht.grad.numpy(), rtol=1e-10, atol=1e-14)
    assert np.allclose(dW, Wt.grad.numpy(), rtol=1e-10, atol=1e-14)
    if noise > 0.3:
        assert 0.0 < f["metrics"][0] < 1.0          # the case really exercises clipping
    # grad_scale is linear; dw_rows selects rows of the same matrix
    dH2, dW2 = O.grpo_loss_bwd(H, W, y, cs, gs["keep"], f["lse"], f["g"], 2.5, dw_rows=[3, 0, 7])
    assert np.allclose(dH2, 2.5 * dH) and np.allclose(dW2, 2.5 * dW[[3, 0, 7]])


def test_backward_finite_differences_of_own_loss():
    cfg = O.Cfg()
    go, cs, reward, H, W, y, rng = _batch(8, P=3, n=4, d=5, V=9)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.02)   # far from the clip kinks

    def loss_of(Hx, Wx):
        return O.grpo_loss_fwd(cfg, Hx, Wx, y, old, cs, gs["adv"], gs["w"], gs["keep"])["loss"]

    f = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
    dH, dW = O.grpo_loss_bwd(H, W, y, cs, gs["keep"], f["lse"], f["g"])
    h = 1e-6
    for (t, k) in [(0, 0), (3, 2), (H.shape[0] - 1, 4)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[t, k] += h
        Hm[t, k] -= h
        assert dH[t, k] == pytest.approx((loss_of(Hp, W) - loss_of(Hm, W)) / (2 * h), rel=1e-5, abs=1e-9)
    for (v, k) in [(0, 0), (4, 3), (8, 1)]:
        Wp, Wm = W.copy(), W.copy()
        Wp[v, k] += h
        Wm[v, k] -= h
        assert dW[v, k] == pytest.approx((loss_of(H, Wp) - loss_of(H, Wm)) / (2 * h), rel=1e-5, abs=1e-9)


def test_gradient_invariants():
    cfg = O.Cfg()
    go, cs, reward, H, W, y, rng = _batch(9, P=4, n=4, d=7, V=10)
    reward[4:8] = 0.0                                   # an all-incorrect group
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.5)
    f = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
    dH, dW = O.grpo_loss_bwd(H, W, y, cs, gs["keep"], f["lse"], f["g"])
    # sum_v dz_tv = 0  =>  column sums of dW vanish
    assert np.allclose(dW.sum(axis=0), 0.0, atol=1e-12)
    owner = O.token_rollout(cs, H.shape[0])
    # uniform group: zero advantage, zero gradient (Sec. 3.2, Theorem 4.1)
    dead = (owner >= 4) & (owner < 8)
    assert not dH[dead].any() and not f["g"][dead].any() and not f["logp"][dead].any()
    # clipped tokens contribute nothing (Appendix A, final display)
    clipped = (f["ind"] == 0) & (gs["keep"][owner] != 0)
    assert clipped.any() and not dH[clipped].any()
    # dH_t = g_t (W[y_t] - softmax_t @ W)
    z = O.logits(H, W)
    p = np.exp(z - f["lse"][:, None])
    live = gs["keep"][owner] != 0
    ref = f["g"][:, None] * (W[y] - p @ W)
    assert np.allclose(dH[live], ref[live], rtol=1e-10, atol=1e-14)


def test_loss_matches_scalar_loop_statement_of_eq2():
    # Eq. 2 written as nested loops over prompts, rollouts and tokens (sequence-mean mode).
    cfg = O.Cfg(agg=O.AGG_SEQ_MEAN, eps_std=0.0)
    go, cs, reward, H, W, y, rng = _batch(10, P=3, n=4, d=5, V=7)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.3)
    f = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
    surviving = [p for p in range(3) if 0 < reward[go[p]:go[p + 1]].sum() < 4]
    J = 0.0
    for p in surviving:
        r = reward[go[p]:go[p + 1]].astype(np.float64)
        A = (r - r.mean()) / r.std()
        for j, i in enumerate(range(go[p], go[p + 1])):
            acc = 0.0
            for t in range(cs[i], cs[i + 1]):
                zt = W @ H[t]
                lp = zt[y[t]] - math.log(np.exp(zt).sum())
                rho = math.exp(lp - old[t])
                acc += min(rho * A[j], min(max(rho, 0.8), 1.2) * A[j])
            J += acc / (cs[i + 1] - cs[i]) / 4
    J /= len(surviving)
    assert f["loss"] == pytest.approx(-J, rel=1e-12)


# ---------------------------------------------------------------- regularisers (KL, entropy)
def test_entropy_closed_forms_and_library_routine():
    import scipy.stats
    V = 17
    assert np.allclose(O.entropy_rows(np.zeros((3, V))), math.log(V))           # uniform: log V
    z = np.full((1, V), -800.0)
    z[0, 5] = 0.0
    assert O.entropy_rows(z)[0] == pytest.approx(0.0, abs=1e-300)               # one-hot: 0
    rng = np.random.default_rng(3)
    z = rng.standard_normal((6, V)) * 3
    p = np.exp(z - z.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    assert np.allclose(O.entropy_rows(z), scipy.stats.entropy(p, axis=1), rtol=1e-12)
    assert np.allclose(O.entropy_rows(z + 1000.0), O.entropy_rows(z), rtol=1e-9)  # shift invariance


def test_kl_estimator_properties():
    rng = np.random.default_rng(4)
    logp = -np.abs(rng.standard_normal(50)) - 0.1
    D, dD = O.kl_to_reference(logp, logp)
    assert not D.any() and not dD.any()                                        # same policy: zero, flat
    ref = logp + rng.standard_normal(50)
    D, dD = O.kl_to_reference(logp, ref)
    assert (D > 0).all()
    h = 1e-6
    Dp, _ = O.kl_to_reference(logp + h, ref)
    Dm, _ = O.kl_to_reference(logp - h, ref)
    assert np.allclose((Dp - Dm) / (2 * h), dD, rtol=1e-6, atol=1e-8)
    # in expectation under pi_theta the estimator is the KL divergence: exact sum over a small vocabulary
    z, zr = rng.standard_normal(9), rng.standard_normal(9)
    lp, lr = z - np.log(np.exp(z).sum()), zr - np.log(np.exp(zr).sum())
    D_all, _ = O.kl_to_reference(lp, lr)
    assert np.sum(np.exp(lp) * D_all) == pytest.approx(np.sum(np.exp(lp) * (lp - lr)), rel=1e-12)


@pytest.mark.parametrize("kl_beta,ent_coef", [(0.0, 0.0), (0.04, 0.0), (0.0, 1e-3), (0.3, 0.2)])
def test_regularised_backward_equals_autograd_of_library_statement(kl_beta, ent_coef):
    go, cs, reward, H, W, y, rng = _batch(7, d=12, V=23)
    cfg = O.Cfg(eps_std=0.0, kl_beta=kl_beta, ent_coef=ent_coef)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.3)
    ref_lp = old + 0.2 * rng.standard_normal(len(old))
    f = O.grpo_loss_reg_fwd(cfg, H, W, y, old, ref_lp, cs, gs["adv"], gs["w"], gs["keep"])
    dH, dW = O.grpo_loss_reg_bwd(cfg, H, W, y, cs, gs["keep"], f["lse"], f["g"], f["entropy"], gs["w"])
    if kl_beta == 0.0 and ent_coef == 0.0:            # reduces to the unregularised functions
        f0 = O.grpo_loss_fwd(cfg, H, W, y, old, cs, gs["adv"], gs["w"], gs["keep"])
        dH0, dW0 = O.grpo_loss_bwd(H, W, y, cs, gs["keep"], f0["lse"], f0["g"])
        assert f["loss"] == f0["loss"]
        assert np.allclose(dH, dH0, rtol=1e-12, atol=1e-15) and np.allclose(dW, dW0, rtol=1e-12, atol=1e-15)
    # independent statement in torch: log_softmax, Categorical entropy, autograd
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    owner = torch.tensor(O.token_rollout(cs, H.shape[0]))
    keep_t = torch.tensor(gs["keep"].astype(bool))[owner]
    A = torch.tensor(gs["adv"])[owner]
    w = torch.tensor(gs["w"])[owner]
    lsm = torch.log_softmax(Ht @ Wt.T, dim=1)
    lp = lsm[torch.arange(H.shape[0]), torch.tensor(y).long()]
    rho = torch.exp(lp - torch.tensor(old))
    surr = torch.minimum(rho * A, torch.clamp(rho, 0.8, 1.2) * A)
    q = torch.tensor(ref_lp) - lp
    ent = torch.distributions.Categorical(logits=lsm).entropy()
    per_tok = -surr + kl_beta * (torch.exp(q) - q - 1) - ent_coef * ent
    loss = (w * per_tok)[keep_t].sum()
    loss.backward()
    assert f["loss"] == pytest.approx(loss.item(), rel=1e-11, abs=1e-14)
    assert np.allclose(dH, Ht.grad.numpy(), rtol=1e-9, atol=1e-13)
    assert np.allclose(dW, Wt.grad.numpy(), rtol=1e-9, atol=1e-13)


def test_regularised_gradient_invariants():
    go, cs, reward, H, W, y, rng = _batch(8, d=10, V=19)
    cfg = O.Cfg(eps_std=0.0, kl_beta=0.1, ent_coef=0.05)
    gs, old = _with_old(cfg, go, cs, reward, H, W, y, rng, 0.2)
    f = O.grpo_loss_reg_fwd(cfg, H, W, y, old, old, cs, gs["adv"], gs["w"], gs["keep"])
    _, dW = O.grpo_loss_reg_bwd(cfg, H, W, y, cs, gs["keep"], f["lse"], f["g"], f["entropy"], gs["w"])
    # each row of dz still sums to zero (sum_v p (log p + H) = 0), so the columns of dW do too
    assert np.abs(dW.sum(axis=0)).max() < 1e-12
    assert (f["entropy"] >= 0).all() and (f["kl"] >= 0).all()
