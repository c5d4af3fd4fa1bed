"""GPU parity tests: the CUDA library, called through its C ABI, against the fp64 oracle
on the same seeded inputs.  Tolerances are the ones the path is specified with:
integer outputs bit-exact; per-token log-probs abs <= 1e-2; loss rel <= 1e-3; dH and dW
relative L2 <= 1e-2 (bf16 path).  The fp32 path is held to 1e-4."""
import numpy as np
import pytest
import torch

from oracle import aero_oracle as O
from paper_2602_14338_b200 import binding as B
from paper_2602_14338_b200 import synth
from tests import aero_testlib as TL

pytestmark = pytest.mark.gpu

LOGP_ABS, LOSS_REL, GRAD_L2 = 1e-2, 1e-3, 1e-2


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    assert c.last_status() == 0
    c.close()


# ------------------------------------------------------------------ stage (a)
GROUP_MODES = [
    dict(),
    dict(uniform_policy=O.UNIFORM_BAYES),
    dict(uniform_policy=O.UNIFORM_BAYES, rejection=1),
    dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, k_ratio=2, agg=O.AGG_SEQ_MEAN),
    dict(rejection=1, stats_over=O.STATS_ALL, denom=O.DENOM_ALL),
    dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, rescue_S=4, n_keep_uniform=0, agg=O.AGG_SEQ_MEAN, denom=O.DENOM_ALL),
    dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, reject_high=1),
    dict(rejection=1, reject_high=1, k_ratio=2, stats_over=O.STATS_ALL),
]


@pytest.mark.parametrize("config", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("mode", range(len(GROUP_MODES)))
def test_group_stats_matches_oracle(ctx, config, mode):
    wl = synth.WORKLOADS[config]
    st = synth.make_structure(wl)
    ocfg = O.Cfg(seed=wl.seed, **GROUP_MODES[mode])
    ref = O.group_stats(ocfg, st.go, st.reward, st.cs, key=st.key, alpha_in=st.alpha, beta_in=st.beta)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
    TL.check_group(out, ref, len(st.reward), len(st.go) - 1)
    assert ctx.last_status() == 0


def test_group_stats_default_key_and_keep_in(ctx):
    wl = synth.scaled(synth.WORKLOADS[3], P=300, n_lo=1, n_hi=40, seed=77)   # groups longer than a team
    st = synth.make_structure(wl)
    rng = np.random.default_rng(5)
    keep_in = (rng.random(len(st.reward)) < 0.8).astype(np.uint8)
    ocfg = O.Cfg(seed=991, uniform_policy=O.UNIFORM_BAYES, rejection=1)
    ref = O.group_stats(ocfg, st.go, st.reward, st.cs, keep_in=keep_in, alpha_in=st.alpha, beta_in=st.beta)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st, use_key=False, keep_in=TL.dev(keep_in))
    TL.check_group(out, ref, len(st.reward), len(st.go) - 1)


def test_group_stats_ties_and_small_groups(ctx):
    wl = synth.scaled(synth.WORKLOADS[3], P=500, n_lo=1, n_hi=6, seed=78)
    st = synth.make_structure(wl)
    st.key[:] = st.key % 3            # heavy ties: the index must break them
    ocfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, n_keep_uniform=2)
    ref = O.group_stats(ocfg, st.go, st.reward, st.cs, key=st.key, alpha_in=st.alpha, beta_in=st.beta)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
    TL.check_group(out, ref, len(st.reward), len(st.go) - 1)


@pytest.mark.parametrize("high", [0, 1])
def test_group_stats_groups_larger_than_a_tile(ctx, high):
    """Groups of thousands of rollouts do not fit the shared-memory staging of a tile and take the
    path that walks global memory; small groups around them take the staged path.  Heavy key ties."""
    rng = np.random.default_rng(91)
    sizes = np.concatenate([rng.integers(1, 9, 30), [2600], rng.integers(1, 9, 25), [3100, 2400, 2500], rng.integers(1, 9, 20)])
    P, R = len(sizes), int(sizes.sum())
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    reward = (rng.random(R) < 0.5).astype(np.float32)
    big = np.nonzero(sizes > 1000)[0]
    reward[go[big[0]]:go[big[0] + 1]] = 0.0                                               # uniform: keep 4 of 2600
    reward[go[big[1]]:go[big[1] + 1]] = (rng.random(sizes[big[1]]) < 0.1).astype(np.float32)   # low success: rejection
    reward[go[big[2]]:go[big[2] + 1]] = (rng.random(sizes[big[2]]) < 0.8).astype(np.float32)   # high success
    lens = rng.integers(1, 50, R)
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    key = rng.integers(0, 200, R).astype(np.uint32)
    st = synth.Structure(go, cs, reward, key, None, None, None, None)
    ocfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, reject_high=high, agg=O.AGG_SEQ_MEAN if high else O.AGG_TOKEN_MEAN)
    ref = O.group_stats(ocfg, go, reward, cs, key=key)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
    TL.check_group(out, ref, R, P)
    assert ctx.last_status() == 0


def test_group_stats_very_long_rollouts(ctx):
    """Rollouts of 2^22 tokens and more leave the staged path (its staging word holds 22 bits of length),
    and a chunk with one of 2^26 or more takes the 64-bit scan of the second pass; token totals pass 2^32."""
    rng = np.random.default_rng(17)
    sizes = rng.integers(1, 17, 400)
    P, R = len(sizes), int(sizes.sum())
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    reward = (rng.random(R) < 0.4).astype(np.float32)
    lens = rng.integers(1, 3000, R).astype(np.int64)
    lens[rng.integers(0, R, 25)] = rng.integers(1 << 22, 1 << 23, 25)
    lens[rng.integers(0, R, 10)] = rng.integers(1 << 26, 1 << 30, 10)
    lens[[0, R - 1]] = [(1 << 31) - 1, 1 << 22]
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    assert cs[-1] > 1 << 32
    key = rng.integers(0, 1 << 32, R, dtype=np.uint64).astype(np.uint32)
    st = synth.Structure(go, cs, reward, key, None, None, None, None)
    for over in (dict(), dict(agg=O.AGG_SEQ_MEAN, denom=O.DENOM_ALL)):
        ocfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, **over)
        ref = O.group_stats(ocfg, go, reward, cs, key=key)
        _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
        TL.check_group(out, ref, R, P)
    assert ctx.last_status() == 0


def test_group_stats_offsets_that_are_no_partition(ctx):
    """Group offsets that go backwards or past R raise AERO_ST_BAD_OFFSETS; every index the kernels use is
    clamped into the arrays (ranges into [0, R], compacted positions below R), so the call completes and
    the next one on good inputs is exact again."""
    rng = np.random.default_rng(23)
    P, R = 700, 5000
    go = np.sort(rng.integers(0, R + 1, P + 1)).astype(np.int32)
    go[0], go[-1] = 0, R
    bad = go.copy()
    bad[100] = R + 50            # past the end
    bad[300] = -7                # negative
    bad[500:520] = bad[500:520][::-1].copy()      # backwards
    bad[640] = 0                 # a share that starts over: overlaps everything before it
    reward = (rng.random(R) < 0.5).astype(np.float32)
    lens = rng.integers(1, 40, R)
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    key = rng.integers(0, 1 << 32, R, dtype=np.uint64).astype(np.uint32)
    cfg = B.cfg_default(uniform_policy=B.AERO_UNIFORM_BAYES, rejection=1)
    ctx.group_stats(cfg, TL.dev(bad), TL.dev(reward), TL.dev(cs), key=TL.dev(key.view(np.int32)))
    torch.cuda.synchronize()
    assert ctx.last_status() & B.AERO_ST_BAD_OFFSETS
    assert ctx.last_status() == 0
    st = synth.Structure(go, cs, reward, key, None, None, None, None)
    ocfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1)
    ref = O.group_stats(ocfg, go, reward, cs, key=key)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
    TL.check_group(out, ref, R, P)


def test_group_stats_empty_inputs_and_status_bits(ctx):
    cfg = B.cfg_default()
    go = torch.zeros(1, dtype=torch.int32, device="cuda")
    cs = torch.zeros(1, dtype=torch.int64, device="cuda")
    rw = torch.zeros(0, dtype=torch.float32, device="cuda")
    out = ctx.group_stats(cfg, go, rw, cs)
    assert out["counters"].cpu().tolist() == [0] * 8 and int(out["kept_tok_off"][0]) == 0
    # empty groups among real ones
    go = torch.tensor([0, 0, 3, 3], dtype=torch.int32, device="cuda")
    rw = torch.tensor([1, 0, 0], dtype=torch.float32, device="cuda")
    cs = torch.tensor([0, 2, 4, 6], dtype=torch.int64, device="cuda")
    out = ctx.group_stats(cfg, go, rw, cs)
    ref = O.group_stats(O.Cfg(), go.cpu().numpy(), rw.cpu().numpy(), cs.cpu().numpy())
    TL.check_group(out, ref, 3, 3)
    assert ctx.last_status() == 0
    # a non-binary reward and an empty rollout raise status bits and nothing traps
    rw2 = torch.tensor([1, 0.25, 0], dtype=torch.float32, device="cuda")
    cs2 = torch.tensor([0, 2, 2, 6], dtype=torch.int64, device="cuda")
    ctx.group_stats(cfg, go, rw2, cs2)
    bits = ctx.last_status()
    assert bits & B.AERO_ST_BAD_REWARD and bits & B.AERO_ST_EMPTY_ROLLOUT
    assert ctx.last_status() == 0


def test_group_stats_large_properties(ctx):
    """2^20 prompts (too many for the oracle's loops): exact invariants plus sampled prompts."""
    wl = synth.scaled(synth.WORKLOADS[3], P=1 << 20, seed=4242, len_median=64.0, len_cap=256)
    st = synth.make_structure(wl)
    ocfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1)
    _, out = TL.run_group_gpu(ctx, TL.lib_cfg(ocfg, "bf16"), st)
    g = {k: v.cpu().numpy() for k, v in out.items()}
    R, P = len(st.reward), wl.P
    lens = st.cs[1:] - st.cs[:-1]
    keep = g["keep"][:R].astype(bool)
    assert g["counters"][0] == keep.sum() and g["counters"][1] == lens[keep].sum()
    assert np.array_equal(g["kept_ids"][:keep.sum()], np.nonzero(keep)[0])
    assert np.array_equal(g["kept_tok_off"][1:keep.sum() + 1], np.cumsum(lens[keep]))
    assert abs(float((g["w"][:R].astype(np.float64) * lens).sum()) - 1.0) < 1e-4
    rng = np.random.default_rng(0)
    for p in rng.integers(0, P, 200):
        a, b = st.go[p], st.go[p + 1]
        sub_go = np.array([0, b - a], np.int32)
        sub_cs = (st.cs[a:b + 1] - st.cs[a]).astype(np.int64)
        ref = O.group_stats(ocfg, sub_go, st.reward[a:b], sub_cs, key=st.key[a:b],
                            alpha_in=st.alpha[p:p + 1], beta_in=st.beta[p:p + 1])
        assert np.array_equal(g["keep"][a:b], ref["keep"])
        np.testing.assert_allclose(g["adv"][a:b], ref["adv"], rtol=2e-5, atol=1e-6)
        assert g["cat"][p] == ref["cat"][0]


# ------------------------------------------------------------------ allocation controller (simulated)
ALLOC_CASES = [
    # P, Beta(a, b) of the hidden success rates, cfg overrides, alloc overrides
    (1000, 0.5, 0.5, dict(uniform_policy=O.UNIFORM_BAYES, rejection=1), dict()),
    (777, 0.3, 2.0, dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, k_ratio=2), dict(n_budget=10)),       # budget binds
    (513, 0.4, 1.5, dict(rejection=1, reject_high=1, rescue_S=2), dict(n_extra=3, k_max=4, n_max=17)),
    (300, 5.0, 0.2, dict(uniform_policy=O.UNIFORM_BAYES), dict(k_max=0)),
    (257, 0.05, 5.0, dict(uniform_policy=O.UNIFORM_BAYES, rejection=1, n_explore=4), dict(n_budget=5, n_extra=1)),
]


@pytest.mark.parametrize("case", range(len(ALLOC_CASES)))
def test_allocation_controller_matches_oracle(ctx, case):
    P, ba, bb, cover, aover = ALLOC_CASES[case]
    thr = synth.success_thresholds(P, ba, bb, seed=600 + case)
    ocfg = O.Cfg(seed=900 + case, **cover)
    oa = O.AllocCfg(**aover)
    ref = O.allocate_sim(ocfg, oa, thr)
    out = ctx.allocate_sim(TL.lib_cfg(ocfg, "bf16"), B.alloc_cfg_default(**aover), TL.dev(thr.view(np.int32)))
    for k in ("n_gen", "c", "n_train"):
        assert np.array_equal(out[k][:P].cpu().numpy(), ref[k]), k
    assert out["counters"].cpu().tolist() == ref["counters"].tolist()
    if case == 1:
        assert ref["counters"][6] < 2                 # the budget really ran out
    assert ctx.last_status() == 0


def test_allocation_controller_large_properties(ctx):
    """2^20 prompts: budget and cap invariants, and the geometric closed forms of the rescue process."""
    P, u = 1 << 20, 0.12
    thr = np.full(P, int(u * 2 ** 32), np.uint32)
    ocfg = O.Cfg(seed=77, uniform_policy=O.UNIFORM_BAYES, rejection=1)
    out = ctx.allocate_sim(TL.lib_cfg(ocfg, "bf16"), B.alloc_cfg_default(), TL.dev(thr.view(np.int32)))
    n, c, nt = (out[k][:P].cpu().numpy().astype(np.int64) for k in ("n_gen", "c", "n_train"))
    cnt = out["counters"].cpu().numpy()
    assert n.min() >= 8 and n.max() <= 32 and n.sum() <= 16 * P and (nt <= n).all()
    assert cnt[0] == n.sum() and cnt[1] == nt.sum() and cnt[3] == (c == 0).sum() and cnt[6] == 16 * P - n.sum()
    p0 = (1 - u) ** 8
    assert abs(cnt[2] / P - p0) < 5 * np.sqrt(p0 * (1 - p0) / P)
    pr = 1 - (1 - u) ** 20
    assert abs(cnt[4] / cnt[2] - pr) < 5 * np.sqrt(pr * (1 - pr) / cnt[2])
    sample = np.random.default_rng(1).integers(0, P, 300)
    for p in sample:                                   # sampled prompts, draw by draw
        draws = [O.default_key(ocfg.seed, int(p) * 32 + j) < int(thr[p]) for j in range(int(n[p]))]
        assert sum(draws) == c[p] and nt[p] == O.curated_size(ocfg, int(n[p]), int(c[p]))
        if n[p] > 8:
            assert not any(draws[:int(n[p]) - 2])


# ------------------------------------------------------------------ stage (b)
def run_fwd_bwd(ctx, batch, dtype, grad_scale=1.0, chunk_tokens=None):
    cfg = TL.lib_cfg(batch.ocfg, dtype)
    dv = batch.to_device()
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    dH, dW = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                               grad_scale=grad_scale, chunk_tokens=chunk_tokens)
    torch.cuda.synchronize()
    return cfg, dv, f, dH, dW


def check_fwd(batch, f, ref, logp_abs, loss_rel, g_rtol):
    T = batch.T
    owner = O.token_rollout(batch.st.cs, T)
    kept = batch.ref_g["keep"][owner] != 0
    logp = f["logp"][:T].cpu().numpy()
    lse = f["lse"][:T].cpu().numpy()
    g = f["g"][:T].cpu().numpy()
    assert np.abs(logp - ref["logp"]).max() <= logp_abs
    assert np.abs(lse - ref["lse"]).max() <= logp_abs
    assert not logp[~kept].any() and not g[~kept].any() and not lse[~kept].any()
    assert (logp[kept] <= 1e-6).all()
    loss = float(f["loss"].item())
    assert abs(loss - ref["loss"]) <= loss_rel * abs(ref["loss"]) + 1e-7
    # clip indicators may legitimately flip when rho sits within rounding of a clip edge
    rho = ref["rho"]
    edge = (np.abs(rho - (1 + batch.ocfg.clip_hi)) < 1e-3) | (np.abs(rho - (1 - batch.ocfg.clip_lo)) < 1e-3)
    ok = ~edge
    np.testing.assert_allclose(g[ok], ref["g"][ok], rtol=g_rtol, atol=1e-12)
    met = f["metrics"].cpu().numpy()
    assert met[3] == kept.sum()
    assert abs(met[0] - ref["metrics"][0]) <= (edge.sum() + 0.5) / max(kept.sum(), 1)
    assert abs(met[1] - ref["metrics"][1]) < 1e-3


def test_tiny_workload_fp32(ctx):
    wl = synth.WORKLOADS[0]
    batch = TL.Batch(wl, TL.cfg_for(wl))
    assert batch.ref_g["gmask"][0] == 0 and batch.ref_g["gmask"][1] == 0      # forced uniform groups
    ref = batch.oracle_fwd()
    cfg, dv, f, dH, dW = run_fwd_bwd(ctx, batch, "fp32", grad_scale=1.5)
    check_fwd(batch, f, ref, 1e-4, 1e-4, 1e-3)
    rdH, rdW = batch.oracle_bwd(ref, 1.5)
    assert TL.rel_l2(dH.cpu().numpy(), rdH) < 1e-4
    assert TL.rel_l2(dW.cpu().numpy(), rdW) < 1e-4
    assert ctx.last_status() == 0


BF16_CASES = {
    # name: (workload overrides, cfg overrides, peak strength)
    "tiny_bf16": (dict(dtype="bf16"), dict(), 0.0),
    "ragged_tail": (dict(P=6, n_lo=3, n_hi=9, d=128, V=1000, len_median=70.0, len_cap=300, dtype="bf16", seed=11),
                    dict(), 0.0),
    "aero_dropped": (dict(P=24, n_lo=2, n_hi=12, d=192, V=3001, len_median=40.0, len_cap=160, dtype="bf16",
                          aero=True, old_noise=0.15, seed=12), dict(uniform_policy=O.UNIFORM_BAYES, rejection=1), 0.0),
    "seq_mean_clipped": (dict(P=8, n_lo=4, n_hi=4, d=256, V=2048, len_median=50.0, len_cap=100, dtype="bf16",
                              old_noise=0.25, seed=13), dict(agg=O.AGG_SEQ_MEAN), 0.0),
    "peaked": (dict(P=6, n_lo=4, n_hi=8, d=128, V=4096, len_median=60.0, len_cap=200, dtype="bf16", seed=14),
               dict(), 45.0),
}


@pytest.mark.parametrize("name", list(BF16_CASES))
def test_bf16_tensor_core_path(ctx, name):
    over, cover, peak = BF16_CASES[name]
    base = synth.WORKLOADS[0] if name == "tiny_bf16" else synth.WORKLOADS[1]
    wl = synth.scaled(base, **over)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **cover), peak=peak)
    ref = batch.oracle_fwd()
    cfg, dv, f, dH, dW = run_fwd_bwd(ctx, batch, "bf16")
    assert ctx.last_status() == 0
    check_fwd(batch, f, ref, LOGP_ABS, LOSS_REL, 2e-2)
    # backward from the oracle's own lse and g, so that only the backward is under test ...
    rdH, rdW = batch.oracle_bwd(ref)
    dH2, dW2 = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"],
                                 TL.dev(ref["lse"], torch.float32), TL.dev(ref["g"], torch.float32))
    assert TL.rel_l2(dH2.float().cpu().numpy(), rdH) < GRAD_L2
    assert TL.rel_l2(dW2.cpu().numpy(), rdW) < GRAD_L2
    # ... and end to end from the library's forward outputs
    assert TL.rel_l2(dH.float().cpu().numpy(), rdH) < GRAD_L2
    assert TL.rel_l2(dW.cpu().numpy(), rdW) < GRAD_L2
    # invariants: columns of dW sum to zero; dropped rows of dH are zero
    owner = O.token_rollout(batch.st.cs, batch.T)
    dropped = batch.ref_g["keep"][owner] == 0
    assert not dH.float().cpu().numpy()[dropped].any()
    col = np.abs(dW.double().cpu().numpy().sum(axis=0)).max()
    assert col <= 2e-2 * np.abs(rdW).sum(axis=0).max() + 1e-9
    if peak > 0:
        # the softmax part alone (one-hot part removed) must also agree: it is what a kernel
        # that dropped the softmax term would get wrong
        Wm, y, g = batch.W, batch.st.y, ref["g"]
        soft_ref = rdH - g[:, None] * Wm[y]
        soft_gpu = dH2.float().cpu().numpy() - g[:, None] * Wm[y]
        live = g != 0
        assert np.linalg.norm(soft_ref[live]) > 0.05 * np.linalg.norm(rdH[live])
        assert TL.rel_l2(soft_gpu[live], soft_ref[live]) < 3e-2
        never_hit = np.setdiff1d(np.arange(wl.V), y)
        assert TL.rel_l2(dW2.cpu().numpy()[never_hit], rdW[never_hit]) < GRAD_L2


@pytest.mark.parametrize("vsplit", [2, 4])
def test_vocabulary_split_between_cta_pairs(ctx, vsplit):
    """At large d several CTA pairs share a token tile and split the vocabulary (running states merged by
    a second kernel).  Forced here on small shapes: all forward modes and the backward against the
    oracle, and bit-identical log-probs between a split and an unsplit run of the log-prob pass."""
    over, cover, peak = BF16_CASES["peaked"]
    wl = synth.scaled(synth.WORKLOADS[1], **over)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, kl_beta=0.1, ent_coef=0.2, **cover), peak=peak)
    ocfg, rg = batch.ocfg, batch.ref_g
    adv32 = rg["adv"].astype(np.float32).astype(np.float64)
    w32 = rg["w"].astype(np.float32).astype(np.float64)
    ref_lp = (batch.old + 0.2).astype(np.float32)
    ref = O.grpo_loss_reg_fwd(ocfg, batch.H, batch.W, batch.st.y, batch.old, ref_lp, batch.st.cs, adv32, w32, rg["keep"])
    rdH, rdW = O.grpo_loss_reg_bwd(ocfg, batch.H, batch.W, batch.st.y, batch.st.cs, rg["keep"], ref["lse"], ref["g"],
                                   ref["entropy"], w32)
    cfg = TL.lib_cfg(ocfg, "bf16")
    dv = batch.to_device()
    plain = ctx.logprob_fwd(cfg, dv["H"], dv["W"], dv["y"], entropy=True)
    ctx.set_tuning(vsplit=vsplit)
    try:
        f = ctx.grpo_loss_reg_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], TL.dev(ref_lp), dv["cs"], dv["adv"], dv["w"],
                                  dv["keep"])
        dH, dW = ctx.grpo_loss_reg_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                       f["entropy"], dv["w"], logp=f["logp"])
        f0 = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
        split = ctx.logprob_fwd(cfg, dv["H"], dv["W"], dv["y"], entropy=True)
        torch.cuda.synchronize()
    finally:
        ctx.set_tuning()
    assert ctx.last_status() == 0
    T = batch.T
    assert np.abs(f["logp"][:T].cpu().numpy() - ref["logp"]).max() <= LOGP_ABS
    assert np.abs(f["entropy"][:T].cpu().numpy() - ref["entropy"]).max() <= LOGP_ABS
    assert abs(f["loss"].item() - ref["loss"]) <= LOSS_REL * abs(ref["loss"]) + 1e-7
    rho = ref["rho"]
    edge = (np.abs(rho - 1.2) < 1e-3) | (np.abs(rho - 0.8) < 1e-3)
    assert TL.rel_l2(dH.float().cpu().numpy()[~edge], rdH[~edge]) < GRAD_L2
    if not edge.any():
        assert TL.rel_l2(dW.cpu().numpy(), rdW) < GRAD_L2
    check_fwd(batch, f0, O.grpo_loss_fwd(O.Cfg(seed=wl.seed, **cover), batch.H, batch.W, batch.st.y, batch.old,
                                          batch.st.cs, adv32, w32, rg["keep"]), LOGP_ABS, LOSS_REL, 2e-2)
    # the split changes only the order in which a row's tiles are merged
    assert np.abs((split["logp"][:T] - plain["logp"][:T]).cpu().numpy()).max() < 1e-5
    assert np.abs((split["entropy"][:T] - plain["entropy"][:T]).cpu().numpy()).max() < 1e-4
    # the L2 eviction priority of the W loads changes no arithmetic: same bits either way, in the
    # forward (hint on by default) and in the one-call step (off by default)
    outs = []
    for hint in (0, 1):
        ctx.set_tuning(w_hint=hint)
        try:
            lp = ctx.logprob_fwd(cfg, dv["H"], dv["W"], dv["y"], entropy=True)
            f1, dH1, dW1 = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"],
                                                 dv["keep"])
            torch.cuda.synchronize()
        finally:
            ctx.set_tuning()
        outs.append((lp["logp"].clone(), f1["logp"].clone(), dH1.clone(), f1["loss"].clone()))
    assert ctx.last_status() == 0
    assert torch.equal(outs[0][0], plain["logp"]) and torch.equal(outs[1][0], plain["logp"])
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2]) and torch.equal(outs[0][3], outs[1][3])
    # walking d always forwards (instead of forwards and backwards in turn) only reorders a logit's fp32 sums
    ctx.set_tuning(k_zigzag=0)
    try:
        fwd_only = ctx.logprob_fwd(cfg, dv["H"], dv["W"], dv["y"], entropy=True)
        f2, dH2, dW2 = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
        torch.cuda.synchronize()
    finally:
        ctx.set_tuning()
    assert ctx.last_status() == 0
    assert np.abs((fwd_only["logp"][:T] - plain["logp"][:T]).cpu().numpy()).max() < 1e-5
    assert np.abs(f2["logp"][:T].cpu().numpy() - ref["logp"]).max() <= LOGP_ABS
    assert TL.rel_l2(dH2.float().cpu().numpy(), outs[0][2].float().cpu().numpy()) < 5e-3    # bf16 roundings that flip


@pytest.mark.parametrize("name", list(BF16_CASES) + ["tiny_fp32"])
def test_forward_and_backward_in_one_call(ctx, name):
    """aero_grpo_loss_fwd_bwd (the forward leaves exp(z - c_t) of each chunk, the backward rescales it
    instead of recomputing the logits) against the oracle, in one chunk and in 128-row chunks, with the
    row factors applied in the backward GEMMs or by the rewriting pass, and with a forced vocabulary split."""
    if name == "tiny_fp32":
        wl, cover, peak, dtype = synth.WORKLOADS[0], {}, 0.0, "fp32"
    else:
        over, cover, peak = BF16_CASES[name]
        wl = synth.scaled(synth.WORKLOADS[0] if name == "tiny_bf16" else synth.WORKLOADS[1], **over)
        dtype = "bf16"
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **cover), peak=peak)
    ref = batch.oracle_fwd()
    rdH, rdW = batch.oracle_bwd(ref, 0.75)
    cfg = TL.lib_cfg(batch.ocfg, dtype)
    dv = batch.to_device()
    tol = (1e-4, 1e-4, 1e-4) if dtype == "fp32" else (LOGP_ABS, LOSS_REL, GRAD_L2)
    rho = ref["rho"]
    edge = (np.abs(rho - (1 + batch.ocfg.clip_hi)) < 1e-3) | (np.abs(rho - (1 - batch.ocfg.clip_lo)) < 1e-3)
    # (row factors in the backward GEMMs, with two splits sharing one shift per row; rowscale 0: the pass
    # that rewrites the block, with a shift per split)
    # (the last entries also pace the producers of the backward products -- same results, another schedule --
    # and run them on single CTAs instead of CTA pairs)
    for chunk, vsplit, rowscale, gsync, pairs in ((None, 0, -1, -1, -1), (128, 0, -1, -1, -1), (128, 0, 0, 3, -1), (128, 2, -1, 2, -1),
                                                  (128, 2, 0, -1, -1), (None, 0, -1, 5, 0), (128, 0, -1, 0, 0), (384, 2, 0, 2, 0)):
        ctx.set_tuning(vsplit=vsplit, rowscale=rowscale, gemm_sync=gsync, gemm_pairs=pairs)
        try:
            ws = None
            if chunk:
                ws = torch.empty(ctx.fwd_bwd_workspace_bytes(batch.T, wl.d, wl.V, batch.R, chunk), dtype=torch.uint8, device="cuda")
            f, dH, dW = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"],
                                              dv["keep"], grad_scale=0.75, workspace=ws)
            torch.cuda.synchronize()
        finally:
            ctx.set_tuning()
        assert ctx.last_status() == 0
        check_fwd(batch, f, ref, tol[0], tol[1], 2e-2 if dtype == "bf16" else 1e-3)
        assert TL.rel_l2(dH.float().cpu().numpy()[~edge], rdH[~edge]) < tol[2]
        if not edge.any():
            assert TL.rel_l2(dW.cpu().numpy(), rdW) < tol[2]
        owner = O.token_rollout(batch.st.cs, batch.T)
        assert not dH.float().cpu().numpy()[batch.ref_g["keep"][owner] == 0].any()
        if peak > 0:          # the softmax part alone
            g = ref["g"] * 0.75
            soft_ref = rdH - g[:, None] * batch.W[batch.st.y]
            soft_gpu = dH.float().cpu().numpy() - g[:, None] * batch.W[batch.st.y]
            live = (g != 0) & ~edge
            assert TL.rel_l2(soft_gpu[live], soft_ref[live]) < 3e-2


def test_one_call_step_redoes_rows_with_a_logit_out_of_range(ctx):
    """The one-call step stores exp(z - c_t) in bf16 with c_t taken from the row's first 32 logits; a logit more
    than about 127 above them cannot be held.  Such a row is listed by the forward and its dz row recomputed
    from H and W, so its gradient must agree with the two-call path like any other row and no status bit is left."""
    wl = synth.scaled(synth.WORKLOADS[1], P=4, n_lo=3, n_hi=6, d=128, V=2000, len_median=40.0, len_cap=120, dtype="bf16",
                      seed=57)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed), peak=0.0)
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    dv = batch.to_device()
    owner = O.token_rollout(batch.st.cs, batch.T)
    kept = np.nonzero(batch.ref_g["keep"][owner] != 0)[0]
    rows = [int(kept[3]), int(kept[-5])]
    H, W = dv["H"].clone(), dv["W"].clone()
    for t in rows:
        H[t] = 2.0                             # z[t, 1500] = 128 * 2 * 1.5 = 384; the first 32 logits of the row stay small
    W[1500] = 1.5
    W[:32] *= 0.01
    y = dv["y"].clone()
    y[rows[1]] = 1500                          # one of the rows has the huge logit as its target (p_y = 1 to rounding)
    # old log-probs of the two rows follow their new ones (about -384 and 0), so that the ratio stays near 1
    f2 = ctx.grpo_loss_fwd(cfg, H, W, y, dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    old = dv["old"].clone()
    old[rows] = f2["logp"][rows] + 0.01
    f2 = ctx.grpo_loss_fwd(cfg, H, W, y, old, dv["cs"], dv["adv"], dv["w"], dv["keep"])
    dH2, dW2 = ctx.grpo_loss_bwd(cfg, H, W, y, dv["cs"], dv["keep"], f2["lse"], f2["g"], logp=f2["logp"])
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for rowscale in (-1, 0):
        ctx.set_tuning(rowscale=rowscale)
        try:
            f, dH, dW = ctx.grpo_loss_fwd_bwd(cfg, H, W, y, old, dv["cs"], dv["adv"], dv["w"], dv["keep"])
            torch.cuda.synchronize()
        finally:
            ctx.set_tuning()
        assert ctx.last_status() == 0
        assert torch.isfinite(f["logp"]).all() and torch.isfinite(dH.float()).all() and torch.isfinite(dW).all()
        np.testing.assert_allclose(f["logp"][:batch.T].cpu().numpy(), f2["logp"][:batch.T].cpu().numpy(), atol=2e-5)
        a, b = dH.float().cpu().numpy(), dH2.float().cpu().numpy()
        live = np.linalg.norm(b, axis=1) > 0
        assert live[rows[0]]
        err = np.linalg.norm(a - b, axis=1)[live] / np.linalg.norm(b, axis=1)[live]
        assert err.max() < GRAD_L2
        assert TL.rel_l2(dW.cpu().numpy(), dW2.cpu().numpy()) < GRAD_L2
    # the same with the entropy term, whose part of a redone row's dz is recomputed from the logits too
    ecfg = TL.lib_cfg(O.Cfg(seed=wl.seed, ent_coef=0.5), "bf16")
    fe = ctx.grpo_loss_reg_fwd(ecfg, H, W, y, old, None, dv["cs"], dv["adv"], dv["w"], dv["keep"], entropy=True)
    dHe, dWe = ctx.grpo_loss_reg_bwd(ecfg, H, W, y, dv["cs"], dv["keep"], fe["lse"], fe["g"], fe["entropy"], dv["w"],
                                     logp=fe["logp"])
    f, dH, dW = ctx.grpo_loss_fwd_bwd(ecfg, H, W, y, old, dv["cs"], dv["adv"], dv["w"], dv["keep"], entropy=True)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert torch.isfinite(dH.float()).all() and torch.isfinite(dW).all()
    np.testing.assert_allclose(f["entropy"][:batch.T].cpu().numpy(), fe["entropy"][:batch.T].cpu().numpy(), atol=2e-5)
    a, b = dH.float().cpu().numpy(), dHe.float().cpu().numpy()
    nb = np.linalg.norm(b, axis=1)
    live = nb > 0
    # (rows where one column holds all of the probability have H_t = 0 and a gradient of rounding size on both
    # paths, each with its own noise: a row is compared against its own norm or a twentieth of the typical row's,
    # whichever is larger -- an entropy term taken from a rounded logarithm would miss that by a factor of 500)
    err = np.linalg.norm(a - b, axis=1)[live] / np.maximum(nb[live], 0.05 * np.median(nb[live]))
    assert err.max() < GRAD_L2
    assert nb[rows[0]] > 0.05 * np.median(nb[live])
    assert TL.rel_l2(dW.cpu().numpy(), dWe.cpu().numpy()) < GRAD_L2
    assert TL.rel_l2(dHe.float().cpu().numpy(), dH2.float().cpu().numpy()) > 5 * GRAD_L2      # the term carries weight


def _row_err(a, b, rows):
    """Relative L2 error of each listed row of a against b."""
    a, b = np.asarray(a, np.float64)[rows], np.asarray(b, np.float64)[rows]
    return np.linalg.norm(a - b, axis=1) / np.linalg.norm(b, axis=1)


def test_confident_tokens_row_by_row(ctx):
    """Rows whose target has probability 0.97, 0.999 and 0.9999: Eq. 3's factor (1 - p) is then tiny, the
    one-hot and the softmax part of the row's gradient cancel to that size, and a whole-matrix norm cannot
    see an error in them.  Every live row of dH is compared with the oracle by itself, for the two-call path
    and both forms of the one-call step; the columns of dW must still sum to zero."""
    wl = synth.scaled(synth.WORKLOADS[1], P=6, n_lo=4, n_hi=8, d=256, V=4096, len_median=60.0, len_cap=200, dtype="bf16",
                      seed=61)
    st = synth.make_structure(wl)
    T = int(st.cs[-1])
    strength = np.array([38.0, 50.0, 57.0])[np.arange(T) % 3]
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed), peak=strength, st=st)
    ref = batch.oracle_fwd()
    one_minus_p = -np.expm1(ref["logp"])
    owner = O.token_rollout(st.cs, T)
    kept = batch.ref_g["keep"][owner] != 0
    for k, (lo, hi) in enumerate([(5e-3, 1e-1), (1e-4, 5e-3), (1e-5, 8e-4)]):   # the three strengths land where intended
        band = one_minus_p[kept & (np.arange(T) % 3 == k)]
        assert np.median(band) > lo and np.median(band) < hi
    rdH, rdW = batch.oracle_bwd(ref, 0.75)
    rho = ref["rho"]
    edge = (np.abs(rho - 1.2) < 1e-3) | (np.abs(rho - 0.8) < 1e-3)
    live = np.nonzero((ref["g"] != 0) & ~edge)[0]
    assert len(live) > 500
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    dv = batch.to_device()
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    # the log-prob itself keeps its relative accuracy when it is tiny
    lp = f["logp"][:T].cpu().numpy()
    assert np.abs(lp[live] - ref["logp"][live]).max() <= LOGP_ABS
    assert (np.abs(lp[live] - ref["logp"][live]) <= 5e-3 * np.abs(ref["logp"][live]) + 1e-7).all()
    results = {}
    results["two calls"] = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                             grad_scale=0.75, logp=f["logp"])
    for name, rowscale in (("one call, row factors", -1), ("one call, rewriting pass", 0)):
        ctx.set_tuning(rowscale=rowscale)
        try:
            _, dH, dW = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"],
                                              dv["keep"], grad_scale=0.75)
            torch.cuda.synchronize()
        finally:
            ctx.set_tuning()
        results[name] = (dH, dW)
    assert ctx.last_status() == 0
    for name, (dH, dW) in results.items():
        err = _row_err(dH.float().cpu().numpy(), rdH, live)
        assert err.max() < GRAD_L2, (name, float(err.max()), int(live[err.argmax()]), float(one_minus_p[live[err.argmax()]]))
        if not edge.any():
            assert TL.rel_l2(dW.cpu().numpy(), rdW) < GRAD_L2, name
        col = np.abs(dW.double().cpu().numpy().sum(axis=0)).max()
        assert col <= 1e-2 * np.abs(rdW).sum(axis=0).max() + 1e-12, name


PEAKED_FULL_WIDTH = {
    # name: (workload, overrides, strengths the rows cycle through)
    "qwen1p5b_2048_tokens": (1, dict(P=4, n_lo=8, n_hi=8, len_median=64.0, len_cap=96, seed=71), (10.0, 14.0, 20.0, 26.0)),
    "qwen7b_split_vocabulary": (2, dict(P=1, n_lo=6, n_hi=6, len_median=56.0, len_cap=80, seed=72), (6.0, 9.0, 12.0, 17.0)),
}


@pytest.mark.parametrize("name", list(PEAKED_FULL_WIDTH))
def test_peaked_logits_at_full_width(ctx, name):
    """Peaked logits at the full widths of the benchmark workloads (d = 1536 with V = 151936 on about 2048 tokens;
    d = 3584 with V = 152064, where two CTA pairs split the vocabulary, on 256 tokens and more): with the
    N(0,1) / N(0,0.02) inputs the softmax part of dH and dW is under 1 % of the one-hot part and no tolerance
    would see it missing.  Here the rows' target probabilities spread from a few per cent to above 0.999, the
    softmax part is isolated (one-hot part removed), and every live row is compared by itself."""
    base, over, strengths = PEAKED_FULL_WIDTH[name]
    wl = synth.scaled(synth.WORKLOADS[base], **over)
    st = synth.make_structure(wl)
    T = int(st.cs[-1])
    assert T >= (1900 if base == 1 else 256)
    strength = np.array(strengths)[np.arange(T) % len(strengths)]
    # (uniform groups keep all their rollouts with the Bayesian advantage, so that every row is live)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, uniform_policy=O.UNIFORM_BAYES, n_keep_uniform=0), peak=strength, st=st)
    ref = batch.oracle_fwd()
    p_y = np.exp(ref["logp"])
    owner = O.token_rollout(st.cs, T)
    kept = batch.ref_g["keep"][owner] != 0
    assert kept.any() and p_y[kept].min() < 0.2 and p_y[kept].max() > 0.999
    rho = ref["rho"]
    edge = (np.abs(rho - 1.2) < 1e-3) | (np.abs(rho - 0.8) < 1e-3)
    live = np.nonzero((ref["g"] != 0) & ~edge)[0]
    hit = np.unique(st.y[kept])
    rows = np.unique(np.concatenate([hit[:256], np.random.default_rng(3).integers(0, wl.V, 768)]))
    rdH, rdW = batch.oracle_bwd(ref, dw_rows=rows)
    never_hit = ~np.isin(rows, hit)
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    dv = batch.to_device()
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    check_fwd(batch, f, ref, LOGP_ABS, LOSS_REL, 2e-2)
    results = {"two calls": ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                               logp=f["logp"])}
    _, dH1, dW1 = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    results["one call"] = (dH1, dW1)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    g = ref["g"]
    onehot = g[:, None] * batch.W[st.y]
    soft_ref = rdH - onehot
    assert np.linalg.norm(soft_ref[live]) > 0.3 * np.linalg.norm(rdH[live])       # the softmax part carries weight here
    for name2, (dH, dW) in results.items():
        dHc = dH.float().cpu().numpy()
        err = _row_err(dHc, rdH, live)
        assert err.max() < GRAD_L2, (name2, float(err.max()), float(p_y[live[err.argmax()]]))
        assert TL.rel_l2((dHc - onehot)[live], soft_ref[live]) < GRAD_L2, name2
        dWc = dW.cpu().numpy()[rows]
        assert TL.rel_l2(dWc, rdW) < GRAD_L2, name2
        assert np.linalg.norm(rdW[never_hit]) > 0 and TL.rel_l2(dWc[never_hit], rdW[never_hit]) < GRAD_L2, name2


def test_bwd_chunking_and_accumulation(ctx):
    over, cover, _ = BF16_CASES["aero_dropped"]
    wl = synth.scaled(synth.WORKLOADS[1], **over)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **cover))
    cfg, dv, f, dH, dW = run_fwd_bwd(ctx, batch, "bf16")
    # one 128-row tile per chunk: many chunks, dW accumulated across them
    dH1, dW1 = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                 chunk_tokens=128, workspace=torch.empty(
                                     ctx.bwd_workspace_bytes(batch.T, wl.d, wl.V, batch.R, 128), dtype=torch.uint8, device="cuda"))
    assert torch.equal(dH1, dH)
    assert TL.rel_l2(dW1.cpu().numpy(), dW.cpu().numpy()) < 1e-5
    # the same products on single CTAs (the default runs them on CTA pairs: units of 256 rows, with an odd
    # number of row tiles in the last pair of a chunk)
    ctx.set_tuning(gemm_pairs=0)
    try:
        for chunk in (None, 128, 384):
            ws = None if chunk is None else torch.empty(ctx.bwd_workspace_bytes(batch.T, wl.d, wl.V, batch.R, chunk),
                                                        dtype=torch.uint8, device="cuda")
            dHp, dWp = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                         chunk_tokens=chunk, workspace=ws)
            assert torch.equal(dHp, dH)
            assert TL.rel_l2(dWp.cpu().numpy(), dW.cpu().numpy()) < 1e-5
    finally:
        ctx.set_tuning()
    # accumulate_dW adds to what is there
    dW2 = dW.clone()
    ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"], dW=dW2, accumulate_dW=True)
    assert TL.rel_l2(dW2.cpu().numpy(), 2 * dW.cpu().numpy()) < 1e-5
    # the loss reduction is order-fixed: identical bits on a second run; accumulate adds
    f2 = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"])
    assert torch.equal(f2["loss"], f["loss"]) and torch.equal(f2["logp"], f["logp"])
    ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"],
                      out=f2, accumulate=True)
    assert abs(f2["loss"].item() - 2 * f["loss"].item()) <= 1e-6 * abs(f["loss"].item()) + 1e-9
    assert ctx.last_status() == 0


def test_all_dropped_and_bad_target(ctx):
    wl = synth.scaled(synth.WORKLOADS[1], P=3, n_lo=4, n_hi=4, d=64, V=300, len_median=30.0, len_cap=64, seed=21)
    batch = TL.Batch(wl, O.Cfg())
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    dv = batch.to_device()
    zero_keep = torch.zeros_like(dv["keep"])
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], zero_keep)
    dH, dW = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], zero_keep, f["lse"], f["g"])
    assert f["loss"].item() == 0.0 and not dH.float().abs().sum().item() and not dW.abs().sum().item()
    assert ctx.last_status() == 0
    # an out-of-range target is reported and its row skipped
    keep = torch.ones_like(dv["keep"])
    y = dv["y"].clone()
    y[5] = wl.V + 7
    f = ctx.grpo_loss_fwd(cfg, dv["H"], dv["W"], y, dv["old"], dv["cs"], dv["adv"], dv["w"], keep)
    assert ctx.last_status() & B.AERO_ST_BAD_TARGET
    assert f["g"][5].item() == 0.0 and f["logp"][5].item() == 0.0


def test_full_width_qwen_1p5b_shape(ctx):
    """Full d = 1536 and V = 151936 of the Qwen2.5-Math-1.5B workload on a batch the oracle can
    finish: 8 rollouts of ~80 tokens (several row tiles, 594 vocabulary tiles with the ragged
    last one).  Every output against the oracle; dW on the target rows plus 1024 random rows."""
    wl = synth.scaled(synth.WORKLOADS[1], P=2, n_lo=4, n_hi=4, len_median=80.0, len_cap=200, seed=31)
    batch = TL.Batch(wl, TL.cfg_for(wl, uniform_policy=O.UNIFORM_BAYES))
    assert batch.T >= 384
    ref = batch.oracle_fwd()
    cfg, dv, f, dH, dW = run_fwd_bwd(ctx, batch, "bf16")
    assert ctx.last_status() == 0
    check_fwd(batch, f, ref, LOGP_ABS, LOSS_REL, 2e-2)
    rows = np.unique(np.concatenate([batch.st.y[:64], np.random.default_rng(1).integers(0, wl.V, 1024)]))
    rdH, rdW = batch.oracle_bwd(ref, dw_rows=rows)
    assert TL.rel_l2(dH.float().cpu().numpy(), rdH) < GRAD_L2
    assert TL.rel_l2(dW.cpu().numpy()[rows], rdW) < GRAD_L2


def test_full_width_qwen_7b_shape(ctx):
    """Full d = 3584 and V = 152064 of the Qwen2.5-7B shaped workloads, AERO mode with ragged groups
    and per-prompt priors, on a batch the oracle can finish.  Every output against the oracle; dW on
    the target rows plus 512 random rows."""
    wl = synth.scaled(synth.WORKLOADS[3], P=3, n_lo=2, n_hi=6, len_median=48.0, len_cap=120, seed=33)
    batch = TL.Batch(wl, TL.cfg_for(wl))
    assert batch.T >= 256 and batch.ref_g["keep"].sum() < batch.R
    ref = batch.oracle_fwd()
    cfg, dv, f, dH, dW = run_fwd_bwd(ctx, batch, "bf16")
    assert ctx.last_status() == 0
    check_fwd(batch, f, ref, LOGP_ABS, LOSS_REL, 2e-2)
    rows = np.unique(np.concatenate([batch.st.y[:64], np.random.default_rng(2).integers(0, wl.V, 512)]))
    rdH, rdW = batch.oracle_bwd(ref, dw_rows=rows)
    assert TL.rel_l2(dH.float().cpu().numpy(), rdH) < GRAD_L2
    assert TL.rel_l2(dW.cpu().numpy()[rows], rdW) < GRAD_L2


REG_CASES = {
    # name: (dtype, workload overrides, cfg overrides, peak, use reference log-probs)
    "tiny_fp32_kl_entropy": ("fp32", dict(), dict(kl_beta=0.04, ent_coef=1e-3), 0.0, True),
    "bf16_entropy_only": ("bf16", dict(P=6, n_lo=3, n_hi=9, d=128, V=1000, len_median=70.0, len_cap=300, dtype="bf16",
                                       seed=41), dict(ent_coef=0.5), 45.0, False),
    "bf16_kl_only": ("bf16", dict(P=6, n_lo=3, n_hi=9, d=128, V=3001, len_median=50.0, len_cap=200, dtype="bf16",
                                  seed=42), dict(kl_beta=0.5), 0.0, True),
    "bf16_peaked_kl_entropy": ("bf16", dict(P=6, n_lo=4, n_hi=8, d=128, V=4096, len_median=60.0, len_cap=200,
                                            dtype="bf16", aero=True, seed=43),
                               dict(kl_beta=0.2, ent_coef=0.3, uniform_policy=O.UNIFORM_BAYES, rejection=1), 45.0, True),
}


@pytest.mark.parametrize("name", list(REG_CASES))
def test_regularised_objective(ctx, name):
    """Eq. 2's KL term and the entropy bonus of Table 9 through aero_grpo_loss_reg_fwd / _bwd against
    the oracle.  The coefficients are larger than the paper's so that both terms carry weight in
    every tolerance; the peaked case makes the entropy gradient comparable to the policy gradient."""
    dtype, over, cover, peak, use_ref = REG_CASES[name]
    base = synth.WORKLOADS[0] if dtype == "fp32" else synth.WORKLOADS[1]
    wl = synth.scaled(base, **over)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **cover), peak=peak)
    ocfg = batch.ocfg
    rg = batch.ref_g
    rng = np.random.default_rng(5)
    ref_lp = (batch.old.astype(np.float64) + 0.3 * rng.standard_normal(batch.T)).astype(np.float32) if use_ref else None
    adv32 = rg["adv"].astype(np.float32).astype(np.float64)
    w32 = rg["w"].astype(np.float32).astype(np.float64)
    ref = O.grpo_loss_reg_fwd(ocfg, batch.H, batch.W, batch.st.y, batch.old, ref_lp, batch.st.cs, adv32, w32, rg["keep"])
    rdH, rdW = O.grpo_loss_reg_bwd(ocfg, batch.H, batch.W, batch.st.y, batch.st.cs, rg["keep"], ref["lse"], ref["g"],
                                   ref["entropy"], w32)
    cfg = TL.lib_cfg(ocfg, dtype)
    dv = batch.to_device()
    want_ent = ocfg.ent_coef != 0.0
    f = ctx.grpo_loss_reg_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], TL.dev(ref_lp) if use_ref else None,
                              dv["cs"], dv["adv"], dv["w"], dv["keep"], entropy=want_ent)
    if want_ent:
        dH, dW = ctx.grpo_loss_reg_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"],
                                       f["entropy"], dv["w"])
    else:
        dH, dW = ctx.grpo_loss_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["cs"], dv["keep"], f["lse"], f["g"])
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    tol = (1e-4, 1e-4, 1e-4) if dtype == "fp32" else (LOGP_ABS, LOSS_REL, GRAD_L2)
    owner = O.token_rollout(batch.st.cs, batch.T)
    kept = rg["keep"][owner] != 0
    assert np.abs(f["logp"][:batch.T].cpu().numpy() - ref["logp"]).max() <= tol[0]
    if want_ent:
        ent = f["entropy"][:batch.T].cpu().numpy()
        assert np.abs(ent - ref["entropy"]).max() <= tol[0] and not ent[~kept].any()
        assert ref["entropy"][kept].min() > 0.05          # the term is not vacuous
    assert abs(f["loss"].item() - ref["loss"]) <= tol[1] * abs(ref["loss"]) + 1e-7
    rho = ref["rho"]
    edge = (np.abs(rho - (1 + ocfg.clip_hi)) < 1e-3) | (np.abs(rho - (1 - ocfg.clip_lo)) < 1e-3)
    np.testing.assert_allclose(f["g"][:batch.T].cpu().numpy()[~edge], ref["g"][~edge], rtol=2e-2, atol=1e-9)
    assert TL.rel_l2(dH.float().cpu().numpy()[~edge], rdH[~edge]) < tol[2]
    if not edge.any():
        assert TL.rel_l2(dW.cpu().numpy(), rdW) < tol[2]
    # the regulariser changes the answer by more than the tolerance: the test can see it
    plain = O.grpo_loss_fwd(ocfg, batch.H, batch.W, batch.st.y, batch.old, batch.st.cs, adv32, w32, rg["keep"])
    pdH, _ = O.grpo_loss_bwd(batch.H, batch.W, batch.st.y, batch.st.cs, rg["keep"], plain["lse"], plain["g"])
    assert TL.rel_l2(pdH, rdH) > 5 * tol[2]
    # the same objective through the one-call step (aero_grpo_loss_reg_fwd_bwd): the entropy term of dz
    # takes log p back from the stored exp(z - c_t); unsplit and with the vocabulary split in two
    for vsplit in ((0,) if dtype == "fp32" else (0, 2)):
        ctx.set_tuning(vsplit=vsplit)
        try:
            f1, dH1, dW1 = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"],
                                                 dv["keep"], ref_logp=TL.dev(ref_lp) if use_ref else None,
                                                 entropy=want_ent)
            torch.cuda.synchronize()
        finally:
            ctx.set_tuning()
        assert ctx.last_status() == 0
        assert np.abs(f1["logp"][:batch.T].cpu().numpy() - ref["logp"]).max() <= tol[0]
        if want_ent:
            ent1 = f1["entropy"][:batch.T].cpu().numpy()
            assert np.abs(ent1 - ref["entropy"]).max() <= tol[0] and not ent1[~kept].any()
        assert abs(f1["loss"].item() - ref["loss"]) <= tol[1] * abs(ref["loss"]) + 1e-7
        np.testing.assert_allclose(f1["g"][:batch.T].cpu().numpy()[~edge], ref["g"][~edge], rtol=2e-2, atol=1e-9)
        assert TL.rel_l2(dH1.float().cpu().numpy()[~edge], rdH[~edge]) < tol[2]
        if not edge.any():
            assert TL.rel_l2(dW1.cpu().numpy(), rdW) < tol[2]
            if want_ent:
                # the entropy part on its own: rows of dW that no token has as its target
                never_hit = np.setdiff1d(np.arange(wl.V), batch.st.y)
                if never_hit.size:
                    assert TL.rel_l2(dW1.cpu().numpy()[never_hit], rdW[never_hit]) < 2 * tol[2]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_kl_term_in_the_one_call_step(ctx, dtype):
    """aero_grpo_loss_kl_fwd_bwd: Eq. 2's KL term through the one-call step (it only changes loss and g_t)
    against the oracle, and against the two-call path with the same term."""
    base = synth.WORKLOADS[0] if dtype == "fp32" else synth.scaled(
        synth.WORKLOADS[1], P=6, n_lo=3, n_hi=9, d=256, V=3001, len_median=50.0, len_cap=200, dtype="bf16", seed=31)
    batch = TL.Batch(base, O.Cfg(seed=base.seed, kl_beta=0.5), peak=0.0)
    ocfg, rg = batch.ocfg, batch.ref_g
    rng = np.random.default_rng(6)
    ref_lp = (batch.old.astype(np.float64) + 0.3 * rng.standard_normal(batch.T)).astype(np.float32)
    adv32 = rg["adv"].astype(np.float32).astype(np.float64)
    w32 = rg["w"].astype(np.float32).astype(np.float64)
    ref = O.grpo_loss_reg_fwd(ocfg, batch.H, batch.W, batch.st.y, batch.old, ref_lp, batch.st.cs, adv32, w32, rg["keep"])
    rdH, rdW = O.grpo_loss_reg_bwd(ocfg, batch.H, batch.W, batch.st.y, batch.st.cs, rg["keep"], ref["lse"], ref["g"],
                                   ref["entropy"], w32)
    cfg = TL.lib_cfg(ocfg, dtype)
    dv = batch.to_device()
    f, dH, dW = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], dv["adv"], dv["w"], dv["keep"],
                                      ref_logp=TL.dev(ref_lp))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    tol = (1e-4, 1e-4, 1e-4) if dtype == "fp32" else (LOGP_ABS, LOSS_REL, GRAD_L2)
    assert np.abs(f["logp"][:batch.T].cpu().numpy() - ref["logp"]).max() <= tol[0]
    assert abs(f["loss"].item() - ref["loss"]) <= tol[1] * abs(ref["loss"]) + 1e-7
    rho = ref["rho"]
    edge = (np.abs(rho - (1 + ocfg.clip_hi)) < 1e-3) | (np.abs(rho - (1 - ocfg.clip_lo)) < 1e-3)
    np.testing.assert_allclose(f["g"][:batch.T].cpu().numpy()[~edge], ref["g"][~edge], rtol=2e-2, atol=1e-9)
    assert TL.rel_l2(dH.float().cpu().numpy()[~edge], rdH[~edge]) < tol[2]
    if not edge.any():
        assert TL.rel_l2(dW.cpu().numpy(), rdW) < tol[2]
    # the term is not vacuous: without it the gradient differs by far more than the tolerance
    plain = O.grpo_loss_fwd(ocfg, batch.H, batch.W, batch.st.y, batch.old, batch.st.cs, adv32, w32, rg["keep"])
    pdH, _ = O.grpo_loss_bwd(batch.H, batch.W, batch.st.y, batch.st.cs, rg["keep"], plain["lse"], plain["g"])
    assert TL.rel_l2(pdH, rdH) > 5 * tol[2]
    # the two-call path with the same term gives the same per-token coefficients
    f2 = ctx.grpo_loss_reg_fwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], TL.dev(ref_lp), dv["cs"], dv["adv"], dv["w"],
                               dv["keep"], entropy=False)
    np.testing.assert_allclose(f["g"][:batch.T].cpu().numpy(), f2["g"][:batch.T].cpu().numpy(), rtol=1e-4, atol=1e-9)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_logprob_pass_alone(ctx, dtype):
    """aero_logprob_fwd over all rows (no groups, no objective): the pass that produces old and
    reference log-probs, against log_softmax of the oracle's logits; entropy output included."""
    if dtype == "fp32":
        wl = synth.WORKLOADS[0]
    else:
        wl = synth.scaled(synth.WORKLOADS[1], P=5, n_lo=2, n_hi=6, d=192, V=5003, len_median=45.0, len_cap=150, seed=51)
    st = synth.make_structure(wl)
    T = int(st.cs[-1])
    H, W = synth.make_tensors(wl, T, device="cpu")
    z = O.logits(H.double().numpy(), W.double().numpy())
    lp, lse = O.log_softmax_pick(z, st.y)
    cfg = B.cfg_default(dtype=B.AERO_BF16 if dtype == "bf16" else B.AERO_FP32)
    o = ctx.logprob_fwd(cfg, H.cuda(), W.cuda(), TL.dev(st.y), entropy=True)
    tol = 1e-4 if dtype == "fp32" else LOGP_ABS
    assert np.abs(o["logp"][:T].cpu().numpy() - lp).max() <= tol
    assert np.abs(o["lse"][:T].cpu().numpy() - lse).max() <= tol
    assert np.abs(o["entropy"][:T].cpu().numpy() - O.entropy_rows(z)).max() <= tol
    o2 = ctx.logprob_fwd(cfg, H.cuda(), W.cuda(), TL.dev(st.y))
    assert torch.equal(o2["logp"][:T], o["logp"][:T])
    assert ctx.last_status() == 0


def test_step_from_host_buffers_matches_device_calls(ctx):
    over, cover, _ = BF16_CASES["aero_dropped"]
    wl = synth.scaled(synth.WORKLOADS[1], **over)
    batch = TL.Batch(wl, O.Cfg(seed=wl.seed, **cover))
    st = batch.st
    cfg = TL.lib_cfg(batch.ocfg, "bf16")
    dv = batch.to_device()
    gi, g = TL.run_group_gpu(ctx, cfg, st)
    f, dH, dW = ctx.grpo_loss_fwd_bwd(cfg, dv["H"], dv["W"], dv["y"], dv["old"], dv["cs"], g["adv"], g["w"], g["keep"])
    l0 = ctx.launch_count()
    dH2, dW2 = torch.empty_like(dH), torch.empty_like(dW)
    ws = torch.empty(ctx.step_workspace_bytes(batch.P, batch.R, batch.T, wl.d, wl.V, 1024, cfg.dtype),
                     dtype=torch.uint8, device="cuda")
    h = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    loss, counters, metrics = ctx.grpo_step_host(
        cfg, h(st.go), h(st.reward), h(st.cs), h(st.key.view(np.int32)), h(st.alpha), h(st.beta),
        batch.H_t.pin_memory(), h(st.y), h(batch.old), dv["W"], dH2, dW2, ws)
    assert ctx.launch_count() > l0
    assert loss.item() == f["loss"].item()
    assert counters.tolist() == g["counters"].cpu().tolist()
    assert torch.equal(dH2, dH)
    assert TL.rel_l2(dW2.cpu().numpy(), dW.cpu().numpy()) < 1e-5
    assert metrics[7].item() == f["metrics"][3].item()
    assert ctx.last_status() == 0


@pytest.mark.parametrize("config", [1, 2, 3, 4])
def test_full_size_workload_in_bench_configuration(ctx, config):
    """A whole benchmark workload (1: Qwen2.5-Math-1.5B shape, ~283k tokens; 2: Qwen2.5-7B shape,
    ~850k; 3: the AERO-curated ragged batch; 4: the ~4.5M-token stress batch) in the launch
    configuration bench.py times.  The oracle cannot produce all of it, so: the group stage is
    compared in full; 96 sampled token rows are compared one by one (log-prob, lse, g, dH row);
    the loss and sampled rows of dW are checked through identities that hold at any size."""
    wl = synth.WORKLOADS[config]
    st = synth.make_structure(wl)
    P, R, T = len(st.go) - 1, len(st.reward), int(st.cs[-1])
    ocfg = TL.cfg_for(wl)
    cfg = TL.lib_cfg(ocfg, "bf16")
    H, W = synth.make_tensors(wl, T, device="cuda")
    ref_g = O.group_stats(ocfg, st.go, st.reward, st.cs, key=st.key, alpha_in=st.alpha, beta_in=st.beta)
    gi, g = TL.run_group_gpu(ctx, cfg, st)
    TL.check_group(g, ref_g, R, P)

    owner = O.token_rollout(st.cs, T)
    kept_rows = np.nonzero(ref_g["keep"][owner] != 0)[0]
    rng = np.random.default_rng(7)
    sample = np.unique(np.concatenate([kept_rows[:2], kept_rows[-2:], rng.choice(kept_rows, 92, replace=False)]))
    W64 = W.double().cpu().numpy()
    Hs = H[torch.from_numpy(sample).cuda()].double().cpu().numpy()
    zs = O.logits(Hs, W64)
    lp_s, lse_s = O.log_softmax_pick(zs, st.y[sample])
    # old log-probs: model-independent constant for the bulk, oracle log-prob + noise on the sample,
    # with a few large perturbations so that both clip edges are exercised
    old = np.full(T, -12.2, np.float32) + st.noise
    pert = st.noise[sample].astype(np.float64)
    pert[::7] *= 8.0
    old[sample] = (lp_s + pert).astype(np.float32)

    y, cs, oldd = TL.dev(st.y), TL.dev(st.cs), TL.dev(old)
    f = ctx.grpo_loss_fwd(cfg, H, W, y, oldd, cs, g["adv"], g["w"], g["keep"])
    chunk = 4 * 148 * 128
    ws = torch.empty(ctx.bwd_workspace_bytes(T, wl.d, wl.V, R, chunk), dtype=torch.uint8, device="cuda")
    dH, dW = ctx.grpo_loss_bwd(cfg, H, W, y, cs, g["keep"], f["lse"], f["g"], workspace=ws)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0

    # --- sampled rows against the oracle
    adv32 = g["adv"][:R].cpu().numpy().astype(np.float64)
    w32 = g["w"][:R].cpu().numpy().astype(np.float64)
    s_ref, g_ref, rho_ref, ind_ref = O.surrogate(ocfg, lp_s, old[sample].astype(np.float64),
                                                 adv32[owner[sample]], w32[owner[sample]])
    logp = f["logp"][:T].cpu().numpy()
    lse = f["lse"][:T].cpu().numpy()
    gg = f["g"][:T].cpu().numpy()
    assert np.abs(logp[sample] - lp_s).max() <= LOGP_ABS
    assert np.abs(lse[sample] - lse_s).max() <= LOGP_ABS
    edge = (np.abs(rho_ref - 1.2) < 1e-3) | (np.abs(rho_ref - 0.8) < 1e-3)
    np.testing.assert_allclose(gg[sample][~edge], g_ref[~edge], rtol=2e-2, atol=1e-14)
    assert (ind_ref == 0).any() and (ind_ref == 1).any()
    mini_cs = np.arange(len(sample) + 1, dtype=np.int64)
    rdH, _ = O.grpo_loss_bwd(Hs, W64, st.y[sample], mini_cs, np.ones(len(sample), np.uint8), lse_s, g_ref,
                             dw_rows=[0])
    dHs = dH[torch.from_numpy(sample).cuda()].float().cpu().numpy()
    live = (g_ref != 0) & ~edge
    assert TL.rel_l2(dHs[live], rdH[live]) < GRAD_L2
    assert not dHs[(g_ref == 0) & ~edge].any()
    # dropped rows: zero outputs
    dropped = torch.from_numpy(np.nonzero(ref_g["keep"][owner] == 0)[0][::97].copy()).cuda()
    assert not dH[dropped].float().abs().sum().item() and not f["g"][dropped].abs().sum().item()

    # --- identities at full size (test-side arithmetic on the library's outputs)
    kept = ref_g["keep"][owner] != 0
    A_t, w_t = adv32[owner], w32[owner]
    rho = np.exp(logp.astype(np.float64) - old.astype(np.float64))
    surr = np.minimum(rho * A_t, np.clip(rho, 1 - ocfg.clip_lo, 1 + ocfg.clip_hi) * A_t)
    loss_re = -float(np.sum((w_t * surr)[kept]))
    assert abs(f["loss"].item() - loss_re) <= 1e-4 * abs(loss_re) + 1e-8
    assert (logp[kept] <= 1e-6).all() and not logp[~kept].any()
    # columns of dW sum to zero because each row of dz does
    colsum = dW.double().sum(dim=0).abs().max().item()
    assert colsum <= 1e-2 * dW.double().abs().sum(dim=0).max().item()
    # rows of dW from the definition, with the library's own lse and g (fp64 on the device)
    vrows = np.unique(np.concatenate([st.y[kept_rows[:8]], rng.integers(0, wl.V, 24)]))
    vr = torch.from_numpy(vrows).cuda()
    Wv = W[vr].double()
    ref_rows = torch.zeros((len(vrows), wl.d), dtype=torch.float64, device="cuda")
    for a in range(0, T, 1 << 18):                       # row blocks bound the fp64 copies of H
        b = min(T, a + (1 << 18))
        H64 = H[a:b].double()
        dz = -torch.exp(H64 @ Wv.T - f["lse"][a:b].double()[:, None])
        dz += (y[a:b, None] == vr[None, :].to(y.dtype)).double()
        dz *= f["g"][a:b].double()[:, None]
        ref_rows += dz.T @ H64
        del H64, dz
    assert TL.rel_l2(dW[vr].cpu().numpy(), ref_rows.cpu().numpy()) < GRAD_L2
    # a different chunking gives the same dH bits and the same dW up to fp32 summation order
    ws2 = torch.empty(ctx.bwd_workspace_bytes(T, wl.d, wl.V, R, 148 * 128), dtype=torch.uint8, device="cuda")
    dH2, dW2 = ctx.grpo_loss_bwd(cfg, H, W, y, cs, g["keep"], f["lse"], f["g"], workspace=ws2)
    assert torch.equal(dH2, dH)
    assert ((dW2 - dW).double().norm() / dW.double().norm()).item() < 1e-4
    assert ctx.last_status() == 0
    del dH2, dW2, ws2, ws
    torch.cuda.empty_cache()
    # forward and backward in one call, as bench.py times the step: same forward up to rounding, gradients within the
    # tolerance of the two-call path (the stored exponentials are rounded to bf16 before, not after, the scaling)
    # and of the oracle on the sampled rows
    ws3 = torch.empty(ctx.fwd_bwd_workspace_bytes(T, wl.d, wl.V, R, chunk), dtype=torch.uint8, device="cuda")
    f3, dH3, dW3 = ctx.grpo_loss_fwd_bwd(cfg, H, W, y, oldd, cs, g["adv"], g["w"], g["keep"], workspace=ws3)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    # (the two forward modes add the exponentials of a row in a different order)
    assert (f3["logp"][:T] - f["logp"][:T]).abs().max().item() < 2e-5
    assert abs(f3["loss"].item() - f["loss"].item()) <= 1e-5 * abs(f["loss"].item())
    assert np.abs(f3["logp"][:T].cpu().numpy()[sample] - lp_s).max() <= LOGP_ABS
    dHs3 = dH3[torch.from_numpy(sample).cuda()].float().cpu().numpy()
    assert TL.rel_l2(dHs3[live], rdH[live]) < GRAD_L2
    assert not dH3[dropped].float().abs().sum().item()
    num = den = 0.0
    for a in range(0, T, 1 << 18):                       # row blocks bound the fp32 copies
        b = min(T, a + (1 << 18))
        x, x3 = dH[a:b].float(), dH3[a:b].float()
        num += float((x3 - x).pow(2).sum())
        den += float(x.pow(2).sum())
        del x, x3
    assert (num / den) ** 0.5 < GRAD_L2
    assert ((dW3 - dW).double().norm() / dW.double().norm()).item() < GRAD_L2
    assert TL.rel_l2(dW3[vr].cpu().numpy(), ref_rows.cpu().numpy()) < GRAD_L2
