"""Pins for the oracle's allocation-controller simulation: hand cases, closed forms of the
geometric rescue process, invariants of the budget rules, and consistency of the curated
sizes with the (separately pinned) group stage.  CPU only."""
import numpy as np

from oracle import aero_oracle as O

FULL = 2 ** 32 - 1


def _thr(u):
    return np.minimum(np.floor(np.asarray(u, np.float64) * 2 ** 32), FULL).astype(np.uint64)


def test_never_and_always_correct_prompts():
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, seed=1)
    a = O.AllocCfg(n_budget=40)                       # budget never binds: 8 + 10 * 2 = 28 <= 32
    out = O.allocate_sim(cfg, a, np.zeros(5, np.uint64))
    assert (out["n_gen"] == 28).all() and not out["c"].any() and (out["n_train"] == 4).all()
    assert out["counters"].tolist() == [140, 20, 5, 5, 0, 10, 60, 5]
    out = O.allocate_sim(cfg, a, np.full(5, FULL + 1, np.uint64))     # every draw succeeds
    assert (out["n_gen"] == 8).all() and (out["c"] == 8).all() and (out["n_train"] == 4).all()
    assert out["counters"][5] == 0
    # per-prompt cap: n_max = 11 allows one full increment and one of a single rollout
    out = O.allocate_sim(cfg, O.AllocCfg(n_budget=40, n_max=11), np.zeros(3, np.uint64))
    assert (out["n_gen"] == 11).all()
    # plain GRPO masking: uniform groups train on nothing
    out = O.allocate_sim(O.Cfg(seed=1), a, np.zeros(3, np.uint64))
    assert not out["n_train"].any()


def test_short_budget_is_granted_in_prompt_order():
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, n_explore=8)
    # 3 prompts, budget 9 per prompt: 3 rollouts left after exploration; increments of 2
    out = O.allocate_sim(cfg, O.AllocCfg(n_budget=9), np.zeros(3, np.uint64))
    assert out["n_gen"].tolist() == [10, 8, 8]        # only the first request fits; then 1 < 2 is left
    assert out["counters"][5] == 1 and out["counters"][6] == 1


def test_rescued_prompt_trains_on_one_correct_one_incorrect():
    # Sec. 4.4: a rescued query yields a group of 2 (one correct, one incorrect)
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1)
    for n in (10, 12, 28):
        assert O.curated_size(cfg, n, 1) == 2
    assert O.curated_size(cfg, 16, 0) == 4 and O.curated_size(cfg, 16, 16) == 4      # Strategy 2
    assert O.curated_size(cfg, 8, 5) == 8                                             # high accuracy keeps all
    assert O.curated_size(O.Cfg(rejection=1, reject_high=1), 8, 5) == 6               # appendix ablation: 3 + 3


def test_curated_size_equals_group_stage_keep_count():
    rng = np.random.default_rng(2)
    for _ in range(200):
        n = int(rng.integers(1, 20))
        c = int(rng.integers(0, n + 1))
        cfg = O.Cfg(uniform_policy=int(rng.integers(0, 2)), rejection=int(rng.integers(0, 2)),
                    k_ratio=int(rng.integers(1, 4)), reject_high=int(rng.integers(0, 2)),
                    rescue_S=int(rng.integers(0, 3)), n_keep_uniform=int(rng.integers(0, 6)))
        reward = np.array([1.0] * c + [0.0] * (n - c), np.float32)
        g = O.group_stats(cfg, np.array([0, n], np.int32), reward, np.arange(n + 1, dtype=np.int64))
        assert int(g["keep"].sum()) == O.curated_size(cfg, n, c)


def test_invariants_and_early_exit():
    rng = np.random.default_rng(3)
    u = rng.beta(0.5, 0.5, 600)
    thr = _thr(u)
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, seed=17)
    a = O.AllocCfg()
    out = O.allocate_sim(cfg, a, thr)
    n, c, nt = out["n_gen"], out["c"], out["n_train"]
    assert (n >= cfg.n_explore).all() and (n <= a.n_max).all() and n.sum() <= a.n_budget * len(u)
    assert (nt <= n).all() and (c <= n).all()
    assert out["counters"][0] == n.sum() and out["counters"][1] == nt.sum()
    for p in np.nonzero(n > cfg.n_explore)[0]:
        draws = [O.default_key(cfg.seed, int(p) * a.n_max + j) < int(thr[p]) for j in range(int(n[p]))]
        assert not any(draws[:int(n[p]) - a.n_extra])              # nothing correct before the last increment
        assert sum(draws) == c[p]
    assert out["counters"][4] == ((n > cfg.n_explore) & (c > 0)).sum()


def test_rates_match_the_geometric_closed_forms():
    # all prompts share u: zero after exploration with probability (1-u)^8; a zero prompt is rescued
    # within 10 increments of 2 with probability 1 - (1-u)^20; the budget (16 per prompt) does not bind
    u, P = 0.15, 6000
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, seed=23)
    out = O.allocate_sim(cfg, O.AllocCfg(), _thr(np.full(P, u)))
    p0 = (1 - u) ** 8
    zero_before, zero_after, rescued = (int(v) for v in out["counters"][2:5])
    assert abs(zero_before / P - p0) < 4 * np.sqrt(p0 * (1 - p0) / P)
    pr = 1 - (1 - u) ** 20
    assert abs(rescued / zero_before - pr) < 4 * np.sqrt(pr * (1 - pr) / zero_before)
    assert zero_after == zero_before - rescued
    # expected extra rollouts of a zero prompt: 2 * sum_{i<10} (1-u)^(2i)
    extra = (int(out["n_gen"].sum()) - 8 * P) / zero_before
    q = (1 - u) ** 2
    assert abs(extra - 2 * (1 - q ** 10) / (1 - q)) < 0.25
