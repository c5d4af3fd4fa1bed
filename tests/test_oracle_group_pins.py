"""Pins for the oracle's group stage: values and closed forms fixed by the paper
and by elementary statistics, plus brute force on small inputs.  CPU only."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import aero_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


def _one_group(n, c, lens=None):
    go = np.array([0, n], dtype=np.int32)
    reward = np.array([1.0] * c + [0.0] * (n - c), dtype=np.float32)
    lens = np.full(n, 5) if lens is None else np.asarray(lens)
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    return go, reward, cs


def test_splitmix64_published_vectors():
    # First outputs of SplitMix64 seeded with 0 (reference implementation by Vigna).
    assert O.default_key(0, 0) == 0xE220A8397B1DCDAF >> 32
    assert O.default_key(0, 1) == 0x6E789E6AA1B965F4 >> 32
    assert O.default_key(0, 2) == 0x06C45D188009454F >> 32


@pytest.mark.parametrize("row", _rows("paper_worked_counts.txt"))
def test_paper_kept_counts(row):
    n, c, k, up, rej, expected = (int(v) for v in row[:6])
    high = int(row[6]) if len(row) > 6 else 0
    cfg = O.Cfg(uniform_policy=up, rejection=rej, k_ratio=k, reject_high=high, seed=7)
    go, reward, cs = _one_group(n, c)
    out = O.group_stats(cfg, go, reward, cs)
    assert int(out["keep"].sum()) == expected
    assert int(out["counters"][0]) == expected
    if 0 < c < n and not high:
        # every correct rollout of a mixed group survives (Sec. 4.2 Strategy 3)
        assert out["keep"][:c].all()
    if 0 < c < n and high and 2 * c >= n:
        # the ablation keeps every incorrect rollout and as many correct ones: advantages are +-1
        assert out["keep"][c:].all() and int(out["keep"][:c].sum()) == min(k * (n - c), c)
        if k == 1 and n - c <= c:
            assert np.allclose(np.abs(out["adv"][out["keep"] != 0]), 1.0, atol=1e-5)


@pytest.mark.parametrize("row", _rows("paper_posterior.txt"))
def test_paper_posterior_mean(row):
    n, c, a0, b0, expected = row
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, alpha0=a0, beta0=b0)
    go, reward, cs = _one_group(int(n), int(c))
    out = O.group_stats(cfg, go, reward, cs)
    assert out["u_tilde"][0] == pytest.approx(expected, rel=1e-14)
    assert out["alpha_out"][0] == a0 + c and out["beta_out"][0] == b0 + n - c
    assert 0.0 < out["u_tilde"][0] < 1.0


def test_posterior_uses_per_prompt_prior_and_all_rollouts():
    # n is counted before the keep-4 subsample; priors are per prompt.
    go = np.array([0, 8, 16], np.int32)
    reward = np.zeros(16, np.float32)
    reward[8:] = 1.0
    cs = np.arange(17, dtype=np.int64) * 3
    out = O.group_stats(O.Cfg(uniform_policy=O.UNIFORM_BAYES), go, reward, cs,
                        alpha_in=[2.0, 0.5], beta_in=[3.0, 1.5])
    assert out["u_tilde"][0] == pytest.approx(2.0 / 13.0)
    assert out["u_tilde"][1] == pytest.approx(8.5 / 10.0)
    assert out["keep"].sum() == 8


@pytest.mark.parametrize("n,c", [(8, 0), (8, 8), (3, 3), (1, 0)])
def test_uniform_group_zero_advantage_under_mask(n, c):
    # Sec. 3.2: identical rewards collapse the advantage to zero.
    go, reward, cs = _one_group(n, c)
    out = O.group_stats(O.Cfg(), go, reward, cs)
    assert not out["adv"].any() and not out["keep"].any() and out["gmask"][0] == 0
    assert not out["w"].any()
    assert out["cat"][0] == (O.CAT_ZERO if c == 0 else O.CAT_PERFECT)


@pytest.mark.parametrize("n,c,k", [(8, 1, 1), (8, 2, 1), (8, 3, 1), (16, 2, 2), (16, 3, 4), (9, 4, 1), (8, 5, 1)])
def test_advantage_closed_form_binary(n, c, k):
    # Proof of Theorem 4.1: mu = c/(c+m), sigma^2 = mu(1-mu), a+ = (1-mu)/sigma, a- = -mu/sigma
    # which simplifies to a+ = sqrt(m/c), a- = -sqrt(c/m).
    cfg = O.Cfg(rejection=1, k_ratio=k, eps_std=0.0, uniform_policy=O.UNIFORM_BAYES)
    go, reward, cs = _one_group(n, c)
    out = O.group_stats(cfg, go, reward, cs)
    low = 2 * c < n
    m = min(k * c, n - c) if low else n - c
    keep = out["keep"].astype(bool)
    assert keep[:c].all() and keep[c:].sum() == m
    a = out["adv"]
    assert np.allclose(a[:c], math.sqrt(m / c), rtol=1e-13)
    assert np.allclose(a[c:][keep[c:]], -math.sqrt(c / m), rtol=1e-13)
    assert not a[~keep].any()
    # standardisation invariants over the surviving subset
    assert abs(a[keep].sum()) < 1e-12
    assert a[keep] @ a[keep] == pytest.approx(c + m, rel=1e-13)
    if k == 1 and low:
        assert np.allclose(np.abs(a[keep]), 1.0)


def test_advantage_matches_numpy_population_std_real_rewards_all_mode():
    # Eq. 1 with the population standard deviation == numpy mean/std with ddof=0.
    rng = np.random.default_rng(0)
    go = np.array([0, 5, 12, 20], np.int32)
    reward = rng.integers(0, 2, 20).astype(np.float32)
    reward[0:5] = [1, 0, 0, 1, 0]
    reward[5:12] = [0, 0, 1, 0, 0, 0, 1]
    reward[12:20] = [1, 1, 1, 0, 1, 1, 0, 1]
    cs = np.arange(21, dtype=np.int64) * 2
    out = O.group_stats(O.Cfg(eps_std=0.0), go, reward, cs)
    for p in range(3):
        r = reward[go[p]:go[p + 1]].astype(np.float64)
        ref = (r - r.mean()) / r.std()
        assert np.allclose(out["adv"][go[p]:go[p + 1]], ref, rtol=1e-13)


def test_stats_all_differs_from_kept_and_matches_full_group():
    cfg = O.Cfg(rejection=1, eps_std=0.0, stats_over=O.STATS_ALL)
    go, reward, cs = _one_group(8, 2)
    out = O.group_stats(cfg, go, reward, cs)
    mu, sd = 0.25, math.sqrt(0.25 * 0.75)
    keep = out["keep"].astype(bool)
    assert keep.sum() == 4
    assert np.allclose(out["adv"][:2], (1 - mu) / sd)
    assert np.allclose(out["adv"][2:][keep[2:]], -mu / sd)


def test_bayes_advantage_for_uniform_groups_reading():
    # Reading taken where the paper is silent: denominator sqrt(u~(1-u~)).
    # Flat prior, n = 8: u~ = 0.1 / 0.9 -> advantage -1/3 (all wrong) / +1/3 (all right).
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, eps_std=0.0)
    for c, expect in [(0, -1.0 / 3.0), (8, 1.0 / 3.0)]:
        go, reward, cs = _one_group(8, c)
        out = O.group_stats(cfg, go, reward, cs)
        keep = out["keep"].astype(bool)
        assert keep.sum() == 4
        assert np.allclose(out["adv"][keep], expect, rtol=1e-13)
        assert (out["adv"][keep] != 0).all()      # "guaranteeing a non-zero advantage"


def test_categories_integer_thresholds():
    # Appendix C: Zero c=0; Partial 0<c/n<0.5; Good 0.5<=c/n<1; Perfect c=n.
    for n in range(1, 13):
        for c in range(n + 1):
            go, reward, cs = _one_group(n, c)
            cat = O.group_stats(O.Cfg(), go, reward, cs)["cat"][0]
            u = c / n
            want = (O.CAT_ZERO if c == 0 else O.CAT_PERFECT if c == n
                    else O.CAT_PARTIAL if u < 0.5 else O.CAT_GOOD)
            assert cat == want, (n, c)


def test_keep_mask_is_the_m_smallest_keys_brute_force():
    # Brute force: an incorrect rollout is kept iff fewer than m incorrect rollouts
    # precede it in (key, index) order -- counted, not sorted.
    rng = np.random.default_rng(3)
    for trial in range(40):
        n = int(rng.integers(2, 20))
        c = int(rng.integers(1, max(2, n // 2)))
        reward = np.zeros(n, np.float32)
        reward[rng.permutation(n)[:c]] = 1.0
        key = rng.integers(0, 4, n).astype(np.uint32)      # many ties -> index tie-break matters
        go = np.array([0, n], np.int32)
        cs = np.arange(n + 1, dtype=np.int64)
        cfg = O.Cfg(rejection=1, k_ratio=int(rng.integers(1, 4)), uniform_policy=O.UNIFORM_BAYES)
        out = O.group_stats(cfg, go, reward, cs, key=key)
        low = 2 * c < n
        m = min(cfg.k_ratio * c, n - c) if low else n - c
        for i in range(n):
            if reward[i] > 0.5:
                assert out["keep"][i] == 1
            else:
                before = sum(1 for j in range(n) if reward[j] < 0.5 and
                             (key[j] < key[i] or (key[j] == key[i] and j < i)))
                assert out["keep"][i] == (1 if before < m else 0)


def test_default_key_used_when_no_key_given():
    n = 12
    go, reward, cs = _one_group(n, 0)
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, seed=123)
    out = O.group_stats(cfg, go, reward, cs)
    keys = [O.default_key(123, i) for i in range(n)]
    expect = set(sorted(range(n), key=lambda i: (keys[i], i))[:4])
    assert set(np.nonzero(out["keep"])[0]) == expect


def test_keep_in_removes_rollouts_before_counting():
    go = np.array([0, 8], np.int32)
    reward = np.array([1, 1, 0, 0, 0, 0, 0, 0], np.float32)
    cs = np.arange(9, dtype=np.int64) * 4
    keep_in = np.array([1, 0, 1, 1, 0, 0, 1, 1], np.uint8)   # present: 1 correct, 4 wrong
    out = O.group_stats(O.Cfg(rejection=1, uniform_policy=O.UNIFORM_BAYES), go, reward, cs, keep_in=keep_in)
    assert out["keep"][1] == 0 and out["keep"][0] == 1
    assert out["keep"].sum() == 2 and not (out["keep"] & (1 - keep_in)).any()
    assert out["beta_out"][0] == 1 + 4


def test_weights_and_offsets():
    go = np.array([0, 4, 8, 12], np.int32)
    reward = np.array([1, 0, 0, 0, 0, 0, 0, 0, 1, 1, 0, 1], np.float32)
    lens = np.array([3, 5, 7, 2, 4, 4, 4, 4, 6, 1, 9, 2])
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    # token mean over kept tokens
    out = O.group_stats(O.Cfg(), go, reward, cs)
    keep = out["keep"].astype(bool)
    assert list(keep) == [True] * 4 + [False] * 4 + [True] * 4
    T_kept = lens[keep].sum()
    assert np.allclose(out["w"][keep], 1.0 / T_kept) and not out["w"][~keep].any()
    assert (out["w"] * lens).sum() == pytest.approx(1.0)
    assert list(out["kept_ids"]) == [0, 1, 2, 3, 8, 9, 10, 11]
    assert list(out["kept_tok_off"][:9]) == list(np.concatenate([[0], np.cumsum(lens[keep])]))
    assert out["counters"][0] == 8 and out["counters"][1] == T_kept and out["counters"][2] == 2
    assert out["counters"][7] == lens.sum()
    # Eq. 2: 1/N sum_i 1/|o_i| sum_t, averaged over surviving prompts
    out = O.group_stats(O.Cfg(agg=O.AGG_SEQ_MEAN), go, reward, cs)
    assert np.allclose(out["w"][keep], 1.0 / (2 * 4 * lens[keep]))
    assert (out["w"] * lens).sum() == pytest.approx(1.0)
    # counting masked prompts in the denominator shrinks the batch gradient (Sec. 3.1)
    out = O.group_stats(O.Cfg(agg=O.AGG_SEQ_MEAN, denom=O.DENOM_ALL), go, reward, cs)
    assert (out["w"] * lens).sum() == pytest.approx(2.0 / 3.0)
    out = O.group_stats(O.Cfg(denom=O.DENOM_ALL), go, reward, cs)
    assert (out["w"] * lens).sum() == pytest.approx(T_kept / lens.sum())


def test_zero_accuracy_ratio_metric():
    # x^zero = (# prompts with all rewards 0)/P   (Sec. 3.2)
    go = np.array([0, 2, 4, 6, 8], np.int32)
    reward = np.array([0, 0, 1, 0, 0, 0, 1, 1], np.float32)
    cs = np.arange(9, dtype=np.int64)
    out = O.group_stats(O.Cfg(), go, reward, cs)
    assert out["metrics"][0] == pytest.approx(0.5)
    assert list(out["counters"][3:7]) == [2, 0, 1, 1]


def test_group_metrics_hand_values():
    # Three prompts with token lengths chosen by hand; AERO curation with k = 1, Bayesian uniform groups keep 2.
    #   prompt 0: rewards 1 0 0 0 (lengths 2 4 6 8), keys put rollout 3 first among the incorrect ones
    #             -> keep rollouts 0 and 3, advantages +1 and -1
    #   prompt 1: rewards 0 0 0 (lengths 1 1 1), flat prior -> u~ = 1/5, keep the two smallest keys (1 and 2),
    #             advantage (0 - 0.2)/sqrt(0.2 * 0.8) = -0.5 each
    #   prompt 2: rewards 1 1 0 (lengths 3 3 3): c = 2 of 3 is not low-success -> keep all;
    #             mean 2/3, population std sqrt(2)/3 -> advantages +1/sqrt(2), +1/sqrt(2), -sqrt(2)
    go = np.array([0, 4, 7, 10], np.int32)
    reward = np.array([1, 0, 0, 0, 0, 0, 0, 1, 1, 0], np.float32)
    lens = np.array([2, 4, 6, 8, 1, 1, 1, 3, 3, 3])
    cs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    key = np.array([9, 7, 8, 1, 5, 2, 3, 0, 0, 0], np.uint32)
    cfg = O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, n_keep_uniform=2, eps_std=0.0)
    out = O.group_stats(cfg, go, reward, cs, key=key)
    assert list(out["keep"]) == [1, 0, 0, 1, 0, 1, 1, 1, 1, 1]
    abs_adv = [1.0, 1.0, 0.5, 0.5, 1 / math.sqrt(2), 1 / math.sqrt(2), math.sqrt(2)]
    assert out["metrics"][1] == pytest.approx(sum(abs_adv) / 7, rel=1e-12)       # mean |advantage| over kept rollouts
    assert out["metrics"][2] == pytest.approx(7 / 10, rel=1e-12)                 # kept rollouts / present rollouts
    assert out["metrics"][3] == pytest.approx((2 + 8 + 1 + 1 + 9) / 32, rel=1e-12)   # kept tokens / present tokens
    assert out["metrics"][0] == pytest.approx(1 / 3)
    # absent rollouts leave the denominators of both fractions
    keep_in = np.array([1, 1, 1, 1, 1, 1, 1, 1, 1, 0], np.uint8)                 # prompt 2 becomes all-correct
    out = O.group_stats(cfg, go, reward, cs, key=key, keep_in=keep_in)
    assert int(out["keep"].sum()) == 6
    assert out["metrics"][2] == pytest.approx(6 / 9, rel=1e-12)
    assert out["metrics"][3] == pytest.approx((2 + 8 + 1 + 1 + 6) / 29, rel=1e-12)


def test_balance_factor_lemma():
    # Lemma 4.2: c*m/(c+m)^2 is maximal iff m = c; it equals the variance of the kept group.
    for c in range(1, 6):
        vals = {m: c * m / (c + m) ** 2 for m in range(1, 4 * c + 1)}
        assert max(vals, key=vals.get) == c
        go, reward, cs = _one_group(c + 4 * c, c)
        out = O.group_stats(O.Cfg(rejection=1, eps_std=0.0), go, reward, cs)
        keep = out["keep"].astype(bool)
        r = reward[keep].astype(np.float64)
        assert r.var() == pytest.approx(0.25)          # k = 1 -> m = c -> the maximum 1/4


def test_rescue_threshold_extends_low_set():
    # S > 0: groups with c/n <= S/n_explore are curated like low-success ones (Strategy 1/Alg. 1).
    go, reward, cs = _one_group(8, 4)                 # u = 0.5 -> Good, normally keep all
    out = O.group_stats(O.Cfg(rejection=1), go, reward, cs)
    assert out["keep"].sum() == 8
    out = O.group_stats(O.Cfg(rejection=1, rescue_S=4, n_explore=8), go, reward, cs)
    assert out["keep"].sum() == 8                     # m = min(4, 4): still all
    go, reward, cs = _one_group(10, 5)
    out = O.group_stats(O.Cfg(rejection=1, rescue_S=4, n_explore=8, k_ratio=1), go, reward, cs)
    assert out["keep"].sum() == 10


def test_rescue_threshold_decides_between_the_two_rejection_rules():
    # For k >= 1 a group with 2c >= n keeps all its incorrect rollouts under the low-success rule anyway
    # (m = min(k c, n - c) = n - c), so the threshold S can only matter where another rule would apply
    # instead: with the high-success down-sampling on, a group of 5 correct / 3 incorrect is cut to 3 + 3,
    # unless S puts it into the low-success set (5 * 8 <= 5 * 8), where it keeps all 8.
    go, reward, cs = _one_group(8, 5)
    cut = O.group_stats(O.Cfg(rejection=1, reject_high=1, rescue_S=4, n_explore=8), go, reward, cs)
    assert cut["keep"].sum() == 6                     # 5 * 8 > 4 * 8: not in the low-success set
    low = O.group_stats(O.Cfg(rejection=1, reject_high=1, rescue_S=5, n_explore=8), go, reward, cs)
    assert low["keep"].sum() == 8
    # inside the range the paper gives (S <= n_explore / 2) the threshold adds only groups with u = 1/2 exactly
    go, reward, cs = _one_group(8, 4)
    at_half = O.group_stats(O.Cfg(rejection=1, reject_high=1, rescue_S=4, n_explore=8), go, reward, cs)
    assert at_half["keep"].sum() == 8


def test_empty_group_and_empty_batch():
    go = np.array([0, 0, 3], np.int32)
    reward = np.array([1, 0, 0], np.float32)
    cs = np.array([0, 2, 4, 6], np.int64)
    out = O.group_stats(O.Cfg(), go, reward, cs)
    assert out["cat"][0] == O.CAT_EMPTY and out["gmask"][0] == 0 and out["gmask"][1] == 1
    assert out["u_tilde"][0] == pytest.approx(0.5)
    out = O.group_stats(O.Cfg(), np.array([0], np.int32), np.zeros(0, np.float32), np.array([0], np.int64))
    assert out["counters"][0] == 0 and out["counters"][1] == 0


def test_high_success_downsampling_brute_force():
    """reject_high: which correct rollouts survive, by counting predecessors in (key, index) order;
    low-success groups and uniform groups are untouched by the switch."""
    rng = np.random.default_rng(11)
    for _ in range(40):
        n = int(rng.integers(2, 14))
        c = int(rng.integers(0, n + 1))
        reward = np.zeros(n, np.float32)
        reward[rng.permutation(n)[:c]] = 1.0
        key = rng.integers(0, 5, n).astype(np.uint32)          # few distinct keys: ties by index matter
        go = np.array([0, n], np.int32)
        cs = np.arange(n + 1, dtype=np.int64) * 2
        k = int(rng.integers(1, 3))
        base = O.group_stats(O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, k_ratio=k), go, reward, cs, key=key)
        out = O.group_stats(O.Cfg(uniform_policy=O.UNIFORM_BAYES, rejection=1, k_ratio=k, reject_high=1), go, reward,
                            cs, key=key)
        if c == 0 or c == n or 2 * c < n:
            assert np.array_equal(out["keep"], base["keep"])
            continue
        m = min(k * (n - c), c)
        for i in range(n):
            if reward[i] < 0.5:
                assert out["keep"][i] == 1            # every incorrect rollout stays
            else:
                # counted, not sorted: kept iff fewer than m correct rollouts precede it in (key, index) order
                before = sum(1 for j in range(n) if reward[j] > 0.5 and
                             (key[j] < key[i] or (key[j] == key[i] and j < i)))
                assert out["keep"][i] == (1 if before < m else 0)
