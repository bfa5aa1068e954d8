"""Pins for the reward side of the CPU oracle: Eq. 5, Eq. 6 and the running
normalisation of Appendix A, against identities, exact rational arithmetic, the
appendix's bounds and its convergence lemma."""
from fractions import Fraction

import numpy as np

import oracle


def test_draft_reward_is_plus_minus_one():
    f = np.array([1, 0, 0, 1, 1], np.uint8)
    assert oracle.reward_draft(f).tolist() == [1.0, -1.0, -1.0, 1.0, 1.0]


def test_refine_reward_closed_form_and_range():
    # tanh(log rho) = (rho^2 - 1) / (rho^2 + 1); with rational rho the right side is exact
    best = np.array([2, 1, 3, 1, 5, 1, 7], np.float32)
    lat = np.array([1, 2, 1, 1, 4, 8, 7], np.float32)
    got = oracle.reward_refine(best, lat, np.ones(7, np.uint8))
    for g, b, l in zip(got, best, lat):
        rho = Fraction(int(b), int(l))
        want = (rho * rho - 1) / (rho * rho + 1)
        assert abs(g - float(want)) < 1e-15
    assert got[3] == 0.0 and got[0] == -got[1]          # no change -> 0; antisymmetric in log rho
    # corollary: every feasible reward lies strictly inside (-1, 1); infeasible is exactly -1
    rng = np.random.default_rng(0)
    b = rng.lognormal(0, 1, 5000).astype(np.float32)
    l = rng.lognormal(0, 1, 5000).astype(np.float32)
    feas = (rng.random(5000) < 0.7).astype(np.uint8)
    r = oracle.reward_refine(b, l, feas)
    ok = feas == 1
    assert np.all(r[~ok] == -1.0)
    assert np.all(np.abs(r[ok]) < 1.0)
    assert np.all((r[ok] > 0) == (b[ok] > l[ok]))         # positive exactly when the kernel got faster
    # a faster kernel earns more: monotone in the speed-up
    l2 = np.sort(rng.lognormal(0, 1, 100).astype(np.float32))
    r2 = oracle.reward_refine(np.ones(100, np.float32), l2, np.ones(100, np.uint8))
    assert np.all(np.diff(r2) <= 0)


def test_normalize_exact_small_sequence():
    # raw = 1/2, -1/2, 1/4, 1: the first two pass through; then mu_2 = 0, sigma_2 = 1/2;
    # mu_3 = 1/12, sigma_3^2 = (1/4 + 1/4 + 1/16)/3 - 1/144 = 13/72
    raw = np.array([0.5, -0.5, 0.25, 1.0], np.float32)
    got = oracle.reward_normalize([], raw, 1e-3)
    assert got[0] == 0.5 and got[1] == -0.5 and got[2] == 0.5
    want3 = float(1 - Fraction(1, 12)) / float(Fraction(13, 72)) ** 0.5
    assert abs(got[3] - want3) < 1e-14


def test_normalize_uses_statistics_before_each_reward_and_splits_cleanly():
    rng = np.random.default_rng(1)
    raw = np.tanh(rng.standard_normal(300)).astype(np.float32)
    whole = oracle.reward_normalize([], raw, 0.05)
    # numpy's own mean / population std over the prefix, independent of the oracle's loops
    for t in (2, 3, 57, 299):
        mu, sd = raw[:t].astype(np.float64).mean(), raw[:t].astype(np.float64).std()
        assert abs(whole[t] - (float(raw[t]) - mu) / max(sd, 0.05)) < 1e-12
    for cut in (0, 1, 2, 150):
        a = oracle.reward_normalize([], raw[:cut], 0.05)
        b = oracle.reward_normalize(raw[:cut].astype(np.float64), raw[cut:], 0.05)
        np.testing.assert_allclose(np.concatenate([a, b]), whole, rtol=0, atol=1e-13)


def test_normalize_bounds_of_the_appendix():
    # rewards in (-1, 1): a variance floor bounds |R_t| by 2 / sigma_min; clipping bounds it by B
    rng = np.random.default_rng(2)
    raw = np.where(rng.random(400) < 0.9, 0.3, np.tanh(rng.standard_normal(400))).astype(np.float32)
    for smin in (0.5, 0.1):
        r = oracle.reward_normalize([], raw, smin)
        assert np.max(np.abs(r[2:])) <= 2.0 / smin
    r = oracle.reward_normalize([], raw, 1e-6, clip=3.0)
    assert np.max(np.abs(r)) <= 3.0
    # a constant stream has sigma = 0: the floor keeps the output finite (and zero)
    r = oracle.reward_normalize([], np.full(50, 0.25, np.float32), 0.1)
    assert np.all(np.isfinite(r)) and np.all(r[2:] == 0.0)


def test_normalize_converges_to_the_stationary_map():
    # lemma: with i.i.d. input, (r - mu_t) / sigma_t -> (r - mu) / sigma
    rng = np.random.default_rng(3)
    mu, sigma = 0.2, 0.3
    raw = (mu + sigma * rng.standard_normal(3000)).astype(np.float32)
    r = oracle.reward_normalize([], raw, 1e-3)
    tail = slice(2500, 3000)
    want = (raw[tail].astype(np.float64) - mu) / sigma
    assert np.max(np.abs(r[tail] - want)) < 0.12
    assert abs(r[tail].mean()) < 0.15 and abs(r[tail].std() - 1) < 0.1
