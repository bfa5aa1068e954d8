"""Pins of the oracle's pool z-score variant of phase 2 (a variant of this library, absent
from the paper): what z-scoring fixes by definition, a worked example and scipy's zscore."""
import numpy as np
import pytest
from scipy import stats

import oracle


def _pool(rng, n, k1, n_bank=500):
    ids = np.full(k1, -1, np.int32)
    ids[:n] = rng.choice(n_bank, size=n, replace=False)
    sims = np.full(k1, -np.inf)
    sims[:n] = np.sort(rng.normal(0.0, 0.05, n))[::-1]
    q = rng.random(n_bank).astype(np.float32)
    return ids, sims, q


def test_worked_example():
    # sims 3, 2, 1: mean 2, population std sqrt(2/3); values 0, 1, 1/2: mean 1/2, std sqrt(1/6)
    ids = np.array([0, 1, 2], np.int32)
    sims = np.array([3.0, 2.0, 1.0])
    q = np.array([0.0, 1.0, 0.5], np.float32)
    r = np.sqrt(1.5)                                  # z-scores: +r, 0, -r and -r, +r, 0
    got_ids, got_sc = oracle.phase2(ids, sims, q, 0.5, 3, zscore=True)
    assert got_ids[0].tolist() == [1, 0, 2]
    np.testing.assert_allclose(got_sc[0], [0.5 * r, 0.0, -0.5 * r], rtol=0, atol=1e-15)
    got_ids, got_sc = oracle.phase2(ids, sims, q, 0.25, 3, zscore=True)
    np.testing.assert_allclose(sorted(got_sc[0]), sorted([0.75 * r - 0.25 * r, 0.25 * r, -0.75 * r]), atol=1e-15)


@pytest.mark.parametrize("w", [0.0, 0.3, 0.5, 1.0])
def test_against_scipy_zscore(w):
    rng = np.random.default_rng(3)
    for n, k1 in [(64, 64), (17, 32), (2, 8)]:
        ids, sims, q = _pool(rng, n, k1)
        want = (1 - w) * stats.zscore(sims[:n], ddof=0) + w * stats.zscore(q[ids[:n]].astype(np.float64), ddof=0)
        order = sorted(range(n), key=lambda i: (-want[i], -sims[i], ids[i]))
        got_ids, got_sc = oracle.phase2(ids, sims, q, w, k1, zscore=True)
        assert got_ids[0, :n].tolist() == [int(ids[i]) for i in order]
        np.testing.assert_allclose(got_sc[0, :n], want[order], rtol=1e-12, atol=1e-12)
        assert np.all(got_ids[0, n:] == -1) and np.all(np.isneginf(got_sc[0, n:]))


def test_zero_mean_unit_variance_and_special_weights():
    rng = np.random.default_rng(4)
    ids, sims, q = _pool(rng, 48, 48)
    for w in (0.0, 1.0):
        _, sc = oracle.phase2(ids, sims, q, w, 48, zscore=True)
        assert abs(sc[0].mean()) < 1e-12 and abs(sc[0].var() - 1.0) < 1e-12
    # w = 0 keeps the similarity order, w = 1 is the paper's rule: the pool ranked by Q alone
    assert oracle.phase2(ids, sims, q, 0.0, 8, zscore=True)[0].tolist() == oracle.phase2(ids, sims, q, 0.0, 8)[0].tolist()
    assert oracle.phase2(ids, sims, q, 1.0, 8, zscore=True)[0].tolist() == oracle.phase2(ids, sims, q, 1.0, 8)[0].tolist()


def test_invariant_under_positive_affine_change_of_values():
    rng = np.random.default_rng(5)
    ids, sims, _ = _pool(rng, 40, 40)
    q = (rng.integers(0, 64, 500) / 64.0).astype(np.float32)      # few mantissa bits: 4 q + 1/2 is exact
    a_ids, a_sc = oracle.phase2(ids, sims, q, 0.4, 40, zscore=True)
    b_ids, b_sc = oracle.phase2(ids, sims, (4.0 * q + 0.5).astype(np.float32), 0.4, 40, zscore=True)
    assert a_ids.tolist() == b_ids.tolist()
    np.testing.assert_allclose(a_sc, b_sc, rtol=1e-12, atol=1e-12)
    # the raw mix is not invariant: the same change reorders it
    assert oracle.phase2(ids, sims, q, 0.4, 40)[0].tolist() != \
        oracle.phase2(ids, sims, (4.0 * q + 0.5).astype(np.float32), 0.4, 40)[0].tolist()


def test_constant_column_counts_as_zero():
    rng = np.random.default_rng(6)
    ids, sims, _ = _pool(rng, 30, 32)
    q = np.full(500, 0.25, np.float32)
    got_ids, got_sc = oracle.phase2(ids, sims, q, 0.5, 32, zscore=True)
    assert got_ids[0, :30].tolist() == ids[:30].tolist()            # similarity order (the pool's own)
    np.testing.assert_allclose(got_sc[0, :30], 0.5 * stats.zscore(sims[:30]), rtol=1e-12)
    # one entry: both columns constant
    one_ids, one_sc = oracle.phase2(ids[:1], sims[:1], q, 0.5, 4, zscore=True)
    assert one_ids[0].tolist() == [int(ids[0]), -1, -1, -1] and one_sc[0, 0] == 0.0


def test_explore_with_zscores_draws_the_same_entries():
    rng = np.random.default_rng(7)
    ids, sims, q = _pool(rng, 24, 24)
    raw = oracle.explore(ids, sims, q, 0.5, 6, 1.0, seed=11, step=3)
    zs = oracle.explore(ids, sims, q, 0.5, 6, 1.0, seed=11, step=3, zscore=True)
    assert raw[2].all() and zs[2].all() and raw[0].tolist() == zs[0].tolist()
    full_ids, full_sc = oracle.phase2(ids, sims, q, 0.5, 24, zscore=True)
    score_of = dict(zip(full_ids[0].tolist(), full_sc[0].tolist()))
    np.testing.assert_allclose(zs[1][0], [score_of[i] for i in zs[0][0].tolist()], rtol=1e-12, atol=1e-15)
    greedy = oracle.explore(ids, sims, q, 0.5, 6, 0.0, seed=11, step=3, zscore=True)
    assert greedy[0].tolist() == full_ids[:, :6].tolist()
