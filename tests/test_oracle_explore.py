"""Pins for the exploration side of the CPU oracle: the counter-based generator against
its published known answers, and the epsilon-greedy choice against its special cases and
the statistics of uniform sampling without replacement."""
import numpy as np

import oracle


def test_philox_known_answers():
    # known-answer vectors distributed with the reference implementation of Philox4x32-10
    cases = [
        ([0, 0, 0, 0], [0, 0], [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]),
        ([0xffffffff] * 4, [0xffffffff] * 2, [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]),
        ([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], [0xa4093822, 0x299f31d0],
         [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]),
    ]
    for ctr, key, want in cases:
        assert oracle.philox4x32_10(ctr, key).tolist() == want


def _pools(rng, b, k1, n, n_valid=None):
    ids = np.stack([rng.permutation(n)[:k1] for _ in range(b)]).astype(np.int32)
    sims = -np.sort(-rng.random((b, k1)), axis=1)
    if n_valid is not None:
        ids[:, n_valid:] = -1
        sims[:, n_valid:] = -np.inf
    return ids, sims, rng.random(n).astype(np.float32)


def test_epsilon_zero_is_greedy_and_one_always_explores():
    rng = np.random.default_rng(0)
    ids, sims, q = _pools(rng, 50, 32, 400)
    g_ids, g_sc = oracle.phase2(ids, sims, q, 0.7, 6)
    e_ids, e_sc, ex = oracle.explore(ids, sims, q, 0.7, 6, 0.0, seed=5, step=9)
    assert not ex.any() and np.array_equal(e_ids, g_ids) and np.array_equal(e_sc, g_sc)
    e_ids, e_sc, ex = oracle.explore(ids, sims, q, 0.7, 6, 1.0, seed=5, step=9)
    assert ex.all()
    for b in range(50):
        assert len(set(e_ids[b].tolist())) == 6 and set(e_ids[b].tolist()) <= set(ids[b].tolist())
        pos = {int(i): j for j, i in enumerate(ids[b])}
        for i, s in zip(e_ids[b], e_sc[b]):
            assert s == (1 - 0.7) * sims[b, pos[int(i)]] + 0.7 * float(q[i])
    # reproducible in (seed, step, query); different steps give different draws
    again = oracle.explore(ids, sims, q, 0.7, 6, 1.0, seed=5, step=9)
    assert np.array_equal(again[0], e_ids)
    other = oracle.explore(ids, sims, q, 0.7, 6, 1.0, seed=5, step=10)
    assert not np.array_equal(other[0], e_ids)
    # a query's draw depends on its global index, not on the batch it arrives in
    tail = oracle.explore(ids[20:], sims[20:], q, 0.7, 6, 1.0, seed=5, step=9, first_query=20)
    assert np.array_equal(tail[0], e_ids[20:])


def test_exploration_rate_and_uniformity():
    rng = np.random.default_rng(1)
    b, k1, k2 = 20000, 16, 4
    ids1, sims1, q = _pools(rng, 1, k1, 100)
    ids, sims = np.repeat(ids1, b, axis=0), np.repeat(sims1, b, axis=0)
    _, _, ex = oracle.explore(ids, sims, q, 0.5, k2, 0.3, seed=11, step=0)
    assert abs(ex.mean() - 0.3) < 4 * (0.3 * 0.7 / b) ** 0.5
    e_ids, _, ex = oracle.explore(ids, sims, q, 0.5, k2, 1.0, seed=11, step=0)
    # every pool entry is equally likely in every draw slot: chi-square over 16 cells, 15 dof
    for slot in range(k2):
        counts = np.array([(e_ids[:, slot] == i).sum() for i in ids1[0]])
        chi2 = ((counts - b / k1) ** 2 / (b / k1)).sum()
        assert chi2 < 45.0          # P(chi2_15 > 45) < 1e-4
    # and pairs of slots never repeat an entry
    assert all(len(set(r.tolist())) == k2 for r in e_ids[:2000])


def test_short_pools_and_padding():
    rng = np.random.default_rng(2)
    ids, sims, q = _pools(rng, 8, 12, 60, n_valid=3)
    e_ids, e_sc, ex = oracle.explore(ids, sims, q, 0.5, 5, 1.0, seed=1, step=1)
    assert ex.all()
    for b in range(8):
        assert sorted(e_ids[b, :3].tolist()) == sorted(ids[b, :3].tolist())      # a permutation of the 3
        assert e_ids[b, 3:].tolist() == [-1, -1] and np.all(np.isneginf(e_sc[b, 3:]))
    ids[:, :] = -1
    e_ids, _, ex = oracle.explore(ids, sims, q, 0.5, 5, 1.0, seed=1, step=1)
    assert not ex.any() and np.all(e_ids == -1)
