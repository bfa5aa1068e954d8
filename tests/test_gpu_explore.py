"""Epsilon-greedy retrieval on the GPU against the CPU oracle: the draws come from the
same counter-based generator on both sides, so the chosen ids must be identical."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def evk():
    from paper_2603_10846_b200 import evk as _evk
    return _evk


def _bank(evk, n, d, seed):
    bank = synth.gaussian_unit(n, d, seed, DEV)
    q_tab = np.random.default_rng(seed).random((2, n)).astype(np.float32)
    mem = evk.evk_mem_create(d, n)
    evk.evk_mem_insert(mem, bank)
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(DEV))
    return mem, q_tab


@pytest.mark.parametrize("eps", [0.0, 0.35, 1.0])
def test_explore_matches_oracle_draws(evk, eps):
    n, d, b, k1, k2, w = 30000, 256, 300, 48, 6, 0.5
    mem, q_tab = _bank(evk, n, d, 7)
    queries = synth.gaussian_unit(b, d, 8, DEV)
    greedy = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 1, k1, k2, w, return_pool=True)]
    for step in (0, 1, 2 ** 40 + 3):
        out = evk.evk_retrieve_explore(mem, queries, 1, k1, k2, w, eps, seed=0xABCDEF0123, step=step,
                                       return_pool=True)
        ids, scores, explored, pool_ids, pool_sims = [x.cpu().numpy() for x in out]
        assert evk.evk_last_status(mem) == 0
        assert np.array_equal(pool_ids, greedy[2]) and np.array_equal(pool_sims, greedy[3])
        o_ids, o_sc, o_ex = oracle.explore(pool_ids, pool_sims.astype(np.float64), q_tab[1], w, k2, eps,
                                           seed=0xABCDEF0123, step=step)
        assert np.array_equal(explored, o_ex)                      # same decisions
        ex = explored.astype(bool)
        assert np.array_equal(ids[ex], o_ids[ex])                  # same draws, in draw order
        np.testing.assert_allclose(scores[ex], o_sc[ex], rtol=2e-3, atol=1e-5)
        assert np.array_equal(ids[~ex], greedy[0][~ex]) and np.array_equal(scores[~ex], greedy[1][~ex])
        if eps == 0.0:
            assert not ex.any()
        if eps == 1.0:
            assert ex.all()


def test_explore_short_pool_and_arguments(evk):
    mem, q_tab = _bank(evk, 5, 64, 9)
    queries = synth.gaussian_unit(40, 64, 10, DEV)
    ids, scores, explored = [x.cpu().numpy() for x in
                             evk.evk_retrieve_explore(mem, queries, 0, 16, 8, 0.5, 1.0, seed=1, step=1)]
    assert explored.all()
    for row_i, row_s in zip(ids, scores):
        assert sorted(row_i[:5].tolist()) == [0, 1, 2, 3, 4] and row_i[5:].tolist() == [-1] * 3
        assert np.all(np.isneginf(row_s[5:]))
    for eps in (-0.1, 1.5, float("nan")):
        with pytest.raises(evk.EvkError):
            evk.evk_retrieve_explore(mem, queries, 0, 16, 8, 0.5, eps, seed=1, step=1)
