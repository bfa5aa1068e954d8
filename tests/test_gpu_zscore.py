"""Pool z-score variant of phase 2 on the GPU against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def evk():
    from paper_2603_10846_b200 import evk as _evk
    return _evk


def _bank(evk, n, d, seed):
    bank = synth.gaussian_unit(n, d, seed, DEV).to(torch.bfloat16)
    q_tab = np.random.default_rng(seed).random((2, n)).astype(np.float32)
    mem = evk.evk_mem_create(d, n)
    evk.evk_mem_insert(mem, bank)
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(DEV))
    return mem, synth.bf16_bits(bank), q_tab


@pytest.mark.parametrize("n,d,b,k1,k2,w", [(40000, 256, 96, 64, 8, 0.5), (5000, 128, 33, 200, 200, 0.3),
                                           (3000, 64, 20, 17, 5, 1.0), (3000, 64, 20, 17, 5, 0.0)])
def test_zscore_retrieve_matches_oracle(evk, n, d, b, k1, k2, w):
    mem, bank_bits, q_tab = _bank(evk, n, d, 21)
    queries = synth.gaussian_unit(b, d, 22, DEV).to(torch.bfloat16)
    raw = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 1, k1, k2, w, return_pool=True)]
    evk.evk_mem_set_score_norm(mem, evk.EVK_NORM_POOL_ZSCORE)
    out = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 1, k1, k2, w, return_pool=True)]
    assert evk.evk_last_status(mem) == 0
    assert np.array_equal(out[2], raw[2]) and np.array_equal(out[3], raw[3])        # phase 1 is untouched
    exact_pool, exact_final = parity.check_retrieve(bank_bits, synth.bf16_bits(queries), q_tab[1], k1, k2, w, out,
                                                    zscore=True)
    assert exact_pool >= 0.9 and exact_final >= 0.9
    if w in (0.0, 1.0):
        assert np.array_equal(out[0], raw[0])            # the order at the two ends does not depend on the mode
    # back to the raw mix: bit-identical to before
    evk.evk_mem_set_score_norm(mem, evk.EVK_NORM_NONE)
    again = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 1, k1, k2, w, return_pool=True)]
    assert all(np.array_equal(a, r) for a, r in zip(again, raw))


def test_zscore_short_pool_constant_values_and_bad_mode(evk):
    mem, bank_bits, q_tab = _bank(evk, 6, 64, 23)
    evk.evk_q_write(mem, 0, torch.full((6,), 0.5, device=DEV))
    evk.evk_mem_set_score_norm(mem, evk.EVK_NORM_POOL_ZSCORE)
    queries = synth.gaussian_unit(9, 64, 24, DEV).to(torch.bfloat16)
    out = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 0, 16, 8, 0.5, return_pool=True)]
    q0 = np.full(6, 0.5, np.float32)
    parity.check_retrieve(bank_bits, synth.bf16_bits(queries), q0, 16, 8, 0.5, out, zscore=True)
    assert np.array_equal(out[0][:, :6], out[2][:, :6])              # constant values: the similarity order
    for mode in (-1, 2):
        with pytest.raises(evk.EvkError):
            evk.evk_mem_set_score_norm(mem, mode)


@pytest.mark.parametrize("eps", [0.4, 1.0])
def test_zscore_explore_matches_oracle(evk, eps):
    n, d, b, k1, k2, w = 20000, 128, 150, 40, 6, 0.5
    mem, bank_bits, q_tab = _bank(evk, n, d, 25)
    evk.evk_mem_set_score_norm(mem, evk.EVK_NORM_POOL_ZSCORE)
    queries = synth.gaussian_unit(b, d, 26, DEV).to(torch.bfloat16)
    greedy = [x.cpu().numpy() for x in evk.evk_retrieve(mem, queries, 0, k1, k2, w)]
    out = evk.evk_retrieve_explore(mem, queries, 0, k1, k2, w, eps, seed=99, step=5, return_pool=True)
    ids, scores, explored, pool_ids, pool_sims = [x.cpu().numpy() for x in out]
    o_ids, o_sc, o_ex = oracle.explore(pool_ids, pool_sims.astype(np.float64), q_tab[0], w, k2, eps, seed=99, step=5,
                                       zscore=True)
    assert np.array_equal(explored, o_ex)
    ex = explored.astype(bool)
    assert np.array_equal(ids[ex], o_ids[ex])
    np.testing.assert_allclose(scores[ex], o_sc[ex], rtol=2e-3, atol=1e-4)
    assert np.array_equal(ids[~ex], greedy[0][~ex]) and np.array_equal(scores[~ex], greedy[1][~ex])
