"""Reward kernels (Eq. 5, Eq. 6, running normalisation) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def evk():
    from paper_2603_10846_b200 import evk as _evk
    return _evk


def test_draft_and_refine_rewards(evk):
    rng = np.random.default_rng(0)
    n = 100003
    feas = (rng.random(n) < 0.6).astype(np.uint8)
    best = rng.lognormal(0, 1, n).astype(np.float32)
    lat = rng.lognormal(0, 1, n).astype(np.float32)
    lat[:10] = best[:10]                                      # no change -> exactly 0
    f_t, b_t, l_t = (torch.from_numpy(x).to(DEV) for x in (feas, best, lat))
    got = evk.evk_reward_draft(f_t).cpu().numpy()
    assert np.array_equal(got, oracle.reward_draft(feas).astype(np.float32))      # exact: +-1
    got = evk.evk_reward_refine(b_t, l_t, f_t).cpu().numpy().astype(np.float64)
    want = oracle.reward_refine(best, lat, feas)
    # fp32 log and tanh against fp64: a few units in the last place of numbers <= 1
    assert np.max(np.abs(got - want)) <= 2e-6
    assert np.all(got[feas == 0] == -1.0) and np.all(got[:10][feas[:10] == 1] == 0.0)
    assert np.all(np.abs(got) <= 1.0)


def test_running_normalisation_across_calls(evk):
    rng = np.random.default_rng(1)
    raw = np.tanh(0.3 + 0.8 * rng.standard_normal(2500)).astype(np.float32)
    want = oracle.reward_normalize([], raw, 0.05, clip=4.0)
    state = evk.evk_reward_norm_state(DEV)
    got = []
    for a, b in zip([0, 1, 2, 3, 1027, 2051], [1, 2, 3, 1027, 2051, 2500]):   # ragged calls, chunks > 1024
        got.append(evk.evk_reward_normalize(state, torch.from_numpy(raw[a:b]).to(DEV), 0.05, 4.0).cpu().numpy())
    got = np.concatenate(got).astype(np.float64)
    # fp64 prefix sums against the definition recomputed per step; the result is rounded to fp32
    assert np.max(np.abs(got - want) / np.maximum(1.0, np.abs(want))) <= 1e-6
    assert got[0] == raw[0] and got[1] == raw[1]
    st = state.cpu().numpy()
    assert st[0] == 2500 and abs(st[1] - raw.astype(np.float64).sum()) < 1e-9
    # the variance floor and a constant stream
    state = evk.evk_reward_norm_state(DEV)
    out = evk.evk_reward_normalize(state, torch.full((100,), 0.25, device=DEV), 0.1).cpu().numpy()
    assert np.all(out[2:] == 0.0)
    for bad in (dict(sigma_min=0.0), dict(sigma_min=0.1, clip=-1.0)):
        with pytest.raises(evk.EvkError):
            evk.evk_reward_normalize(state, torch.zeros(4, device=DEV), bad["sigma_min"], bad.get("clip", 0.0))


def test_rewards_feed_the_update_bit_exactly(evk):
    # whatever the reward kernels produce is an ordinary fp32 array to evk_q_update
    from paper_2603_10846_b200 import synth
    from tests import parity
    n = 2000
    rng = np.random.default_rng(2)
    q0 = rng.random((2, n)).astype(np.float32)
    mem = evk.evk_mem_create(64, n)
    evk.evk_mem_insert(mem, synth.gaussian_unit(n, 64, 3, DEV))
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q0[s]).to(DEV))
    ids = rng.integers(0, n, 600).astype(np.int32)
    best = torch.from_numpy(rng.lognormal(0, 0.5, 600).astype(np.float32)).to(DEV)
    lat = torch.from_numpy(rng.lognormal(0, 0.5, 600).astype(np.float32)).to(DEV)
    feas = torch.from_numpy((rng.random(600) < 0.8).astype(np.uint8)).to(DEV)
    r = evk.evk_reward_normalize(evk.evk_reward_norm_state(DEV), evk.evk_reward_refine(best, lat, feas), 0.1)
    evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 1, r, 0.1)
    parity.check_update(q0[1], ids, r.cpu().numpy(), 0.1, evk.evk_q_read(mem, 1).cpu().numpy())
