"""The decreasing-step value update on the GPU against the CPU oracle: bit-exact tables and
visit counts, small (one launch) and large (radix-sorted) batches, across calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_decay_update_bits_and_counts():
    from paper_2603_10846_b200 import evk
    n = 3000
    rng = np.random.default_rng(0)
    q0 = rng.standard_normal((2, n)).astype(np.float32)
    mem = evk.evk_mem_create(64, n)
    evk.evk_mem_insert(mem, synth.gaussian_unit(n, 64, 1, DEV))
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q0[s]).to(DEV))
    q, v = q0[1].copy(), np.zeros(n, np.uint32)
    for m in (1, 700, 8192, 8193, 40000):                       # both kernels, hot ids, several calls
        ids = np.where(rng.random(m) < 0.3, 11, rng.integers(0, n, m)).astype(np.int32)
        r = rng.standard_normal(m).astype(np.float32)
        evk.evk_q_update_decay(mem, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(r).to(DEV))
        q, v = oracle.q_update_decay(q, v, ids, r)
        got_q = evk.evk_q_read(mem, 1).cpu().numpy()
        got_v = evk.evk_visits_read(mem, 1).cpu().numpy().view(np.uint32)
        assert evk.evk_last_status(mem) == 0
        assert np.array_equal(got_q.view(np.uint32), q.view(np.uint32))
        assert np.array_equal(got_v, v)
    # the other stage and the constant-step update leave the counts alone
    assert np.all(evk.evk_visits_read(mem, 0).cpu().numpy() == 0)
    evk.evk_q_update(mem, torch.tensor([11, 11], dtype=torch.int32, device=DEV), 1, torch.ones(2, device=DEV), 0.5)
    assert np.array_equal(evk.evk_visits_read(mem, 1).cpu().numpy().view(np.uint32), v)
    # a rejected batch changes nothing
    evk.evk_q_update_decay(mem, torch.tensor([1, n], dtype=torch.int32, device=DEV), 1, torch.ones(2, device=DEV))
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    assert np.array_equal(evk.evk_visits_read(mem, 1).cpu().numpy().view(np.uint32), v)
