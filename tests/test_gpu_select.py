"""Start-point selection by value against the CPU oracle (the pool cut of Section 3.2 with
w = 1 over a caller-given id list ranks by Q alone, ties by id)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_select_by_value_matches_oracle():
    from paper_2603_10846_b200 import evk
    n = 50000
    rng = np.random.default_rng(0)
    q_tab = rng.random((2, n)).astype(np.float32)
    q_tab[1, ::7] = 0.5                                   # many exact ties -> id order decides
    mem = evk.evk_mem_create(64, n)
    evk.evk_mem_insert(mem, synth.gaussian_unit(n, 64, 1, DEV))
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(DEV))
    lens = [0, 1, 3, 40, 257, 4096, 1000]
    cands = [rng.permutation(n)[:L].astype(np.int32) for L in lens]
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    flat = torch.from_numpy(np.concatenate(cands)).to(DEV)
    for k in (1, 5, 300):
        ids, q = evk.evk_select_by_value(mem, flat, torch.from_numpy(offsets).to(DEV), 1, k)
        ids, q = ids.cpu().numpy(), q.cpu().numpy()
        assert evk.evk_last_status(mem) == 0
        for t, c in enumerate(cands):
            want_ids, want_q = oracle.phase2(c, np.zeros(len(c)), q_tab[1], 1.0, k)
            assert ids[t].tolist() == want_ids[0].tolist()
            assert np.array_equal(q[t].astype(np.float64), want_q[0])
    # bad input is reported, not dereferenced
    bad = torch.tensor([1, 2, n], dtype=torch.int32, device=DEV)
    ids, _ = evk.evk_select_by_value(mem, bad, torch.tensor([0, 3], dtype=torch.int32, device=DEV), 0, 2)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE and ids.cpu().tolist() == [[-1, -1]]
    long = torch.arange(0, 5000, dtype=torch.int32, device=DEV)
    evk.evk_select_by_value(mem, long, torch.tensor([0, 5000], dtype=torch.int32, device=DEV), 0, 2)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_UNSUPPORTED
