"""The stored oracle results for the tiny workload: the oracle still reproduces them (CPU),
and the CUDA library returns the same ids and update bits on the same inputs (GPU)."""
import json
import os
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2603_10846_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.join(HERE, "golden"))


def _stored():
    with open(os.path.join(HERE, "golden", "tiny_oracle.json")) as f:
        return json.load(f)


def test_oracle_reproduces_stored_values():
    import make_tiny_golden
    now, stored = make_tiny_golden.compute(), _stored()
    assert now == stored


@pytest.mark.gpu
def test_library_matches_stored_values():
    from paper_2603_10846_b200 import evk
    stored = _stored()
    wl = synth.WORKLOADS["tiny"]
    bank = synth.make_bank(wl, "cpu")              # the same CPU-drawn fp32 inputs as the script
    queries = synth.make_queries(wl, wl.batches[0], "cpu")
    assert int(oracle.bf16_round(bank.numpy()).astype(np.uint64).sum()) == stored["checksum_bank"]
    q_tab = synth.make_q_tables(wl)
    mem = evk.evk_mem_create(wl.d, wl.n)
    evk.evk_mem_insert(mem, bank.cuda())
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).cuda())
    for stage in (0, 1):
        ids, scores, pool_ids, _ = evk.evk_retrieve(mem, queries.cuda(), stage, wl.k1, wl.k2, wl.w, return_pool=True)
        want = stored[f"stage{stage}"]
        assert ids.cpu().tolist() == want["ids"]
        assert [sorted(r) for r in pool_ids.cpu().tolist()] == [sorted(r) for r in want["pool_ids"]]
        want_sc = np.array([[float.fromhex(x) for x in row] for row in want["scores_hex"]])
        np.testing.assert_allclose(scores.cpu().numpy(), want_sc, rtol=2e-3, atol=1e-5)
    u = stored["update"]
    ids = np.array(u["ids"], np.int32)
    evk.evk_q_update(mem, torch.from_numpy(ids).cuda(), 0, torch.tensor(u["rewards"], dtype=torch.float32).cuda(),
                     wl.alpha)
    got = evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32)[np.unique(ids)]
    assert got.tolist() == u["q_after_bits"]
