"""A bank saved to a file and loaded back answers retrievals and updates with the same bits."""
import numpy as np
import pytest
import torch

from paper_2603_10846_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_save_load_round_trip_and_filtered_bank(tmp_path):
    from paper_2603_10846_b200 import checkpoint, evk
    n, d = 6000, 128
    rng = np.random.default_rng(0)
    mem = evk.evk_mem_create(d, n + 100)
    evk.evk_mem_insert(mem, synth.gaussian_unit(n, d, 1, DEV, dtype=torch.float32))      # rounded at insert
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(rng.random(n).astype(np.float32)).to(DEV))
    ids = torch.from_numpy(rng.integers(0, n, 500).astype(np.int32)).to(DEV)
    evk.evk_q_update_decay(mem, ids, 0, torch.rand(500, device=DEV))
    path = str(tmp_path / "bank.npz")
    checkpoint.save(mem, path)
    back = checkpoint.load(path, DEV, capacity=n + 7)
    assert evk.evk_mem_size(back) == n
    assert torch.equal(evk.evk_bank_read(back).view(torch.int16), evk.evk_bank_read(mem).view(torch.int16))
    for s in range(2):
        assert torch.equal(evk.evk_q_read(back, s), evk.evk_q_read(mem, s))
        assert torch.equal(evk.evk_visits_read(back, s), evk.evk_visits_read(mem, s))
    queries = synth.gaussian_unit(9, d, 2, DEV)
    for a, b in zip(evk.evk_retrieve(mem, queries, 1, 32, 4, 0.5), evk.evk_retrieve(back, queries, 1, 32, 4, 0.5)):
        assert torch.equal(a, b)
    evk.evk_q_update_decay(mem, ids, 0, torch.ones(500, device=DEV))
    evk.evk_q_update_decay(back, ids, 0, torch.ones(500, device=DEV))
    assert torch.equal(evk.evk_q_read(back, 0), evk.evk_q_read(mem, 0))
    # a filtered bank: kept entries are renumbered in order, their rows and values carried over
    keep = np.sort(rng.choice(n, 1000, replace=False))
    part = checkpoint.load(path, DEV, keep=keep)
    assert evk.evk_mem_size(part) == 1000
    full_rows = evk.evk_bank_read(checkpoint.load(path, DEV)).view(torch.int16).cpu().numpy()
    assert np.array_equal(evk.evk_bank_read(part).view(torch.int16).cpu().numpy(), full_rows[keep])
    assert np.array_equal(evk.evk_visits_read(part, 0).cpu().numpy(), evk.evk_visits_read(mem, 0).cpu().numpy()[keep] * 0
                          + evk.evk_visits_read(checkpoint.load(path, DEV), 0).cpu().numpy()[keep])
    with pytest.raises(ValueError):
        checkpoint.load(path, DEV, keep=[5, 3])
