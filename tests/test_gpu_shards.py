"""A bank split by rows: three shards held as three handles on one GPU (run one after the
other, nothing waits on anything) must give exactly what the unsplit bank gives — the same
pool, the same final ids and scores — and owner-applied updates the same table bits."""
import numpy as np
import pytest
import torch

from paper_2603_10846_b200 import parallel, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_row_shards_equal_the_unsplit_bank():
    from paper_2603_10846_b200 import evk
    n, d, b, k1, k2, w = 50000, 256, 37, 96, 7, 0.4
    bank = synth.gaussian_unit(n, d, 1, DEV)
    bank[40000] = bank[123]                       # a tie across two shards: the smaller global id wins
    queries = torch.cat([synth.gaussian_unit(b - 1, d, 2, DEV), bank[123:124]])
    q_tab = np.random.default_rng(0).random((2, n)).astype(np.float32)

    def make(rows, q):
        mem = evk.evk_mem_create(d, max(rows.shape[0], 1))
        if rows.shape[0]:
            evk.evk_mem_insert(mem, rows)
            for s in range(2):
                evk.evk_q_write(mem, s, torch.from_numpy(np.ascontiguousarray(q[s])).to(DEV))
        return mem

    whole = make(bank, q_tab)
    want = evk.evk_retrieve(whole, queries, 1, k1, k2, w, return_pool=True)
    bounds = [0, 20000, 20010, n]                 # uneven shards; the middle one is smaller than k1
    shards = [make(bank[a:e], q_tab[:, a:e]) for a, e in zip(bounds[:-1], bounds[1:])]
    parts = [evk.evk_retrieve_local(m, queries, 1, k1, a) for m, a in zip(shards, bounds[:-1])]
    g, s, q = (torch.stack([p[i] for p in parts]) for i in range(3))
    ids, scores, pool_g, pool_s = evk.evk_merge_shards(g, s, q, k2, w, return_pool=True)
    assert torch.equal(pool_g, want[2]) and torch.equal(pool_s, want[3])
    assert torch.equal(ids, want[0]) and torch.equal(scores, want[1])
    assert pool_g[-1, :2].tolist() == [123, 40000]
    # the single-process path of the helper: one shard that is the whole bank
    ids1, scores1 = parallel.retrieve_row_sharded(evk, whole, queries, 1, k1, k2, w, 0)
    assert torch.equal(ids1, want[0]) and torch.equal(scores1, want[1])

    # updates: every shard applies the pairs it owns, in array order
    rng = np.random.default_rng(1)
    u_ids = torch.from_numpy(np.where(rng.random(30000) < 0.2, 20005, rng.integers(0, n, 30000)).astype(np.int32)).to(DEV)
    u_r = torch.from_numpy(rng.standard_normal(30000).astype(np.float32)).to(DEV)
    evk.evk_q_update(whole, u_ids, 1, u_r, 0.1)
    got = []
    for m, a, e in zip(shards, bounds[:-1], bounds[1:]):
        li, lr = parallel.own_updates(u_ids, u_r, a, e)
        evk.evk_q_update(m, li, 1, lr, 0.1)
        got.append(evk.evk_q_read(m, 1))
    assert torch.equal(torch.cat(got), evk.evk_q_read(whole, 1))


def test_merge_shards_argument_checks():
    from paper_2603_10846_b200 import evk
    g = torch.zeros((2, 3, 8), dtype=torch.int32, device=DEV)
    s = torch.zeros((2, 3, 8), device=DEV)
    for k2, w in ((9, 0.5), (0, 0.5), (2, 1.5)):
        with pytest.raises(evk.EvkError):
            evk.evk_merge_shards(g, s, s, k2, w)
