"""Entries dropped from a live bank, and banks carried over through export / import, against the
CPU oracle's live mask (which is pinned by retrieval on the compacted bank)."""
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


@pytest.fixture(params=["stream", "tensor"])
def scoring(request, evk):
    return {"stream": evk.EVK_SCORING_STREAM, "tensor": evk.EVK_SCORING_TENSOR}[request.param]


def _bank(evk, n, d, seed, scoring=None, capacity=None):
    bank = synth.gaussian_unit(n, d, seed, DEV)
    q_tab = np.random.default_rng(seed).random((2, n)).astype(np.float32)
    mem = evk.evk_mem_create(d, capacity or n)
    if scoring is not None:
        evk.evk_mem_set_scoring(mem, scoring)
    evk.evk_mem_insert(mem, bank)
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(DEV))
    return bank, q_tab, mem


def _retrieve(evk, mem, queries, stage, k1, k2, w):
    out = evk.evk_retrieve(mem, queries, stage, k1, k2, w, return_pool=True)
    torch.cuda.synchronize()
    assert evk.evk_last_status(mem) == 0
    return [x.cpu().numpy() for x in out]


@pytest.mark.parametrize("n,d,b,k1,k2", [
    (30000, 256, 7, 64, 8),        # one query tile, thresholds started off by the scan itself (bank rows on the lanes)
    (30000, 256, 50, 64, 8),       # ... queries on the lanes, resident in shared memory
    (30000, 1024, 100, 64, 8),     # ... queries on the lanes, streamed through the ring
    (70000, 128, 200, 96, 8),      # a pair of query tiles: sampled thresholds, some sampled rows dropped
    (900, 64, 3, 40, 5),           # a small bank
])
def test_dropped_entries_are_never_retrieved(evk, scoring, n, d, b, k1, k2):
    bank, q_tab, mem = _bank(evk, n, d, 300 + n % 7, scoring)
    queries = synth.gaussian_unit(b, d, 301, DEV)
    before = _retrieve(evk, mem, queries, 0, k1, k2, 0.5)
    rng = np.random.default_rng(302)
    live = np.ones(n, np.uint8)
    # drop a random third, every 4th row (the strided sample of a paired scan falls on such rows), and
    # each query's best three entries, so that every pool changes
    drop = np.unique(np.concatenate([rng.choice(n, n // 3, replace=False), np.arange(0, n, 4),
                                     before[2][:, :3].reshape(-1)])).astype(np.int32)
    live[drop] = 0
    evk.evk_mem_tombstone(mem, torch.from_numpy(np.concatenate([drop, drop[:50]])).to(DEV))   # some ids twice
    out = _retrieve(evk, mem, queries, 0, k1, k2, 0.5)
    ep, ef = parity.check_retrieve(synth.bf16_bits(bank), synth.bf16_bits(queries), q_tab[0], k1, k2, 0.5, out,
                                   sample=list(range(min(b, 24))) + [b - 1], live=live)
    assert ep >= 0.9 and ef >= 0.9
    assert not np.isin(out[2], drop).any() and not np.isin(out[0], drop).any()
    st = evk.evk_mem_stats(mem)
    assert st["entries"] == n and st["live_entries"] == int(live.sum()) and st["dropped_entries"] == drop.size
    # dropping them again changes nothing
    evk.evk_mem_tombstone(mem, torch.from_numpy(drop[:100]).to(DEV))
    again = _retrieve(evk, mem, queries, 0, k1, k2, 0.5)
    assert all(np.array_equal(x, y) for x, y in zip(out, again))
    assert evk.evk_mem_stats(mem)["live_entries"] == int(live.sum())


def test_fewer_live_entries_than_the_pool_and_a_tie(evk, scoring):
    n, d = 3000, 128
    bank = synth.gaussian_unit(n, d, 310, DEV)
    bank[1234] = bank[17]
    bank[2999] = bank[17]
    mem = evk.evk_mem_create(d, n)
    evk.evk_mem_set_scoring(mem, scoring)
    evk.evk_mem_insert(mem, bank)
    queries = bank[17:18].clone()
    out = _retrieve(evk, mem, queries, 0, 8, 3, 0.0)
    assert out[2][0, :3].tolist() == [17, 1234, 2999]
    evk.evk_mem_tombstone(mem, torch.tensor([1234], dtype=torch.int32, device=DEV))       # the middle one of the tie
    out = _retrieve(evk, mem, queries, 0, 8, 3, 0.0)
    assert out[2][0, :2].tolist() == [17, 2999] and 1234 not in out[2][0]
    # all but five entries go: pools of 40 hold five entries and padding
    keep = np.array([5, 17, 100, 2000, 2999])
    drop = np.setdiff1d(np.arange(n), keep).astype(np.int32)
    evk.evk_mem_tombstone(mem, torch.from_numpy(drop).to(DEV))
    q2 = synth.gaussian_unit(4, d, 311, DEV)
    out = _retrieve(evk, mem, q2, 1, 40, 8, 0.5)
    assert np.all(np.sort(out[2][:, :5], axis=1) == keep) and np.all(out[2][:, 5:] == -1)
    assert np.all(out[0][:, 5:] == -1) and np.all(np.isneginf(out[1][:, 5:]))
    live = np.zeros(n, np.uint8)
    live[keep] = 1
    parity.check_retrieve(synth.bf16_bits(bank), synth.bf16_bits(q2), np.zeros(n, np.float32), 40, 8, 0.5, out, live=live)
    # and the last five
    evk.evk_mem_tombstone(mem, torch.from_numpy(keep.astype(np.int32)).to(DEV))
    out = _retrieve(evk, mem, q2, 1, 40, 8, 0.5)
    assert np.all(out[2] == -1) and np.all(out[0] == -1)


def test_a_bad_id_leaves_the_bank_untouched_and_start_points_skip_dropped_entries(evk):
    n, d = 5000, 64
    bank, q_tab, mem = _bank(evk, n, d, 320)
    queries = synth.gaussian_unit(5, d, 321, DEV)
    before = _retrieve(evk, mem, queries, 0, 32, 4, 0.5)
    evk.evk_mem_tombstone(mem, torch.tensor([3, 4, n, 5], dtype=torch.int32, device=DEV))
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    evk.evk_mem_tombstone(mem, torch.tensor([-1], dtype=torch.int32, device=DEV))
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    after = _retrieve(evk, mem, queries, 0, 32, 4, 0.5)
    assert all(np.array_equal(x, y) for x, y in zip(before, after))
    assert evk.evk_mem_stats(mem)["live_entries"] == n
    # start points: a task's candidates minus the dropped ones, by value
    cand = np.arange(100, 160, dtype=np.int32)
    drop = cand[np.argsort(-q_tab[1][cand])[:3]].astype(np.int32)          # the three most valuable go
    evk.evk_mem_tombstone(mem, torch.from_numpy(drop).to(DEV))
    ids, q = evk.evk_select_by_value(mem, torch.from_numpy(cand).to(DEV), torch.tensor([0, 60], dtype=torch.int32, device=DEV), 1, 5)
    left = np.setdiff1d(cand, drop)
    want = left[np.lexsort((left, -q_tab[1][left]))][:5]
    assert ids.cpu().numpy()[0].tolist() == want.tolist()


def test_export_import_carries_rows_values_counts_and_marks(evk, tmp_path):
    from paper_2603_10846_b200 import checkpoint
    n, d = 8000, 128
    bank, q_tab, mem = _bank(evk, n, d, 330, capacity=n + 50)
    rng = np.random.default_rng(331)
    upd = torch.from_numpy(rng.integers(0, n, 700).astype(np.int32)).to(DEV)
    evk.evk_q_update_decay(mem, upd, 1, torch.rand(700, device=DEV))
    drop = np.sort(rng.choice(n, 2500, replace=False)).astype(np.int32)
    evk.evk_mem_tombstone(mem, torch.from_numpy(drop).to(DEV))
    rows, q, visits, live = evk.evk_mem_export(mem)
    assert live.cpu().numpy().sum() == n - 2500 and not live.cpu().numpy()[drop].any()
    # the same bank rebuilt in two imports
    twin = evk.evk_mem_create(d, n + 3)
    ids0 = evk.evk_mem_import(twin, rows[:3001], q[:, :3001].contiguous(), visits[:, :3001].contiguous(), live[:3001],
                              return_ids=True)
    evk.evk_mem_import(twin, rows[3001:], q[:, 3001:].contiguous(), visits[:, 3001:].contiguous(), live[3001:])
    assert ids0.cpu().tolist() == list(range(3001)) and evk.evk_mem_size(twin) == n
    assert evk.evk_mem_stats(twin)["live_entries"] == n - 2500
    for a, b in zip(evk.evk_mem_export(mem), evk.evk_mem_export(twin)):
        assert torch.equal(a.view(torch.uint8) if a.dtype == torch.bfloat16 else a,
                           b.view(torch.uint8) if b.dtype == torch.bfloat16 else b)
    queries = synth.gaussian_unit(6, d, 332, DEV)
    for x, y in zip(_retrieve(evk, mem, queries, 1, 48, 6, 0.5), _retrieve(evk, twin, queries, 1, 48, 6, 0.5)):
        assert np.array_equal(x, y)
    with pytest.raises(evk.EvkError) as e:
        evk.evk_mem_import(twin, rows[:10])
    assert e.value.status == evk.EVK_ERR_CAPACITY
    # through a file: as it was, and compacted (the filtered bank that is handed on)
    path = str(tmp_path / "bank.npz")
    checkpoint.save(mem, path)
    same = checkpoint.load(path, DEV)
    for x, y in zip(_retrieve(evk, mem, queries, 1, 48, 6, 0.5), _retrieve(evk, same, queries, 1, 48, 6, 0.5)):
        assert np.array_equal(x, y)
    compact = checkpoint.load(path, DEV, drop_dead=True)
    kept = np.setdiff1d(np.arange(n), drop)
    assert evk.evk_mem_size(compact) == kept.size and evk.evk_mem_stats(compact)["live_entries"] == kept.size
    out_full = _retrieve(evk, mem, queries, 1, 48, 6, 0.5)
    out_compact = _retrieve(evk, compact, queries, 1, 48, 6, 0.5)
    assert np.array_equal(kept[out_compact[2]], out_full[2]) and np.array_equal(out_compact[3], out_full[3])
    assert np.array_equal(kept[out_compact[0]], out_full[0]) and np.array_equal(out_compact[1], out_full[1])


def test_counters(evk):
    n, d, b, k1 = 60000, 128, 10, 64
    bank, q_tab, mem = _bank(evk, n, d, 340, scoring=evk.EVK_SCORING_TENSOR)
    queries = synth.gaussian_unit(b, d, 341, DEV)
    st0 = evk.evk_mem_stats(mem)
    assert st0["retrieve_calls"] == 0 and st0["candidates_filed"] == 0 and st0["insert_calls"] == 1
    _retrieve(evk, mem, queries, 0, k1, 8, 0.5)
    st = evk.evk_mem_stats(mem)
    assert st["retrieve_calls"] == 1 and st["candidates_filed"] >= b * k1 and st["kernel_launches"] > st0["kernel_launches"]
    ids = np.where(np.arange(30000) % 3 == 0, 777, np.arange(30000) % n).astype(np.int32)
    evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 0, torch.ones(30000, device=DEV), 0.1)
    st = evk.evk_mem_stats(mem)
    assert st["update_calls"] == 1 and st["longest_update_run"] == int((ids == 777).sum())
    # too small a bank for sampled thresholds and only a few bank splits per query tile: every row passes,
    # the candidate lists fill and are cut back, and that is counted
    bank2 = synth.gaussian_unit(16000, 64, 342, DEV)
    mem2 = evk.evk_mem_create(64, 16000)
    evk.evk_mem_set_scoring(mem2, evk.EVK_SCORING_TENSOR)
    evk.evk_mem_insert(mem2, bank2)
    evk.evk_retrieve(mem2, synth.gaussian_unit(2000, 64, 343, DEV), 0, 100, 10, 0.5)
    assert evk.evk_last_status(mem2) == 0
    assert evk.evk_mem_stats(mem2)["list_cutbacks"] > 0
