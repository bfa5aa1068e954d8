"""Parity of the CUDA library (through the C ABI) against the CPU oracle, on the five
synthetic bank shapes and on edge cases.  All tests here need a B200."""
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
    """Both phase-1 kernels are forced in turn."""
    return {"stream": evk.EVK_SCORING_STREAM, "tensor": evk.EVK_SCORING_TENSOR}[request.param]


def tensor_unsupported(evk, scoring, d, k1):
    return scoring == evk.EVK_SCORING_TENSOR and (d < 64 or k1 > 512)


def host_bits(t):
    return synth.bf16_bits(t)


def make_mem(evk, bank, q_tables, capacity=None, scoring=None):
    """Create a bank, insert the rows (stage tables written afterwards), return the handle."""
    n, d = bank.shape
    mem = evk.evk_mem_create(d, capacity or max(n, 1), n_stages=q_tables.shape[0])
    if scoring is not None:
        evk.evk_mem_set_scoring(mem, scoring)
    if n:
        evk.evk_mem_insert(mem, bank)
        for s in range(q_tables.shape[0]):
            evk.evk_q_write(mem, s, torch.from_numpy(q_tables[s]).to(DEV))
    return mem


def run_retrieve(evk, mem, queries, stage, k1, k2, w):
    out = evk.evk_retrieve(mem, queries, stage, k1, k2, w, return_pool=True)
    torch.cuda.synchronize()
    assert evk.evk_last_status(mem) == 0
    return [x.cpu().numpy() for x in out]


def sample_of(b, n, seed=0):
    if b <= n:
        return list(range(b))
    return sorted(np.random.default_rng(seed).choice(b, n, replace=False).tolist())


# ---------------------------------------------------------------------------
# the five workloads
# ---------------------------------------------------------------------------

def test_tiny_fp32_bank_both_stages_then_updates(evk):
    wl = synth.WORKLOADS["tiny"]
    bank32 = synth.make_bank(wl, DEV)                       # fp32: the library rounds to bf16
    queries32 = synth.make_queries(wl, wl.batches[0], DEV)
    q_tab = synth.make_q_tables(wl)
    mem = make_mem(evk, bank32, q_tab)
    # the insert boundary: stored bits = the oracle's own nearest-even rounding
    bank_bits = host_bits(evk.evk_bank_read(mem))
    assert np.array_equal(bank_bits, oracle.bf16_round(bank32.cpu().numpy()))
    q_bits = oracle.bf16_round(queries32.cpu().numpy())
    for stage in (0, 1):
        out = run_retrieve(evk, mem, queries32, stage, wl.k1, wl.k2, wl.w)
        ep, ef = parity.check_retrieve(bank_bits, q_bits, q_tab[stage], wl.k1, wl.k2, wl.w, out)
        assert ep == 1.0 and ef == 1.0
    ids, r = synth.make_updates(wl)
    evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 0, torch.from_numpy(r).to(DEV), wl.alpha)
    q_after = evk.evk_q_read(mem, 0).cpu().numpy()
    assert evk.evk_last_status(mem) == 0
    parity.check_update(q_tab[0], ids, r, wl.alpha, q_after)
    # the other stage's table keeps its bits, and its retrieval is unchanged
    assert np.array_equal(evk.evk_q_read(mem, 1).cpu().numpy().view(np.uint32), q_tab[1].view(np.uint32))
    out = run_retrieve(evk, mem, queries32, 0, wl.k1, wl.k2, wl.w)
    parity.check_retrieve(bank_bits, q_bits, q_after, wl.k1, wl.k2, wl.w, out)


def tile_sample(b, per_tile, seed=0, tile=128):
    """Query indices that hit every 128-query tile of the batch (so both blocks of every pair of
    tiles): per tile its first and last row, then random rows, `per_tile` in all."""
    rng = np.random.default_rng(seed)
    picked = []
    for t0 in range(0, b, tile):
        rows = np.arange(t0, min(b, t0 + tile))
        must = [rows[0], rows[-1]][:per_tile]
        rest = np.setdiff1d(rows, must)
        extra = rng.choice(rest, min(max(per_tile - len(must), 0), rest.size), replace=False)
        picked += sorted(set(int(x) for x in must) | set(int(x) for x in extra))
    return picked


def _workload_case(evk, name, b, sample, stage=0, scoring=None, n=None, label=None):
    wl = synth.WORKLOADS[name]
    bank = synth.make_bank(wl, DEV, n=n)
    queries = synth.make_queries(wl, b, DEV)
    q_tab = synth.make_q_tables(wl, n=n)
    mem = make_mem(evk, bank, q_tab, scoring=scoring)
    out = run_retrieve(evk, mem, queries, stage, wl.k1, wl.k2, wl.w)
    bank_bits, q_bits = host_bits(bank), host_bits(queries)
    ep, ef = parity.check_retrieve(bank_bits, q_bits, q_tab[stage], wl.k1, wl.k2, wl.w, out, sample=sample)
    n_judged = b if sample is None else len(sample)
    parity.record(label or f"{name} B={b}", scoring, n_judged, b, ep, ef)
    assert ep >= 0.9 and ef >= 0.9
    return wl, mem, q_tab


def test_mid_bank_retrieve_and_lognormal_updates(evk, scoring):
    # every one of the 256 queries is judged
    wl, mem, q_tab = _workload_case(evk, "mid", 256, None, stage=1, scoring=scoring)
    ids, r = synth.make_updates(wl)
    evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(r).to(DEV), wl.alpha)
    parity.check_update(q_tab[1], ids, r, wl.alpha, evk.evk_q_read(mem, 1).cpu().numpy())


def test_clustered_bank(evk, scoring):
    # 128 of the 1,024 queries: 16 in each of the 8 query tiles
    _workload_case(evk, "clustered", 1024, tile_sample(1024, 16, seed=2), scoring=scoring)


@pytest.mark.parametrize("b", [1, 8, 64])
def test_large_bank_small_batches(evk, b, scoring):
    _workload_case(evk, "large_hbm", b, None, scoring=scoring)     # every query is judged


def test_large_bank_interleaved_retrievals_and_zipf_updates(evk, scoring):
    """The streaming protocol as configured: rounds of retrieve (4,096 fresh queries) -> update
    (65,536 popularity-skewed ids), the stage alternating by round.  From round 2 on a retrieval
    reads a value table that an earlier round's update wrote (Section 3.2's phase 2 fed by Eq. 4).
    The oracle keeps its own tables, advanced by its own binary32 update; nothing the library
    returns ever goes into them."""
    wl = synth.WORKLOADS["large_compute"]
    b = max(wl.batches)
    bank = synth.make_bank(wl, DEV)
    q_orc = synth.make_q_tables(wl)                      # the oracle's tables
    mem = make_mem(evk, bank, q_orc, scoring=scoring)
    bank_bits = host_bits(bank)
    del bank
    for rnd in range(4):
        stage = rnd % 2
        queries = synth.make_queries(wl, b, DEV, salt=rnd)
        out = run_retrieve(evk, mem, queries, stage, wl.k1, wl.k2, wl.w)
        # one query in each of the 32 query tiles: the first row of tile 0, the last row of the last
        # tile, a row of this round's own choice elsewhere
        sample = tile_sample(b, 1, seed=10 + rnd)
        sample[-1] = b - 1
        ep, ef = parity.check_retrieve(bank_bits, host_bits(queries), q_orc[stage], wl.k1, wl.k2, wl.w, out,
                                       sample=sample, workers=6)
        parity.record(f"large_compute round {rnd} (stage {stage})", scoring, len(sample), b, ep, ef)
        assert ep >= 0.9 and ef >= 0.9
        ids, r = synth.make_updates(wl, round_idx=rnd)
        evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), stage, torch.from_numpy(r).to(DEV), wl.alpha)
        got = evk.evk_q_read(mem, stage).cpu().numpy()
        parity.check_update(q_orc[stage], ids, r, wl.alpha, got)          # whole table, bit for bit
        q_orc[stage] = oracle.q_update_f32(q_orc[stage], ids, r, wl.alpha)
        other = evk.evk_q_read(mem, 1 - stage).cpu().numpy()
        assert np.array_equal(other.view(np.uint32), q_orc[1 - stage].view(np.uint32))
        assert evk.evk_last_status(mem) == 0


def test_retrieved_items_are_updated_and_retrieved_again(evk, scoring):
    """The method's own loop on one stage: retrieve a context, reward it, update exactly the
    retrieved items (Eq. 4), retrieve again.  Every later retrieval ranks pools whose values an
    update wrote.  The oracle follows with its own tables; the ids that get updated on BOTH sides
    are the oracle's own retrieval (the library's result has just been checked against it), so
    nothing the library returned flows into an expected value."""
    n, d, b, k1, k2, w, alpha = 50000, 256, 96, 48, 6, 0.7, 0.25
    bank = synth.gaussian_unit(n, d, 201, DEV)
    queries = synth.gaussian_unit(b, d, 202, DEV)          # the same tasks come back every round
    q_orc = np.random.default_rng(203).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_orc, scoring=scoring)
    bank_bits, q_bits = host_bits(bank), host_bits(queries)
    rng = np.random.default_rng(204)
    moved = 0
    first_ids = None
    for rnd in range(6):
        out = run_retrieve(evk, mem, queries, 1, k1, k2, w)
        ep, ef = parity.check_retrieve(bank_bits, q_bits, q_orc[1], k1, k2, w, out)
        assert ep >= 0.9 and ef >= 0.9
        if first_ids is None:
            first_ids = out[0].copy()
        else:
            moved += int((out[0] != first_ids).any(axis=1).sum())
        # one reward per query, shared by the k2 items of its context
        r_q = (rng.random(b) < 0.4).astype(np.float32) * 2 - 1
        ids = oracle.retrieve(bank_bits, q_bits, q_orc[1], k1, k2, w)[0].reshape(-1).astype(np.int32)
        r = np.repeat(r_q, k2).astype(np.float32)
        evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 1, torch.from_numpy(r).to(DEV), alpha)
        got = evk.evk_q_read(mem, 1).cpu().numpy()
        parity.check_update(q_orc[1], ids, r, alpha, got)
        q_orc[1] = oracle.q_update_f32(q_orc[1], ids, r, alpha)
    assert moved > 0          # the updates did change later retrievals
    parity.record("retrieve-update loop, 6 rounds", scoring, b, b, ep, ef)


# ---------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------

def _random_case(evk, n, d, b, k1, k2, w, seed, capacity=None, scoring=None):
    bank = synth.gaussian_unit(n, d, seed, DEV)
    queries = synth.gaussian_unit(b, d, seed + 1, DEV)
    q_tab = np.random.default_rng(seed).random((2, max(n, 1))).astype(np.float32)[:, :n]
    mem = make_mem(evk, bank, np.ascontiguousarray(q_tab), capacity=capacity, scoring=scoring)
    if tensor_unsupported(evk, scoring, d, k1):
        with pytest.raises(evk.EvkError) as e:
            evk.evk_retrieve(mem, queries, 0, k1, k2, w)
        assert e.value.status == evk.EVK_ERR_UNSUPPORTED
        return mem, None
    out = run_retrieve(evk, mem, queries, 0, k1, k2, w)
    if n:
        ep, ef = parity.check_retrieve(host_bits(bank), host_bits(queries), q_tab[0], k1, k2, w, out)
        assert ep >= 0.9 and ef >= 0.9
    return mem, out


@pytest.mark.parametrize("n,d,b,k1,k2", [
    (1, 64, 3, 8, 2),            # single entry, pool mostly padding
    (37, 8, 5, 64, 64),          # bank smaller than k1, narrowest rows, k2 = k1
    (1000, 776, 7, 100, 10),     # width not a multiple of 256, ragged row count
    (30000, 200, 140, 40, 6),    # width not a multiple of 64 (zero-filled last slice), sampled thresholds, two query tiles
    (4097, 2048, 2, 1024, 16),   # widest rows, largest pool
    (70001, 256, 9, 33, 5),      # several tiles per block plus a tail
    (20000, 1024, 4, 1, 1),      # k1 = k2 = 1: plain argmax
    (300, 64, 130, 16, 4),       # two query tiles, the second nearly empty; bank just over one tile
    (66000, 128, 150, 512, 32),  # sampled thresholds, two query tiles, widest pool of the tensor path
    (40000, 128, 330, 96, 8),    # three query tiles: the second pair of blocks has one tile of queries only
    (90000, 128, 16, 48, 6),     # the last batch size of one chunk of queries on the N side (bank rows on the lanes)
    (90000, 192, 17, 48, 6),     # ... two chunks, the second with one query; three 64-column slices
    (90000, 64, 32, 200, 9),     # ... the largest batch of that layout
    (90000, 64, 33, 200, 9),     # the first batch with the queries back on the M side
])
def test_edge_shapes(evk, n, d, b, k1, k2, scoring):
    _random_case(evk, n, d, b, k1, k2, 0.5, seed=n, scoring=scoring)


def test_empty_bank_and_empty_batch(evk, scoring):
    mem = evk.evk_mem_create(64, 128)
    evk.evk_mem_set_scoring(mem, scoring)
    queries = synth.gaussian_unit(4, 64, 1, DEV)
    ids, scores, pool_ids, pool_sims = run_retrieve(evk, mem, queries, 0, 16, 4, 0.5)
    assert np.all(ids == -1) and np.all(np.isneginf(scores))
    assert np.all(pool_ids == -1) and np.all(np.isneginf(pool_sims))
    out = evk.evk_retrieve(mem, queries[:0], 0, 16, 4, 0.5)
    assert out[0].shape == (0, 4)
    evk.evk_q_update(mem, torch.empty(0, dtype=torch.int32, device=DEV), 0,
                     torch.empty(0, dtype=torch.float32, device=DEV), 0.5)
    assert evk.evk_last_status(mem) == 0


def test_orthonormal_bank_is_exact(evk, scoring):
    # sims are exact powers of two: no tolerance anywhere
    d = 64
    perm = np.random.default_rng(0).permutation(d)
    bank = torch.eye(d, dtype=torch.float32)[perm].to(DEV)
    q = (2.0 ** -torch.arange(d, dtype=torch.float32))[None, :].to(DEV)
    mem = make_mem(evk, bank, np.zeros((2, d), np.float32), scoring=scoring)
    ids, scores, pool_ids, pool_sims = run_retrieve(evk, mem, q, 0, 10, 10, 0.0)
    inv = np.argsort(perm)
    assert pool_ids[0].tolist() == [int(inv[i]) for i in range(10)]
    assert pool_sims[0].tolist() == [2.0 ** -i for i in range(10)]
    assert ids[0].tolist() == pool_ids[0].tolist()


def test_ties_break_by_id_and_degenerate_scores(evk, scoring):
    # duplicate rows tie exactly; a zero query makes every similarity equal
    d, n = 128, 3000
    bank = synth.gaussian_unit(n, d, 5, DEV)
    bank[1234] = bank[17]
    bank[2999] = bank[17]
    q_tab = np.zeros((2, n), np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=scoring)
    queries = torch.cat([bank[17:18], torch.zeros((1, d), dtype=torch.bfloat16, device=DEV)])
    ids, scores, pool_ids, pool_sims = run_retrieve(evk, mem, queries, 0, 40, 8, 0.0)
    assert pool_ids[0, :3].tolist() == [17, 1234, 2999]
    assert pool_ids[1].tolist() == list(range(40)) and np.all(pool_sims[1] == 0.0)
    assert ids[1].tolist() == list(range(8))
    parity.check_retrieve(host_bits(bank), host_bits(queries), q_tab[0], 40, 8, 0.0,
                          (ids, scores, pool_ids, pool_sims))


@pytest.mark.parametrize("n", [50000, 3000])
def test_bank_sorted_against_the_scan(evk, scoring, n):
    # similarities increase with the row index, so every row beats the running threshold:
    # the worst case for candidate-list upkeep.
    d = 256
    q = synth.gaussian_unit(1, d, 9, DEV)
    bank = synth.gaussian_unit(n, d, 10, DEV)
    sims = (bank.float() @ q.float().T).squeeze(1)
    bank = bank[torch.argsort(sims)].contiguous()
    q_tab = np.random.default_rng(1).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=scoring)
    out = run_retrieve(evk, mem, q, 1, 256, 16, 0.5)
    parity.check_retrieve(host_bits(bank), host_bits(q), q_tab[1], 256, 16, 0.5, out)


def test_special_weights_and_stage_separation(evk, scoring):
    n, d, b, k1, k2 = 5000, 128, 6, 32, 5
    bank = synth.gaussian_unit(n, d, 21, DEV)
    queries = synth.gaussian_unit(b, d, 22, DEV)
    q_tab = np.random.default_rng(2).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=scoring)
    ids0, sc0, pool_ids, pool_sims = run_retrieve(evk, mem, queries, 0, k1, k2, 0.0)
    assert np.array_equal(ids0, pool_ids[:, :k2]) and np.array_equal(sc0, pool_sims[:, :k2])
    for stage in (0, 1):
        ids1, sc1, pool_ids1, _ = run_retrieve(evk, mem, queries, stage, k1, k2, 1.0)
        assert np.array_equal(pool_ids1, pool_ids)      # the pool does not depend on the stage
        for i in range(b):
            order = np.argsort(-q_tab[stage][pool_ids[i]], kind="stable")[:k2]
            assert ids1[i].tolist() == pool_ids[i][order].tolist()
            assert np.array_equal(sc1[i], q_tab[stage][pool_ids[i][order]])
    ids_all, _, _, _ = run_retrieve(evk, mem, queries, 0, k1, k1, 0.37)
    assert np.array_equal(np.sort(ids_all, axis=1), np.sort(pool_ids, axis=1))
    # an update of stage 0 cannot change a stage-1 retrieval
    before = run_retrieve(evk, mem, queries, 1, k1, k2, 0.6)
    upd = torch.arange(0, n, dtype=torch.int32, device=DEV)
    evk.evk_q_update(mem, upd, 0, torch.ones(n, device=DEV), 0.5)
    after = run_retrieve(evk, mem, queries, 1, k1, k2, 0.6)
    for x, y in zip(before, after):
        assert np.array_equal(x, y)


def test_fp32_queries_equal_pre_rounded_bf16_queries(evk, scoring):
    n, d = 3000, 512
    bank = synth.gaussian_unit(n, d, 31, DEV)
    q32 = synth.gaussian_unit(5, d, 32, DEV, dtype=torch.float32)
    mem = make_mem(evk, bank, np.zeros((2, n), np.float32), scoring=scoring)
    a = run_retrieve(evk, mem, q32, 0, 50, 7, 0.5)
    b = run_retrieve(evk, mem, q32.to(torch.bfloat16), 0, 50, 7, 0.5)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_incremental_inserts_match_one_insert(evk):
    n, d = 9000, 128
    bank = synth.gaussian_unit(n, d, 41, DEV)
    queries = synth.gaussian_unit(3, d, 42, DEV)
    q0 = torch.rand(n, device=DEV)
    whole = evk.evk_mem_create(d, n)
    ids = evk.evk_mem_insert(whole, bank, evk.EVK_STAGE_DRAFT, q_init=q0, return_ids=True)
    assert ids.cpu().tolist() == list(range(n))
    parts = evk.evk_mem_create(d, n, q_default=0.25)
    cuts = [0, 1, 64, 65, 4000, n]
    for a, b in zip(cuts[:-1], cuts[1:]):
        evk.evk_mem_insert(parts, bank[a:b], evk.EVK_STAGE_DRAFT, q_init=q0[a:b])
        assert evk.evk_mem_size(parts) == b
        mid = run_retrieve(evk, parts, queries, 0, 16, 4, 0.5)          # cold start: sizes grow
        assert np.all(mid[2][:, :min(16, b)] < b)
    assert torch.equal(evk.evk_q_read(parts, 0), q0)
    assert torch.all(evk.evk_q_read(parts, 1) == 0.25) and torch.all(evk.evk_q_read(whole, 1) == 0.0)
    for x, y in zip(run_retrieve(evk, whole, queries, 0, 16, 4, 0.5),
                    run_retrieve(evk, parts, queries, 0, 16, 4, 0.5)):
        assert np.array_equal(x, y)
    with pytest.raises(evk.EvkError) as e:
        evk.evk_mem_insert(parts, bank[:1])
    assert e.value.status == evk.EVK_ERR_CAPACITY


def test_update_duplicates_split_and_order(evk):
    n, m = 1000, 50000
    rng = np.random.default_rng(51)
    ids = np.where(rng.random(m) < 0.5, 7, rng.integers(0, n, m)).astype(np.int32)   # one very hot id
    r = rng.standard_normal(m).astype(np.float32)
    q0 = rng.standard_normal(n).astype(np.float32)
    bank = synth.gaussian_unit(n, 64, 52, DEV)
    results = []
    for cuts in ([0, m], [0, 1, 2047, 2048, 2049, 30000, m]):
        mem = make_mem(evk, bank, np.stack([q0, q0]))
        for a, b in zip(cuts[:-1], cuts[1:]):
            evk.evk_q_update(mem, torch.from_numpy(ids[a:b]).to(DEV), 1, torch.from_numpy(r[a:b]).to(DEV), 0.3)
        results.append(evk.evk_q_read(mem, 1).cpu().numpy())
        assert evk.evk_last_status(mem) == 0
    parity.check_update(q0, ids, r, 0.3, results[0])
    assert np.array_equal(results[0].view(np.uint32), results[1].view(np.uint32))
    # alpha = 1 is not special-cased: q + (r - q) in binary32
    mem = make_mem(evk, bank, np.stack([q0, q0]))
    evk.evk_q_update(mem, torch.from_numpy(ids).to(DEV), 0, torch.from_numpy(r).to(DEV), 1.0)
    parity.check_update(q0, ids, r, 1.0, evk.evk_q_read(mem, 0).cpu().numpy())


@pytest.mark.parametrize("m", [2047, 2048, 2049, 9000, 65536, 65537, 150000])
def test_update_paths_by_batch_length(evk, m):
    # the single-block kernel (up to 2,048 updates), the one-cluster sort (up to 65,536) and the
    # multi-launch sort beyond: each at its edges, with a hot id, a run that crosses every block
    # boundary of the cluster, both step-size rules, and a rejected batch that must change nothing
    n = 1 << 20
    rng = np.random.default_rng(m)
    ids = rng.integers(0, n, m)
    ids[rng.random(m) < 0.3] = 777777                       # ~30 % of the batch on one entry
    ids[::97] = 5                                            # and a run spread evenly over the batch
    ids = ids.astype(np.int32)
    r = rng.standard_normal(m).astype(np.float32)
    q0 = rng.standard_normal((2, n)).astype(np.float32)
    bank = torch.zeros((n, 64), device=DEV, dtype=torch.bfloat16)
    mem = make_mem(evk, bank, q0)
    t_ids, t_r = torch.from_numpy(ids).to(DEV), torch.from_numpy(r).to(DEV)
    bad = t_ids.clone()
    bad[m - 1] = n
    evk.evk_q_update(mem, bad, 0, t_r, 0.2)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    bad_r = t_r.clone()
    bad_r[m // 2] = float("inf")
    evk.evk_q_update(mem, t_ids, 0, bad_r, 0.2)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_NONFINITE
    assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q0[0].view(np.uint32))
    evk.evk_q_update(mem, t_ids, 0, t_r, 0.2)
    assert evk.evk_last_status(mem) == 0
    parity.check_update(q0[0], ids, r, 0.2, evk.evk_q_read(mem, 0).cpu().numpy())
    evk.evk_q_update_decay(mem, t_ids, 1, t_r)
    want, visits = oracle.q_update_decay(q0[1], np.zeros(n, np.uint32), ids, r)
    assert np.array_equal(evk.evk_q_read(mem, 1).cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert np.array_equal(evk.evk_visits_read(mem, 1).cpu().numpy().view(np.uint32), visits)


def test_bad_updates_are_rejected_before_any_write(evk):
    n = 500
    bank = synth.gaussian_unit(n, 64, 61, DEV)
    q0 = np.random.default_rng(3).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q0)
    good = torch.arange(0, 100, dtype=torch.int32, device=DEV)
    for bad_ids, bad_r, code in (
            (torch.tensor([1, 2, n, 3], dtype=torch.int32), torch.zeros(4), evk.EVK_ERR_RANGE),
            (torch.tensor([1, -1, 3], dtype=torch.int32), torch.zeros(3), evk.EVK_ERR_RANGE),
            (torch.tensor([1, 2, 3], dtype=torch.int32), torch.tensor([0.0, float("nan"), 1.0]), evk.EVK_ERR_NONFINITE),
            (torch.tensor([1, 2, 3], dtype=torch.int32), torch.tensor([0.0, float("inf"), 1.0]), evk.EVK_ERR_NONFINITE)):
        evk.evk_q_update(mem, bad_ids.to(DEV), 0, bad_r.to(DEV), 0.5)
        assert evk.evk_last_status(mem) == code
        assert evk.evk_last_status(mem) == 0                       # read clears
        assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q0[0].view(np.uint32))
    evk.evk_q_update(mem, good, 0, torch.ones(100, device=DEV), 0.5)       # the handle still works
    assert evk.evk_last_status(mem) == 0
    parity.check_update(q0[0], good.cpu().numpy(), np.ones(100, np.float32), 0.5,
                        evk.evk_q_read(mem, 0).cpu().numpy())
    # host-side argument checks return before anything is enqueued
    queries = synth.gaussian_unit(2, 64, 62, DEV)
    for kwargs in (dict(k1=8, k2=9, w=0.5), dict(k1=0, k2=1, w=0.5), dict(k1=2000, k2=1, w=0.5),
                   dict(k1=8, k2=2, w=1.5), dict(k1=8, k2=2, w=-0.1)):
        with pytest.raises(evk.EvkError) as e:
            evk.evk_retrieve(mem, queries, 0, kwargs["k1"], kwargs["k2"], kwargs["w"])
        assert e.value.status == evk.EVK_ERR_INVALID
    for alpha in (0.0, -0.5, 1.5, float("nan")):
        with pytest.raises(evk.EvkError):
            evk.evk_q_update(mem, good, 0, torch.ones(100, device=DEV), alpha)
    with pytest.raises(evk.EvkError):
        evk.evk_retrieve(mem, queries, 2, 8, 2, 0.5)               # stage out of range


def test_runs_are_bitwise_repeatable(evk, scoring):
    n, d = 40000, 512
    bank = synth.gaussian_unit(n, d, 71, DEV)
    queries = synth.gaussian_unit(11, d, 72, DEV)
    q_tab = np.random.default_rng(4).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=scoring)
    a = run_retrieve(evk, mem, queries, 0, 128, 8, 0.5)
    for _ in range(3):
        b = run_retrieve(evk, mem, queries, 0, 128, 8, 0.5)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)


def test_host_buffer_entry_points(evk):
    n, d, b, k1, k2 = 20000, 256, 8, 64, 8
    bank = synth.gaussian_unit(n, d, 81, DEV)
    queries = synth.gaussian_unit(b, d, 82, DEV)
    q_tab = np.random.default_rng(5).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab)
    want = run_retrieve(evk, mem, queries, 0, k1, k2, 0.5)
    q_host = queries.cpu().pin_memory()
    ids_h = torch.empty((b, k2), dtype=torch.int32).pin_memory()
    sc_h = torch.empty((b, k2), dtype=torch.float32).pin_memory()
    evk.evk_retrieve_host(mem, q_host, 0, k1, k2, 0.5, ids_h, sc_h)
    assert np.array_equal(ids_h.numpy(), want[0]) and np.array_equal(sc_h.numpy(), want[1])
    ids = ids_h.reshape(-1).clone().pin_memory()
    r = torch.ones(ids.numel()).pin_memory()
    evk.evk_q_update_host(mem, ids, 0, r, 0.25)
    parity.check_update(q_tab[0], ids.numpy(), r.numpy(), 0.25, evk.evk_q_read(mem, 0).cpu().numpy())


@pytest.mark.parametrize("b,k2", [(64, 16), (300, 8), (2100, 32)])
def test_kernels_of_one_stream_wait_for_one_another(evk, b, k2):
    """The kernels of a retrieval and of the update behind it are chained so that one may start while
    its predecessor still runs; each must wait before it reads what the predecessor writes.  Buffers
    are filled with garbage first, so that a kernel that ran ahead would read garbage: the scratch of
    the retrieval (stale thresholds, counters and candidate lists) and the result ids that the update
    consumes (1,024 ids: the single-block update; 2,400: the one-cluster sort; 67,200: the
    multi-launch sort)."""
    n, d, k1 = 50000, 64, 64
    bank = synth.gaussian_unit(n, d, 401, DEV)
    q_tab = np.random.default_rng(402).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    queries = [synth.gaussian_unit(b, d, 403 + j, DEV) for j in range(3)]
    clean = []
    for qs in queries:
        clean.append(evk.evk_retrieve(mem, qs, 0, k1, k2, 0.5)[0].clone())
        torch.cuda.synchronize()
    ids = torch.empty((b, k2), dtype=torch.int32, device=DEV)
    scores = torch.empty((b, k2), dtype=torch.float32, device=DEV)
    rewards = torch.from_numpy(np.random.default_rng(404).random(b * k2).astype(np.float32)).to(DEV)
    q_orc = q_tab[1].copy()
    for it in range(12):
        ids.fill_(0x7f7f7f7f)
        mem._ws["retrieve"].fill_(0x7f)
        evk.evk_retrieve(mem, queries[it % 3], 0, k1, k2, 0.5, out=(ids, scores))
        evk.evk_q_update(mem, ids.reshape(-1), 1, rewards, 0.2)
        assert evk.evk_last_status(mem) == 0, it
        assert torch.equal(ids, clean[it % 3]), it
        q_orc = oracle.q_update_f32(q_orc, ids.reshape(-1).cpu().numpy(), rewards.cpu().numpy(), 0.2)
    assert np.array_equal(evk.evk_q_read(mem, 1).cpu().numpy().view(np.uint32), q_orc.view(np.uint32))


@pytest.mark.parametrize("d,dtype", [(1024, torch.bfloat16), (64, torch.bfloat16), (2048, torch.float32)])
def test_a_retrieval_sees_the_rows_appended_just_before_it(evk, d, dtype):
    """The scan is launched so that it may start while the kernels before it still run (and those before
    them: every kernel of the library lets its successor be scheduled at once).  Rows appended by the
    insert just before it, or two calls ago, and fp32 queries, which the library converts in a kernel of its
    own, must be loaded only once those kernels are done: on a bank of one or two tiles the first loads would
    otherwise meet rows that are still being written (seen: a third of 400 rounds returned a stale
    neighbour).  400 rounds of insert 16 rows -> retrieve them, nothing synchronises; the three cases run
    in one process on purpose (recycled memory holds garbage where a row is not yet written)."""
    n0, rounds, n_new = 40, 400, 16
    mem = evk.evk_mem_create(d, n0 + rounds * n_new + 64)
    evk.evk_mem_insert(mem, synth.gaussian_unit(n0, d, 1, DEV))
    rows = synth.gaussian_unit(rounds * n_new, d, 2, DEV)
    queries = rows.to(dtype)
    outs = torch.empty((rounds, n_new), dtype=torch.int32, device=DEV)
    sc = torch.empty((n_new, 1), dtype=torch.float32, device=DEV)
    busy = torch.empty(1 << 28, dtype=torch.uint8, device=DEV)
    torch.cuda.synchronize()
    for _ in range(4):
        busy.zero_()          # the launches below queue up behind this and then run back to back
    for r in range(rounds):
        evk.evk_mem_insert(mem, rows[r * n_new:(r + 1) * n_new])
        evk.evk_retrieve(mem, queries[r * n_new:(r + 1) * n_new], 0, 8, 1, 0.0, out=(outs[r].view(n_new, 1), sc))
    torch.cuda.synchronize()
    assert evk.evk_last_status(mem) == 0
    want = (torch.arange(rounds * n_new, device=DEV, dtype=torch.int32) + n0).view(rounds, n_new)
    assert torch.equal(outs, want)


def test_host_buffer_calls_check_arguments_before_copying(evk):
    # a refused call enqueues nothing: no kernel is launched, the outputs keep their contents
    n, d, b, k1, k2 = 5000, 128, 4, 32, 4
    bank = synth.gaussian_unit(n, d, 83, DEV)
    q_tab = np.random.default_rng(6).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab)
    q_host = synth.gaussian_unit(b, d, 84, "cpu").pin_memory()
    ids_h = torch.full((b, k2), -7, dtype=torch.int32).pin_memory()
    sc_h = torch.full((b, k2), -7.0, dtype=torch.float32).pin_memory()
    before = evk.evk_launch_count(mem)
    for stage, kk1, kk2, w in ((2, k1, k2, 0.5), (-1, k1, k2, 0.5), (0, k1, k2, 1.5), (0, k1, k2, float("nan")),
                              (0, k1, k1 + 1, 0.5), (0, 0, 1, 0.5), (0, evk.EVK_MAX_K1 + 1, 1, 0.5)):
        with pytest.raises(evk.EvkError) as e:
            evk.evk_retrieve_host(mem, q_host, stage, kk1, kk2, w, ids_h, sc_h)
        assert e.value.status == evk.EVK_ERR_INVALID
    ids = torch.arange(10, dtype=torch.int32).pin_memory()
    r = torch.ones(10).pin_memory()
    for stage, alpha in ((2, 0.5), (-1, 0.5), (0, 0.0), (0, 1.5), (0, float("nan"))):
        with pytest.raises(evk.EvkError) as e:
            evk.evk_q_update_host(mem, ids, stage, r, alpha)
        assert e.value.status == evk.EVK_ERR_INVALID
    torch.cuda.synchronize()
    assert evk.evk_launch_count(mem) == before
    assert torch.all(ids_h == -7) and torch.all(sc_h == -7.0)
    assert np.array_equal(evk.evk_q_read(mem, 0).cpu().numpy().view(np.uint32), q_tab[0].view(np.uint32))
    # a device-detected error still leaves the stream drained and the handle usable
    bad = torch.tensor([1, n + 5, 2], dtype=torch.int32).pin_memory()
    evk.evk_q_update_host(mem, bad, 0, torch.ones(3).pin_memory(), 0.5)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_RANGE
    evk.evk_retrieve_host(mem, q_host, 0, k1, k2, 0.5, ids_h, sc_h)
    assert torch.all(ids_h >= 0)


def test_both_kernels_return_the_same_pool(evk):
    # the two phase-1 kernels sum in different orders, so similarities may differ in the last
    # bits; the id sets agree except where two entries are within rounding of the boundary
    n, d, b, k1 = 200000, 768, 40, 128
    bank = synth.gaussian_unit(n, d, 91, DEV)
    queries = synth.gaussian_unit(b, d, 92, DEV)
    q_tab = np.random.default_rng(6).random((2, n)).astype(np.float32)
    outs = []
    for mode in (evk.EVK_SCORING_STREAM, evk.EVK_SCORING_TENSOR, evk.EVK_SCORING_AUTO):
        mem = make_mem(evk, bank, q_tab, scoring=mode)
        kind, launches = evk.evk_retrieve_plan(mem, b, k1)
        assert kind == (evk.EVK_SCORING_STREAM if mode == evk.EVK_SCORING_STREAM else evk.EVK_SCORING_TENSOR)
        outs.append(run_retrieve(evk, mem, queries, 0, k1, 8, 0.5))
    same = sum(set(outs[0][2][i].tolist()) == set(outs[1][2][i].tolist()) for i in range(b))
    assert same >= b - 2
    np.testing.assert_allclose(np.sort(outs[0][3], axis=1), np.sort(outs[1][3], axis=1), rtol=1e-4, atol=1e-6)
    for x, y in zip(outs[1], outs[2]):
        assert np.array_equal(x, y)


def test_sample_rows_recompute_to_the_same_bits(evk):
    # the starting threshold of the tensor path is a similarity computed in a separate pass over
    # sampled rows; the scan must reproduce it exactly, or a query could end up short of k1
    # candidates (the library would then report EVK_ERR_INCOMPLETE)
    n, d = 120000, 1024
    bank = synth.gaussian_unit(n, d, 93, DEV)
    queries = synth.gaussian_unit(133, d, 94, DEV)
    mem = make_mem(evk, bank, np.zeros((2, n), np.float32), scoring=evk.EVK_SCORING_TENSOR)
    for k1 in (1, 7, 512):
        out = evk.evk_retrieve(mem, queries, 0, k1, 1, 0.0, return_pool=True)
        assert evk.evk_last_status(mem) == 0
        assert int((out[2] >= 0).sum()) == 133 * k1


def test_tensor_path_candidate_lists_overflow_and_are_cut_back(evk):
    # too small a bank for sampled thresholds and only a few bank splits per query tile: every
    # row passes the initial threshold, so each query's list fills and is cut back several times
    n, d, b, k1 = 16000, 64, 2000, 100
    bank = synth.gaussian_unit(n, d, 95, DEV)
    queries = synth.gaussian_unit(b, d, 96, DEV)
    q_tab = np.random.default_rng(8).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    out = run_retrieve(evk, mem, queries, 0, k1, 10, 0.5)
    ep, ef = parity.check_retrieve(host_bits(bank), host_bits(queries), q_tab[0], k1, 10, 0.5, out,
                                   sample=sample_of(b, 96))
    assert ep >= 0.9 and ef >= 0.9
    # and the same with one query whose similarities rise along the scan
    q1 = queries[:1]
    order = torch.argsort((bank.float() @ q1.float().T).squeeze(1))
    bank2 = bank[order].contiguous()
    mem2 = make_mem(evk, bank2, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    out2 = run_retrieve(evk, mem2, queries, 0, k1, 10, 0.5)
    parity.check_retrieve(host_bits(bank2), host_bits(queries), q_tab[0], k1, 10, 0.5, out2, sample=[0, 1, 1999])


@pytest.mark.parametrize("b", [3, 40])
def test_one_query_tile_lists_overflow_and_are_cut_back(evk, b):
    # a bank sorted against the scan for query 0 makes every row of every tile pass, so that its lists fill
    # and are cut back: 3 queries in the layout with the bank rows on the accumulator lanes, 40 in the one
    # with the queries there
    n, d, k1 = 250000, 64, 100
    bank = synth.gaussian_unit(n, d, 97, DEV)
    queries = synth.gaussian_unit(b, d, 98, DEV)
    order = torch.argsort((bank.float() @ queries[:1].float().T).squeeze(1))
    bank = bank[order].contiguous()
    q_tab = np.random.default_rng(8).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    before = evk.evk_mem_stats(mem)["list_cutbacks"]
    out = run_retrieve(evk, mem, queries, 0, k1, 10, 0.5)
    assert evk.evk_mem_stats(mem)["list_cutbacks"] > before
    ep, ef = parity.check_retrieve(host_bits(bank), host_bits(queries), q_tab[0], k1, 10, 0.5, out,
                                   sample=[0, 1, b - 1] + sample_of(b, 5, seed=4))
    assert ep == 1.0 and ef == 1.0


def test_more_query_tiles_than_sms(evk):
    # 149 query tiles: each gets a single bank split and blocks take several jobs in turn
    n, d, b, k1 = 3000, 64, 149 * 128 - 5, 20
    bank = synth.gaussian_unit(n, d, 97, DEV)
    queries = synth.gaussian_unit(b, d, 98, DEV)
    q_tab = np.random.default_rng(9).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    out = run_retrieve(evk, mem, queries, 1, k1, 5, 0.5)
    ep, ef = parity.check_retrieve(host_bits(bank), host_bits(queries), q_tab[1], k1, 5, 0.5, out,
                                   sample=[0, 127, 128, 9000, b - 1] + sample_of(b, 40, seed=3))
    assert ep >= 0.9 and ef >= 0.9


@pytest.mark.parametrize("b", [5, 20, 200, 330])
def test_bounded_wait_runs_out_and_the_handle_survives(evk, b):
    # failure detection without a fault: the producer of one scan issues no loads, the consumer's
    # wait expires, every block backs out, and the status word says so.  5 queries: single blocks with
    # the bank rows on the accumulator lanes (four epilogue warps leave together); 20: single blocks;
    # 200: one pair of blocks per tile; 330: a second pair whose other block has a tile of padding
    n, d = 40000, 256
    bank = synth.gaussian_unit(n, d, 101, DEV)
    queries = synth.gaussian_unit(b, d, 102, DEV)
    q_tab = np.random.default_rng(10).random((2, n)).astype(np.float32)
    mem = make_mem(evk, bank, q_tab, scoring=evk.EVK_SCORING_TENSOR)
    good = run_retrieve(evk, mem, queries, 0, 64, 8, 0.5)
    evk.evk_mem_inject_stall(mem)
    out = evk.evk_retrieve(mem, queries, 0, 64, 8, 0.5, return_pool=True)
    assert evk.evk_last_status(mem) == evk.EVK_ERR_DEVICE_TIMEOUT
    assert torch.all(out[0] == -1) and torch.all(out[2] == -1)
    again = run_retrieve(evk, mem, queries, 0, 64, 8, 0.5)          # one-shot: the next call is normal
    for x, y in zip(good, again):
        assert np.array_equal(x, y)
