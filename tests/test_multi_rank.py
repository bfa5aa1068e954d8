"""The multi-process exchange step on CPU (gloo, world_size 2): update batches are
all-gathered in rank order, so replicas that apply them end up with identical tables,
equal to one process applying rank 0's batch and then rank 1's.  The update arithmetic
here is the CPU oracle's (the CUDA kernel is checked against it elsewhere)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_10846_b200 import parallel


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _batch(rank, n, m):
    rng = np.random.default_rng(100 + rank)
    ids = np.where(rng.random(m) < 0.3, 5, rng.integers(0, n, m)).astype(np.int32)   # rank-shared hot id
    return ids, rng.standard_normal(m).astype(np.float32)


def _worker(rank, world, port, n, sizes, out_dir):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q = np.random.default_rng(7).random(n).astype(np.float32)      # identical replicas
    for rnd, m in enumerate(sizes[rank]):
        ids, r = _batch(rank + 10 * rnd, n, m)
        all_ids, all_r = parallel.gather_update_batches(torch.from_numpy(ids), torch.from_numpy(r))
        q = oracle.q_update_f32(q, all_ids.numpy(), all_r.numpy(), 0.1)
    np.save(os.path.join(out_dir, f"q{rank}.npy"), q)
    dist.destroy_process_group()


def test_replicas_stay_bit_identical(tmp_path):
    import oracle
    n, world = 500, 2
    sizes = [[300, 0, 128], [300, 77, 200]]           # equal, empty-vs-ragged, ragged
    mp.spawn(_worker, args=(world, _free_port(), n, sizes, str(tmp_path)), nprocs=world, join=True)
    q0 = np.load(tmp_path / "q0.npy")
    q1 = np.load(tmp_path / "q1.npy")
    assert np.array_equal(q0.view(np.uint32), q1.view(np.uint32))
    want = np.random.default_rng(7).random(n).astype(np.float32)
    for rnd in range(3):
        for rank in range(world):
            ids, r = _batch(rank + 10 * rnd, n, sizes[rank][rnd])
            want = oracle.q_update_f32(want, ids, r, 0.1)
    assert np.array_equal(q0.view(np.uint32), want.view(np.uint32))


def test_query_shards_cover_the_batch():
    for n, world in ((4096, 8), (10, 3), (2, 4), (0, 2)):
        spans = [parallel.shard_queries(n, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(spans[:-1], spans[1:]))
        assert max(e - b for b, e in spans) - min(e - b for b, e in spans) <= 1


def test_row_shards_partition_updates_in_order():
    # owner-applied updates (ids made local, order kept) give the bits of one unsplit table
    import oracle
    n, world, m = 1000, 3, 5000
    rng = np.random.default_rng(3)
    ids = np.where(rng.random(m) < 0.3, 400, rng.integers(0, n, m)).astype(np.int32)
    r = rng.standard_normal(m).astype(np.float32)
    q0 = rng.random(n).astype(np.float32)
    want = oracle.q_update_f32(q0, ids, r, 0.2)
    got = []
    for rank in range(world):
        a, e = parallel.row_shard(n, rank, world)
        li, lr = parallel.own_updates(torch.from_numpy(ids), torch.from_numpy(r), a, e)
        assert li.numel() == int(((ids >= a) & (ids < e)).sum())
        got.append(oracle.q_update_f32(q0[a:e], li.numpy(), lr.numpy(), 0.2))
    assert np.array_equal(np.concatenate(got).view(np.uint32), want.view(np.uint32))
    spans = [parallel.row_shard(n, rk, world) for rk in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == n and all(x[1] == y[0] for x, y in zip(spans[:-1], spans[1:]))


# ---- the row-sharded retrieval's gather (two gloo ranks, a stand-in for the CUDA library) ----

class _StubEvk:
    """Plays the two library calls of the row-sharded retrieval on the CPU with the oracle, and
    records what reaches the merge.  Only the plumbing between them (parallel.retrieve_row_sharded)
    is under test here."""

    def __init__(self, bank_bits, q_stage, begin, end):
        self.bank_bits, self.q_stage, self.begin, self.end = bank_bits, q_stage, begin, end
        self.seen = None

    def evk_retrieve_local(self, mem, queries, stage, k1, id_offset):
        import oracle
        assert id_offset == self.begin
        ids, sims = oracle.phase1(self.bank_bits[self.begin:self.end], queries.numpy().view(np.uint16), k1)
        gids = np.where(ids >= 0, ids + id_offset, -1).astype(np.int32)
        qs = np.where(ids >= 0, self.q_stage[np.clip(gids, 0, None)], 0.0).astype(np.float32)
        return torch.from_numpy(gids), torch.from_numpy(sims.astype(np.float32)), torch.from_numpy(qs)

    def evk_merge_shards(self, gids, sims, qs, k2, w):
        import oracle
        self.seen = (gids.clone(), sims.clone(), qs.clone())
        g, b, k1 = gids.shape
        ids_out = np.empty((b, k2), np.int32)
        sc_out = np.empty((b, k2), np.float64)
        for i in range(b):
            cand_g = gids[:, i, :].reshape(-1).numpy()
            cand_s = sims[:, i, :].reshape(-1).numpy().astype(np.float64)
            order = np.lexsort((cand_g, -cand_s))
            order = [j for j in order if cand_g[j] >= 0][:k1]
            pool_g = np.full(k1, -1, np.int32)
            pool_s = np.full(k1, -np.inf)
            pool_g[:len(order)], pool_s[:len(order)] = cand_g[order], cand_s[order]
            q_lookup = np.zeros(int(cand_g.max()) + 1, np.float32)
            q_lookup[cand_g[cand_g >= 0]] = qs[:, i, :].reshape(-1).numpy()[cand_g >= 0]
            a, s = oracle.phase2(pool_g, pool_s, q_lookup, w, k2)
            ids_out[i], sc_out[i] = a[0], s[0]
        return torch.from_numpy(ids_out), torch.from_numpy(sc_out)


def _sharded_worker(rank, world, port, n, d, b, k1, k2, w, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(11)
    bank_bits = (rng.integers(0, 1 << 14, (n, d)).astype(np.uint16) | 0x3c00)      # bf16 values in [1, 2)
    bank_bits[rng.random((n, d)) < 0.5] |= 0x8000                                   # random signs
    q_bits = bank_bits[rng.integers(0, n, b)].copy()
    q_stage = rng.random(n).astype(np.float32)
    begin, end = parallel.row_shard(n, rank, world)
    stub = _StubEvk(bank_bits, q_stage, begin, end)
    queries = torch.from_numpy(q_bits.view(np.int16))
    ids, scores = parallel.retrieve_row_sharded(stub, None, queries, 0, k1, k2, w, begin)
    g, s, q = stub.seen
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), ids=ids.numpy(), scores=scores.numpy(), g=g.numpy(),
             s=s.numpy(), q=q.numpy(), bank=bank_bits, queries=q_bits, q_stage=q_stage)
    dist.destroy_process_group()


def _run_sharded(tmp_path, n, d, b, k1, k2, w):
    import oracle
    world = 2
    mp.spawn(_sharded_worker, args=(world, _free_port(), n, d, b, k1, k2, w, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = np.load(tmp_path / "r0.npz"), np.load(tmp_path / "r1.npz")
    spans = [parallel.row_shard(n, r, world) for r in range(world)]
    for r in (r0, r1):
        # what reaches the merge: [world][B][k1], shard g's candidates from shard g's id range only
        assert r["g"].shape == (world, b, k1) and r["s"].shape == (world, b, k1) and r["q"].shape == (world, b, k1)
        for gi, (a, e) in enumerate(spans):
            real = r["g"][gi][r["g"][gi] >= 0]
            assert real.size == b * min(k1, e - a) and real.min() >= a and real.max() < e
            assert np.array_equal(r["q"][gi][r["g"][gi] >= 0], r["q_stage"][real])
    # both ranks hold the same gathered arrays and the same answer
    for key in ("g", "s", "q", "ids", "scores"):
        assert np.array_equal(r0[key], r1[key])
    # and the answer is the unsplit bank's
    want = oracle.retrieve(r0["bank"], r0["queries"], r0["q_stage"], k1, k2, w)
    n_real = min(k2, n)
    assert np.array_equal(r0["ids"][:, :n_real], want[0][:, :n_real])


def test_row_sharded_retrieval_gathers_shards_in_id_order_equal_shards(tmp_path):
    _run_sharded(tmp_path, n=600, d=32, b=5, k1=24, k2=4, w=0.5)


def test_row_sharded_retrieval_unequal_and_short_shards(tmp_path):
    _run_sharded(tmp_path, n=51, d=16, b=3, k1=40, k2=6, w=1.0)       # 26 + 25 rows, both shorter than k1
