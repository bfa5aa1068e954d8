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
