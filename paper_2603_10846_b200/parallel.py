"""Several GPUs, one process each: replicated bank, sharded query batches.

Every rank holds the whole bank and both value tables and retrieves for its own share
of the query batches, so retrieval needs no communication.  The one exchange step is
the value update: a rank's rewards change entries that every other rank will read, so
the (id, reward) batches of all ranks are all-gathered and every rank applies the
concatenation in rank order.  Eq. 4 is order-dependent in binary32, and a fixed global
order keeps the replicas' tables bit-identical without ever comparing them.

This module only moves the batches (torch.distributed: NCCL on GPUs, gloo on CPU); the
update itself is the library's kernel.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_queries(n_queries: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced [begin, end) share of a global batch for one rank."""
    base, extra = divmod(n_queries, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def gather_update_batches(ids: torch.Tensor, rewards: torch.Tensor,
                          group: Optional[dist.ProcessGroup] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All ranks' (ids, rewards), concatenated in rank order; batch lengths may differ."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return ids, rewards
    world = dist.get_world_size(group)
    n_local = torch.tensor([ids.numel()], dtype=torch.int64, device=ids.device)
    counts = [torch.zeros_like(n_local) for _ in range(world)]
    dist.all_gather(counts, n_local, group=group)
    counts = [int(c.item()) for c in counts]
    n_max = max(counts)
    if all(c == n_max for c in counts):
        all_ids = torch.empty(world * n_max, dtype=ids.dtype, device=ids.device)
        all_r = torch.empty(world * n_max, dtype=rewards.dtype, device=rewards.device)
        dist.all_gather_into_tensor(all_ids, ids.contiguous(), group=group)
        dist.all_gather_into_tensor(all_r, rewards.contiguous(), group=group)
        return all_ids, all_r
    # ragged: pad to the longest batch, gather, cut the padding out again
    pad_ids = torch.zeros(n_max, dtype=ids.dtype, device=ids.device)
    pad_r = torch.zeros(n_max, dtype=rewards.dtype, device=rewards.device)
    pad_ids[:ids.numel()] = ids
    pad_r[:rewards.numel()] = rewards
    ids_l = [torch.empty_like(pad_ids) for _ in range(world)]
    r_l = [torch.empty_like(pad_r) for _ in range(world)]
    dist.all_gather(ids_l, pad_ids, group=group)
    dist.all_gather(r_l, pad_r, group=group)
    return (torch.cat([t[:c] for t, c in zip(ids_l, counts)]),
            torch.cat([t[:c] for t, c in zip(r_l, counts)]))


# ---- banks too large for one GPU: split by rows -----------------------------------------

def row_shard(n_entries: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [begin, end) id range of one rank; ranges ascend with the rank."""
    return shard_queries(n_entries, rank, world)


def own_updates(ids: torch.Tensor, rewards: torch.Tensor, begin: int, end: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """The (id, reward) pairs a shard owns, in array order, with ids made local.  Every rank sees
    the whole batch; an entry's updates all land on its owner in their original order, so the
    stored bits equal those of one unsplit table."""
    mine = (ids >= begin) & (ids < end)
    return (ids[mine] - begin).to(ids.dtype).contiguous(), rewards[mine].contiguous()


def retrieve_row_sharded(evk, mem, queries: torch.Tensor, stage: int, k1: int, k2: int, w: float,
                         id_offset: int, group: Optional[dist.ProcessGroup] = None):
    """Retrieval over a row-sharded bank: local phase 1, one all-gather of the tagged pools
    (B * k1 * 12 bytes per rank), merge + phase 2 on every rank.  Returns global ids and scores."""
    gids, sims, qs = evk.evk_retrieve_local(mem, queries, stage, k1, id_offset)
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return evk.evk_merge_shards(gids[None], sims[None], qs[None], k2, w)
    # gathered along the first axis (rank-major), then viewed as [world][B][k1]
    b = gids.shape[0]
    all_g = torch.empty((world * b,) + tuple(gids.shape[1:]), dtype=gids.dtype, device=gids.device)
    all_s = torch.empty((world * b,) + tuple(sims.shape[1:]), dtype=sims.dtype, device=sims.device)
    all_q = torch.empty((world * b,) + tuple(qs.shape[1:]), dtype=qs.dtype, device=qs.device)
    dist.all_gather_into_tensor(all_g, gids.contiguous(), group=group)
    dist.all_gather_into_tensor(all_s, sims.contiguous(), group=group)
    dist.all_gather_into_tensor(all_q, qs.contiguous(), group=group)
    shape = (world,) + tuple(gids.shape)
    return evk.evk_merge_shards(all_g.view(shape), all_s.view(shape), all_q.view(shape), k2, w)
