"""Saving a memory bank to a file and loading it back.

The method carries a memory from one run into the next (a bank learned on one level of
tasks initialises the next, a bank is handed to another generator).  A checkpoint holds
what the library stores per entry: the bf16 embedding rows, every stage's value table and
the per-stage update counts, plus the shape.  Loading builds a new bank (optionally with a
larger capacity, or keeping only a subset of the entries) through the library's own
insert and write calls; ids of kept entries are renumbered in their old order.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import evk

FORMAT = "evk-checkpoint-1"


def save(mem: "evk.EvkMem", path: str) -> None:
    """Write bank rows (as uint16 bit patterns), value tables and update counts to `path` (.npz)."""
    n = evk.evk_mem_size(mem)
    rows = evk.evk_bank_read(mem).view(torch.int16).cpu().numpy().view(np.uint16)
    q = np.stack([evk.evk_q_read(mem, s).cpu().numpy() for s in range(mem.n_stages)]) if n else \
        np.zeros((mem.n_stages, 0), np.float32)
    visits = np.stack([evk.evk_visits_read(mem, s).cpu().numpy().view(np.uint32) for s in range(mem.n_stages)]) \
        if n else np.zeros((mem.n_stages, 0), np.uint32)
    with open(path, "wb") as f:
        np.savez(f, format=np.array(FORMAT), d=np.int64(mem.d), n_stages=np.int64(mem.n_stages),
                 size=np.int64(n), rows=rows, q=q, visits=visits)


def load(path: str, device="cuda", capacity: Optional[int] = None,
         keep: Optional[Sequence[int]] = None) -> "evk.EvkMem":
    """Build a bank from a checkpoint.  `keep`: ascending entry ids to retain (a filtered bank).

    Update counts of the decreasing-step update are restored only when every entry is kept
    in place (they are positional state of the arena); a filtered bank starts its counts at 0."""
    with np.load(path) as z:
        if str(z["format"]) != FORMAT:
            raise ValueError(f"{path}: not an {FORMAT} file")
        d, n_stages, size = int(z["d"]), int(z["n_stages"]), int(z["size"])
        rows, q, visits = z["rows"], z["q"], z["visits"]
    if keep is not None:
        keep = np.asarray(keep, dtype=np.int64)
        if keep.size and (np.any(np.diff(keep) <= 0) or keep[0] < 0 or keep[-1] >= size):
            raise ValueError("keep must be ascending entry ids of the checkpoint")
        rows, q, visits = rows[keep], q[:, keep], None
        size = int(keep.size)
    cap = max(capacity or size, size, 1)
    mem = evk.evk_mem_create(d, cap, n_stages=n_stages, device=device)
    if size:
        emb = torch.from_numpy(rows.view(np.int16)).to(device).view(torch.bfloat16)
        evk.evk_mem_insert(mem, emb)
        for s in range(n_stages):
            evk.evk_q_write(mem, s, torch.from_numpy(np.ascontiguousarray(q[s])).to(device))
        if visits is not None and visits.any():
            evk.evk_visits_write(mem, visits, device)
    return mem
