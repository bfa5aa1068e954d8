"""Saving a memory bank to a file and loading it back.

The method carries a memory from one run into the next (a bank learned on one level of
tasks initialises the next, a filtered bank is handed to another generator).  A checkpoint
holds what the library stores per entry: the bf16 embedding rows, every stage's value table,
the per-stage update counts and the marks of dropped entries, plus the shape.  This module
only moves those arrays between the library's export / import calls and a file; which
entries survive a filtered load is decided by the marks the library keeps.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import evk

FORMAT = "evk-checkpoint-2"


def save(mem: "evk.EvkMem", path: str) -> None:
    """Write bank rows (as uint16 bit patterns), value tables, update counts and live marks to `path` (.npz)."""
    rows, q, visits, live = evk.evk_mem_export(mem)
    with open(path, "wb") as f:
        np.savez(f, format=np.array(FORMAT), d=np.int64(mem.d), n_stages=np.int64(mem.n_stages),
                 size=np.int64(rows.shape[0]), rows=rows.view(torch.int16).cpu().numpy().view(np.uint16),
                 q=q.cpu().numpy(), visits=visits.cpu().numpy().view(np.uint32), live=live.cpu().numpy())


def load(path: str, device="cuda", capacity: Optional[int] = None,
         keep: Optional[Sequence[int]] = None, drop_dead: bool = False) -> "evk.EvkMem":
    """Build a bank from a checkpoint through evk_mem_import.

    By default every entry comes back at its old id, dropped ones still dropped.  `drop_dead`
    leaves dropped entries out of the file's arrays, `keep` (ascending entry ids) retains only
    those: either way the survivors are renumbered in their old order (a compact, filtered bank)."""
    with np.load(path) as z:
        if str(z["format"]) != FORMAT:
            raise ValueError(f"{path}: not an {FORMAT} file")
        d, n_stages, size = int(z["d"]), int(z["n_stages"]), int(z["size"])
        rows, q, visits, live = z["rows"], z["q"], z["visits"], z["live"]
    sel = None
    if keep is not None:
        sel = np.asarray(keep, dtype=np.int64)
        if sel.size and (np.any(np.diff(sel) <= 0) or sel[0] < 0 or sel[-1] >= size):
            raise ValueError("keep must be ascending entry ids of the checkpoint")
    if drop_dead:
        alive = np.nonzero(live)[0]
        sel = alive if sel is None else np.intersect1d(sel, alive)
    if sel is not None:
        rows, q, visits, live = rows[sel], q[:, sel], visits[:, sel], live[sel]
        size = int(sel.size)
    mem = evk.evk_mem_create(d, max(capacity or size, size, 1), n_stages=n_stages, device=device)
    if size:
        evk.evk_mem_import(
            mem, torch.from_numpy(np.ascontiguousarray(rows).view(np.int16)).to(device).view(torch.bfloat16),
            torch.from_numpy(np.ascontiguousarray(q)).to(device),
            torch.from_numpy(np.ascontiguousarray(visits).view(np.int32)).to(device),
            torch.from_numpy(np.ascontiguousarray(live)).to(device))
    return mem
