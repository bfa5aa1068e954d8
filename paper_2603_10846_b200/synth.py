"""Seeded synthetic workloads shaped like the experience banks of the method.

This module only draws inputs (embeddings, queries, value tables, update
batches).  It holds none of the retrieval or update arithmetic and is the one
module shared by the CUDA path's tests and the CPU checker's tests.

Large embedding matrices are drawn with a seeded ``torch.Generator`` on the
device they are needed on (the bits differ between a CPU and a CUDA generator;
a test always hands the *same* tensor, copied, to both sides).  Small arrays
(value tables, update batches) come from ``numpy.random.Generator(PCG64)``.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n: int                       # bank entries
    d: int                       # embedding width
    emb_dtype: str               # "fp32" (library rounds to bf16 at insert) or "bf16"
    bank: str                    # "gaussian" | "mixture"
    batches: Sequence[int]       # query batch sizes
    k1: int
    k2: int
    w: float
    q_dist: str                  # "uniform" | "beta25"
    seed: int
    n_updates: int = 0
    update_ids: str = "uniform"  # "uniform" | "zipf"
    rewards: str = "bernoulli"   # "bernoulli" | "lognormal"
    reward_p: float = 0.3
    alpha: float = 0.1
    rounds: int = 1
    notes: str = ""


# The five bank shapes: a tiny fp32 bank, a mid bf16 bank, a clustered bank
# queried across tasks, a large bank scanned by small batches (bandwidth-bound)
# and a larger bank scanned by big batches with streaming updates.
WORKLOADS = {
    "tiny": Workload("tiny", 1024, 768, "fp32", "gaussian", (16,), 32, 4, 0.5, "uniform", 0,
                     n_updates=64, update_ids="uniform", rewards="bernoulli", reward_p=0.3, alpha=0.1),
    "mid": Workload("mid", 65536, 1024, "bf16", "gaussian", (256,), 64, 8, 0.3, "beta25", 1,
                    n_updates=4096, update_ids="uniform", rewards="lognormal", alpha=0.1),
    "clustered": Workload("clustered", 262144, 1024, "bf16", "mixture", (1024,), 128, 8, 0.5,
                          "uniform", 2),
    "large_hbm": Workload("large_hbm", 1048576, 1024, "bf16", "gaussian", (1, 8, 64), 256, 16, 0.5,
                          "uniform", 3),
    "large_compute": Workload("large_compute", 4194304, 768, "bf16", "gaussian", (4096,), 128, 8, 0.5,
                              "uniform", 4, n_updates=65536, update_ids="zipf", rewards="bernoulli",
                              reward_p=0.4, alpha=0.05, rounds=100),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _unit_rows(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=1, keepdim=True).clamp_min(1e-30)


def gaussian_unit(n: int, d: int, seed: int, device="cpu", dtype=torch.bfloat16,
                  chunk: int = 1 << 16) -> torch.Tensor:
    """n rows drawn i.i.d. N(0, I_d), scaled to unit L2 norm, cast to `dtype`."""
    g = _gen(seed, device)
    out = torch.empty((n, d), dtype=dtype, device=device)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = torch.randn((e - s, d), generator=g, device=device, dtype=torch.float32)
        out[s:e] = _unit_rows(x).to(dtype)
    return out


def mixture_means(n_comp: int, d: int, seed: int, device="cpu") -> torch.Tensor:
    """Component means: Gaussian directions scaled onto the unit sphere (fp32)."""
    g = _gen(seed, device)
    return _unit_rows(torch.randn((n_comp, d), generator=g, device=device, dtype=torch.float32))


def mixture_unit(n: int, means: torch.Tensor, std: float, seed: int, dtype=torch.bfloat16,
                 chunk: int = 1 << 16):
    """Rows = mean[c] + std*N(0,I), c uniform over the components, then unit norm.

    Returns (rows, component index per row)."""
    device = means.device
    g = _gen(seed, device)
    n_comp, d = means.shape
    out = torch.empty((n, d), dtype=dtype, device=device)
    comp = torch.empty((n,), dtype=torch.int64, device=device)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        c = torch.randint(0, n_comp, (e - s,), generator=g, device=device)
        x = means[c] + std * torch.randn((e - s, d), generator=g, device=device, dtype=torch.float32)
        out[s:e] = _unit_rows(x).to(dtype)
        comp[s:e] = c
    return out, comp


def make_bank(wl: Workload, device="cpu", n: Optional[int] = None) -> torch.Tensor:
    """The bank's embeddings for a workload (optionally only the first n rows' worth)."""
    n = wl.n if n is None else n
    dtype = torch.float32 if wl.emb_dtype == "fp32" else torch.bfloat16
    if wl.bank == "gaussian":
        return gaussian_unit(n, wl.d, 1000 + wl.seed, device, dtype)
    means = mixture_means(64, wl.d, 3000 + wl.seed, device)
    rows, _ = mixture_unit(n, means, 0.15, 1000 + wl.seed, dtype)
    return rows


def make_queries(wl: Workload, b: int, device="cpu", salt: int = 0) -> torch.Tensor:
    """A batch of b queries from the workload's query distribution."""
    dtype = torch.float32 if wl.emb_dtype == "fp32" else torch.bfloat16
    seed = 2000 + wl.seed + 7919 * salt
    if wl.bank == "gaussian":
        return gaussian_unit(b, wl.d, seed, device, dtype)
    # clustered: 90% of queries from the bank's 64 components, 10% from 8 held-out ones
    means = mixture_means(64, wl.d, 3000 + wl.seed, device)
    held = mixture_means(8, wl.d, 4000 + wl.seed, device)
    n_held = b // 10
    q_in, _ = mixture_unit(b - n_held, means, 0.15, seed, dtype)
    if n_held == 0:
        return q_in
    q_out, _ = mixture_unit(n_held, held, 0.15, seed + 1, dtype)
    q = torch.cat([q_in, q_out], dim=0)
    perm = torch.randperm(b, generator=_gen(seed + 2, "cpu")).to(q.device)
    return q[perm].contiguous()


def make_q_tables(wl: Workload, n: Optional[int] = None, n_stages: int = 2) -> np.ndarray:
    """Initial value tables [n_stages][n], fp32: U(0,1) or Beta(2,5)."""
    n = wl.n if n is None else n
    rng = np.random.Generator(np.random.PCG64(5000 + wl.seed))
    if wl.q_dist == "uniform":
        q = rng.random((n_stages, n), dtype=np.float64)
    elif wl.q_dist == "beta25":
        q = rng.beta(2.0, 5.0, size=(n_stages, n))
    else:
        raise ValueError(wl.q_dist)
    return q.astype(np.float32)


def zipf_bounded_ids(rng: np.random.Generator, n: int, m: int, s: float,
                     perm_seed: int) -> np.ndarray:
    """m draws from the bounded Zipf law P(rank=i) ∝ i^-s on ranks 1..n (exact
    normalised pmf, fp64 CDF, inverse-CDF sampling), ranks mapped to entry ids by a
    seeded permutation."""
    pmf = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(pmf)
    cdf /= cdf[-1]
    ranks = np.searchsorted(cdf, rng.random(m), side="right")
    ranks = np.minimum(ranks, n - 1)
    perm = np.random.Generator(np.random.PCG64(perm_seed)).permutation(n)
    return perm[ranks].astype(np.int32)


def make_updates(wl: Workload, round_idx: int = 0, n: Optional[int] = None,
                 m: Optional[int] = None):
    """One update batch: (ids int32 [m], rewards fp32 [m])."""
    n = wl.n if n is None else n
    m = wl.n_updates if m is None else m
    rng = np.random.Generator(np.random.PCG64([6000 + wl.seed, round_idx]))
    if wl.update_ids == "uniform":
        ids = rng.integers(0, n, size=m, dtype=np.int64).astype(np.int32)
    elif wl.update_ids == "zipf":
        ids = zipf_bounded_ids(rng, n, m, 1.1, 7000 + wl.seed)
    else:
        raise ValueError(wl.update_ids)
    if wl.rewards == "bernoulli":
        r = (rng.random(m) < wl.reward_p).astype(np.float32)
    elif wl.rewards == "lognormal":
        r = np.clip(rng.lognormal(0.0, 0.5, size=m), 0.0, 10.0).astype(np.float32)
    else:
        raise ValueError(wl.rewards)
    return ids, r


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The bit patterns of a bf16 tensor as a host uint16 array (a plain copy)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
