"""CPU oracle for the value-driven memory — TEST INFRASTRUCTURE, not the product.

A ctypes front for ``evk_oracle.c`` (plain C, fp64): exact two-phase retrieval
(Section 3.2) and the unified value update (Eq. 4 / Eq. 8).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; it
imports nothing from the CUDA package and is never given a value that came from
it.  Inputs are numpy arrays; embeddings and queries are bfloat16 bit patterns
held as ``uint16``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "evk_oracle.c")
_LIB = os.path.join(_HERE, "libevk_oracle.so")

_CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-fexcess-precision=standard"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c_i32, c_i64, c_f32, c_f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_double
    p = ctypes.c_void_p
    lib.evk_oracle_bf16_round.argtypes = [p, p, c_i64]
    lib.evk_oracle_bf16_round.restype = None
    lib.evk_oracle_bf16_decode.argtypes = [p, p, c_i64]
    lib.evk_oracle_bf16_decode.restype = None
    lib.evk_oracle_threads.argtypes = []
    lib.evk_oracle_threads.restype = ctypes.c_int
    lib.evk_oracle_sims.argtypes = [p, c_i64, c_i32, p, p]
    lib.evk_oracle_sims.restype = None
    lib.evk_oracle_rank.argtypes = [p, c_i64, c_i32, p, p]
    lib.evk_oracle_rank.restype = c_i32
    lib.evk_oracle_rank_live.argtypes = [p, p, c_i64, c_i32, p, p]
    lib.evk_oracle_rank_live.restype = c_i32
    lib.evk_oracle_phase1.argtypes = [p, c_i64, c_i32, p, c_i32, p, p]
    lib.evk_oracle_phase1.restype = c_i32
    lib.evk_oracle_phase2.argtypes = [p, p, c_i32, p, c_f64, c_i32, p, p]
    lib.evk_oracle_phase2.restype = c_i32
    lib.evk_oracle_phase2_zscore.argtypes = [p, p, c_i32, p, c_f64, c_i32, p, p]
    lib.evk_oracle_phase2_zscore.restype = c_i32
    lib.evk_oracle_q_update_f64.argtypes = [p, p, p, c_i64, c_f64]
    lib.evk_oracle_q_update_f64.restype = None
    lib.evk_oracle_q_update_f32.argtypes = [p, p, p, c_i64, c_f32]
    lib.evk_oracle_q_update_f32.restype = None
    lib.evk_oracle_reward_draft.argtypes = [p, c_i64, p]
    lib.evk_oracle_reward_draft.restype = None
    lib.evk_oracle_reward_refine.argtypes = [p, p, p, c_i64, p]
    lib.evk_oracle_reward_refine.restype = None
    lib.evk_oracle_reward_normalize.argtypes = [p, c_i64, p, c_i64, c_f64, c_f64, p]
    lib.evk_oracle_reward_normalize.restype = None
    lib.evk_oracle_philox4x32_10.argtypes = [p, p, p]
    lib.evk_oracle_philox4x32_10.restype = None
    lib.evk_oracle_explore.argtypes = [p, p, c_i32, p, c_f64, c_i32, c_f32, ctypes.c_uint64, ctypes.c_uint64,
                                       ctypes.c_uint32, p, p]
    lib.evk_oracle_explore.restype = c_i32
    lib.evk_oracle_explore_zscore.argtypes = lib.evk_oracle_explore.argtypes
    lib.evk_oracle_explore_zscore.restype = c_i32
    lib.evk_oracle_q_update_decay_f64.argtypes = [p, p, p, p, c_i64]
    lib.evk_oracle_q_update_decay_f64.restype = None
    lib.evk_oracle_q_update_decay_f32.argtypes = [p, p, p, p, c_i64]
    lib.evk_oracle_q_update_decay_f32.restype = None
    _lib = lib
    return lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def threads() -> int:
    """Host threads the similarity scan spreads bank rows over."""
    return int(_load().evk_oracle_threads())


def bf16_round(x) -> np.ndarray:
    """fp32 -> bfloat16 bits, round to nearest even (the insert boundary)."""
    x = _c(x, np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().evk_oracle_bf16_round(_ptr(x), _ptr(out), x.size)
    return out


def bf16_decode(bits) -> np.ndarray:
    """bfloat16 bits -> fp64, exact."""
    bits = _c(bits, np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().evk_oracle_bf16_decode(_ptr(bits), _ptr(out), bits.size)
    return out


def sims(bank_bits, query_bits) -> np.ndarray:
    """Inner products of one query with every bank row, fp64 (phase 1 scores)."""
    bank_bits = _c(bank_bits, np.uint16)
    query_bits = _c(query_bits, np.uint16)
    size, d = bank_bits.shape
    assert query_bits.shape == (d,)
    out = np.empty(size, dtype=np.float64)
    _load().evk_oracle_sims(_ptr(bank_bits), size, d, _ptr(query_bits), _ptr(out))
    return out


def rank(sims_row, k1: int, live=None):
    """The ranking step of phase 1 on one query's similarities (entry id = index): the first k1
    by (similarity desc, id asc) after a full sort.  live (uint8 per entry, optional): entries
    marked 0 have been dropped from the memory and are left out.  ids int32 [k1], sims fp64 [k1]."""
    sims_row = _c(sims_row, np.float64)
    assert sims_row.ndim == 1
    ids = np.empty(k1, dtype=np.int32)
    sm = np.empty(k1, dtype=np.float64)
    if live is None:
        _load().evk_oracle_rank(_ptr(sims_row), sims_row.size, k1, _ptr(ids), _ptr(sm))
    else:
        live = _c(live, np.uint8)
        assert live.shape == sims_row.shape
        _load().evk_oracle_rank_live(_ptr(sims_row), _ptr(live), sims_row.size, k1, _ptr(ids), _ptr(sm))
    return ids, sm


def phase1(bank_bits, query_bits, k1: int, live=None):
    """Top-k1 pool per query by (similarity desc, id asc): ids int32, sims fp64.  live: see rank."""
    bank_bits = _c(bank_bits, np.uint16)
    query_bits = _c(query_bits, np.uint16)
    if query_bits.ndim == 1:
        query_bits = query_bits[None, :]
    size, d = bank_bits.shape
    b = query_bits.shape[0]
    assert query_bits.shape[1] == d
    ids = np.empty((b, k1), dtype=np.int32)
    sm = np.empty((b, k1), dtype=np.float64)
    lib = _load()
    for i in range(b):
        if live is None:
            lib.evk_oracle_phase1(_ptr(bank_bits), size, d, _ptr(query_bits[i]), k1,
                                  _ptr(ids[i]), _ptr(sm[i]))
        else:
            ids[i], sm[i] = rank(sims(bank_bits, query_bits[i]) if size else np.zeros(0), k1, live)
    return ids, sm


def phase2(pool_ids, pool_sims, q_stage, w: float, k2: int, zscore: bool = False):
    """Cut each pool to k2 by (1-w)*sim + w*Q (score desc, sim desc, id asc); with zscore the
    two terms are first replaced by their z-scores over the pool."""
    pool_ids = _c(pool_ids, np.int32)
    pool_sims = _c(pool_sims, np.float64)
    q_stage = _c(q_stage, np.float32)
    if pool_ids.ndim == 1:
        pool_ids, pool_sims = pool_ids[None, :], pool_sims[None, :]
    b, k1 = pool_ids.shape
    ids = np.empty((b, k2), dtype=np.int32)
    sc = np.empty((b, k2), dtype=np.float64)
    lib = _load()
    fn = lib.evk_oracle_phase2_zscore if zscore else lib.evk_oracle_phase2
    for i in range(b):
        fn(_ptr(pool_ids[i]), _ptr(pool_sims[i]), k1, _ptr(q_stage), float(w), k2, _ptr(ids[i]), _ptr(sc[i]))
    return ids, sc


def retrieve(bank_bits, query_bits, q_stage, k1: int, k2: int, w: float, zscore: bool = False, live=None):
    """Both phases; returns (ids, scores, pool_ids, pool_sims).  live: see rank."""
    pool_ids, pool_sims = phase1(bank_bits, query_bits, k1, live)
    ids, sc = phase2(pool_ids, pool_sims, q_stage, w, k2, zscore)
    return ids, sc, pool_ids, pool_sims


def q_update_f64(q_stage, ids, rewards, alpha: float) -> np.ndarray:
    """Eq. 4 applied in array order, fp64; returns the new table (input untouched)."""
    q = np.array(q_stage, dtype=np.float64, order="C", copy=True)
    ids = _c(ids, np.int32)
    rewards = _c(rewards, np.float32)
    assert ids.shape == rewards.shape and ids.ndim == 1
    if ids.size:
        assert ids.min() >= 0 and ids.max() < q.size
    _load().evk_oracle_q_update_f64(_ptr(q), _ptr(ids), _ptr(rewards), ids.size, float(alpha))
    return q


def q_update_f32(q_stage, ids, rewards, alpha) -> np.ndarray:
    """Eq. 4 in binary32, three separately rounded operations per step, array order."""
    q = np.array(q_stage, dtype=np.float32, order="C", copy=True)
    ids = _c(ids, np.int32)
    rewards = _c(rewards, np.float32)
    assert ids.shape == rewards.shape and ids.ndim == 1
    if ids.size:
        assert ids.min() >= 0 and ids.max() < q.size
    _load().evk_oracle_q_update_f32(_ptr(q), _ptr(ids), _ptr(rewards), ids.size,
                                    float(np.float32(alpha)))
    return q


def reward_draft(feasible) -> np.ndarray:
    """Eq. 5: +1 if feasible else -1 (fp64)."""
    f = _c(feasible, np.uint8)
    out = np.empty(f.shape, dtype=np.float64)
    _load().evk_oracle_reward_draft(_ptr(f), f.size, _ptr(out))
    return out


def reward_refine(best_latency, latency, feasible) -> np.ndarray:
    """Eq. 6: -1 if infeasible else tanh(log b - log l) (fp64)."""
    b = _c(best_latency, np.float32)
    l = _c(latency, np.float32)
    f = _c(feasible, np.uint8)
    assert b.shape == l.shape == f.shape
    out = np.empty(b.shape, dtype=np.float64)
    _load().evk_oracle_reward_refine(_ptr(b), _ptr(l), _ptr(f), b.size, _ptr(out))
    return out


def reward_normalize(history, raw, sigma_min: float, clip: float = 0.0) -> np.ndarray:
    """Running z-score with the statistics of everything seen before each reward."""
    h = _c(history, np.float64)
    r = _c(raw, np.float32)
    out = np.empty(r.shape, dtype=np.float64)
    _load().evk_oracle_reward_normalize(_ptr(h), h.size, _ptr(r), r.size, float(sigma_min), float(clip), _ptr(out))
    return out


def philox4x32_10(counter, key) -> np.ndarray:
    """One block of Philox4x32-10: counter 4 x uint32, key 2 x uint32 -> 4 x uint32."""
    c = _c(counter, np.uint32)
    k = _c(key, np.uint32)
    out = np.empty(4, dtype=np.uint32)
    _load().evk_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def explore(pool_ids, pool_sims, q_stage, w: float, k2: int, epsilon: float, seed: int, step: int,
            first_query: int = 0, zscore: bool = False):
    """Epsilon-greedy choice per query over canonical pools; returns (ids, scores, explored)."""
    pool_ids = _c(pool_ids, np.int32)
    pool_sims = _c(pool_sims, np.float64)
    q_stage = _c(q_stage, np.float32)
    if pool_ids.ndim == 1:
        pool_ids, pool_sims = pool_ids[None, :], pool_sims[None, :]
    b, k1 = pool_ids.shape
    ids = np.empty((b, k2), dtype=np.int32)
    sc = np.empty((b, k2), dtype=np.float64)
    explored = np.zeros(b, dtype=np.uint8)
    lib = _load()
    fn = lib.evk_oracle_explore_zscore if zscore else lib.evk_oracle_explore
    for i in range(b):
        explored[i] = fn(_ptr(pool_ids[i]), _ptr(pool_sims[i]), k1, _ptr(q_stage), float(w), k2,
                                             float(np.float32(epsilon)), int(seed), int(step), first_query + i,
                                             _ptr(ids[i]), _ptr(sc[i]))
    return ids, sc, explored


def q_update_decay(q_stage, visits, ids, rewards, dtype=np.float32):
    """Eq. 8 with alpha_t = 1/visits (running mean); returns (new table, new visit counts)."""
    q = np.array(q_stage, dtype=dtype, order="C", copy=True)
    v = np.array(visits, dtype=np.uint32, order="C", copy=True)
    ids = _c(ids, np.int32)
    rewards = _c(rewards, np.float32)
    assert ids.shape == rewards.shape and ids.ndim == 1 and q.shape == v.shape
    if ids.size:
        assert ids.min() >= 0 and ids.max() < q.size
    fn = _load().evk_oracle_q_update_decay_f32 if dtype == np.float32 else _load().evk_oracle_q_update_decay_f64
    fn(_ptr(q), _ptr(v), _ptr(ids), _ptr(rewards), ids.size)
    return q, v
