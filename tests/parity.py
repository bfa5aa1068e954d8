"""Comparison rules between the CUDA library and the CPU oracle.

Similarities: the library multiplies bf16 operands exactly and accumulates in fp32
in an order of its own; the oracle accumulates in fp64.  The bound is
    |s_lib - s_orc| <= REL * |s_orc| + ABS * ||q|| * ||e||
with REL = 2e-3 and ABS = 1e-5 (unit-norm Gaussian vectors give |sim| ~ 1/sqrt(d)
with many values near zero, where a purely relative bound means nothing).

Id sets: ranks whose oracle scores lie within that bound of the k-th score are
legitimately ambiguous, so a set is accepted when (a) every oracle entry scoring
above the k-th score by more than the bound is present, and (b) every returned
entry scores no less than the k-th score minus the bound.
"""
from __future__ import annotations

import numpy as np

import oracle

REL = 2e-3
ABS = 1e-5

# Realised exact-match rates, one line per judged case; printed at the end of the test run.
REPORT = []


def record(case, scoring, judged, batch, exact_pool, exact_final):
    kind = {None: "auto", 1: "stream", 2: "tensor"}.get(scoring, str(scoring))
    REPORT.append(f"{case:44s} kernel={kind:6s} judged {judged:4d} of {batch:4d}: "
                  f"pool ids exact {100 * exact_pool:6.2f} %, result ids exact {100 * exact_final:6.2f} %")


def tol(score, scale=1.0):
    return REL * np.abs(score) + ABS * scale


def check_pool(bank_bits, query_bits, k1, pool_ids, pool_sims, norm_scale=1.0, sims=None, live=None):
    """Phase 1 of one query.  Returns True if the id set equals the oracle's exactly.
    sims: this query's oracle similarities if the caller already has them; live: uint8 per entry,
    0 for entries dropped from the memory."""
    size = bank_bits.shape[0]
    n_pool = min(k1, size if live is None else int(np.count_nonzero(live)))
    if sims is None:
        sims = oracle.sims(bank_bits, query_bits) if size else np.zeros(0)
    o_ids, o_sims = oracle.rank(sims, k1, live)
    pool_ids = np.asarray(pool_ids)
    pool_sims = np.asarray(pool_sims, dtype=np.float64)
    # shape of the answer: n_pool real entries, then padding
    assert np.all(pool_ids[:n_pool] >= 0) and np.all(pool_ids[:n_pool] < size), "pool id out of range"
    assert np.all(pool_ids[n_pool:] == -1) and np.all(np.isneginf(pool_sims[n_pool:])), "bad padding"
    real = pool_ids[:n_pool]
    assert len(set(real.tolist())) == n_pool, "duplicate ids in pool"
    assert live is None or np.all(live[real] != 0), "a dropped entry is in the pool"
    if n_pool == 0:
        return True
    # similarities of the returned ids
    want = sims[real]
    err = np.abs(pool_sims[:n_pool] - want)
    assert np.all(err <= tol(want, norm_scale)), f"pool sim error {err.max():.3e}"
    # the library's own order: (sim desc, id asc)
    s = pool_sims[:n_pool]
    assert np.all((s[:-1] > s[1:]) | ((s[:-1] == s[1:]) & (real[:-1] < real[1:]))), "pool not ordered"
    # band rule at the k1 boundary
    s_star = o_sims[n_pool - 1]
    t = tol(s_star, norm_scale)
    must = set(o_ids[:n_pool][o_sims[:n_pool] > s_star + t].tolist())
    assert must <= set(real.tolist()), "pool misses an entry clearly above the boundary"
    assert np.all(want >= s_star - t), "pool holds an entry clearly below the boundary"
    return set(real.tolist()) == set(o_ids[:n_pool].tolist())


def check_final(bank_bits, query_bits, q_stage, w, k2, pool_ids, ids, scores, norm_scale=1.0, zscore=False,
                sims=None):
    """Phase 2 of one query, judged on the library's own pool.  zscore: the pool z-score variant."""
    pool_ids = np.asarray(pool_ids)
    ids = np.asarray(ids)
    scores = np.asarray(scores, dtype=np.float64)
    real = pool_ids[pool_ids >= 0]
    n_out = min(k2, real.size)
    assert np.all(ids[n_out:] == -1) and np.all(np.isneginf(scores[n_out:])), "bad padding"
    if n_out == 0:
        return True
    if sims is None:
        sims = oracle.sims(bank_bits, query_bits)
    o_ids, o_sc = oracle.phase2(real, sims[real], q_stage, w, real.size, zscore)   # the whole pool, ranked
    o_ids, o_sc = o_ids[0], o_sc[0]
    score_of = dict(zip(o_ids.tolist(), o_sc.tolist()))
    got = ids[:n_out]
    assert len(set(got.tolist())) == n_out, "duplicate ids in result"
    assert set(got.tolist()) <= set(real.tolist()), "result id not in pool"
    want = np.array([score_of[i] for i in got.tolist()])
    scale = (1 - w) * norm_scale + w * float(np.max(np.abs(q_stage[real]))) if real.size else 1.0
    if zscore:
        # a similarity off by ABS * ||q|| ||e|| moves its z-score by that over the pool's std
        sd = float(np.std(sims[real]))
        scale = (1 - w) * norm_scale / max(sd, 1e-6) + w
    err = np.abs(scores[:n_out] - want)
    assert np.all(err <= tol(want, max(scale, 1e-30))), f"score error {err.max():.3e}"
    assert np.all(scores[:n_out][:-1] >= scores[:n_out][1:]), "result not ordered by score"
    s_star = o_sc[n_out - 1]
    t = tol(s_star, scale)
    must = set(o_ids[:n_out][o_sc[:n_out] > s_star + t].tolist())
    assert must <= set(got.tolist()), "result misses an entry clearly above the boundary"
    assert np.all(want >= s_star - t), "result holds an entry clearly below the boundary"
    return got.tolist() == o_ids[:n_out].tolist()


def check_retrieve(bank_bits, queries_bits, q_stage, k1, k2, w, out, sample=None, norm_scale=1.0, zscore=False,
                   workers=4, live=None):
    """out = (ids, scores, pool_ids, pool_sims) as host arrays; sample = query indices to judge.
    Returns the share of judged queries whose pool, and whose result, equal the oracle's exactly.
    Each judged query costs the oracle one scan of the bank and one full sort; `workers` queries are
    judged side by side (threads: the oracle's C calls release the interpreter lock)."""
    ids, scores, pool_ids, pool_sims = [np.asarray(x) for x in out]
    b = queries_bits.shape[0]
    sample = list(range(b) if sample is None else sample)
    size = bank_bits.shape[0]

    def judge(i):
        sims = oracle.sims(bank_bits, queries_bits[i]) if size else np.zeros(0)
        ep = bool(check_pool(bank_bits, queries_bits[i], k1, pool_ids[i], pool_sims[i], norm_scale, sims=sims,
                             live=live))
        ef = bool(check_final(bank_bits, queries_bits[i], q_stage, w, k2, pool_ids[i], ids[i], scores[i],
                              norm_scale, zscore, sims=sims))
        return ep, ef

    if workers > 1 and len(sample) > 1 and size * bank_bits.shape[1] > (1 << 22):
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(workers) as pool:
            res = list(pool.map(judge, sample))
    else:
        res = [judge(i) for i in sample]
    n = max(len(res), 1)
    return sum(r[0] for r in res) / n, sum(r[1] for r in res) / n


def check_update(q_before, ids, rewards, alpha, q_after):
    """Stored bits equal the sequential binary32 recurrence; values track the fp64 truth."""
    want32 = oracle.q_update_f32(q_before, ids, rewards, alpha)
    got = np.asarray(q_after, dtype=np.float32)
    bad = np.nonzero(want32.view(np.uint32) != got.view(np.uint32))[0]
    if bad.size:
        # mismatch report: count, share, largest absolute and relative error, index range
        diff = np.abs(got[bad].astype(np.float64) - want32[bad])
        rel = diff / np.maximum(np.abs(want32[bad]), 1e-30)
        raise AssertionError(
            f"{bad.size} of {got.size} entries differ ({100.0 * bad.size / got.size:.3f}%), "
            f"max_abs {diff.max():.3e}, max_rel {rel.max():.3e}, ids {bad.min()}..{bad.max()}")
    # Each step commits three binary32 roundings of relative size u = 2^-24 on numbers no
    # larger than `scale`, and the recurrence shrinks earlier errors by (1 - alpha) per step,
    # so the distance to the fp64 recurrence stays below 4 u scale / alpha.
    a32 = float(np.float32(alpha))
    want64 = oracle.q_update_f64(q_before, ids, rewards, a32)
    scale = max(1.0, float(np.max(np.abs(q_before), initial=0.0)), float(np.max(np.abs(rewards), initial=0.0)))
    assert np.max(np.abs(got - want64), initial=0.0) <= 4 * 2.0 ** -24 * scale / a32
