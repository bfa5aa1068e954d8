"""Pins for the CPU oracle: each check ties an oracle function to something other
than itself — exact rational arithmetic, closed forms and lemmas of Appendix A,
library routines on special cases, invariants, and hand-built banks whose result
is known without computing anything."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits_of(x):
    """bf16 bits through torch's own converter (independent of the oracle's)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


# --------------------------------------------------------------------------
# bfloat16 boundary
# --------------------------------------------------------------------------

def test_bf16_round_known_bit_patterns():
    # 1.0 = 0x3F80; bf16 has 7 explicit mantissa bits, so 1 + 2^-7 is the next value.
    x = np.array([1.0, 1 + 2 ** -7, 1 + 2 ** -8, 1 + 3 * 2 ** -8, 1 + 2 ** -8 + 2 ** -20,
                  -2.5, 0.0, np.inf, -np.inf, 3.3895314e38, 3.4028235e38], dtype=np.float32)
    want = [0x3F80, 0x3F81, 0x3F80, 0x3F82, 0x3F81, 0xC020, 0x0000, 0x7F80, 0xFF80, 0x7F7F, 0x7F80]
    assert oracle.bf16_round(x).tolist() == want
    # halfway cases go to the even neighbour; just above halfway goes up; the largest
    # bf16 value stays, the largest fp32 value rounds up to infinity.


def test_bf16_round_matches_torch_converter():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.standard_normal(200000).astype(np.float32),
                        (rng.standard_normal(1000) * 1e-38).astype(np.float32),  # subnormals
                        rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32).view(np.float32)])
    x = x[~np.isnan(x)]
    assert np.array_equal(oracle.bf16_round(x), bits_of(x))


def test_bf16_decode_is_exact_widening():
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    f = (bits.astype(np.uint32) << 16).view(np.float32)
    got = oracle.bf16_decode(bits)
    ok = ~np.isnan(f)
    assert np.array_equal(got[ok], f[ok].astype(np.float64))
    assert np.all(np.isnan(got[~ok]))


# --------------------------------------------------------------------------
# Phase 1 (dense retrieval of the top-K pool, Section 3.2)
# --------------------------------------------------------------------------

def test_sims_exact_against_rational_arithmetic():
    # small dyadic values: every product and partial sum is exact in fp64, so the
    # result must equal the rational inner product exactly.
    rng = np.random.default_rng(5)
    bank = rng.integers(-64, 65, size=(37, 24)).astype(np.float32) / 32
    q = rng.integers(-64, 65, size=24).astype(np.float32) / 16
    got = oracle.sims(bits_of(bank), bits_of(q))
    for i in range(bank.shape[0]):
        want = sum(Fraction(float(a)) * Fraction(float(b)) for a, b in zip(bank[i], q))
        assert Fraction(float(got[i])) == want


def test_sims_matches_blas_on_random_bf16():
    rng = np.random.default_rng(6)
    bank = bits_of(rng.standard_normal((513, 96)))
    q = bits_of(rng.standard_normal(96))
    got = oracle.sims(bank, q)
    want = oracle.bf16_decode(bank) @ oracle.bf16_decode(q)   # BLAS dgemv, other sum order
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def test_phase1_orthonormal_bank_closed_form():
    # e_i = unit basis vectors (i < d), query = sum_i 2^-i e_i  =>  sim_i = 2^-i exactly,
    # so the pool is ids 0..k1-1 in order, with those powers of two, no tolerance.
    d, n, k1 = 64, 64, 10
    bank = np.eye(n, d, dtype=np.float32)
    q = (2.0 ** -np.arange(d)).astype(np.float32)
    perm = np.random.default_rng(0).permutation(n)          # hide the order in the rows
    ids, sm = oracle.phase1(bits_of(bank[perm]), bits_of(q), k1)
    inv = np.argsort(perm)
    assert ids[0].tolist() == [int(inv[i]) for i in range(k1)]
    assert sm[0].tolist() == [2.0 ** -i for i in range(k1)]


def test_phase1_transposed_operand_would_fail():
    # asymmetric construction: bank row i has a single 1 at column (i+3) mod d, the query
    # is one-hot at column 5: only row 2 scores 1, everything else 0 (ties by id asc).
    d = 16
    bank = np.zeros((d, d), dtype=np.float32)
    for i in range(d):
        bank[i, (i + 3) % d] = 1.0
    q = np.zeros(d, dtype=np.float32)
    q[5] = 1.0
    ids, sm = oracle.phase1(bits_of(bank), bits_of(q), 4)
    assert ids[0].tolist() == [2, 0, 1, 3]
    assert sm[0].tolist() == [1.0, 0.0, 0.0, 0.0]


def test_phase1_brute_force_against_lexsort():
    rng = np.random.default_rng(7)
    bank = bits_of(rng.standard_normal((700, 48)))
    bank[100] = bank[3]            # exact duplicates: equal sims, id-ascending tie-break
    bank[650] = bank[3]
    qs = bits_of(rng.standard_normal((5, 48)))
    ids, sm = oracle.phase1(bank, qs, 64)
    e = oracle.bf16_decode(bank)
    for b in range(5):
        s = e @ oracle.bf16_decode(qs[b])
        np.testing.assert_allclose(oracle.sims(bank, qs[b]), s, rtol=0, atol=1e-12)
        s = oracle.sims(bank, qs[b])  # ordering below is numpy's lexsort, not the oracle's qsort
        order = np.lexsort((np.arange(700), -s))[:64]
        assert ids[b].tolist() == order.tolist()
        assert np.array_equal(sm[b], s[order])
    # the duplicated rows appear in id order wherever they land
    for b in range(5):
        row = list(ids[b])
        if 3 in row and 100 in row and 650 in row:
            assert row.index(3) < row.index(100) < row.index(650)
    # a query equal to the duplicated row puts all three copies at the head of its pool
    ids, sm = oracle.phase1(bank, bank[3], 4)
    assert ids[0, :3].tolist() == [3, 100, 650] and sm[0, 0] == sm[0, 1] == sm[0, 2]


def test_rank_step_is_a_lexsort_with_ties_and_padding():
    # the ranking step taken alone, on similarities with many exact ties
    rng = np.random.default_rng(70)
    s = rng.integers(-3, 4, 500).astype(np.float64) / 4.0
    ids, sm = oracle.rank(s, 120)
    order = np.lexsort((np.arange(500), -s))[:120]
    assert ids.tolist() == order.tolist() and np.array_equal(sm, s[order])
    ids, sm = oracle.rank(s[:7], 10)
    assert ids[7:].tolist() == [-1] * 3 and np.all(np.isneginf(sm[7:]))
    assert ids[:7].tolist() == np.lexsort((np.arange(7), -s[:7])).tolist()
    ids, sm = oracle.rank(np.zeros(0), 3)
    assert ids.tolist() == [-1] * 3
    # and phase 1 is exactly sims followed by rank
    bank = bits_of(rng.standard_normal((300, 24)))
    q = bits_of(rng.standard_normal(24))
    a = oracle.phase1(bank, q, 17)
    b = oracle.rank(oracle.sims(bank, q), 17)
    assert np.array_equal(a[0][0], b[0]) and np.array_equal(a[1][0], b[1])


def test_dropped_entries_equal_retrieval_on_the_compacted_bank():
    # Dropping entries from the memory is the same as never having stored them: retrieval over
    # the bank with a live mask equals retrieval over the bank with those rows removed, once the
    # compacted ids are mapped back.  (Exact ties included: rows 3, 100 and 650 are one vector.)
    rng = np.random.default_rng(71)
    n, d, k1, k2 = 700, 40, 50, 6
    bank = bits_of(rng.standard_normal((n, d)))
    bank[100] = bank[3]
    bank[650] = bank[3]
    qs = np.concatenate([bits_of(rng.standard_normal((4, d))), bank[3:4]])
    q_stage = rng.random(n).astype(np.float32)
    live = (rng.random(n) < 0.6).astype(np.uint8)
    live[3], live[100], live[650] = 1, 0, 1          # the middle copy of the tie is gone
    kept = np.nonzero(live)[0]
    got = oracle.retrieve(bank, qs, q_stage, k1, k2, 0.4, live=live)
    want = oracle.retrieve(bank[kept], qs, q_stage[kept], k1, k2, 0.4)
    assert np.array_equal(got[2], kept[want[2]]) and np.array_equal(got[3], want[3])
    assert np.array_equal(got[0], kept[want[0]]) and np.array_equal(got[1], want[1])
    assert got[2][4, :2].tolist() == [3, 650]          # the query equal to the tied rows: 100 is skipped
    # nothing dropped: the plain retrieval; everything dropped: padding only; fewer live than k1
    all_live = oracle.retrieve(bank, qs, q_stage, k1, k2, 0.4, live=np.ones(n, np.uint8))
    plain = oracle.retrieve(bank, qs, q_stage, k1, k2, 0.4)
    assert all(np.array_equal(a, b) for a, b in zip(all_live, plain))
    none = oracle.phase1(bank, qs[0], 5, live=np.zeros(n, np.uint8))
    assert none[0].tolist() == [[-1] * 5] and np.all(np.isneginf(none[1]))
    few = np.zeros(n, np.uint8)
    few[[9, 500, 77]] = 1
    ids, sm = oracle.phase1(bank, qs[1], 8, live=few)
    assert sorted(ids[0, :3].tolist()) == [9, 77, 500] and ids[0, 3:].tolist() == [-1] * 5
    # the ranking step alone, against a lexsort restricted to the live entries
    s = rng.integers(-3, 4, 300).astype(np.float64)
    lv = (rng.random(300) < 0.5).astype(np.uint8)
    ids, sm = oracle.rank(s, 40, live=lv)
    order = [i for i in np.lexsort((np.arange(300), -s)) if lv[i]][:40]
    assert ids.tolist() == order and np.array_equal(sm, s[order])


def test_phase1_k1_equals_size_is_a_permutation_and_padding():
    rng = np.random.default_rng(8)
    bank = bits_of(rng.standard_normal((33, 16)))
    q = bits_of(rng.standard_normal(16))
    ids, sm = oracle.phase1(bank, q, 33)
    assert sorted(ids[0].tolist()) == list(range(33))
    assert np.all(np.diff(sm[0]) <= 0)
    ids, sm = oracle.phase1(bank, q, 40)      # pool larger than the bank: cold start
    assert sorted(ids[0, :33].tolist()) == list(range(33))
    assert ids[0, 33:].tolist() == [-1] * 7 and np.all(np.isneginf(sm[0, 33:]))


def test_phase1_row_permutation_permutes_ids_only():
    rng = np.random.default_rng(9)
    bank = bits_of(rng.standard_normal((257, 32)))
    q = bits_of(rng.standard_normal(32))
    perm = rng.permutation(257)
    ids_a, sm_a = oracle.phase1(bank, q, 20)
    ids_b, sm_b = oracle.phase1(bank[perm], q, 20)
    assert np.array_equal(sm_a, sm_b)
    assert perm[ids_b[0]].tolist() == ids_a[0].tolist()


# --------------------------------------------------------------------------
# Phase 2 (value filter of the pool, Section 3.2)
# --------------------------------------------------------------------------

def _pool(rng, n=500, k1=40):
    ids = rng.permutation(n)[:k1].astype(np.int32)
    sims = np.sort(rng.standard_normal(k1))[::-1].copy()
    q = rng.random(n).astype(np.float32)
    return ids, sims, q


def test_phase2_w1_is_the_papers_rule_rank_by_q_alone():
    rng = np.random.default_rng(20)
    ids, sims, q = _pool(rng)
    out_ids, out_sc = oracle.phase2(ids, sims, q, 1.0, 7)
    want = ids[np.argsort(-q[ids].astype(np.float64), kind="stable")][:7]
    assert out_ids[0].tolist() == want.tolist()
    assert np.array_equal(out_sc[0], q[want].astype(np.float64))


def test_phase2_w0_and_equal_q_reduce_to_similarity_ranking():
    rng = np.random.default_rng(21)
    ids, sims, q = _pool(rng)
    out_ids, out_sc = oracle.phase2(ids, sims, q, 0.0, 9)
    assert out_ids[0].tolist() == ids[:9].tolist()
    assert np.array_equal(out_sc[0], sims[:9])
    # equal Q for every entry: any w < 1 keeps the similarity order ...
    qc = np.full_like(q, 0.625)
    for w in (0.25, 0.5, 0.875):
        out_ids, _ = oracle.phase2(ids, sims, qc, w, 9)
        assert out_ids[0].tolist() == ids[:9].tolist()
    # ... and w = 1 makes every score equal, where the secondary key (sim desc) decides.
    out_ids, out_sc = oracle.phase2(ids, sims, qc, 1.0, 9)
    assert out_ids[0].tolist() == ids[:9].tolist()
    assert np.all(out_sc[0] == 0.625)


def test_phase2_equal_q_large_offset_collapses_scores_but_keeps_order():
    # adding a large equal Q swallows differences of 1e-17 between scores; the secondary
    # key keeps similarity order.
    ids = np.arange(6, dtype=np.int32)
    sims = np.array([0.5, 0.5 - 1e-17, 0.25, 0.25 - 1e-18, 0.1, 0.0])
    q = np.full(6, 1024.0, dtype=np.float32)
    out_ids, _ = oracle.phase2(ids, sims, q, 0.5, 6)
    assert out_ids[0].tolist() == [0, 1, 2, 3, 4, 5]
    out_ids, _ = oracle.phase2(ids[::-1].copy(), sims[::-1].copy(), q, 0.5, 6)
    assert out_ids[0].tolist() == [0, 1, 2, 3, 4, 5]


def test_phase2_k2_equals_k1_keeps_the_id_set():
    rng = np.random.default_rng(22)
    ids, sims, q = _pool(rng)
    for w in (0.0, 0.3, 1.0):
        out_ids, _ = oracle.phase2(ids, sims, q, w, len(ids))
        assert sorted(out_ids[0].tolist()) == sorted(ids.tolist())


def test_phase2_hand_worked_example_exact():
    # dyadic numbers, w = 1/4: score = 3/4 sim + 1/4 Q, computed here with rationals.
    ids = np.array([7, 2, 9, 4, 0], dtype=np.int32)
    sims = np.array([0.875, 0.75, 0.5, 0.25, 0.125])
    q = np.zeros(10, dtype=np.float32)
    q[[7, 2, 9, 4, 0]] = [0.0, 0.5, 1.0, 0.25, 1.0]
    w = Fraction(1, 4)
    sc = {int(i): (1 - w) * Fraction(float(s)) + w * Fraction(float(q[i])) for i, s in zip(ids, sims)}
    # 7: 21/32, 2: 22/32, 9: 20/32, 4: 8/32, 0: 11/32
    assert sc == {7: Fraction(21, 32), 2: Fraction(22, 32), 9: Fraction(20, 32),
                  4: Fraction(8, 32), 0: Fraction(11, 32)}
    out_ids, out_sc = oracle.phase2(ids, sims, q, 0.25, 3)
    assert out_ids[0].tolist() == [2, 7, 9]
    assert [Fraction(float(x)) for x in out_sc[0]] == [Fraction(22, 32), Fraction(21, 32), Fraction(20, 32)]


def test_phase2_monotone_in_q_and_ignores_padding():
    rng = np.random.default_rng(23)
    ids, sims, q = _pool(rng)
    base_ids, _ = oracle.phase2(ids, sims, q, 0.5, len(ids))
    target = int(base_ids[0, 20])
    q2 = q.copy()
    q2[target] += 0.5
    new_ids, _ = oracle.phase2(ids, sims, q2, 0.5, len(ids))
    assert list(new_ids[0]).index(target) <= 20
    # padded pool slots (id -1) never reach the output
    pid = np.concatenate([ids[:5], np.full(3, -1, np.int32)])
    ps = np.concatenate([sims[:5], np.full(3, -np.inf)])
    out_ids, out_sc = oracle.phase2(pid, ps, q, 0.5, 8)
    assert sorted(out_ids[0, :5].tolist()) == sorted(ids[:5].tolist())
    assert out_ids[0, 5:].tolist() == [-1, -1, -1] and np.all(np.isneginf(out_sc[0, 5:]))


def test_retrieve_is_phase1_then_phase2_and_stage_tables_are_separate():
    rng = np.random.default_rng(24)
    bank = bits_of(rng.standard_normal((300, 32)))
    qs = bits_of(rng.standard_normal((3, 32)))
    q_tab = rng.random((2, 300)).astype(np.float32)
    r0 = oracle.retrieve(bank, qs, q_tab[0], 16, 4, 1.0)
    r1 = oracle.retrieve(bank, qs, q_tab[1], 16, 4, 1.0)
    assert np.array_equal(r0[2], r1[2])          # the pool does not depend on the stage
    for b in range(3):
        assert r0[0][b].tolist() == r0[2][b][np.argsort(-q_tab[0][r0[2][b]], kind="stable")][:4].tolist()
        assert r1[0][b].tolist() == r1[2][b][np.argsort(-q_tab[1][r1[2][b]], kind="stable")][:4].tolist()


# --------------------------------------------------------------------------
# Eq. 4 / Eq. 8 (unified value update) and Appendix A
# --------------------------------------------------------------------------

def test_update_exact_rational_recurrence():
    # alpha = 1/4 and dyadic rewards: every step is exact in fp64 for a few steps, so the
    # oracle must equal the rational recurrence Q + a(r - Q) exactly.
    ids = np.array([3, 1, 3, 3, 0, 1, 3], dtype=np.int32)
    r = np.array([1.0, -1.0, 0.5, 1.0, 0.25, 1.0, -1.0], dtype=np.float32)
    q0 = np.array([0.0, 0.5, 0.125, -0.75], dtype=np.float32)
    got = oracle.q_update_f64(q0, ids, r, 0.25)
    want = [Fraction(float(x)) for x in q0]
    a = Fraction(1, 4)
    for i, rv in zip(ids, r):
        want[i] = want[i] + a * (Fraction(float(rv)) - want[i])
    assert [Fraction(float(x)) for x in got] == want
    # binary32 can also hold these exactly
    got32 = oracle.q_update_f32(q0, ids, r, 0.25)
    assert [Fraction(float(x)) for x in got32] == want


def test_update_golden_dyadic_sequence():
    # Eq. 4 with alpha = 1/2, Q0 = 0, r = 1 every step: 1/2, 3/4, 7/8, ... = 1 - 2^-t.
    with open(os.path.join(GOLDEN, "eq4_dyadic.json")) as f:
        g = json.load(f)
    q = np.zeros(1, dtype=np.float32)
    for t, want in enumerate(g["q_after_step"], start=1):
        q64 = oracle.q_update_f64(np.zeros(1, np.float32), np.zeros(t, np.int32),
                                  np.ones(t, np.float32), g["alpha"])
        assert q64[0] == want == 1 - 2.0 ** -t
    q = oracle.q_update_f32(q, np.zeros(len(g["q_after_step"]), np.int32),
                            np.ones(len(g["q_after_step"]), np.float32), g["alpha"])
    assert float(q[0]) == g["q_after_step"][-1]


def test_update_closed_form_constant_reward_and_unrolled_form():
    # Lemma (constant step size), unrolled: Q_t = (1-a)^t Q_0 + a sum_k (1-a)^(t-1-k) R_k.
    rng = np.random.default_rng(30)
    a32 = np.float32(0.1)
    a = float(a32)
    t = 200
    r = rng.standard_normal(t).astype(np.float32)
    q0 = np.array([0.3], dtype=np.float32)
    got = oracle.q_update_f64(q0, np.zeros(t, np.int32), r, a)[0]
    want = (1 - a) ** t * float(q0[0]) + a * sum((1 - a) ** (t - 1 - k) * float(r[k]) for k in range(t))
    assert abs(got - want) < 1e-12
    # constant reward: r + (1-a)^t (Q0 - r)
    got = oracle.q_update_f64(q0, np.zeros(t, np.int32), np.full(t, 0.75, np.float32), a)[0]
    assert abs(got - (0.75 + (1 - a) ** t * (float(q0[0]) - 0.75))) < 1e-12


def test_update_stays_in_convex_hull():
    # Lemma (bounded rewards imply bounded values): each step is a convex combination.
    rng = np.random.default_rng(31)
    n, m = 50, 5000
    ids = rng.integers(0, n, m).astype(np.int32)
    r = rng.uniform(-1, 1, m).astype(np.float32)
    q0 = rng.uniform(-1, 1, n).astype(np.float32)
    for a in (0.05, 0.5, 1.0):
        q64 = oracle.q_update_f64(q0, ids, r, a)
        q32 = oracle.q_update_f32(q0, ids, r, a)
        assert np.all(np.abs(q64) <= 1.0) and np.all(np.abs(q32) <= 1.0 + 1e-6)
        for i in range(n):
            vals = np.concatenate([[q0[i]], r[ids == i]]).astype(np.float64)
            assert vals.min() - 1e-12 <= q64[i] <= vals.max() + 1e-12
    # alpha = 1 replaces the value by the last reward of each entry (in exact arithmetic)
    q64 = oracle.q_update_f64(q0, ids, r, 1.0)
    for i in range(n):
        hits = np.nonzero(ids == i)[0]
        if hits.size:
            assert abs(q64[i] - float(r[hits[-1]])) < 1e-15


def test_update_order_split_and_commutation():
    rng = np.random.default_rng(32)
    n, m = 20, 400
    ids = rng.integers(0, n, m).astype(np.int32)
    r = rng.standard_normal(m).astype(np.float32)
    q0 = rng.standard_normal(n).astype(np.float32)
    a = np.float32(0.3)
    whole = oracle.q_update_f32(q0, ids, r, a)
    for cut in (0, 1, 137, m):
        part = oracle.q_update_f32(oracle.q_update_f32(q0, ids[:cut], r[:cut], a), ids[cut:], r[cut:], a)
        assert np.array_equal(whole.view(np.uint32), part.view(np.uint32))
    # a stable regrouping by entry (which keeps each entry's own order) changes nothing ...
    order = np.argsort(ids, kind="stable")
    regroup = oracle.q_update_f32(q0, ids[order], r[order], a)
    assert np.array_equal(whole.view(np.uint32), regroup.view(np.uint32))
    # ... but reversing the order of one entry's rewards does (order matters within an entry)
    i0 = np.bincount(ids).argmax()
    hits = np.nonzero(ids == i0)[0]
    r_rev = r.copy()
    r_rev[hits] = r[hits][::-1]
    assert oracle.q_update_f64(q0, ids, r_rev, float(a))[i0] != oracle.q_update_f64(q0, ids, r, float(a))[i0]
    # entries that are not named keep their bits
    q_small = oracle.q_update_f32(q0, np.array([4, 4], np.int32), np.array([1, 0], np.float32), a)
    mask = np.arange(n) != 4
    assert np.array_equal(q_small[mask].view(np.uint32), q0[mask].view(np.uint32))


def test_update_f32_matches_numpy_float32_scalar_arithmetic():
    # numpy float32 scalars round after every operation: an independent binary32 machine.
    rng = np.random.default_rng(33)
    n, m = 64, 3000
    ids = rng.integers(0, n, m).astype(np.int32)
    r = rng.lognormal(0, 0.5, m).astype(np.float32)
    q0 = rng.random(n).astype(np.float32)
    for a in (np.float32(0.1), np.float32(0.05), np.float32(1.0)):
        got = oracle.q_update_f32(q0, ids, r, a)
        want = q0.copy()
        for i, rv in zip(ids, r):
            diff = np.float32(rv - want[i])
            step = np.float32(a * diff)
            want[i] = np.float32(want[i] + step)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # a fused multiply-add would differ somewhere on this stream: make sure the check bites
    n_diff = 0
    a = np.float32(0.1)
    want = q0.copy()
    for i, rv in zip(ids, r):
        diff = np.float32(rv - want[i])
        fma = np.float32(float(want[i]) + float(a) * float(diff))     # single rounding
        want[i] = np.float32(want[i] + np.float32(a * diff))
        n_diff += int(fma != want[i])
    assert n_diff > 0


def test_update_f32_tracks_f64_truth():
    rng = np.random.default_rng(34)
    n, m = 100, 20000
    ids = rng.integers(0, n, m).astype(np.int32)
    r = (rng.random(m) < 0.4).astype(np.float32)
    q0 = rng.random(n).astype(np.float32)
    a = np.float32(0.05)
    q32 = oracle.q_update_f32(q0, ids, r, a)
    q64 = oracle.q_update_f64(q0, ids, r, float(a))
    assert np.max(np.abs(q32 - q64)) < 1e-6


def test_update_ema_statistics():
    # Lemma (EMA dynamics): E[Q_t] -> mu, Var(Q_t) -> alpha/(2-alpha) sigma_R^2.
    rng = np.random.default_rng(35)
    n, steps, a = 4000, 300, 0.2
    mu, sigma = 0.3, 0.7
    ids = np.tile(np.arange(n, dtype=np.int32), steps)
    r = (mu + sigma * rng.standard_normal(n * steps)).astype(np.float32)
    q = oracle.q_update_f64(np.zeros(n, np.float32), ids, r, a)
    assert abs(q.mean() - mu) < 0.02
    assert abs(q.var() / (a / (2 - a) * sigma ** 2) - 1) < 0.1


# --------------------------------------------------------------------------
# Decreasing step size (Appendix A, Robbins-Monro lemma): alpha_t = 1 / visits
# --------------------------------------------------------------------------

def test_decay_update_is_the_running_mean():
    # with alpha_t = 1/t the first update overwrites Q_0 and Q_t is the mean of the rewards so far
    rng = np.random.default_rng(40)
    n, m = 30, 2000
    ids = rng.integers(0, n, m).astype(np.int32)
    r = (rng.integers(-8, 9, m) / 8).astype(np.float32)
    q0 = rng.standard_normal(n).astype(np.float32)
    q64, v = oracle.q_update_decay(q0, np.zeros(n, np.uint32), ids, r, dtype=np.float64)
    assert v.tolist() == np.bincount(ids, minlength=n).tolist()
    for i in range(n):
        hits = r[ids == i]
        want = Fraction(0)
        for x in hits:
            want += Fraction(float(x))
        if len(hits):
            assert abs(q64[i] - float(want / len(hits))) < 1e-12
        else:
            assert q64[i] == q0[i]
    # continuing from stored counts equals one long batch; alpha_t satisfies sum = inf, sum of squares < inf
    qa, va = oracle.q_update_decay(q0, np.zeros(n, np.uint32), ids[:700], r[:700], dtype=np.float32)
    qb, vb = oracle.q_update_decay(qa, va, ids[700:], r[700:], dtype=np.float32)
    qc, vc = oracle.q_update_decay(q0, np.zeros(n, np.uint32), ids, r, dtype=np.float32)
    assert np.array_equal(qb.view(np.uint32), qc.view(np.uint32)) and np.array_equal(vb, vc)
    assert np.max(np.abs(qc - q64)) < 1e-5


def test_decay_update_f32_matches_numpy_scalars_and_converges():
    rng = np.random.default_rng(41)
    n, m = 8, 4000
    ids = rng.integers(0, n, m).astype(np.int32)
    r = (0.3 + 0.5 * rng.standard_normal(m)).astype(np.float32)
    q0 = np.zeros(n, np.float32)
    got, _ = oracle.q_update_decay(q0, np.zeros(n, np.uint32), ids, r)
    want, cnt = q0.copy(), np.zeros(n, np.int64)
    for i, rv in zip(ids, r):
        cnt[i] += 1
        alpha = np.float32(1.0) / np.float32(cnt[i])
        want[i] = np.float32(want[i] + np.float32(alpha * np.float32(rv - want[i])))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.max(np.abs(got - 0.3)) < 0.1          # lemma: Q_t -> mu
