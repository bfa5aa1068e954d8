/*
 * evk_oracle.c — TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of what the value-driven memory computes:
 * the two-phase retrieval of Section 3.2 ("Memory Architecture and Value-Driven
 * Retrieval") and the unified value update of Eq. 4 (restated as Eq. 8 in
 * Appendix A).  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  It shares no code with the CUDA library and never sees a
 * value the CUDA library produced.
 *
 * Stored embeddings and queries are bfloat16 bit patterns (uint16_t); they are
 * widened to fp64 exactly, so every product below is exact and every sum is a
 * plain left-to-right fp64 sum over the embedding dimension.
 *
 * Every function here is pinned by tests/test_oracle_*.py against closed forms,
 * invariants, library routines and brute force; none is "parity unpinned" except
 * the general mixing weight 0 < w < 1 of evk_oracle_phase2, whose formula is a
 * reading (the paper's own rule is w = 1) and is pinned only through its special
 * cases, a hand-worked exact example and monotonicity, and the pool z-score
 * variant evk_oracle_phase2_zscore, which the paper does not have at all.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- bfloat16 <-> IEEE ------------------------------------------------- */

/* bfloat16 is the upper half of an IEEE binary32; widening is exact. */
static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Round-to-nearest-even narrowing of binary32 to bfloat16 (the storage
 * precision of the bank; the rounding is part of the insert boundary). */
static uint16_t f32_to_bf16(float x) {
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) /* NaN: keep sign, force quiet */
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

void evk_oracle_bf16_round(const float *x, uint16_t *out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16(x[i]);
}

void evk_oracle_bf16_decode(const uint16_t *bits, double *out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_f64(bits[i]);
}

int evk_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- Phase 1: dense retrieval (Section 3.2) ----------------------------- */

/* sim[i] = <q, e_i> for every stored entry i < size.  Rows are independent, so
 * they may be spread over host threads; each row's sum is sequential. */
void evk_oracle_sims(const uint16_t *bank, int64_t size, int32_t d,
                     const uint16_t *query, double *sims) {
    double *q = (double *)malloc((size_t)d * sizeof(double));
    for (int32_t j = 0; j < d; ++j) q[j] = bf16_to_f64(query[j]);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < size; ++i) {
        const uint16_t *e = bank + i * (int64_t)d;
        double acc = 0.0;
        for (int32_t j = 0; j < d; ++j) acc += q[j] * bf16_to_f64(e[j]);
        sims[i] = acc;
    }
    free(q);
}

typedef struct {
    double key;  /* primary, descending   */
    double key2; /* secondary, descending */
    int32_t id;  /* last, ascending       */
} ranked_t;

static int ranked_cmp(const void *a, const void *b) {
    const ranked_t *x = (const ranked_t *)a, *y = (const ranked_t *)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    if (x->key2 > y->key2) return -1;
    if (x->key2 < y->key2) return 1;
    return (x->id > y->id) - (x->id < y->id);
}

/* Ranking step of the candidate pool: the `size` similarities sims[] (entry id = index) are
 * fully sorted by (similarity descending, id ascending); the first min(k1, n_live) are the
 * pool.  live[] (may be NULL: every entry is live) marks entries that have been dropped from
 * the memory with 0: a dropped entry is simply not there (it takes no place in the order and
 * cannot be returned), while the ids of the others stay what they were.  Unused slots get id -1
 * and similarity -inf.  Returns the pool length. */
int32_t evk_oracle_rank_live(const double *sims, const uint8_t *live, int64_t size, int32_t k1,
                             int32_t *pool_ids, double *pool_sims) {
    for (int32_t j = 0; j < k1; ++j) { pool_ids[j] = -1; pool_sims[j] = -INFINITY; }
    if (size <= 0) return 0;
    ranked_t *r = (ranked_t *)malloc((size_t)size * sizeof(ranked_t));
    int64_t n = 0;
    for (int64_t i = 0; i < size; ++i) {
        if (live && !live[i]) continue;
        r[n].key = sims[i]; r[n].key2 = 0.0; r[n].id = (int32_t)i;
        ++n;
    }
    qsort(r, (size_t)n, sizeof(ranked_t), ranked_cmp);
    int32_t n_pool = (int32_t)((int64_t)k1 < n ? (int64_t)k1 : n);
    for (int32_t j = 0; j < n_pool; ++j) { pool_ids[j] = r[j].id; pool_sims[j] = r[j].key; }
    free(r);
    return n_pool;
}

int32_t evk_oracle_rank(const double *sims, int64_t size, int32_t k1,
                        int32_t *pool_ids, double *pool_sims) {
    return evk_oracle_rank_live(sims, NULL, size, k1, pool_ids, pool_sims);
}

/* The top-K candidate pool C(x): every stored entry's similarity (evk_oracle_sims), then the
 * ranking step above. */
int32_t evk_oracle_phase1(const uint16_t *bank, int64_t size, int32_t d,
                          const uint16_t *query, int32_t k1,
                          int32_t *pool_ids, double *pool_sims) {
    if (size <= 0) return evk_oracle_rank(NULL, 0, k1, pool_ids, pool_sims);
    double *sims = (double *)malloc((size_t)size * sizeof(double));
    evk_oracle_sims(bank, size, d, query, sims);
    const int32_t n_pool = evk_oracle_rank(sims, size, k1, pool_ids, pool_sims);
    free(sims);
    return n_pool;
}

/* ---- Phase 2: value filter (Section 3.2) -------------------------------- */

/* The pool is cut down to the final k2 items with the stage's value estimates.
 * score = (1-w)*sim + w*Q_stage[id]; w = 1 is the paper's rule (rank by Q alone),
 * w = 0 its similarity-only ablation arm.  Order: (score desc, sim desc, id asc).
 * q_stage is the fp32 value table of ONE stage, widened exactly.  Pool slots with
 * id < 0 are padding and are ignored.  Unused outputs get id -1, score -inf. */
int32_t evk_oracle_phase2(const int32_t *pool_ids, const double *pool_sims, int32_t k1,
                          const float *q_stage, double w, int32_t k2,
                          int32_t *ids_out, double *scores_out) {
    ranked_t *r = (ranked_t *)malloc((size_t)(k1 > 0 ? k1 : 1) * sizeof(ranked_t));
    int32_t n = 0;
    for (int32_t j = 0; j < k1; ++j) {
        if (pool_ids[j] < 0) continue;
        double qv = (double)q_stage[pool_ids[j]];
        r[n].key = (1.0 - w) * pool_sims[j] + w * qv;
        r[n].key2 = pool_sims[j];
        r[n].id = pool_ids[j];
        ++n;
    }
    qsort(r, (size_t)n, sizeof(ranked_t), ranked_cmp);
    int32_t n_out = n < k2 ? n : k2;
    for (int32_t j = 0; j < k2; ++j) { ids_out[j] = -1; scores_out[j] = -INFINITY; }
    for (int32_t j = 0; j < n_out; ++j) { ids_out[j] = r[j].id; scores_out[j] = r[j].key; }
    free(r);
    return n_out;
}

/* Pool z-scores: a variant of the value filter with no counterpart in the paper (which
 * normalises rewards, not scores).  Over the valid entries of ONE query's pool, each term
 * is replaced by its z-score, z(x) = (x - mean) / std with the population standard
 * deviation, z = 0 where std <= 1e-6; then score = (1-w)*z(sim) + w*z(Q_stage[id]).
 * Writes the n valid entries' scores, in pool order, to scores[]; returns n. */
static int32_t zscore_pool_scores(const int32_t *pool_ids, const double *pool_sims, int32_t k1,
                                  const float *q_stage, double w, double *scores) {
    int32_t n = 0;
    double mean_s = 0.0, mean_q = 0.0, var_s = 0.0, var_q = 0.0;
    for (int32_t j = 0; j < k1; ++j) {
        if (pool_ids[j] < 0) continue;
        mean_s += pool_sims[j];
        mean_q += (double)q_stage[pool_ids[j]];
        ++n;
    }
    if (n == 0) return 0;
    mean_s /= n;
    mean_q /= n;
    for (int32_t j = 0; j < k1; ++j) {
        if (pool_ids[j] < 0) continue;
        const double ds = pool_sims[j] - mean_s, dq = (double)q_stage[pool_ids[j]] - mean_q;
        var_s += ds * ds;
        var_q += dq * dq;
    }
    const double sd_s = sqrt(var_s / n), sd_q = sqrt(var_q / n);
    int32_t m = 0;
    for (int32_t j = 0; j < k1; ++j) {
        if (pool_ids[j] < 0) continue;
        const double zs = sd_s > 1e-6 ? (pool_sims[j] - mean_s) / sd_s : 0.0;
        const double zq = sd_q > 1e-6 ? ((double)q_stage[pool_ids[j]] - mean_q) / sd_q : 0.0;
        scores[m++] = (1.0 - w) * zs + w * zq;
    }
    return n;
}

/* evk_oracle_phase2 with pool z-scores in place of the raw terms; same order rule and
 * padding.  "Parity unpinned" as a formula (it is this library's variant); pinned through
 * what z-scoring fixes: zero mean and unit variance over the pool, invariance under a
 * positive affine change of Q, the orders at w = 0 and w = 1, a hand-worked example and
 * scipy's zscore. */
int32_t evk_oracle_phase2_zscore(const int32_t *pool_ids, const double *pool_sims, int32_t k1,
                                 const float *q_stage, double w, int32_t k2,
                                 int32_t *ids_out, double *scores_out) {
    ranked_t *r = (ranked_t *)malloc((size_t)(k1 > 0 ? k1 : 1) * sizeof(ranked_t));
    double *sc = (double *)malloc((size_t)(k1 > 0 ? k1 : 1) * sizeof(double));
    const int32_t n = zscore_pool_scores(pool_ids, pool_sims, k1, q_stage, w, sc);
    int32_t m = 0;
    for (int32_t j = 0; j < k1; ++j) {
        if (pool_ids[j] < 0) continue;
        r[m].key = sc[m];
        r[m].key2 = pool_sims[j];
        r[m].id = pool_ids[j];
        ++m;
    }
    qsort(r, (size_t)n, sizeof(ranked_t), ranked_cmp);
    int32_t n_out = n < k2 ? n : k2;
    for (int32_t j = 0; j < k2; ++j) { ids_out[j] = -1; scores_out[j] = -INFINITY; }
    for (int32_t j = 0; j < n_out; ++j) { ids_out[j] = r[j].id; scores_out[j] = r[j].key; }
    free(sc);
    free(r);
    return n_out;
}

/* ---- Eq. 4: unified value update ---------------------------------------- */

/* Q <- Q + alpha*(r - Q) for each (id, reward) strictly in array order, on one
 * stage's table.  fp64 truth. */
void evk_oracle_q_update_f64(double *q_stage, const int32_t *ids, const float *rewards,
                             int64_t m, double alpha) {
    for (int64_t t = 0; t < m; ++t) {
        double q = q_stage[ids[t]];
        q_stage[ids[t]] = q + alpha * ((double)rewards[t] - q);
    }
}

/* The same recurrence in binary32: a subtraction, a multiplication and an
 * addition, each rounded to nearest on its own (this file is compiled with
 * -ffp-contract=off; the volatile temporaries also keep x87-style excess
 * precision and fusing out).  This is the bit-level definition of the stored
 * table after a batch. */
void evk_oracle_q_update_f32(float *q_stage, const int32_t *ids, const float *rewards,
                             int64_t m, float alpha) {
    for (int64_t t = 0; t < m; ++t) {
        volatile float q = q_stage[ids[t]];
        volatile float diff = rewards[t] - q;
        volatile float step = alpha * diff;
        volatile float next = q + step;
        q_stage[ids[t]] = next;
    }
}

/* ---- Rewards (Eq. 5, Eq. 6) and their online normalisation (Appendix A) --------- */

/* Eq. 5: the drafting reward is +1 for a feasible kernel and -1 otherwise. */
void evk_oracle_reward_draft(const uint8_t *feasible, int64_t n, double *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = feasible[i] ? 1.0 : -1.0;
}

/* Eq. 6: -1 for an infeasible kernel, otherwise tanh(log b - log l) with b the best
 * latency so far and l the new one (the speed-up ratio rho = b / l enters as
 * tanh(log rho), Appendix A "Reward definitions by stage"). */
void evk_oracle_reward_refine(const float *best, const float *latency, const uint8_t *feasible,
                              int64_t n, double *out) {
    for (int64_t i = 0; i < n; ++i)
        out[i] = feasible[i] ? tanh(log((double)best[i]) - log((double)latency[i])) : -1.0;
}

/* Running z-score of the raw rewards (Appendix A, "Stability of Online Normalization"):
 *   R_t = (r_t - mu_{t-1}) / max(sigma_{t-1}, sigma_min),   optionally clipped to [-clip, clip],
 * with mu_t the mean and sigma_t the POPULATION standard deviation of r_1..r_t, both
 * recomputed here from their definitions for every t (quadratic work: small inputs only).
 * history[0..n_hist) are the raw rewards of earlier calls.  While fewer than two rewards
 * have been seen the raw reward passes through unchanged.  clip <= 0 disables clipping. */
void evk_oracle_reward_normalize(const double *history, int64_t n_hist, const float *raw, int64_t n,
                                 double sigma_min, double clip, double *out) {
    for (int64_t t = 0; t < n; ++t) {
        const int64_t seen = n_hist + t;
        double r = (double)raw[t];
        if (seen >= 2) {
            double mu = 0.0;
            for (int64_t k = 0; k < seen; ++k) mu += (k < n_hist) ? history[k] : (double)raw[k - n_hist];
            mu /= (double)seen;
            double var = 0.0;
            for (int64_t k = 0; k < seen; ++k) {
                const double v = ((k < n_hist) ? history[k] : (double)raw[k - n_hist]) - mu;
                var += v * v;
            }
            double sigma = sqrt(var / (double)seen);
            if (sigma < sigma_min) sigma = sigma_min;
            r = (r - mu) / sigma;
        }
        if (clip > 0.0) r = r > clip ? clip : (r < -clip ? -clip : r);
        out[t] = r;
    }
}

/* ---- Exploration: epsilon-greedy choice of the context (Section 3.3) ------------- */

/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
 * SC'11): ten rounds of two 32x32->64 multiplications and key bumps. */
void evk_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The j-th 32-bit word of the stream of (seed, step, query): block j/4 of the generator
 * with counter (query, step_lo, step_hi, block) and key (seed_lo, seed_hi). */
static uint32_t explore_word(uint64_t seed, uint64_t step, uint32_t query, uint32_t j) {
    const uint32_t ctr[4] = {query, (uint32_t)step, (uint32_t)(step >> 32), j / 4};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    evk_oracle_philox4x32_10(ctr, key, out);
    return out[j % 4];
}

/* Epsilon-greedy over the pool of one query.  Word 0 of the query's stream decides: with
 * u = (word >> 8) * 2^-24 < epsilon the context is min(k2, n) pool entries drawn uniformly
 * without replacement (a partial Fisher-Yates shuffle of the pool positions, position i
 * swapped with i + floor(word_{i+1} * (n - i) / 2^32)), in draw order, each with its mixed
 * score; otherwise it is the greedy result of evk_oracle_phase2.  The pool must be in its
 * canonical order (similarity descending, id ascending).  Returns 1 if the query explored. */
int32_t evk_oracle_explore(const int32_t *pool_ids, const double *pool_sims, int32_t k1,
                           const float *q_stage, double w, int32_t k2, float epsilon,
                           uint64_t seed, uint64_t step, uint32_t query,
                           int32_t *ids_out, double *scores_out) {
    int32_t n = 0;
    while (n < k1 && pool_ids[n] >= 0) ++n;
    const float u = (float)(explore_word(seed, step, query, 0) >> 8) * (1.0f / 16777216.0f);
    if (!(u < epsilon) || n == 0) {
        evk_oracle_phase2(pool_ids, pool_sims, k1, q_stage, w, k2, ids_out, scores_out);
        return 0;
    }
    int32_t *perm = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    for (int32_t i = 0; i < n; ++i) perm[i] = i;
    const int32_t m = k2 < n ? k2 : n;
    for (int32_t j = 0; j < k2; ++j) { ids_out[j] = -1; scores_out[j] = -INFINITY; }
    for (int32_t i = 0; i < m; ++i) {
        const uint32_t r = explore_word(seed, step, query, (uint32_t)(i + 1));
        const int32_t pick = i + (int32_t)(((uint64_t)r * (uint64_t)(n - i)) >> 32);
        const int32_t tmp = perm[i]; perm[i] = perm[pick]; perm[pick] = tmp;
        const int32_t pos = perm[i];
        ids_out[i] = pool_ids[pos];
        scores_out[i] = (1.0 - w) * pool_sims[pos] + w * (double)q_stage[pool_ids[pos]];
    }
    free(perm);
    return 1;
}

/* evk_oracle_explore with pool z-scores: the same draws, scores from zscore_pool_scores. */
int32_t evk_oracle_explore_zscore(const int32_t *pool_ids, const double *pool_sims, int32_t k1,
                                  const float *q_stage, double w, int32_t k2, float epsilon,
                                  uint64_t seed, uint64_t step, uint32_t query,
                                  int32_t *ids_out, double *scores_out) {
    int32_t n = 0;
    while (n < k1 && pool_ids[n] >= 0) ++n;
    const float u = (float)(explore_word(seed, step, query, 0) >> 8) * (1.0f / 16777216.0f);
    if (!(u < epsilon) || n == 0) {
        evk_oracle_phase2_zscore(pool_ids, pool_sims, k1, q_stage, w, k2, ids_out, scores_out);
        return 0;
    }
    double *sc = (double *)malloc((size_t)k1 * sizeof(double));
    zscore_pool_scores(pool_ids, pool_sims, n, q_stage, w, sc);  /* the first n slots are the valid ones */
    int32_t *perm = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    for (int32_t i = 0; i < n; ++i) perm[i] = i;
    const int32_t m = k2 < n ? k2 : n;
    for (int32_t j = 0; j < k2; ++j) { ids_out[j] = -1; scores_out[j] = -INFINITY; }
    for (int32_t i = 0; i < m; ++i) {
        const uint32_t r = explore_word(seed, step, query, (uint32_t)(i + 1));
        const int32_t pick = i + (int32_t)(((uint64_t)r * (uint64_t)(n - i)) >> 32);
        const int32_t tmp = perm[i]; perm[i] = perm[pick]; perm[pick] = tmp;
        const int32_t pos = perm[i];
        ids_out[i] = pool_ids[pos];
        scores_out[i] = sc[pos];
    }
    free(perm);
    free(sc);
    return 1;
}

/* ---- Decreasing step size (Appendix A, Robbins-Monro lemma) ------------------------ */

/* Eq. 8 with alpha_t = 1 / (number of updates the entry has received, this one included):
 * the stored value becomes the running mean of the entry's rewards.  visits[] counts the
 * updates per entry and is advanced here.  fp64 truth. */
void evk_oracle_q_update_decay_f64(double *q_stage, uint32_t *visits, const int32_t *ids,
                                   const float *rewards, int64_t m) {
    for (int64_t t = 0; t < m; ++t) {
        const int32_t i = ids[t];
        visits[i] += 1;
        const double alpha = 1.0 / (double)visits[i];
        q_stage[i] = q_stage[i] + alpha * ((double)rewards[t] - q_stage[i]);
    }
}

/* The same in binary32: alpha = 1.0f / (float)visits by IEEE division, then the three
 * separately rounded operations of evk_oracle_q_update_f32. */
void evk_oracle_q_update_decay_f32(float *q_stage, uint32_t *visits, const int32_t *ids,
                                   const float *rewards, int64_t m) {
    for (int64_t t = 0; t < m; ++t) {
        const int32_t i = ids[t];
        visits[i] += 1;
        volatile float alpha = 1.0f / (float)visits[i];
        volatile float q = q_stage[i];
        volatile float diff = rewards[t] - q;
        volatile float step = alpha * diff;
        volatile float next = q + step;
        q_stage[i] = next;
    }
}
