// Phase 2 of value-driven retrieval (Section 3.2): the candidate pool of a query
// is cut down to the final k2 items using the stage's value estimates.
//
//   score = (1 - w) * sim + w * Q_stage[id]
//
// w = 1 ranks the pool by Q_stage alone (the rule the method states); w = 0 keeps
// the similarity order.  Results are ordered (score desc, sim desc, id asc).
#pragma once

#include "evk_common.cuh"

namespace evk {

// "a ranks before b": (score, sim) packed as ordered bits, then the smaller id.
__device__ __forceinline__ bool rerank_before(uint64_t ka, int32_t ia, uint64_t kb, int32_t ib) {
    return ka > kb || (ka == kb && (uint32_t)ia < (uint32_t)ib);
}

// One pool entry as the rerank sees it.
struct PoolEntry {
    int32_t id;
    float sim, q;
};

// Block-wide: scores the n entries that fetch(i) returns (any order), sorts them by (score
// desc, sim desc, id asc) and writes the first k2 (padding: id -1, score -inf).
// skey / sid: shared scratch of next_pow2(n) entries each.
template <int NT, class Fetch>
__device__ void rerank_block_with(Fetch fetch, int n, int k2, float w, uint64_t *skey, int32_t *sid,
                                  int32_t *__restrict__ ids_out, float *__restrict__ scores_out) {
    const int tid = threadIdx.x;
    const int np2 = next_pow2(n > 1 ? n : 1);
    const float one_minus_w = 1.0f - w;
    for (int i = tid; i < np2; i += NT) {
        uint64_t key = 0;
        int32_t id = -1;  // padding compares as the largest unsigned id and a zero key: last
        if (i < n) {
            const PoolEntry e = fetch(i);
            id = e.id;
            float score = fmaf(w, e.q, one_minus_w * e.sim);
            score += 0.0f;
            key = ((uint64_t)ordered_bits(score) << 32) | ordered_bits(e.sim + 0.0f);
        }
        skey[i] = key;
        sid[i] = id;
    }
    bool wide_before = true;  // stages with stride <= 32 stay inside a warp's own 64 elements
    for (int size = 2; size <= np2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const bool wide = stride > 32;
            if (wide || wide_before) __syncthreads(); else __syncwarp();
            wide_before = wide;
            for (int t = tid; t < (np2 >> 1); t += NT) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool desc = ((lo & size) == 0);
                const uint64_t ka = skey[lo], kb = skey[hi];
                const int32_t ia = sid[lo], ib = sid[hi];
                if (rerank_before(ka, ia, kb, ib) != desc) {
                    skey[lo] = kb; skey[hi] = ka;
                    sid[lo] = ib; sid[hi] = ia;
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < k2; i += NT) {
        const int32_t id = (i < np2) ? sid[i] : -1;
        float score = -INFINITY;
        if (id >= 0) score = from_ordered_bits((uint32_t)(skey[i] >> 32));
        ids_out[i] = id;
        scores_out[i] = score;
    }
}

// The pool as n ranking keys (similarity, id) in shared memory, values looked up in q_stage.
template <int NT>
__device__ void rerank_block(const uint64_t *pool_keys, int n, int k2, const float *__restrict__ q_stage, float w,
                             uint64_t *skey, int32_t *sid, int32_t *__restrict__ ids_out,
                             float *__restrict__ scores_out) {
    rerank_block_with<NT>(
        [=](int i) {
            PoolEntry e;
            e.id = key_id(pool_keys[i]);
            e.sim = key_sim(pool_keys[i]);
            e.q = q_stage[e.id];
            return e;
        },
        n, k2, w, skey, sid, ids_out, scores_out);
}

}  // namespace evk
