// Phase 2 of value-driven retrieval (Section 3.2): the candidate pool of a query
// is cut down to the final k2 items using the stage's value estimates.
//
//   score = (1 - w) * sim + w * Q_stage[id]
//
// w = 1 ranks the pool by Q_stage alone (the rule the method states); w = 0 keeps
// the similarity order.  Results are ordered (score desc, sim desc, id asc).
//
// Variant (norm = 1, no counterpart in the paper, which normalises rewards only): the two
// terms are made commensurate per query first, each as its z-score over the pool,
//   z(x) = (x - mean_pool(x)) / std_pool(x)   (population std; 0 where the std is <= 1e-6),
//   score = (1 - w) * z(sim) + w * z(Q_stage[id]).
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

// Sum of v over the block, the same bits in every thread.
template <int NT>
__device__ double block_sum_f64(double v) {
    __shared__ double red[NT / 32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();  // earlier readers of red are done
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < NT / 32; ++i) t += red[i];
    return t;
}

// Mean and reciprocal population std of a pool column for the z-score variant.
struct ZStat {
    double mean, inv_std;  // inv_std = 0 for a (nearly) constant column
    __device__ double z(float x) const { return ((double)x - mean) * inv_std; }
};
constexpr double kZStdFloor = 1e-6;
constexpr int kRankByCount = 256;   // pools up to this size are ranked by counting instead of sorted

// Block-wide: scores the n entries that fetch(i) returns (any order), sorts them by (score
// desc, sim desc, id asc) and writes the first k2 (padding: id -1, score -inf).
// skey / sid: shared scratch of next_pow2(n) entries each.  norm: 0 raw mix, 1 pool z-scores.
template <int NT, class Fetch>
__device__ void rerank_block_with(Fetch fetch, int n, int k2, float w, int norm, uint64_t *skey, int32_t *sid,
                                  int32_t *__restrict__ ids_out, float *__restrict__ scores_out) {
    const int tid = threadIdx.x;
    const int np2 = next_pow2(n > 1 ? n : 1);
    const float one_minus_w = 1.0f - w;
    ZStat zs = {0.0, 0.0}, zq = {0.0, 0.0};
    if (norm && n > 0) {
        // two passes in fp64: means, then squared deviations
        double a = 0.0, b = 0.0;
        for (int i = tid; i < n; i += NT) {
            const PoolEntry e = fetch(i);
            a += (double)e.sim;
            b += (double)e.q;
        }
        zs.mean = block_sum_f64<NT>(a) / n;
        zq.mean = block_sum_f64<NT>(b) / n;
        a = 0.0;
        b = 0.0;
        for (int i = tid; i < n; i += NT) {
            const PoolEntry e = fetch(i);
            a += ((double)e.sim - zs.mean) * ((double)e.sim - zs.mean);
            b += ((double)e.q - zq.mean) * ((double)e.q - zq.mean);
        }
        const double sd_s = sqrt(block_sum_f64<NT>(a) / n), sd_q = sqrt(block_sum_f64<NT>(b) / n);
        zs.inv_std = sd_s > kZStdFloor ? 1.0 / sd_s : 0.0;
        zq.inv_std = sd_q > kZStdFloor ? 1.0 / sd_q : 0.0;
    }
    for (int i = tid; i < np2; i += NT) {
        uint64_t key = 0;
        int32_t id = -1;  // padding compares as the largest unsigned id and a zero key: last
        if (i < n) {
            const PoolEntry e = fetch(i);
            id = e.id;
            float score = norm ? (float)((1.0 - (double)w) * zs.z(e.sim) + (double)w * zq.z(e.q))
                               : fmaf(w, e.q, one_minus_w * e.sim);
            score += 0.0f;
            key = ((uint64_t)ordered_bits(score) << 32) | ordered_bits(e.sim + 0.0f);
        }
        skey[i] = key;
        sid[i] = id;
    }
    if (n <= kRankByCount) {
        // A small pool is ranked by counting: every entry counts the entries that rank before it
        // (all threads read the same entry at a time, a broadcast) and, being one of the first k2,
        // writes itself to its place.  No barrier between steps, a fraction of the sorting network's time.
        __syncthreads();
        for (int i = tid; i < n; i += NT) {
            const uint64_t ka = skey[i];
            const int32_t ia = sid[i];
            int rank = 0;
            // eight entries per step, loaded together (padding entries rank behind every real one)
            int j = 0;
            for (; j + 8 <= np2; j += 8) {
                uint64_t kb[8];
                int32_t ib[8];
#pragma unroll
                for (int u = 0; u < 8; u += 2) {
                    const ulonglong2 k2v = *reinterpret_cast<const ulonglong2 *>(skey + j + u);
                    kb[u] = k2v.x;
                    kb[u + 1] = k2v.y;
                }
#pragma unroll
                for (int u = 0; u < 8; u += 4) {
                    const int4 i4 = *reinterpret_cast<const int4 *>(sid + j + u);
                    ib[u] = i4.x; ib[u + 1] = i4.y; ib[u + 2] = i4.z; ib[u + 3] = i4.w;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) rank += rerank_before(kb[u], ib[u], ka, ia) ? 1 : 0;
            }
            for (; j < n; ++j) rank += rerank_before(skey[j], sid[j], ka, ia) ? 1 : 0;
            if (rank < k2) {
                ids_out[rank] = ia;
                scores_out[rank] = from_ordered_bits((uint32_t)(ka >> 32));
            }
        }
        for (int i = n + tid; i < k2; i += NT) {
            ids_out[i] = -1;
            scores_out[i] = -INFINITY;
        }
        return;
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
                             int norm, uint64_t *skey, int32_t *sid, int32_t *__restrict__ ids_out,
                             float *__restrict__ scores_out) {
    rerank_block_with<NT>(
        [=](int i) {
            PoolEntry e;
            e.id = key_id(pool_keys[i]);
            e.sim = key_sim(pool_keys[i]);
            e.q = q_stage[e.id];
            return e;
        },
        n, k2, w, norm, skey, sid, ids_out, scores_out);
}

}  // namespace evk
