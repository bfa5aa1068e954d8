// Phase 2 of value-driven retrieval (Section 3.2): the candidate pool of a query
// is cut down to the final k2 items using the stage's value estimates.
//
//   score = (1 - w) * sim + w * Q_stage[id]
//
// w = 1 ranks the pool by Q_stage alone (the rule the method states); w = 0 keeps
// the similarity order.  Results are ordered (score desc, sim desc, id asc).  One
// thread block per query: gather the k1 values, sort, write the first k2.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;

// "a ranks before b"
__device__ __forceinline__ bool before(uint64_t ka, int32_t ia, uint64_t kb, int32_t ib) {
    return ka > kb || (ka == kb && (uint32_t)ia < (uint32_t)ib);
}

__global__ void __launch_bounds__(kThreads)
rerank_kernel(const int32_t *__restrict__ pool_ids, const float *__restrict__ pool_sims, int k1, int k2,
              const float *__restrict__ q_stage, float w, int32_t *__restrict__ ids_out,
              float *__restrict__ scores_out) {
    __shared__ uint64_t skey[EVK_MAX_K1];  // (score, sim) as ordered bits
    __shared__ int32_t sid[EVK_MAX_K1];    // padding: id -1 compares as the largest unsigned id

    const int tid = threadIdx.x;
    const int q = blockIdx.x;
    const int np2 = next_pow2(k1);
    const float one_minus_w = 1.0f - w;
    for (int i = tid; i < np2; i += kThreads) {
        uint64_t key = 0;
        int32_t id = -1;
        if (i < k1) {
            id = pool_ids[(size_t)q * k1 + i];
            if (id >= 0) {
                const float sim = pool_sims[(size_t)q * k1 + i];
                float score = fmaf(w, q_stage[id], one_minus_w * sim);
                score += 0.0f;
                key = ((uint64_t)ordered_bits(score) << 32) | ordered_bits(sim + 0.0f);
            }
        }
        skey[i] = key;
        sid[i] = id;
    }
    for (int size = 2; size <= np2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = tid; t < (np2 >> 1); t += kThreads) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool desc = ((lo & size) == 0);
                const uint64_t ka = skey[lo], kb = skey[hi];
                const int32_t ia = sid[lo], ib = sid[hi];
                const bool a_first = before(ka, ia, kb, ib);
                if (a_first != desc) {
                    skey[lo] = kb; skey[hi] = ka;
                    sid[lo] = ib; sid[hi] = ia;
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < k2; i += kThreads) {
        const int32_t id = (i < np2) ? sid[i] : -1;
        float score = -INFINITY;
        if (id >= 0) score = from_ordered_bits((uint32_t)(skey[i] >> 32));
        ids_out[(size_t)q * k2 + i] = id;
        scores_out[(size_t)q * k2 + i] = score;
    }
}

}  // namespace

cudaError_t launch_rerank(const int32_t *pool_ids, const float *pool_sims, int B, int k1, int k2,
                          const float *q_stage, float w, int32_t *ids_out, float *scores_out,
                          cudaStream_t stream, int *launches) {
    if (B <= 0) return cudaSuccess;
    rerank_kernel<<<B, kThreads, 0, stream>>>(pool_ids, pool_sims, k1, k2, q_stage, w, ids_out, scores_out);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace evk
