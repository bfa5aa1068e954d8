// Exploration on top of value-driven retrieval (Section 3.3: the drafting context is chosen
// from the pool with an epsilon-greedy policy over Q).  Per query, a counter-based generator
// keyed by (seed, step, query) decides whether to explore; an exploring query's context is
// min(k2, n) pool entries drawn uniformly without replacement, in draw order, instead of the
// greedy top-k2.  Queries that do not explore keep the result the rerank wrote.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

// Philox4x32-10 (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// Word j of the stream of (seed, step, query): block j / 4, counter (query, step, block).
struct WordStream {
    uint2 key;
    uint32_t query, step_lo, step_hi, block;
    uint4 cur;
    __device__ WordStream(uint64_t seed, uint64_t step, uint32_t q)
        : key(make_uint2((uint32_t)seed, (uint32_t)(seed >> 32))), query(q), step_lo((uint32_t)step),
          step_hi((uint32_t)(step >> 32)), block(0xffffffffu), cur(make_uint4(0, 0, 0, 0)) {}
    __device__ uint32_t word(uint32_t j) {
        if (j / 4 != block) {
            block = j / 4;
            cur = philox4x32_10(make_uint4(query, step_lo, step_hi, block), key);
        }
        const uint32_t r = j % 4;
        return r == 0 ? cur.x : (r == 1 ? cur.y : (r == 2 ? cur.z : cur.w));
    }
};

// One warp per query; lane 0 walks the partial shuffle over positions held in shared memory.
__global__ void __launch_bounds__(32)
explore_kernel(const int32_t *__restrict__ pool_ids, const float *__restrict__ pool_sims, int k1, int k2,
               const float *__restrict__ q_stage, float w, int norm, float epsilon, uint64_t seed, uint64_t step,
               int32_t *__restrict__ ids_out, float *__restrict__ scores_out, uint8_t *__restrict__ explored_out) {
    __shared__ int32_t perm[EVK_MAX_K1];
    const int q = blockIdx.x, lane = threadIdx.x;
    pdl_wait();  // the pool and the greedy result come from the kernel before
    const int32_t *ids = pool_ids + (size_t)q * k1;
    const float *sims = pool_sims + (size_t)q * k1;
    int n = 0;
    for (int i = lane; i < k1; i += 32) {
        perm[i] = i;
        n += ids[i] >= 0;
    }
    n = __reduce_add_sync(0xffffffffu, n);
    // z-score variant: pool statistics as the rerank computes them (fp64, two passes)
    double mean_s = 0.0, mean_q = 0.0, inv_s = 0.0, inv_q = 0.0;
    if (norm && n > 0) {
        auto warp_sum = [](double v) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            return v;
        };
        double a = 0.0, b = 0.0;
        for (int i = lane; i < k1; i += 32)
            if (ids[i] >= 0) {
                a += (double)sims[i];
                b += (double)q_stage[ids[i]];
            }
        mean_s = warp_sum(a) / n;
        mean_q = warp_sum(b) / n;
        a = 0.0;
        b = 0.0;
        for (int i = lane; i < k1; i += 32)
            if (ids[i] >= 0) {
                const double ds = (double)sims[i] - mean_s, dq = (double)q_stage[ids[i]] - mean_q;
                a += ds * ds;
                b += dq * dq;
            }
        const double sd_s = sqrt(warp_sum(a) / n), sd_q = sqrt(warp_sum(b) / n);
        inv_s = sd_s > 1e-6 ? 1.0 / sd_s : 0.0;
        inv_q = sd_q > 1e-6 ? 1.0 / sd_q : 0.0;
    }
    __syncwarp();
    if (lane != 0) return;
    WordStream ws(seed, step, (uint32_t)q);
    const float u = (float)(ws.word(0) >> 8) * (1.0f / 16777216.0f);
    const bool explore = (u < epsilon) && n > 0;
    if (explored_out) explored_out[q] = explore ? 1 : 0;
    if (!explore) return;
    const int m = k2 < n ? k2 : n;
    const float one_minus_w = 1.0f - w;
    for (int i = 0; i < k2; ++i) {
        int32_t id = -1;
        float score = -INFINITY;
        if (i < m) {
            const uint32_t r = ws.word((uint32_t)(i + 1));
            const int pick = i + (int)(((uint64_t)r * (uint64_t)(n - i)) >> 32);
            const int32_t tmp = perm[i];
            perm[i] = perm[pick];
            perm[pick] = tmp;
            const int pos = perm[i];
            id = ids[pos];
            if (norm)
                score = (float)((1.0 - (double)w) * (((double)sims[pos] - mean_s) * inv_s) +
                                (double)w * (((double)q_stage[id] - mean_q) * inv_q)) + 0.0f;
            else
                score = fmaf(w, q_stage[id], one_minus_w * sims[pos]) + 0.0f;
        }
        ids_out[(size_t)q * k2 + i] = id;
        scores_out[(size_t)q * k2 + i] = score;
    }
}

}  // namespace

cudaError_t launch_explore(const int32_t *pool_ids, const float *pool_sims, int B, int k1, int k2,
                           const float *q_stage, float w, int norm, float epsilon, uint64_t seed, uint64_t step,
                           int32_t *ids_out, float *scores_out, uint8_t *explored_out, cudaStream_t stream,
                           int *launches) {
    if (B <= 0) return cudaSuccess;
    ++*launches;
    return launch_overlapped(explore_kernel, dim3(B), dim3(32), 0, stream, pool_ids, pool_sims, k1, k2, q_stage, w,
                             norm, epsilon, seed, step, ids_out, scores_out, explored_out);
}

}  // namespace evk
