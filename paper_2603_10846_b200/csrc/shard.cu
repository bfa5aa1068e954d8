// A bank split by rows over several GPUs.  Shard g owns the entries [offset_g, offset_g + size_g)
// and both value tables for them.  Every shard runs phase 1 on its rows for all queries and
// tags each local candidate with its global id and its stage value (tag_pool_kernel); the
// tagged pools of all shards are then gathered on every GPU (a collective in the caller) and
// merged (merge_shards_kernel): the k1 best of the G * k1 candidates are the pool the
// unsplit bank would have produced, because each shard's pool is the exact top-k1 of its
// rows, and phase 2 runs on it with the values that travelled with the candidates.
#include "evk_common.cuh"
#include "evk_kernels.cuh"
#include "rerank.cuh"

namespace evk {

namespace {

constexpr int kTagThreads = 256;

__global__ void __launch_bounds__(kTagThreads)
tag_pool_kernel(const int32_t *__restrict__ pool_ids, int64_t n, int32_t id_offset, const float *__restrict__ q_stage,
                int32_t *__restrict__ gids_out, float *__restrict__ q_out) {
    pdl_wait();
    for (int64_t i = blockIdx.x * (int64_t)kTagThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kTagThreads) {
        const int32_t id = pool_ids[i];
        gids_out[i] = id >= 0 ? id + id_offset : -1;
        q_out[i] = id >= 0 ? q_stage[id] : 0.0f;
    }
}

constexpr int kThreads = 512;
constexpr int kSelPerThread = 8;
constexpr int kCap = kThreads * kSelPerThread;  // 4096 keys
constexpr int kBatch = 2048;

// Candidate records are [shard][query][k1]; a record's source index is shard * k1 + position.
// Shards must be passed in ascending id-range order: among equal similarities a pool lists
// smaller ids first, so source order then equals global-id order and the usual key
// (similarity descending, then the low word ascending) ranks exactly as one bank would.
__global__ void __launch_bounds__(kThreads)
merge_shards_kernel(const int32_t *__restrict__ gids, const float *__restrict__ sims, const float *__restrict__ qs,
                    int n_shards, int B, int k1, int k2, float w, int32_t *__restrict__ ids_out,
                    float *__restrict__ scores_out, int32_t *__restrict__ pool_gids_out,
                    float *__restrict__ pool_sims_out) {
    __shared__ __align__(16) uint64_t keys[kCap];
    __shared__ int hist[256];
    __shared__ uint64_t scal[4];
    __shared__ int count;
    __shared__ uint64_t tau;
    const int tid = threadIdx.x, q = blockIdx.x;
    if (tid == 0) {
        count = 0;
        tau = 0;
    }
    __syncthreads();
    const int total = n_shards * k1;
    auto record = [&](int src) { return ((size_t)(src / k1) * B + q) * k1 + (src % k1); };
    for (int base = 0; base < total; base += kBatch) {
        const uint64_t t = tau;
#pragma unroll
        for (int j = 0; j < kBatch / kThreads; ++j) {
            const int src = base + tid + j * kThreads;
            uint64_t key = 0;
            if (src < total) {
                const size_t r = record(src);
                if (gids[r] >= 0) key = make_key(sims[r], src);
            }
            const bool keep = key > t;
            const int slot = warp_claim_slot(keep, &count);
            if (keep) keys[slot] = key;
        }
        __syncthreads();
        const int n = count;
        if (n > kCap - kBatch && n > k1) {
            const uint64_t kth = block_select_topk<kThreads, kSelPerThread>(keys, n, k1, hist, scal);
            if (tid == 0) {
                count = k1;
                tau = kth;
            }
        }
        __syncthreads();
    }
    int n = count;
    if (n > k1) {
        block_select_topk<kThreads, kSelPerThread>(keys, n, k1, hist, scal);
        n = k1;
    }
    if (pool_gids_out || pool_sims_out) {
        const int np2 = next_pow2(n > 1 ? n : 1);
        for (int i = n + tid; i < np2; i += kThreads) keys[i] = 0;
        __syncthreads();
        block_sort_desc<kThreads>(keys, np2);
        for (int i = tid; i < k1; i += kThreads) {
            int32_t gid = -1;
            float s = -INFINITY;
            if (i < n) {
                gid = gids[record(key_id(keys[i]))];
                s = key_sim(keys[i]);
            }
            if (pool_gids_out) pool_gids_out[(size_t)q * k1 + i] = gid;
            if (pool_sims_out) pool_sims_out[(size_t)q * k1 + i] = s;
        }
    }
    __syncthreads();
    uint64_t *skey = keys + EVK_MAX_K1;
    int32_t *sid = reinterpret_cast<int32_t *>(keys + 2 * EVK_MAX_K1);
    rerank_block_with<kThreads>(
        [&](int i) {
            const size_t r = record(key_id(keys[i]));
            PoolEntry e;
            e.id = gids[r];
            e.sim = key_sim(keys[i]);
            e.q = qs[r];
            return e;
        },
        n, k2, w, 0, skey, sid, ids_out + (size_t)q * k2, scores_out + (size_t)q * k2);
}

}  // namespace

cudaError_t launch_tag_pool(const int32_t *pool_ids, int64_t n, int32_t id_offset, const float *q_stage,
                            int32_t *gids_out, float *q_out, cudaStream_t stream, int *launches) {
    if (n <= 0) return cudaSuccess;
    int64_t grid = (n + kTagThreads - 1) / kTagThreads;
    if (grid > num_sms() * 8) grid = num_sms() * 8;
    ++*launches;
    return launch_overlapped(tag_pool_kernel, dim3((unsigned)grid), dim3(kTagThreads), 0, stream, pool_ids, n,
                             id_offset, q_stage, gids_out, q_out);
}

cudaError_t launch_merge_shards(const int32_t *gids, const float *sims, const float *qs, int n_shards, int B, int k1,
                                int k2, float w, int32_t *ids_out, float *scores_out, int32_t *pool_gids_out,
                                float *pool_sims_out, cudaStream_t stream) {
    if (B <= 0) return cudaSuccess;
    merge_shards_kernel<<<B, kThreads, 0, stream>>>(gids, sims, qs, n_shards, B, k1, k2, w, ids_out, scores_out,
                                                    pool_gids_out, pool_sims_out);
    return cudaGetLastError();
}

}  // namespace evk
