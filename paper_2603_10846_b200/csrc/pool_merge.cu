// The end of a retrieval, one thread block per query:
//
//   1. merge the candidate lists that the scoring kernel left per (query, part) into the
//      pool C(x) of Section 3.2 — the k1 entries of largest similarity, ordered
//      (similarity descending, id ascending);
//   2. phase 2: cut the pool down to k2 with the stage's value estimates (rerank.cuh).
//
// Candidates stream through a shared-memory buffer that is cut back to its best k1 by
// an exact radix select whenever it fills; the survivors are sorted with a bitonic
// network.  Keys are totally ordered and distinct, so the result does not depend on
// the order in which the scoring kernel appended candidates.
#include "evk_common.cuh"
#include "evk_kernels.cuh"
#include "rerank.cuh"

namespace evk {

namespace {

// Two shapes of the same kernel.  Few queries: 512 threads and room for 4,096 keys per query, so that
// one query's merge is as parallel as it can be.  Hundreds of queries and pools of at most 256: blocks
// of 128 threads with a quarter of the buffers, sixteen of which fit on an SM, so that all queries are
// merged in one wave (1,024 queries over the clustered bank: 53 -> about 25 us).
constexpr int kSelPerThread = 8;

template <int kThreads, int kMaxParts>
__global__ void __launch_bounds__(kThreads)
merge_rerank_kernel(const uint64_t *__restrict__ part_keys, const int *__restrict__ part_counts, int nparts,
                    int part_stride, int qt_size, int k1, int expect, const uint32_t *__restrict__ live_count,
                    int32_t *__restrict__ status,
                    int32_t *__restrict__ pool_ids_user, float *__restrict__ pool_sims_user,
                    int k2, const float *__restrict__ q_stage, float w, int norm,
                    int32_t *__restrict__ ids_out, float *__restrict__ scores_out) {
    constexpr int kCap = kThreads * kSelPerThread;   // keys held at once (4,096 = 32 KB, or 1,024)
    constexpr int kBatch = kCap / 2;                 // candidates examined between capacity checks
    constexpr int kPoolMax = kCap / 4;               // largest pool; the rerank's scratch lives behind it
    __shared__ __align__(16) uint64_t keys[kCap];
    __shared__ int offs[kMaxParts + 1];
    __shared__ int hist[256];
    __shared__ uint64_t scal[4];
    __shared__ int count;
    __shared__ uint64_t tau;

    const int tid = threadIdx.x;
    const int q = blockIdx.x;
    pdl_trigger();
    pdl_wait();  // the candidate lists are the scoring kernel's output
    // list of part p: list0 + p * qt_size
    const size_t list0 = (size_t)(q / qt_size) * ((size_t)nparts * qt_size) + (size_t)(q % qt_size);

    if (tid == 0) {
        count = 0;
        tau = 0;
        offs[0] = 0;
    }
    // The first 32 keys of the first kSpec lists of every warp are fetched before the list lengths are
    // known (a list's place does not depend on them), so that lengths and keys cost one trip to memory
    // together.  What lies behind a list's end is read and dropped.
    constexpr int kWarps = kThreads / 32;
    constexpr int kSpec = 10;
    const int warp = tid >> 5, lane = tid & 31;
    uint64_t spec[kSpec];
#pragma unroll
    for (int u = 0; u < kSpec; ++u) {
        const int p = warp + u * kWarps;
        spec[u] = (p < nparts && lane < part_stride) ? part_keys[(list0 + (size_t)p * qt_size) * part_stride + lane] : 0;
    }
    for (int p = tid; p < nparts; p += kThreads) offs[p + 1] = part_counts[list0 + (size_t)p * qt_size];
    __syncthreads();
    if (tid < 32) {
        // inclusive scan of the part counts, 32 at a time
        int carry = 0;
        for (int base = 0; base < nparts; base += 32) {
            const int p = base + tid;
            int v = (p < nparts) ? offs[p + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, off);
                if (tid >= off) v += u;
            }
            if (p < nparts) offs[p + 1] = v + carry;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();
    const int total = offs[nparts];

    if (total <= kCap) {
        // Everything fits at once: each warp copies whole lists to their places, no search per key.
#pragma unroll
        for (int u = 0; u < kSpec; ++u) {
            const int p = warp + u * kWarps;
            if (p < nparts) {
                const int first = offs[p], cnt = offs[p + 1] - first;
                if (lane < cnt) keys[first + lane] = spec[u];
                if (cnt > 32) {
                    const uint64_t *src = part_keys + (list0 + (size_t)p * qt_size) * part_stride;
                    for (int i = 32 + lane; i < cnt; i += 32) keys[first + i] = src[i];
                }
            }
        }
        // Further lists four per warp and step, their loads issued together; a list longer than a warp
        // finishes in the loop behind.
        for (int p0 = warp + kSpec * kWarps; p0 < nparts; p0 += 4 * kWarps) {
            uint64_t v[4];
            int first[4], cnt[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int p = p0 + u * kWarps;
                first[u] = p < nparts ? offs[p] : 0;
                cnt[u] = p < nparts ? offs[p + 1] - first[u] : 0;
                v[u] = lane < cnt[u] ? part_keys[(list0 + (size_t)p * qt_size) * part_stride + lane] : 0;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (lane < cnt[u]) keys[first[u] + lane] = v[u];
                if (cnt[u] > 32) {
                    const uint64_t *src = part_keys + (list0 + (size_t)(p0 + u * kWarps) * qt_size) * part_stride;
                    for (int i = 32 + lane; i < cnt[u]; i += 32) keys[first[u] + i] = src[i];
                }
            }
        }
        if (tid == 0) count = total;
        __syncthreads();
    }
    for (int base = 0; base < total && total > kCap; base += kBatch) {
        const uint64_t t = tau;
#pragma unroll
        for (int j = 0; j < kBatch / kThreads; ++j) {
            const int idx = base + tid + j * kThreads;
            uint64_t key = 0;
            if (idx < total) {
                // part p with offs[p] <= idx < offs[p+1]
                int lo = 0, hi = nparts;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (offs[mid] <= idx) lo = mid; else hi = mid;
                }
                key = part_keys[(list0 + (size_t)lo * qt_size) * part_stride + (idx - offs[lo])];
            }
            const bool keep = idx < total && key > t;
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
    // entries dropped from the memory cannot be found: the pool is as long as the live entries allow
    if (live_count) {
        const int live = (int)min(*live_count, (uint32_t)0x7fffffff);
        expect = expect < live ? expect : live;
    }
    if (n < expect && tid == 0) atomicCAS(status, 0, (int)EVK_ERR_INCOMPLETE);
    if (n > k1) {
        block_select_topk<kThreads, kSelPerThread>(keys, n, k1, hist, scal);
        n = k1;
    }
    if (pool_ids_user || pool_sims_user) {
        // the pool itself is wanted: put it in (similarity descending, id ascending) order
        const int np2 = next_pow2(n > 1 ? n : 1);
        for (int i = n + tid; i < np2; i += kThreads) keys[i] = 0;
        __syncthreads();
        block_sort_desc<kThreads>(keys, np2);
        for (int i = tid; i < k1; i += kThreads) {
            int32_t id = -1;
            float s = -INFINITY;
            if (i < n) {
                id = key_id(keys[i]);
                s = key_sim(keys[i]);
            }
            if (pool_ids_user) pool_ids_user[(size_t)q * k1 + i] = id;
            if (pool_sims_user) pool_sims_user[(size_t)q * k1 + i] = s;
        }
    }
    __syncthreads();
    // phase 2 on the pool keys[0..n) (any order); scratch behind the pool
    uint64_t *skey = keys + kPoolMax;
    int32_t *sid = reinterpret_cast<int32_t *>(keys + 2 * kPoolMax);
    rerank_block<kThreads>(keys, n, k2, q_stage, w, norm, skey, sid, ids_out + (size_t)q * k2, scores_out + (size_t)q * k2);
}

}  // namespace

cudaError_t launch_merge_rerank(const uint64_t *part_keys, const int *part_counts, int nparts,
                                int part_stride, int qt_size, int B, int k1, int expect, const uint32_t *live_count,
                                int32_t *status,
                                int32_t *pool_ids_user, float *pool_sims_user,
                                int k2, const float *q_stage, float w, int norm, int32_t *ids_out, float *scores_out,
                                cudaStream_t stream, int *launches) {
    static_assert(EVK_MAX_K1 * 4 <= 512 * kSelPerThread, "the large shape holds the largest pool");
    if (B <= 0) return cudaSuccess;
    if (nparts > kMergeMaxParts) return cudaErrorInvalidValue;
    ++*launches;
    // the small shape holds 1,024 candidates at a time: pools up to 128 (some 500 candidates per query) fit, a
    // pool of 256 over 74 lists (some 2,000) went through it in batches, 92 us for 256 queries where the
    // large shape takes 55
    if (B >= 256 && k1 <= 128 && nparts <= 255)
        return launch_overlapped(merge_rerank_kernel<128, 255>, dim3(B), dim3(128), 0, stream, part_keys, part_counts,
                                 nparts, part_stride, qt_size, k1, expect, live_count, status, pool_ids_user,
                                 pool_sims_user, k2, q_stage, w, norm, ids_out, scores_out);
    return launch_overlapped(merge_rerank_kernel<512, kMergeMaxParts>, dim3(B), dim3(512), 0, stream, part_keys,
                             part_counts, nparts, part_stride, qt_size, k1, expect, live_count, status, pool_ids_user,
                             pool_sims_user, k2, q_stage, w, norm, ids_out, scores_out);
}

}  // namespace evk
