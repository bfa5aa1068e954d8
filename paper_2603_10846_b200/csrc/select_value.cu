// Start-point selection of the refining stage (Section 3.4): each task keeps a set of
// feasible kernels P(x) stored in the memory; the next start point is chosen by its value
// estimate Q_2.  For every task, the k entries of largest Q_stage among a caller-given id
// list are returned, ordered (Q descending, id ascending).  One thread block per task.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;
constexpr int kSelPerThread = 16;
constexpr int kMaxLen = kThreads * kSelPerThread;  // 4096 candidates per task

__global__ void __launch_bounds__(kThreads)
select_by_value_kernel(const int32_t *__restrict__ cand_ids, const int32_t *__restrict__ offsets, int64_t size,
                       const uint32_t *__restrict__ live_bits,
                       const float *__restrict__ q_stage, int k, int32_t *__restrict__ ids_out,
                       float *__restrict__ q_out, int32_t *__restrict__ status) {
    __shared__ uint64_t keys[kMaxLen];
    __shared__ int hist[256];
    __shared__ uint64_t scal[4];
    __shared__ int bad_s, kept_s;
    const int tid = threadIdx.x, task = blockIdx.x;
    const int begin = offsets[task], end = offsets[task + 1];
    int n = end - begin;
    if (tid == 0) { bad_s = 0; kept_s = 0; }
    __syncthreads();
    int bad = 0;
    if (n < 0 || n > kMaxLen) {
        bad = 1;
        n = 0;
    }
    // candidates that are still in the memory, gathered at the front of `keys` (whole warps step together)
    for (int i0 = 0; i0 < n; i0 += kThreads) {
        const int i = i0 + tid;
        uint64_t key = 0;
        bool keep = false;
        if (i < n) {
            const int32_t id = cand_ids[begin + i];
            if (id < 0 || id >= size) {
                bad = 2;
            } else if (entry_live(live_bits, id)) {   // an entry dropped from the memory is no candidate
                key = make_key(q_stage[id], id);
                keep = true;
            }
        }
        const int slot = warp_claim_slot(keep, &kept_s);
        if (keep) keys[slot] = key;
    }
    if (bad) atomicOr(&bad_s, bad);
    __syncthreads();
    if (bad_s) {
        if (tid == 0) atomicCAS(status, 0, (bad_s & 2) ? (int)EVK_ERR_RANGE : (int)EVK_ERR_UNSUPPORTED);
        n = 0;
    } else {
        n = kept_s;
    }
    if (n > k) {
        block_select_topk<kThreads, kSelPerThread>(keys, n, k, hist, scal);
        n = k;
    }
    const int np2 = next_pow2(n > 1 ? n : 1);
    for (int i = n + tid; i < np2; i += kThreads) keys[i] = 0;
    __syncthreads();
    block_sort_desc<kThreads>(keys, np2);
    for (int i = tid; i < k; i += kThreads) {
        ids_out[(size_t)task * k + i] = (i < n) ? key_id(keys[i]) : -1;
        q_out[(size_t)task * k + i] = (i < n) ? key_sim(keys[i]) : -INFINITY;
    }
}

}  // namespace

cudaError_t launch_select_by_value(const int32_t *cand_ids, const int32_t *offsets, int n_tasks, int64_t size,
                                   const uint32_t *live_bits, const float *q_stage, int k, int32_t *ids_out, float *q_out, int32_t *status,
                                   cudaStream_t stream, int *launches) {
    if (n_tasks <= 0) return cudaSuccess;
    select_by_value_kernel<<<n_tasks, kThreads, 0, stream>>>(cand_ids, offsets, size, live_bits, q_stage, k, ids_out, q_out, status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace evk
