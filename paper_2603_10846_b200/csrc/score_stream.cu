// Phase 1 for small query batches: a streaming scan of the bank.
//
// Dense retrieval of the candidate pool (Section 3.2) needs sim = <q, e_i> for
// every stored entry and the k1 largest per query.  With a handful of queries the
// scan moves 2*d bytes per entry and does almost no arithmetic, so it is bound by
// HBM bandwidth: each warp reads whole bank rows with 128-bit coalesced loads,
// keeps its slice of every query in registers as fp32, multiplies, and reduces
// across the warp with shuffles.  The similarities are never written out: a row
// survives only if it beats the block's current k1-th best for that query, and
// survivors go to a per-query candidate list in shared memory that is cut back to
// the best k1 (exact radix select) whenever it fills.  Each block finally writes
// at most k1 candidates per query; a second kernel merges the blocks' lists.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerWarp = 8;
constexpr int kRowsPerIter = kWarps * kRowsPerWarp;  // rows a block takes per iteration
constexpr int kSelPerThread = 8;                     // capacity <= kThreads * kSelPerThread
constexpr int kMaxCap = kThreads * kSelPerThread;    // 2048

// A bank row is read once per launch: no L1 allocation, and first in line for eviction from L2 so
// that the stream does not push out what is read again (queries, candidate lists).
__device__ __forceinline__ uint4 ldg_stream(const uint4 *p, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}

// QB queries per pass, NCH 16-byte chunks of a row per lane (row width d <= NCH*256).
template <int QB, int NCH>
__global__ void __launch_bounds__(kThreads)
score_stream_kernel(const __nv_bfloat16 *__restrict__ bank, int64_t size, int d,
                    const __nv_bfloat16 *__restrict__ queries, int q_base, int nq, int k1, int cap,
                    int nparts, uint64_t *__restrict__ part_keys, int *__restrict__ part_counts,
                    const uint32_t *__restrict__ live_bits) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t *keys = reinterpret_cast<uint64_t *>(smem_raw);          // [QB][cap]
    uint64_t *scal = keys + (size_t)QB * cap;                         // [4]
    uint64_t *tau_key = scal + 4;                                     // [QB]
    float *tau_sim = reinterpret_cast<float *>(tau_key + QB);         // [QB]
    int *counts = reinterpret_cast<int *>(tau_sim + QB);              // [QB]
    int *hist = counts + QB;                                          // [256]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = d >> 3;  // 16-byte chunks per row

    if (tid < QB) {
        tau_key[tid] = 0;
        tau_sim[tid] = -INFINITY;
        counts[tid] = 0;
    }

    // This lane's slice of every query, widened to fp32 once.
    float qf[QB][NCH * 8];
#pragma unroll
    for (int q = 0; q < QB; ++q) {
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int c = lane + 32 * j;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (q < nq && c < chunks)
                v = *reinterpret_cast<const uint4 *>(queries + (size_t)(q_base + q) * d + c * 8);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                qf[q][j * 8 + 2 * t] = __uint_as_float(w[t] << 16);
                qf[q][j * 8 + 2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u);
            }
        }
    }
    __syncthreads();

    const uint64_t policy = l2_evict_first_policy();
    const int64_t n_iters = (size + kRowsPerIter - 1) / kRowsPerIter;
    for (int64_t it = blockIdx.x; it < n_iters; it += gridDim.x) {
        const int64_t row0 = it * kRowsPerIter + warp * kRowsPerWarp;
#pragma unroll 1
        for (int rr = 0; rr < kRowsPerWarp; rr += 2) {
            uint4 v[2][NCH];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int64_t row = row0 + rr + r;
                const uint4 *src = reinterpret_cast<const uint4 *>(bank + row * d);
#pragma unroll
                for (int j = 0; j < NCH; ++j) {
                    const int c = lane + 32 * j;
                    v[r][j] = (row < size && c < chunks) ? ldg_stream(src + c, policy) : make_uint4(0, 0, 0, 0);
                }
            }
            float acc[2][QB];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
#pragma unroll
                for (int q = 0; q < QB; ++q) acc[r][q] = 0.0f;
#pragma unroll
                for (int j = 0; j < NCH; ++j) {
                    const uint32_t w[4] = {v[r][j].x, v[r][j].y, v[r][j].z, v[r][j].w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float lo = __uint_as_float(w[t] << 16);
                        const float hi = __uint_as_float(w[t] & 0xffff0000u);
#pragma unroll
                        for (int q = 0; q < QB; ++q) {
                            acc[r][q] = fmaf(lo, qf[q][j * 8 + 2 * t], acc[r][q]);
                            acc[r][q] = fmaf(hi, qf[q][j * 8 + 2 * t + 1], acc[r][q]);
                        }
                    }
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int q = 0; q < QB; ++q) acc[r][q] += __shfl_xor_sync(0xffffffffu, acc[r][q], off);
            }
            // lane q (< nq) files row r's similarity for query q.
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int64_t row = row0 + rr + r;
                float s = acc[r][0];
#pragma unroll
                for (int q = 1; q < QB; ++q)
                    if (lane == q) s = acc[r][q];
                if (lane < nq && row < size && s >= tau_sim[lane] && entry_live(live_bits, row)) {
                    const uint64_t key = make_key(s, (int32_t)row);
                    if (key > tau_key[lane]) {
                        const int slot = atomicAdd(&counts[lane], 1);
                        keys[(size_t)lane * cap + slot] = key;
                    }
                }
            }
        }
        __syncthreads();
        // A list that could overflow during the next iteration is cut back to its best k1.
        for (int q = 0; q < nq; ++q) {
            const int n = counts[q];
            if (n > cap - kRowsPerIter) {
                const uint64_t kth = block_select_topk<kThreads, kSelPerThread, false>(keys + (size_t)q * cap, n, k1, hist, scal);
                if (tid == 0) {
                    counts[q] = k1;
                    tau_key[q] = kth;
                    tau_sim[q] = key_sim(kth);
                }
            }
        }
        __syncthreads();
    }

    for (int q = 0; q < nq; ++q) {
        int n = counts[q];
        if (n > k1) {
            block_select_topk<kThreads, kSelPerThread, false>(keys + (size_t)q * cap, n, k1, hist, scal);
            n = k1;
        }
        const size_t list = (size_t)(q_base + q) * nparts + blockIdx.x;
        for (int i = tid; i < n; i += kThreads) part_keys[list * k1 + i] = keys[(size_t)q * cap + i];
        if (tid == 0) part_counts[list] = n;
        __syncthreads();
    }
}

int stream_cap(int k1) {
    int cap = 2 * next_pow2(k1);
    if (cap < 256) cap = 256;
    if (cap > kMaxCap) cap = kMaxCap;
    return cap;
}

size_t stream_smem(int qb, int cap) {
    return (size_t)qb * cap * 8 + 4 * 8 + (size_t)qb * (8 + 4 + 4) + 256 * 4 + 16;
}

template <int QB, int NCH>
cudaError_t launch_one(const __nv_bfloat16 *bank, int64_t size, int d, const __nv_bfloat16 *queries,
                       int q_base, int nq, int k1, const StreamPlan &plan, uint64_t *part_keys,
                       int *part_counts, cudaStream_t stream) {
    auto kern = score_stream_kernel<QB, NCH>;
    const size_t smem = stream_smem(QB, plan.cap);
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<plan.nparts, kThreads, smem, stream>>>(bank, size, d, queries, q_base, nq, k1, plan.cap,
                                                  plan.nparts, part_keys, part_counts, plan.live_bits);
    return cudaGetLastError();
}

template <int NCH>
cudaError_t launch_nch(int qb, const __nv_bfloat16 *bank, int64_t size, int d,
                       const __nv_bfloat16 *queries, int q_base, int nq, int k1, const StreamPlan &plan,
                       uint64_t *part_keys, int *part_counts, cudaStream_t stream) {
    if constexpr (NCH <= 4) {
        if (qb == 4)
            return launch_one<4, NCH>(bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream);
    }
    if (qb == 2)
        return launch_one<2, NCH>(bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream);
    return launch_one<1, NCH>(bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream);
}

// Blocks of this variant that fit on one SM (registers and shared memory), asked of the runtime:
// the grid is sized to exactly one wave of them.
template <int QB, int NCH>
int blocks_per_sm(size_t smem) {
    auto kern = score_stream_kernel<QB, NCH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 1;
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kThreads, smem) != cudaSuccess || n < 1) return 1;
    return n;
}

template <int NCH>
int blocks_per_sm_nch(int qb, size_t smem) {
    if constexpr (NCH <= 4) {
        if (qb == 4) return blocks_per_sm<4, NCH>(smem);
    }
    return qb == 2 ? blocks_per_sm<2, NCH>(smem) : blocks_per_sm<1, NCH>(smem);
}

int blocks_per_sm_for(int qb, int nch, size_t smem) {
    switch (nch) {
        case 1: return blocks_per_sm_nch<1>(qb, smem);
        case 2: return blocks_per_sm_nch<2>(qb, smem);
        case 3: return blocks_per_sm_nch<3>(qb, smem);
        case 4: return blocks_per_sm_nch<4>(qb, smem);
        case 6: return blocks_per_sm_nch<6>(qb, smem);
        case 8: return blocks_per_sm_nch<8>(qb, smem);
        default: return 1;
    }
}

int nch_for(int d) {
    const int chunks = d / 8;
    const int need = (chunks + 31) / 32;
    const int avail[] = {1, 2, 3, 4, 6, 8};
    for (int a : avail)
        if (need <= a) return a;
    return 0;
}

}  // namespace

bool stream_supported(int d) { return d > 0 && d % 8 == 0 && nch_for(d) != 0; }

StreamPlan stream_plan(int64_t size, int d, int B, int k1) {
    StreamPlan p;
    p.live_bits = nullptr;
    const int nch = nch_for(d);
    const int qb_max = (nch <= 4) ? 4 : 2;
    p.qb = B >= 4 ? 4 : (B >= 2 ? 2 : 1);
    if (p.qb > qb_max) p.qb = qb_max;
    p.cap = stream_cap(k1);
    p.smem = stream_smem(p.qb, p.cap);
    // Registers hold the queries, so occupancy falls as qb*nch grows (1-4 blocks per SM); a grid
    // that is not a whole wave of resident blocks leaves a ragged second wave.
    int ctas_per_sm = blocks_per_sm_for(p.qb, nch, p.smem);
    if (ctas_per_sm > 4) ctas_per_sm = 4;
    int64_t iters = (size + kRowsPerIter - 1) / kRowsPerIter;
    int64_t grid = (int64_t)num_sms() * ctas_per_sm;
    if (grid > iters) grid = iters;
    if (grid < 1) grid = 1;
    p.nparts = (int)grid;
    return p;
}

cudaError_t launch_score_stream(const __nv_bfloat16 *bank, int64_t size, int d,
                                const __nv_bfloat16 *queries, int B, int k1, const StreamPlan &plan,
                                uint64_t *part_keys, int *part_counts, cudaStream_t stream, int *launches) {
    const int nch = nch_for(d);
    for (int q_base = 0; q_base < B; q_base += plan.qb) {
        const int nq = (B - q_base < plan.qb) ? (B - q_base) : plan.qb;
        cudaError_t err;
        switch (nch) {
            case 1: err = launch_nch<1>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            case 2: err = launch_nch<2>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            case 3: err = launch_nch<3>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            case 4: err = launch_nch<4>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            case 6: err = launch_nch<6>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            case 8: err = launch_nch<8>(plan.qb, bank, size, d, queries, q_base, nq, k1, plan, part_keys, part_counts, stream); break;
            default: return cudaErrorInvalidValue;
        }
        if (err != cudaSuccess) return err;
        ++*launches;
    }
    return cudaSuccess;
}

}  // namespace evk
