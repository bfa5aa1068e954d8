// The unified value update (Eq. 4; Eq. 8 in Appendix A):
//
//   Q_stage[id] <- Q + alpha * (r - Q)        for each (id, r) of the batch, in array order.
//
// An id may occur many times in one batch (popular entries are retrieved often),
// and binary32 arithmetic is not associative, so the stored bits depend on the
// order in which one entry's rewards are applied.  The order is fixed to array
// order: the batch is sorted by id with a STABLE radix sort (so each entry's
// rewards stay in array order), and one thread then walks each entry's run of
// rewards sequentially with three separately rounded operations.  Entries with
// different ids do not interact, so they run in parallel.
//
// A checking pass runs first; if any id is out of range or any reward is not
// finite, nothing is written and the status word records why.
#include <mutex>

#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPerThread = 8;
constexpr int kTile = kThreads * kPerThread;  // 2048 elements per block and pass

constexpr int kFlagRange = 1, kFlagNonFinite = 2;

__global__ void __launch_bounds__(kThreads)
validate_kernel(const int32_t *__restrict__ ids, const float *__restrict__ rewards, int64_t m, int64_t size,
                int *__restrict__ flags) {
    int bad = 0;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < m; i += (int64_t)gridDim.x * kThreads) {
        const int32_t id = ids[i];
        if (id < 0 || id >= size) bad |= kFlagRange;
        const float r = rewards[i];
        if (!(fabsf(r) <= 3.402823466e38f)) bad |= kFlagNonFinite;
    }
    bad = __reduce_or_sync(0xffffffffu, bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicOr(flags, bad);
}

// Per-block histogram of one 8-bit digit; hist is digit-major: hist[digit * nb + block].
__global__ void __launch_bounds__(kThreads)
radix_hist_kernel(const int32_t *__restrict__ keys, int64_t m, int shift, int nb, const int *__restrict__ flags,
                  int *__restrict__ hist) {
    if (*flags) return;
    __shared__ int h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kTile;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        const int64_t e = base + threadIdx.x + j * kThreads;
        if (e < m) atomicAdd(&h[(keys[e] >> shift) & 0xff], 1);
    }
    __syncthreads();
    hist[threadIdx.x * nb + blockIdx.x] = h[threadIdx.x];
}

// Exclusive scan of n ints in place, one block.
__global__ void __launch_bounds__(1024)
scan_kernel(int *__restrict__ data, int n, const int *__restrict__ flags) {
    if (*flags) return;
    __shared__ int warp_sums[32];
    __shared__ int carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int base = 0; base < n; base += 1024) {
        const int i = base + tid;
        const int v = (i < n) ? data[i] : 0;
        int x = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += u;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int s = warp_sums[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, s, off);
                if (lane >= off) s += u;
            }
            warp_sums[lane] = s;  // inclusive over warps
        }
        __syncthreads();
        const int carry = carry_s;
        const int before = (warp ? warp_sums[warp - 1] : 0) + carry;
        if (i < n) data[i] = before + x - v;
        __syncthreads();
        if (tid == 1023) carry_s = before + x;
        __syncthreads();
    }
}

// Stable scatter of one digit.  Warp w owns the 256 consecutive elements
// [tile + 256w, tile + 256w + 256) and visits them 32 at a time in order, so ranks
// within a digit follow array order inside the warp, warps are ordered by prefix
// sums, and blocks by the scanned histogram.
__global__ void __launch_bounds__(kThreads)
radix_scatter_kernel(const int32_t *__restrict__ keys_in, const float *__restrict__ vals_in, int64_t m,
                     int shift, int nb, const int *__restrict__ flags, const int *__restrict__ offsets,
                     int32_t *__restrict__ keys_out, float *__restrict__ vals_out) {
    if (*flags) return;
    __shared__ int warp_cnt[kWarps][256];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < kWarps * 256; i += kThreads) (&warp_cnt[0][0])[i] = 0;
    __syncthreads();

    const int64_t base = (int64_t)blockIdx.x * kTile + warp * (32 * kPerThread);
    int32_t key[kPerThread];
    float val[kPerThread];
    int rank[kPerThread];
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int r = 0; r < kPerThread; ++r) {
        const int64_t e = base + r * 32 + lane;
        const bool valid = e < m;
        key[r] = valid ? keys_in[e] : 0;
        val[r] = valid ? vals_in[e] : 0.0f;
        const int digit = valid ? ((key[r] >> shift) & 0xff) : 256;
        const uint32_t peers = __match_any_sync(0xffffffffu, digit);
        int old = 0;
        if (valid) old = warp_cnt[warp][digit];
        __syncwarp();
        if (valid && (peers & lt_mask) == 0) warp_cnt[warp][digit] = old + __popc(peers);
        __syncwarp();
        rank[r] = old + __popc(peers & lt_mask);
    }
    __syncthreads();
    {
        // digit `tid`: turn per-warp counts into starting offsets
        int run = offsets[tid * nb + blockIdx.x];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int t = warp_cnt[w][tid];
            warp_cnt[w][tid] = run;
            run += t;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kPerThread; ++r) {
        const int64_t e = base + r * 32 + lane;
        if (e < m) {
            const int digit = (key[r] >> shift) & 0xff;
            const int dst = warp_cnt[warp][digit] + rank[r];
            keys_out[dst] = key[r];
            vals_out[dst] = val[r];
        }
    }
}

// One step of Eq. 4 (Eq. 8 with a decreasing step size when `decay`): three separately rounded
// binary32 operations, never contracted into a fused multiply-add.
__device__ __forceinline__ float value_step(float q, float r, float alpha, bool decay, uint32_t &seen) {
    const float a = decay ? __fdiv_rn(1.0f, __uint2float_rn(++seen)) : alpha;
    const float diff = __fsub_rn(r, q);
    const float step = __fmul_rn(a, diff);
    return __fadd_rn(q, step);
}

// The sorted batch as the run walk sees it: separate id / reward arrays, or (id, reward bits) pairs.
struct SortedArrays {
    const int32_t *ids;
    const float *rewards;
    __device__ __forceinline__ int32_t id(int64_t i) const { return ids[i]; }
    __device__ __forceinline__ float reward(int64_t i) const { return rewards[i]; }
};
struct SortedPairs {
    const uint64_t *pairs;
    __device__ __forceinline__ int32_t id(int64_t i) const { return (int32_t)(uint32_t)pairs[i]; }
    __device__ __forceinline__ float reward(int64_t i) const { return __uint_as_float((uint32_t)(pairs[i] >> 32)); }
};

// Walks the runs of equal ids of a batch sorted by id (each entry's rewards in array order).  One
// thread per element; the thread at a run's first element owns the run.  A run of one element (most
// are) costs one round trip to memory.  A long run (a very popular entry) cannot be split, since the
// order of the rewards is part of the result; it is handed to a whole warp, whose lanes fetch 32
// rewards at a time (the next 32 are in flight meanwhile) and all step through the same recurrence
// on broadcast values, so that the chain of dependent operations never waits for memory.
constexpr int kApplyThreads = 256;
constexpr int kLongRun = 96;       // runs from this length on are walked by a warp
constexpr int kLongSlots = 32;     // long runs a block can hand to its warps (more are walked by their threads)

template <class Sorted>
__global__ void __launch_bounds__(kApplyThreads)
apply_runs_kernel(const Sorted sorted, int64_t m, float alpha, float *__restrict__ q_stage,
                  uint32_t *__restrict__ visits, const int *__restrict__ flags, int32_t *__restrict__ status,
                  uint32_t *__restrict__ longest_run) {
    __shared__ int long_n;
    __shared__ long long long_start[kLongSlots];
    pdl_trigger();
    pdl_wait();
    const int f = *flags;
    if (f) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && *status == 0)
            *status = (f & kFlagRange) ? EVK_ERR_RANGE : EVK_ERR_NONFINITE;
        return;
    }
    const bool decay = visits != nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) long_n = 0;
    __syncthreads();
    const int64_t t = blockIdx.x * (int64_t)kApplyThreads + threadIdx.x;
    if (t < m) {
        const int32_t id = sorted.id(t);
        const int32_t prev = t > 0 ? sorted.id(t - 1) : -1;
        const int32_t next = t + 1 < m ? sorted.id(t + 1) : -1;
        if (prev != id) {
            const float r0 = sorted.reward(t);
            float q = q_stage[id];
            uint32_t seen = decay ? visits[id] : 0;
            bool mine = true;
            if (next == id) {
                // end of the run: first index > t whose id differs (ids are sorted)
                int64_t lo = t + 1, hi = m;  // id(lo) == id, id(hi) != id (or hi == m)
                while (hi - lo > 1) {
                    const int64_t mid = (lo + hi) >> 1;
                    if (sorted.id(mid) == id) lo = mid; else hi = mid;
                }
                const int64_t end = hi;
                if (longest_run && end - t > 8) atomicMax(longest_run, (uint32_t)(end - t));
                if (end - t >= kLongRun) {
                    const int slot = atomicAdd(&long_n, 1);
                    if (slot < kLongSlots) {
                        long_start[slot] = t;
                        mine = false;
                    }
                }
                if (mine) {
                    q = value_step(q, r0, alpha, decay, seen);
                    for (int64_t j = t + 1; j < end; ++j) q = value_step(q, sorted.reward(j), alpha, decay, seen);
                }
            } else {
                q = value_step(q, r0, alpha, decay, seen);
            }
            if (mine) {
                q_stage[id] = q;
                if (decay) visits[id] = seen;
            }
        }
    }
    __syncthreads();
    const int n_long = long_n < kLongSlots ? long_n : kLongSlots;
    for (int s = warp; s < n_long; s += kApplyThreads / 32) {
        const int64_t t0 = long_start[s];
        const int32_t id = sorted.id(t0);
        int64_t lo = t0, hi = m;
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (sorted.id(mid) == id) lo = mid; else hi = mid;
        }
        const int64_t end = hi;
        float q = q_stage[id];
        uint32_t seen = decay ? visits[id] : 0;
        float cur = (t0 + lane < end) ? sorted.reward(t0 + lane) : 0.0f;
        for (int64_t j0 = t0; j0 < end; j0 += 32) {
            const float nxt = (j0 + 32 + lane < end) ? sorted.reward(j0 + 32 + lane) : 0.0f;
            if (end - j0 >= 32) {
#pragma unroll
                for (int j = 0; j < 32; ++j) q = value_step(q, __shfl_sync(0xffffffffu, cur, j), alpha, decay, seen);
            } else {
                const int n = (int)(end - j0);
                for (int j = 0; j < n; ++j) q = value_step(q, __shfl_sync(0xffffffffu, cur, j), alpha, decay, seen);
            }
            cur = nxt;
        }
        if (lane == 0) {
            q_stage[id] = q;
            if (decay) visits[id] = seen;
        }
    }
}

// Small batches (a retrieved context is B*k2 ids) in ONE launch: a single block checks the
// batch, sorts (id, position) pairs in shared memory and walks each entry's run.  Sorting by
// the pair keeps every entry's rewards in array order, as the multi-kernel path does.
constexpr int kSmallThreads = 1024;
constexpr int kSmallMax = 2048;   // above this the cluster sort is faster

__global__ void __launch_bounds__(kSmallThreads)
small_update_kernel(const int32_t *__restrict__ ids, const float *__restrict__ rewards, int m, int n_pow2,
                    int64_t size, float alpha, float *__restrict__ q_stage, uint32_t *__restrict__ visits,
                    int32_t *__restrict__ status, uint32_t *__restrict__ longest_run) {
    extern __shared__ __align__(16) unsigned char small_smem[];
    uint64_t *keys = reinterpret_cast<uint64_t *>(small_smem);        // [n_pow2] (id << 32) | position
    float *r = reinterpret_cast<float *>(keys + n_pow2);               // [m]
    __shared__ int bad_s;
    const int tid = threadIdx.x;
    pdl_trigger();
    pdl_wait();  // ids usually come straight out of the retrieval enqueued before
    if (tid == 0) bad_s = 0;
    __syncthreads();
    int bad = 0;
    for (int i = tid; i < n_pow2; i += kSmallThreads) {
        uint64_t key = ~(uint64_t)0;  // padding sorts last
        if (i < m) {
            const int32_t id = ids[i];
            const float rv = rewards[i];
            if (id < 0 || id >= size) bad |= kFlagRange;
            if (!(fabsf(rv) <= 3.402823466e38f)) bad |= kFlagNonFinite;
            key = ((uint64_t)(uint32_t)id << 32) | (uint32_t)i;
            r[i] = rv;
        }
        keys[i] = key;
    }
    if (bad) atomicOr(&bad_s, bad);
    __syncthreads();
    if (bad_s) {
        if (tid == 0 && *status == 0) *status = (bad_s & kFlagRange) ? EVK_ERR_RANGE : EVK_ERR_NONFINITE;
        return;
    }
    // bitonic sort, ascending
    // (a stage with stride <= 32 stays inside the 64 elements a warp owns: warp sync is enough)
    bool wide_before = true;
    for (int sz = 2; sz <= n_pow2; sz <<= 1) {
        for (int stride = sz >> 1; stride > 0; stride >>= 1) {
            const bool wide = stride > 32;
            if (wide || wide_before) __syncthreads(); else __syncwarp();
            wide_before = wide;
            for (int t = tid; t < (n_pow2 >> 1); t += kSmallThreads) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool asc = ((lo & sz) == 0);
                const uint64_t a = keys[lo], b = keys[hi];
                if ((a > b) == asc) { keys[lo] = b; keys[hi] = a; }
            }
        }
    }
    __syncthreads();
    for (int t = tid; t < m; t += kSmallThreads) {
        const uint32_t id = (uint32_t)(keys[t] >> 32);
        if (t > 0 && (uint32_t)(keys[t - 1] >> 32) == id) continue;  // not the head of its run
        float q = q_stage[id];
        uint32_t seen = visits ? visits[id] : 0;
        int j = t;
        for (; j < m && (uint32_t)(keys[j] >> 32) == id; ++j) {
            // decreasing step size: alpha_t = 1 / (updates this entry has received, this one included)
            q = value_step(q, r[(uint32_t)keys[j]], alpha, visits != nullptr, seen);
        }
        q_stage[id] = q;
        if (visits) visits[id] = seen;
    }
}

// ---- medium batches: the sort in ONE launch of one cluster of thread blocks -----------------
//
// A stable least-significant-digit radix sort of the (id, reward) pairs, 8 bits a pass.  The blocks
// of a cluster are scheduled together by the hardware, so the phases of a pass are separated by
// cluster barriers and the per-block digit counts are read from the partners' shared memory; no
// block ever spins on memory that another block writes.  Element e belongs to warp e / span of the
// cluster, which visits its elements 32 at a time in array order: ranks inside a digit follow array
// order within the warp, warps and blocks are ordered by prefix sums, so every pass is stable and
// an entry's rewards stay in array order.  Inside a block the pairs are first put in digit order in
// shared memory, so that the block writes each digit's pairs to global memory as one contiguous
// piece (a direct scatter of single pairs costs a memory transaction per pair, and a cluster has
// only as many load/store units as it has blocks).
constexpr int kClThreads = 1024;
constexpr int kClWarps = kClThreads / 32;
constexpr int kClusterMax = 65536;   // updates one cluster sorts

__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the value at the same shared-memory address in block `rank` of the cluster
__device__ __forceinline__ int cl_peer_int(const int *p, uint32_t rank) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(p), r;
    int v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(r) : "memory");
    return v;
}

// NB blocks of 1,024 threads sort up to MAXM updates; a warp visits at most ROUNDS = MAXM / (NB * 1024) groups of 32.
// flags_out receives the verdict of the checking pass (0: the batch is sound and pairs_out holds
// it sorted; otherwise nothing else was written).  The sorted batch ends in pairs_a for an odd
// number of passes, in pairs_b for an even one.
template <int NB, int MAXM = kClusterMax>
__global__ void __launch_bounds__(kClThreads, 1)
cluster_sort_kernel(const int32_t *__restrict__ ids, const float *__restrict__ rewards, int m, int64_t size,
                    int *__restrict__ flags_out, uint64_t *pairs_a, uint64_t *pairs_b, int passes) {
    constexpr int ROUNDS = MAXM / (NB * kClThreads);
    extern __shared__ __align__(16) unsigned char cl_smem[];
    uint64_t *local = reinterpret_cast<uint64_t *>(cl_smem);   // [ROUNDS * 1024] this block's pairs in digit order
    __shared__ int warp_cnt[kClWarps][256];   // per warp and digit: count, then offset inside the block's digit
    __shared__ int cta_hist[256];             // this block's count per digit (read by the whole cluster)
    __shared__ int gbase[256];                // where this block's pairs of a digit start in global memory
    __shared__ int lstart[256];               // where they start in `local`
    __shared__ int scan_tmp[2][8];
    __shared__ int flag_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cl_rank();
    pdl_trigger();
    pdl_wait();
    // elements of warp (rank, warp): [first, first + span), visited 32 at a time
    const int span = (((m + NB * kClWarps - 1) / (NB * kClWarps)) + 31) & ~31;
    const int first = ((int)rank * kClWarps + warp) * span;
    const int rounds = span >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;

    // ---- check the batch before anything is written ----
    if (tid == 0) flag_s = 0;
    __syncthreads();
    uint64_t pr[ROUNDS];
    int bad = 0;
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
        const int e = first + r * 32 + lane;
        const bool valid = r < rounds && e < m;
        const int32_t id = valid ? ids[e] : 0;
        const float rv = valid ? rewards[e] : 0.0f;
        if (valid) {
            if (id < 0 || id >= size) bad |= kFlagRange;
            if (!(fabsf(rv) <= 3.402823466e38f)) bad |= kFlagNonFinite;
        }
        pr[r] = ((uint64_t)__float_as_uint(rv) << 32) | (uint32_t)id;
    }
    bad = __reduce_or_sync(0xffffffffu, bad);
    if (lane == 0 && bad) atomicOr(&flag_s, bad);
    __syncthreads();
    cl_sync();
    {
        int all = 0;
#pragma unroll
        for (uint32_t c = 0; c < NB; ++c) all |= cl_peer_int(&flag_s, c);
        if (rank == 0 && tid == 0) *flags_out = all;
        if (all) {        // the same verdict in every block: all leave together
            cl_sync();    // nobody's shared memory goes away while a partner still reads it
            return;
        }
    }

    uint64_t *out = pairs_a;
    for (int pass = 0; pass < passes; ++pass) {
        const int shift = 8 * pass;
        for (int i = tid; i < kClWarps * 256; i += kClThreads) (&warp_cnt[0][0])[i] = 0;
        __syncthreads();
        int rnk[ROUNDS];
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const int e = first + r * 32 + lane;
            const bool valid = r < rounds && e < m;
            const uint32_t digit = ((uint32_t)pr[r] >> shift) & 0xff;
            // lanes of this group with the same digit: one ballot per digit bit
            uint32_t peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const uint32_t bal = __ballot_sync(0xffffffffu, (digit >> b) & 1u);
                peers &= ((digit >> b) & 1u) ? bal : ~bal;
            }
            int old = 0;
            if (valid) old = warp_cnt[warp][digit];
            __syncwarp();
            if (valid && (peers & lt_mask) == 0) warp_cnt[warp][digit] = old + __popc(peers);
            __syncwarp();
            rnk[r] = old + __popc(peers & lt_mask);
        }
        __syncthreads();
        if (tid < 256) {
            // digit `tid`: per-warp counts become offsets inside the block's digit; the total goes on show
            int run = 0;
#pragma unroll 8
            for (int w = 0; w < kClWarps; ++w) {
                const int t = warp_cnt[w][tid];
                warp_cnt[w][tid] = run;
                run += t;
            }
            cta_hist[tid] = run;
        }
        __syncthreads();
        cl_sync();
        if (tid < 256) {
            // Digit `tid` of this block starts, in global memory, behind all smaller digits of the
            // cluster and behind this digit in the blocks before this one; in `local`, behind this
            // block's smaller digits.
            int total = 0, before = 0, h[NB];
#pragma unroll
            for (uint32_t c = 0; c < NB; ++c) h[c] = cl_peer_int(&cta_hist[tid], c);
#pragma unroll
            for (uint32_t c = 0; c < NB; ++c) {
                total += h[c];
                if (c < rank) before += h[c];
            }
            const int mine = cta_hist[tid];
            int incl_t = total, incl_m = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, incl_t, off);
                const int v = __shfl_up_sync(0xffffffffu, incl_m, off);
                if (lane >= off) { incl_t += u; incl_m += v; }
            }
            if (lane == 31) { scan_tmp[0][warp] = incl_t; scan_tmp[1][warp] = incl_m; }
            // (only the first eight warps are here; they meet at a named barrier)
            asm volatile("bar.sync 1, 256;" ::: "memory");
            int base_t = incl_t - total, base_m = incl_m - mine;
            for (int w = 0; w < warp; ++w) { base_t += scan_tmp[0][w]; base_m += scan_tmp[1][w]; }
            gbase[tid] = base_t + before;
            lstart[tid] = base_m;
        }
        __syncthreads();
        // the block's pairs in digit order in shared memory ...
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const int e = first + r * 32 + lane;
            if (r < rounds && e < m) {
                const uint32_t digit = ((uint32_t)pr[r] >> shift) & 0xff;
                local[lstart[digit] + warp_cnt[warp][digit] + rnk[r]] = pr[r];
            }
        }
        __syncthreads();
        // ... and out to global memory, every digit's pairs as one contiguous piece
        const int n_local = lstart[255] + cta_hist[255];
        for (int i = tid; i < n_local; i += kClThreads) {
            const uint64_t v = local[i];
            const uint32_t digit = ((uint32_t)v >> shift) & 0xff;
            out[gbase[digit] + (i - lstart[digit])] = v;
        }
        // the pairs are visible to the whole cluster, and cta_hist may be rewritten
        __syncthreads();
        cl_sync();
        if (pass + 1 < passes) {
#pragma unroll
            for (int r = 0; r < ROUNDS; ++r) {
                const int e = first + r * 32 + lane;
                pr[r] = (r < rounds && e < m) ? out[e] : 0;
            }
            out = (out == pairs_a) ? pairs_b : pairs_a;
        }
    }
}

int num_blocks(int64_t m) { return (int)((m + kTile - 1) / kTile); }

struct UpdateLayout {
    size_t flags, hist, keys_a, vals_a, keys_b, vals_b, total;
};

UpdateLayout layout_for(int64_t m) {
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    UpdateLayout l;
    const size_t nb = (size_t)num_blocks(m > 0 ? m : 1);
    l.flags = 0;
    l.hist = 256;
    l.keys_a = l.hist + align(256 * nb * sizeof(int));
    l.vals_a = l.keys_a + align((size_t)m * 4);
    l.keys_b = l.vals_a + align((size_t)m * 4);
    l.vals_b = l.keys_b + align((size_t)m * 4);
    l.total = l.vals_b + align((size_t)m * 4);
    return l;
}

}  // namespace

size_t q_update_workspace_bytes(int64_t m) { return layout_for(m).total; }

// Launches the cluster sort with NB blocks if the device can co-schedule such a cluster.
template <int NB, int MAXM = kClusterMax>
cudaError_t try_cluster_sort(const int32_t *ids, const float *rewards, int m, int64_t size, int *flags,
                             uint64_t *pairs_a, uint64_t *pairs_b, int passes, cudaStream_t stream, bool *launched) {
    *launched = false;
    auto kern = cluster_sort_kernel<NB, MAXM>;
    const size_t smem = (size_t)(MAXM / NB) * sizeof(uint64_t);
    static int usable = -1;   // -1: not asked yet (asked once; every device of a process is the same part)
    if (usable < 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess && NB > 8) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        int n_clusters = 0;
        if (e == cudaSuccess) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(NB);
            q.blockDim = dim3(kClThreads);
            q.dynamicSmemBytes = smem;
            cudaLaunchAttribute a[1];
            a[0].id = cudaLaunchAttributeClusterDimension;
            a[0].val.clusterDim.x = NB;
            a[0].val.clusterDim.y = 1;
            a[0].val.clusterDim.z = 1;
            q.attrs = a;
            q.numAttrs = 1;
            e = cudaOccupancyMaxActiveClusters(&n_clusters, kern, &q);
        }
        if (e != cudaSuccess) (void)cudaGetLastError();
        usable = (e == cudaSuccess && n_clusters >= 1) ? 1 : 0;
    }
    if (!usable) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(NB);
    cfg.blockDim = dim3(kClThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    // A plain launch, not a programmatic dependent one: on B200 (driver 580) a kernel launched as a
    // cluster with that attribute was seen to run past its griddepcontrol.wait while the kernel before
    // it (the merge that writes the ids) was still running.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = NB;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    *launched = true;
    return cudaLaunchKernelEx(&cfg, kern, ids, rewards, m, size, flags, pairs_a, pairs_b, passes);
}

cudaError_t launch_q_update(float *q_stage, int64_t size, const int32_t *ids, const float *rewards,
                            int64_t m, float alpha, uint32_t *visits, int32_t *status, void *workspace,
                            cudaStream_t stream, int *launches, uint32_t *longest_run) {
    if (m <= 0) return cudaSuccess;
    if (m <= kSmallMax) {
        int n_pow2 = 2;
        while (n_pow2 < m) n_pow2 <<= 1;
        const size_t smem = (size_t)n_pow2 * sizeof(uint64_t) + (size_t)m * sizeof(float);
        ++*launches;
        return launch_overlapped(small_update_kernel, dim3(1), dim3(kSmallThreads), smem, stream, ids, rewards, (int)m,
                                 n_pow2, size, alpha, q_stage, visits, status, longest_run);
    }
    int bits = 0;
    while (bits < 31 && ((int64_t)1 << bits) < size) ++bits;
    int passes = (bits + 7) / 8;
    if (passes < 1) passes = 1;
    const UpdateLayout l = layout_for(m);
    char *ws = static_cast<char *>(workspace);
    int *flags = reinterpret_cast<int *>(ws + l.flags);
    const int apply_grid = (int)((m + kApplyThreads - 1) / kApplyThreads);

    if (m <= kClusterMax) {
        // the four key / value arrays of the multi-launch path double as two arrays of pairs
        uint64_t *pairs_a = reinterpret_cast<uint64_t *>(ws + l.keys_a);
        uint64_t *pairs_b = reinterpret_cast<uint64_t *>(ws + l.keys_b);
        bool launched = false;
        // smaller batches sort in smaller clusters, whose barriers and digit-count exchanges are cheaper:
        // 2,049-8,192 updates in 4 blocks, up to 16,384 in 8 (19-23 us against 25-27 with 16)
        cudaError_t err = cudaSuccess;
        if (m <= 8192)
            err = try_cluster_sort<4, 8192>(ids, rewards, (int)m, size, flags, pairs_a, pairs_b, passes, stream, &launched);
        else if (m <= 16384)
            err = try_cluster_sort<8, 16384>(ids, rewards, (int)m, size, flags, pairs_a, pairs_b, passes, stream, &launched);
        if (err == cudaSuccess && !launched)
            err = try_cluster_sort<16>(ids, rewards, (int)m, size, flags, pairs_a, pairs_b, passes, stream, &launched);
        if (err == cudaSuccess && !launched)
            err = try_cluster_sort<8>(ids, rewards, (int)m, size, flags, pairs_a, pairs_b, passes, stream, &launched);
        if (err != cudaSuccess) return err;
        if (launched) {
            ++*launches;
            SortedPairs sorted;
            sorted.pairs = (passes & 1) ? pairs_a : pairs_b;
            ++*launches;
            return launch_overlapped(apply_runs_kernel<SortedPairs>, dim3(apply_grid), dim3(kApplyThreads), 0, stream,
                                     sorted, m, alpha, q_stage, visits, (const int *)flags, status, longest_run);
        }
    }

    int *hist = reinterpret_cast<int *>(ws + l.hist);
    int32_t *keys[2] = {reinterpret_cast<int32_t *>(ws + l.keys_a), reinterpret_cast<int32_t *>(ws + l.keys_b)};
    float *vals[2] = {reinterpret_cast<float *>(ws + l.vals_a), reinterpret_cast<float *>(ws + l.vals_b)};
    const int nb = num_blocks(m);

    cudaError_t err = cudaMemsetAsync(flags, 0, sizeof(int), stream);
    if (err != cudaSuccess) return err;
    int vgrid = (int)((m + kThreads - 1) / kThreads);
    if (vgrid > num_sms() * 8) vgrid = num_sms() * 8;
    validate_kernel<<<vgrid, kThreads, 0, stream>>>(ids, rewards, m, size, flags);
    ++*launches;

    const int32_t *k_in = ids;
    const float *v_in = rewards;
    for (int p = 0; p < passes; ++p) {
        int32_t *k_out = keys[p & 1];
        float *v_out = vals[p & 1];
        radix_hist_kernel<<<nb, kThreads, 0, stream>>>(k_in, m, 8 * p, nb, flags, hist);
        scan_kernel<<<1, 1024, 0, stream>>>(hist, 256 * nb, flags);
        radix_scatter_kernel<<<nb, kThreads, 0, stream>>>(k_in, v_in, m, 8 * p, nb, flags, hist, k_out, v_out);
        *launches += 3;
        k_in = k_out;
        v_in = v_out;
    }
    SortedArrays sorted;
    sorted.ids = k_in;
    sorted.rewards = v_in;
    apply_runs_kernel<SortedArrays><<<apply_grid, kApplyThreads, 0, stream>>>(sorted, m, alpha, q_stage, visits, flags, status, longest_run);
    ++*launches;
    return cudaGetLastError();
}

// ---- the same update for callers that cannot allocate device memory ------------
//
// Scratch for one batch of at most kStaticMaxUpdates updates, reserved in the
// library image itself.  Every GPU that loads the library carries these bytes
// until the process exits.  All calls on a device share the array.
constexpr int64_t kStaticMaxUpdates = 65536;
constexpr size_t kStaticScratchBytes = 256 + 256 * 32 * sizeof(int) + 4 * (size_t)kStaticMaxUpdates * 4;
static __device__ __align__(256) unsigned char g_q_update_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices];  // device address of g_q_update_scratch, per device ordinal
std::mutex g_scratch_mu;

// The array's name is only a host-side handle here; the address a kernel can use has to
// be asked for, with the device that will run the kernel current.
cudaError_t static_scratch(void **out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        err = cudaGetSymbolAddress(&p, g_q_update_scratch);
        if (err != cudaSuccess) return err;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}
}  // namespace

int64_t q_update_static_max() { return kStaticMaxUpdates; }

cudaError_t launch_q_update_static(float *q_stage, int64_t size, const int32_t *ids, const float *rewards,
                                   int64_t m, float alpha, int32_t *status, cudaStream_t stream, int *launches) {
    if (m <= 0) return cudaSuccess;
    if (m > kStaticMaxUpdates || layout_for(m).total > kStaticScratchBytes) return cudaErrorInvalidValue;
    void *scratch = nullptr;
    cudaError_t err = static_scratch(&scratch);
    if (err != cudaSuccess) return err;
    // launch_q_update clears the flag word itself and overwrites every other part of the
    // scratch it reads, so what the previous call left behind does not matter.
    return launch_q_update(q_stage, size, ids, rewards, m, alpha, nullptr, status, scratch, stream, launches);
}

}  // namespace evk
