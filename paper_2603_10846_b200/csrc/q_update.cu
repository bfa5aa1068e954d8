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

// One thread per run of equal ids (the thread at the run's first element).
__global__ void __launch_bounds__(kThreads)
apply_kernel(const int32_t *__restrict__ ids, const float *__restrict__ rewards, int64_t m, float alpha,
             float *__restrict__ q_stage, uint32_t *__restrict__ visits, const int *__restrict__ flags,
             int32_t *__restrict__ status) {
    const int f = *flags;
    if (f) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && *status == 0)
            *status = (f & kFlagRange) ? EVK_ERR_RANGE : EVK_ERR_NONFINITE;
        return;
    }
    const int64_t t = blockIdx.x * (int64_t)kThreads + threadIdx.x;
    if (t >= m) return;
    const int32_t id = ids[t];
    if (t > 0 && ids[t - 1] == id) return;
    // end of the run: first index > t whose id differs (ids are sorted)
    int64_t end = t + 1;
    if (end < m && ids[end] == id) {
        int64_t lo = end, hi = m;  // ids[lo] == id, ids[hi] != id (or hi == m)
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (ids[mid] == id) lo = mid; else hi = mid;
        }
        end = hi;
    }
    float q = q_stage[id];
    uint32_t seen = visits ? visits[id] : 0;
    for (int64_t j = t; j < end; ++j) {
        const float a = visits ? __fdiv_rn(1.0f, __uint2float_rn(++seen)) : alpha;
        const float diff = __fsub_rn(rewards[j], q);
        const float step = __fmul_rn(a, diff);
        q = __fadd_rn(q, step);
    }
    if (visits) visits[id] = seen;
    q_stage[id] = q;
}

// Small batches (a retrieved context is B*k2 ids) in ONE launch: a single block checks the
// batch, sorts (id, position) pairs in shared memory and walks each entry's run.  Sorting by
// the pair keeps every entry's rewards in array order, as the multi-kernel path does.
constexpr int kSmallThreads = 1024;
constexpr int kSmallMax = 8192;

__global__ void __launch_bounds__(kSmallThreads)
small_update_kernel(const int32_t *__restrict__ ids, const float *__restrict__ rewards, int m, int n_pow2,
                    int64_t size, float alpha, float *__restrict__ q_stage, uint32_t *__restrict__ visits,
                    int32_t *__restrict__ status) {
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
        for (int j = t; j < m && (uint32_t)(keys[j] >> 32) == id; ++j) {
            // decreasing step size: alpha_t = 1 / (updates this entry has received, this one included)
            const float a = visits ? __fdiv_rn(1.0f, __uint2float_rn(++seen)) : alpha;
            const float diff = __fsub_rn(r[(uint32_t)keys[j]], q);
            const float step = __fmul_rn(a, diff);
            q = __fadd_rn(q, step);
        }
        q_stage[id] = q;
        if (visits) visits[id] = seen;
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

cudaError_t launch_q_update(float *q_stage, int64_t size, const int32_t *ids, const float *rewards,
                            int64_t m, float alpha, uint32_t *visits, int32_t *status, void *workspace,
                            cudaStream_t stream, int *launches) {
    if (m <= 0) return cudaSuccess;
    if (m <= kSmallMax) {
        int n_pow2 = 2;
        while (n_pow2 < m) n_pow2 <<= 1;
        const size_t smem = (size_t)n_pow2 * sizeof(uint64_t) + (size_t)m * sizeof(float);
        cudaError_t e = cudaFuncSetAttribute(small_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(kSmallMax * (sizeof(uint64_t) + sizeof(float))));
        if (e != cudaSuccess) return e;
        ++*launches;
        return launch_overlapped(small_update_kernel, dim3(1), dim3(kSmallThreads), smem, stream, ids, rewards, (int)m,
                                 n_pow2, size, alpha, q_stage, visits, status);
    }
    const UpdateLayout l = layout_for(m);
    char *ws = static_cast<char *>(workspace);
    int *flags = reinterpret_cast<int *>(ws + l.flags);
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

    int bits = 0;
    while (bits < 31 && ((int64_t)1 << bits) < size) ++bits;
    int passes = (bits + 7) / 8;
    if (passes < 1) passes = 1;

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
    apply_kernel<<<(int)((m + kThreads - 1) / kThreads), kThreads, 0, stream>>>(k_in, v_in, m, alpha, q_stage, visits, flags, status);
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
