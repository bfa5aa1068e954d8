// Appending experiences to the memory (Eq. 1): embeddings become bf16 rows of the
// bank, and each new entry gets one value estimate per stage.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;

// 8 elements per thread: two 16-byte loads of fp32 (or one of bf16), one 16-byte store.
// (the query conversion; inserts use insert_kernel below)
__global__ void __launch_bounds__(kThreads)
insert_rows_kernel(__nv_bfloat16 *__restrict__ dst, const void *__restrict__ src, int is_bf16, int64_t n_vec) {
    pdl_trigger();
    pdl_wait();
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * kThreads) {
        uint4 out;
        if (is_bf16) {
            out = reinterpret_cast<const uint4 *>(src)[i];
        } else {
            const float4 a = reinterpret_cast<const float4 *>(src)[2 * i];
            const float4 b = reinterpret_cast<const float4 *>(src)[2 * i + 1];
            __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y);
            __nv_bfloat162 p1 = __floats2bfloat162_rn(a.z, a.w);
            __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y);
            __nv_bfloat162 p3 = __floats2bfloat162_rn(b.z, b.w);
            out.x = *reinterpret_cast<uint32_t *>(&p0);
            out.y = *reinterpret_cast<uint32_t *>(&p1);
            out.z = *reinterpret_cast<uint32_t *>(&p2);
            out.w = *reinterpret_cast<uint32_t *>(&p3);
        }
        reinterpret_cast<uint4 *>(dst)[i] = out;
    }
}

// Rows and values of an insert in one launch (an insert of a few rows is all launch latency).
__global__ void __launch_bounds__(kThreads)
insert_kernel(__nv_bfloat16 *__restrict__ dst, const void *__restrict__ src, int is_bf16, int64_t n_vec,
              float *__restrict__ q_tables, uint32_t *__restrict__ visits, uint32_t *__restrict__ live_bits,
              uint32_t *__restrict__ dev, int64_t capacity, int n_stages,
              int64_t first, int64_t n, int stage, const float *__restrict__ q_init, float q_default,
              int32_t *__restrict__ ids_out) {
    pdl_trigger();
    pdl_wait();   // the rows may come out of, and the value slots may still be read by, the kernel before
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * kThreads) {
        uint4 out;
        if (is_bf16) {
            out = reinterpret_cast<const uint4 *>(src)[i];
        } else {
            const float4 a = reinterpret_cast<const float4 *>(src)[2 * i];
            const float4 b = reinterpret_cast<const float4 *>(src)[2 * i + 1];
            __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y);
            __nv_bfloat162 p1 = __floats2bfloat162_rn(a.z, a.w);
            __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y);
            __nv_bfloat162 p3 = __floats2bfloat162_rn(b.z, b.w);
            out.x = *reinterpret_cast<uint32_t *>(&p0);
            out.y = *reinterpret_cast<uint32_t *>(&p1);
            out.z = *reinterpret_cast<uint32_t *>(&p2);
            out.w = *reinterpret_cast<uint32_t *>(&p3);
        }
        reinterpret_cast<uint4 *>(dst)[i] = out;
    }
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) {
        const float v = q_init ? q_init[i] : q_default;
        for (int s = 0; s < n_stages; ++s) {
            q_tables[(int64_t)s * capacity + first + i] = (stage < 0 || s == stage) ? v : q_default;
            visits[(int64_t)s * capacity + first + i] = 0;  // no update seen yet
        }
        atomicOr(live_bits + ((first + i) >> 5), 1u << ((first + i) & 31));   // the entry is in the memory
        if (ids_out) ids_out[i] = (int32_t)(first + i);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(dev + kDevLive, (uint32_t)n);
    // The last block to get here tells the scans that the rows are there.  (Inserts never overlap one
    // another: each waits for the kernel before it, so the ticket counter is back at 0 for the next.)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(dev + kDevInsTicket, 1u) == gridDim.x - 1) {
            dev[kDevInsTicket] = 0;
            __threadfence();
            atomicMax(dev + kDevRowsReady, (uint32_t)(first + n));
        }
    }
}

// ---- entries dropped from a live bank ------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
tombstone_check_kernel(const int32_t *__restrict__ ids, int64_t n, int64_t size, uint32_t *__restrict__ dev) {
    pdl_trigger();
    pdl_wait();
    int bad = 0;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads)
        if (ids[i] < 0 || ids[i] >= size) bad = 1;
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(dev + kDevFlag, 1u);
}

__global__ void __launch_bounds__(kThreads)
tombstone_apply_kernel(const int32_t *__restrict__ ids, int64_t n, uint32_t *__restrict__ live_bits,
                       uint32_t *__restrict__ dev, int32_t *__restrict__ status) {
    pdl_trigger();
    pdl_wait();
    if (dev[kDevFlag]) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(status, 0, (int)EVK_ERR_RANGE);
        return;
    }
    int dropped = 0;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) {
        const uint32_t bit = 1u << (ids[i] & 31);
        const uint32_t old = atomicAnd(live_bits + (ids[i] >> 5), ~bit);
        dropped += (old & bit) ? 1 : 0;      // an id named twice, or dropped before, counts once
    }
    dropped = __reduce_add_sync(0xffffffffu, dropped);
    if ((threadIdx.x & 31) == 0 && dropped) {
        atomicSub(dev + kDevLive, (uint32_t)dropped);
        atomicAdd(dev + kDevDropped, (uint32_t)dropped);
    }
}

__global__ void __launch_bounds__(kThreads)
live_export_kernel(const uint32_t *__restrict__ live_bits, int64_t first, int64_t n, uint8_t *__restrict__ out) {
    pdl_trigger();
    pdl_wait();
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads)
        out[i] = (uint8_t)((live_bits[(first + i) >> 5] >> ((first + i) & 31)) & 1u);
}

__global__ void __launch_bounds__(kThreads)
live_import_kernel(const uint8_t *__restrict__ live, int64_t first, int64_t n, uint32_t *__restrict__ live_bits,
                   uint32_t *__restrict__ dev) {
    pdl_trigger();
    pdl_wait();
    int dropped = 0;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) {
        if (live[i] == 0) {
            const uint32_t bit = 1u << ((first + i) & 31);
            const uint32_t old = atomicAnd(live_bits + ((first + i) >> 5), ~bit);
            dropped += (old & bit) ? 1 : 0;
        }
    }
    dropped = __reduce_add_sync(0xffffffffu, dropped);
    if ((threadIdx.x & 31) == 0 && dropped) {
        atomicSub(dev + kDevLive, (uint32_t)dropped);
        atomicAdd(dev + kDevDropped, (uint32_t)dropped);
    }
}

int grid_for(int64_t work_items) {
    int64_t g = (work_items + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)num_sms() * 8;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

}  // namespace

cudaError_t launch_insert(__nv_bfloat16 *bank, float *q_tables, uint32_t *visits, uint32_t *live_bits, uint32_t *dev,
                          int64_t capacity,
                          int d, int n_stages, int64_t first, int64_t n, const void *emb, int emb_dtype,
                          int stage, const float *q_init, float q_default, int32_t *ids_out,
                          cudaStream_t stream, int *launches) {
    if (n <= 0) return cudaSuccess;
    const int64_t n_vec = n * d / 8;
    ++*launches;
    return launch_overlapped(insert_kernel, dim3(grid_for(n_vec > n ? n_vec : n)), dim3(kThreads), 0, stream,
                             bank + first * d, emb, (int)(emb_dtype == EVK_DTYPE_BF16), n_vec, q_tables, visits, live_bits, dev,
                             capacity,
                             n_stages, first, n, stage, q_init, q_default, ids_out);
}

cudaError_t launch_tombstone(const int32_t *ids, int64_t n, int64_t size, uint32_t *live_bits, uint32_t *dev,
                             int32_t *status, cudaStream_t stream, int *launches) {
    if (n <= 0) return cudaSuccess;
    cudaError_t err = cudaMemsetAsync(dev + kDevFlag, 0, sizeof(uint32_t), stream);
    if (err != cudaSuccess) return err;
    tombstone_check_kernel<<<grid_for(n), kThreads, 0, stream>>>(ids, n, size, dev);
    *launches += 2;
    return launch_overlapped(tombstone_apply_kernel, dim3(grid_for(n)), dim3(kThreads), 0, stream, ids, n, live_bits, dev,
                             status);
}

cudaError_t launch_live_export(const uint32_t *live_bits, int64_t first, int64_t n, uint8_t *out, cudaStream_t stream,
                               int *launches) {
    if (n <= 0) return cudaSuccess;
    ++*launches;
    return launch_overlapped(live_export_kernel, dim3(grid_for(n)), dim3(kThreads), 0, stream, live_bits, first, n, out);
}

cudaError_t launch_live_import(const uint8_t *live, int64_t first, int64_t n, uint32_t *live_bits, uint32_t *dev,
                               cudaStream_t stream, int *launches) {
    if (n <= 0) return cudaSuccess;
    ++*launches;
    return launch_overlapped(live_import_kernel, dim3(grid_for(n)), dim3(kThreads), 0, stream, live, first, n, live_bits,
                             dev);
}

cudaError_t launch_convert_queries(const float *src, __nv_bfloat16 *dst, int64_t n_elems,
                                   cudaStream_t stream, int *launches) {
    if (n_elems <= 0) return cudaSuccess;
    const int64_t n_vec = n_elems / 8;
    ++*launches;
    return launch_overlapped(insert_rows_kernel, dim3(grid_for(n_vec)), dim3(kThreads), 0, stream, dst, src, 0, n_vec);
}

}  // namespace evk
