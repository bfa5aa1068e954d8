// A read-only bandwidth calibration: how fast this GPU can stream a region of device memory into
// shared memory and drop it, with the copy engine the scan uses and nothing else in the way.  The
// measured copy bandwidth (read + write) is not the ceiling of a kernel that only reads; this is.
// One block per SM, one thread issuing 32 KB bulk copies into a ring of four stages, one thread
// consuming them.  Every wait is bounded.
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kChunkBytes = 32768;
constexpr int kProbeStages = 4;
constexpr long long kProbeTimeout = 2000000000LL;

__device__ __forceinline__ uint32_t probe_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool probe_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool probe_wait(uint32_t bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!probe_try_wait(bar, parity))
        if (clock64() - t0 > kProbeTimeout) return false;
    return true;
}

__global__ void __launch_bounds__(64)
read_probe_kernel(const unsigned char *__restrict__ src, size_t n_chunks, int32_t *__restrict__ status) {
    extern __shared__ __align__(128) unsigned char probe_smem[];
    __shared__ uint64_t full[kProbeStages], empty[kProbeStages];
    __shared__ int bad;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kProbeStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(probe_smem_u32(&full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(probe_smem_u32(&empty[s])));
        }
        bad = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t stage = 0, phase = 0;
        for (size_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
            if (!probe_wait(probe_smem_u32(&empty[stage]), phase ^ 1)) { bad = 1; break; }
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(probe_smem_u32(&full[stage])), "r"(kChunkBytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(probe_smem_u32(probe_smem + (size_t)stage * kChunkBytes)), "l"(src + c * kChunkBytes),
                           "r"(kChunkBytes), "r"(probe_smem_u32(&full[stage])) : "memory");
            if (++stage == kProbeStages) { stage = 0; phase ^= 1; }
        }
    } else if (threadIdx.x == 32) {
        uint32_t stage = 0, phase = 0;
        unsigned acc = 0;
        for (size_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
            if (!probe_wait(probe_smem_u32(&full[stage]), phase)) { bad = 1; break; }
            acc ^= *reinterpret_cast<volatile unsigned *>(probe_smem + (size_t)stage * kChunkBytes);
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(probe_smem_u32(&empty[stage])) : "memory");
            if (++stage == kProbeStages) { stage = 0; phase ^= 1; }
        }
        if (acc == 0x9e3779b9u && status) atomicCAS(status, 0, 0);   // keeps the reads alive
    }
    __syncthreads();
    // a copy that was issued has landed or its wait ran out; either way no further copy is in flight
    // once the consumer has seen (or given up on) the last armed stage
    if (threadIdx.x == 0 && bad && status) atomicCAS(status, 0, (int)EVK_ERR_DEVICE_TIMEOUT);
}

}  // namespace

cudaError_t launch_read_probe(const void *src, size_t bytes, int32_t *status, cudaStream_t stream) {
    const size_t n_chunks = bytes / kChunkBytes;
    if (n_chunks == 0) return cudaSuccess;
    const size_t smem = (size_t)kProbeStages * kChunkBytes;
    cudaError_t e = cudaFuncSetAttribute(read_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int grid = num_sms();
    if ((size_t)grid > n_chunks) grid = (int)n_chunks;
    read_probe_kernel<<<grid, 64, smem, stream>>>(static_cast<const unsigned char *>(src), n_chunks, status);
    return cudaGetLastError();
}

}  // namespace evk
