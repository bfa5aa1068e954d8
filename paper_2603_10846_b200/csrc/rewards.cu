// Rewards that feed the value update: the drafting reward (Eq. 5), the refining reward
// (Eq. 6) and its online z-score normalisation (Appendix A, "Stability of Online
// Normalization": running mean and population standard deviation, variance floor or
// output clipping, no rescaling of stored values).
#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
reward_draft_kernel(const uint8_t *__restrict__ feasible, int64_t n, float *__restrict__ out) {
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads)
        out[i] = feasible[i] ? 1.0f : -1.0f;
}

__global__ void __launch_bounds__(kThreads)
reward_refine_kernel(const float *__restrict__ best, const float *__restrict__ latency,
                     const uint8_t *__restrict__ feasible, int64_t n, float *__restrict__ out) {
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads)
        out[i] = feasible[i] ? tanhf(logf(best[i]) - logf(latency[i])) : -1.0f;
}

// state = {count, sum, sum of squares} in fp64, carried from call to call.  Reward t of this call
// is normalised with the statistics of everything before it: the state plus an exclusive
// prefix over this call's rewards, computed by a block-wide scan in chunks of 1024.
constexpr int kNormThreads = 1024;

__global__ void __launch_bounds__(kNormThreads)
reward_normalize_kernel(double *__restrict__ state, const float *__restrict__ raw, int64_t n, double sigma_min,
                        double clip, float *__restrict__ out) {
    __shared__ double warp_s1[32], warp_s2[32];
    __shared__ double carry[3];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 3) carry[tid] = state[tid];
    __syncthreads();
    for (int64_t base = 0; base < n; base += kNormThreads) {
        const int64_t i = base + tid;
        const double r = (i < n) ? (double)raw[i] : 0.0;
        double s1 = r, s2 = r * r;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double u1 = __shfl_up_sync(0xffffffffu, s1, off);
            const double u2 = __shfl_up_sync(0xffffffffu, s2, off);
            if (lane >= off) { s1 += u1; s2 += u2; }
        }
        if (lane == 31) { warp_s1[warp] = s1; warp_s2[warp] = s2; }
        __syncthreads();
        if (warp == 0) {
            double w1 = warp_s1[lane], w2 = warp_s2[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double u1 = __shfl_up_sync(0xffffffffu, w1, off);
                const double u2 = __shfl_up_sync(0xffffffffu, w2, off);
                if (lane >= off) { w1 += u1; w2 += u2; }
            }
            warp_s1[lane] = w1;
            warp_s2[lane] = w2;
        }
        __syncthreads();
        const double before1 = carry[1] + (warp ? warp_s1[warp - 1] : 0.0) + s1 - r;
        const double before2 = carry[2] + (warp ? warp_s2[warp - 1] : 0.0) + s2 - r * r;
        const double seen = carry[0] + (double)tid;
        if (i < n) {
            double v = r;
            if (seen >= 2.0) {
                const double mu = before1 / seen;
                double var = before2 / seen - mu * mu;
                if (var < 0.0) var = 0.0;
                double sigma = sqrt(var);
                if (sigma < sigma_min) sigma = sigma_min;
                v = (r - mu) / sigma;
            }
            if (clip > 0.0) v = v > clip ? clip : (v < -clip ? -clip : v);
            out[i] = (float)v;
        }
        __syncthreads();
        if (tid == kNormThreads - 1) {
            carry[0] += (double)((n - base) < kNormThreads ? (n - base) : kNormThreads);
            carry[1] = before1 + r;
            carry[2] = before2 + r * r;
        }
        __syncthreads();
    }
    if (tid < 3) state[tid] = carry[tid];
}

int grid_for(int64_t n) {
    int64_t g = (n + kThreads - 1) / kThreads;
    if (g > num_sms() * 8) g = num_sms() * 8;
    return (int)(g < 1 ? 1 : g);
}

}  // namespace

cudaError_t launch_reward_draft(const uint8_t *feasible, int64_t n, float *out, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    reward_draft_kernel<<<grid_for(n), kThreads, 0, stream>>>(feasible, n, out);
    return cudaGetLastError();
}

cudaError_t launch_reward_refine(const float *best, const float *latency, const uint8_t *feasible, int64_t n,
                                 float *out, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    reward_refine_kernel<<<grid_for(n), kThreads, 0, stream>>>(best, latency, feasible, n, out);
    return cudaGetLastError();
}

cudaError_t launch_reward_normalize(double *state, const float *raw, int64_t n, float sigma_min, float clip,
                                    float *out, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    reward_normalize_kernel<<<1, kNormThreads, 0, stream>>>(state, raw, n, (double)sigma_min, (double)clip, out);
    return cudaGetLastError();
}

}  // namespace evk
