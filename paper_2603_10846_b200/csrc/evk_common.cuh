// Shared device helpers: ranking keys, block-wide selection, launch plumbing.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "evk.h"

namespace evk {

// Streaming multiprocessors of the current device (cudaDevAttrMultiProcessorCount, asked once per
// device; 148 on a B200: 2 dies x 74).  Grids, bank splits and workspace sizes follow it, so a
// workspace must be sized and used with the same device current.  Falls back to 148 when no
// device can be asked (sizes queried on a machine without a GPU).
int num_sms();
constexpr uint32_t kPadId = 0xffffffffu;

// ---------------------------------------------------------------------------
// Ranking keys.  A candidate (sim, id) is packed into one 64-bit integer so that
// "larger key" means "ranks earlier": similarity descending, then id ascending.
// The float is mapped to an unsigned integer with the same order; the id is
// stored complemented.  Keys of distinct entries are distinct.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ordered_bits(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}
__device__ __forceinline__ uint64_t make_key(float sim, int32_t id) {
    sim += 0.0f;  // -0 -> +0: equal similarities must tie exactly
    return ((uint64_t)ordered_bits(sim) << 32) | (uint32_t)(~(uint32_t)id);
}
__device__ __forceinline__ float key_sim(uint64_t key) { return from_ordered_bits((uint32_t)(key >> 32)); }
__device__ __forceinline__ int32_t key_id(uint64_t key) { return (int32_t)(~(uint32_t)key); }

// Entries dropped from the memory: one bit per entry (1 = live) in 32-bit words.  A null pointer
// means that nothing has ever been dropped.
__device__ __forceinline__ bool entry_live(const uint32_t *live_bits, int64_t id) {
    return !live_bits || ((__ldg(live_bits + (id >> 5)) >> (id & 31)) & 1u);
}

// Per-bank words in device memory (the 256-byte block at the end of the arena).
enum DevWord { kDevStatus = 0, kDevLive = 1, kDevFiledLo = 2, kDevFiledHi = 3, kDevCutbacks = 4, kDevLongestRun = 5,
               kDevFlag = 6, kDevDropped = 7,
               // rows [0, kDevRowsReady) of the bank are in memory: published by every insert once all its
               // blocks have written theirs (kDevInsTicket counts them), read by the scan before it loads a tile
               kDevRowsReady = 8, kDevInsTicket = 9 };

// Claims one slot of a shared counter for every lane whose `want` is set, with a single atomic
// per warp.  Every lane of the warp must call it; returns the lane's slot (undefined if !want).
__device__ __forceinline__ int warp_claim_slot(bool want, int *counter) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t votes = __ballot_sync(0xffffffffu, want);
    int base = 0;
    if (votes && lane == (uint32_t)(__ffs(votes) - 1)) base = atomicAdd(counter, __popc(votes));
    base = __shfl_sync(0xffffffffu, base, votes ? (__ffs(votes) - 1) : 0);
    return base + __popc(votes & ((1u << lane) - 1u));
}

// ---------------------------------------------------------------------------
// Block-wide exact selection.  Keeps the k largest of n distinct 64-bit keys held
// in shared memory and moves them to keys[0..k) (in no particular order).
// Most-significant-digit radix select, 8 bits per pass, followed by an in-place
// compaction through registers.  Every thread of the block must call it with the
// same arguments; n <= NT * PER_THREAD; 0 < k < n.  Returns the k-th largest key.
//   hist: 256 ints of shared memory; scal: 4 uint64 of shared memory.
// ---------------------------------------------------------------------------
//   SKIP_COMMON: look first for the bits all keys agree on and skip their passes.  Pays when
//   the lists are long and similar (the merge of many lists); costs a pass otherwise.
template <int NT, int PER_THREAD, bool SKIP_COMMON = true>
__device__ uint64_t block_select_topk(uint64_t *keys, int n, int k, int *hist, uint64_t *scal) {
    const int tid = threadIdx.x;
    uint64_t prefix = 0, mask = 0;
    int kk = k;
    uint64_t common = 0, varying = ~(uint64_t)0;
    if constexpr (SKIP_COMMON) {
    // Bits on which all keys agree (sign and exponent of similarities in a narrow range, the
    // upper id bits of a small bank) need no pass: every key would fall into one bin, and the
    // shared-memory atomics on that single counter would run one after another.
    if (tid < 4) hist[tid] = (tid < 2) ? -1 : 0;  // and_lo, and_hi, or_lo, or_hi
    __syncthreads();
    {
        uint64_t all_and = ~(uint64_t)0, all_or = 0;
        for (int i = tid; i < n; i += NT) {
            all_and &= keys[i];
            all_or |= keys[i];
        }
        const uint32_t a_lo = __reduce_and_sync(0xffffffffu, (uint32_t)all_and);
        const uint32_t a_hi = __reduce_and_sync(0xffffffffu, (uint32_t)(all_and >> 32));
        const uint32_t o_lo = __reduce_or_sync(0xffffffffu, (uint32_t)all_or);
        const uint32_t o_hi = __reduce_or_sync(0xffffffffu, (uint32_t)(all_or >> 32));
        if ((tid & 31) == 0) {
            atomicAnd(&hist[0], (int)a_lo);
            atomicAnd(&hist[1], (int)a_hi);
            atomicOr(&hist[2], (int)o_lo);
            atomicOr(&hist[3], (int)o_hi);
        }
    }
    __syncthreads();
    common = ((uint64_t)(uint32_t)hist[1] << 32) | (uint32_t)hist[0];
    varying = common ^ (((uint64_t)(uint32_t)hist[3] << 32) | (uint32_t)hist[2]);
    __syncthreads();
    }
    for (int shift = 56; shift >= 0; shift -= 8) {
        if (((varying >> shift) & 0xff) == 0) {
            prefix |= common & ((uint64_t)0xff << shift);
            mask |= (uint64_t)0xff << shift;
            continue;
        }
        for (int i = tid; i < 256; i += NT) hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += NT) {
            const uint64_t key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&hist[(int)((key >> shift) & 0xff)], 1);
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns bins [8l, 8l+8); find the bin holding the kk-th largest, from the top.
            int local[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { local[j] = hist[tid * 8 + j]; sum += local[j]; }
            int incl = sum;  // becomes the total of this lane and every higher lane
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int v = __shfl_down_sync(0xffffffffu, incl, off);
                if (tid + off < 32) incl += v;
            }
            const int above = incl - sum;
            if (above < kk && kk <= above + sum) {  // exactly one lane
                int c = above, digit = tid * 8;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (kk <= c + local[j]) { digit = tid * 8 + j; break; }
                    c += local[j];
                }
                scal[0] = prefix | ((uint64_t)digit << shift);
                scal[1] = (uint64_t)(kk - c);
                scal[3] = (uint64_t)local[digit & 7];  // keys left in the chosen bin
            }
        }
        __syncthreads();
        prefix = scal[0];
        kk = (int)scal[1];
        mask |= (uint64_t)0xff << shift;
        const bool last_one = (scal[3] == 1);
        __syncthreads();
        if (last_one) {
            // a single key is left under this prefix: it is the k-th largest
            for (int i = tid; i < n; i += NT)
                if ((keys[i] & mask) == prefix) scal[0] = keys[i];
            __syncthreads();
            prefix = scal[0];
            __syncthreads();
            break;
        }
    }
    // prefix is now the k-th largest key; exactly k keys are >= prefix.
    uint64_t mine[PER_THREAD];
#pragma unroll
    for (int j = 0; j < PER_THREAD; ++j) {
        int i = tid + j * NT;
        mine[j] = (i < n) ? keys[i] : 0;
    }
    int *counter = reinterpret_cast<int *>(&scal[2]);
    if (tid == 0) *counter = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < PER_THREAD; ++j) {
        const int i = tid + j * NT;
        const bool keep = i < n && mine[j] >= prefix;
        const int slot = warp_claim_slot(keep, counter);
        if (keep) keys[slot] = mine[j];
    }
    __syncthreads();
    return prefix;
}

// Block-wide bitonic sort of n_pow2 keys in shared memory, descending.
template <int NT>
__device__ void block_sort_desc(uint64_t *keys, int n_pow2) {
    // A stage with stride <= 32 stays inside the 64 elements a warp owns, so a warp sync is
    // enough between two such stages.
    bool wide_before = true;
    for (int size = 2; size <= n_pow2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const bool wide = stride > 32;
            if (wide || wide_before) __syncthreads(); else __syncwarp();
            wide_before = wide;
            for (int t = threadIdx.x; t < (n_pow2 >> 1); t += NT) {
                int lo = 2 * t - (t & (stride - 1));
                int hi = lo + stride;
                bool desc = ((lo & size) == 0);
                uint64_t a = keys[lo], b = keys[hi];
                if ((a < b) == desc) { keys[lo] = b; keys[hi] = a; }
            }
        }
    }
    __syncthreads();
}

// Programmatic dependent launch.  A kernel launched through launch_overlapped may be scheduled
// while the kernel enqueued before it on the stream is still running; it must call pdl_wait()
// before it touches anything an earlier kernel wrote or reads anything it will overwrite.
// pdl_wait() returns once the preceding kernel has finished and its writes are visible (at
// once in an ordinary launch).  pdl_trigger() in the earlier kernel lets the next one be
// scheduled from that point on instead of at the earlier kernel's end.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__host__ __device__ __forceinline__ int next_pow2(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

}  // namespace evk
