// Phase 1 on the tensor cores: similarity of a tile of 128 queries against the
// whole bank as a bf16 GEMM with fp32 accumulation (tcgen05.mma, accumulators in
// tensor memory), with the top-k1 selection fused into the epilogue so that the
// B x N similarity matrix of Section 3.2's dense retrieval is never written out.
//
// Layout of one thread block (224 threads, one block per SM, persistent):
//   warp 0     TMA producer: streams 64-column slices of a bank tile (B operand, 256
//              rows) into a shared-memory ring of up to four stages, 128-byte swizzled,
//              K-major (a last slice that reaches beyond the row width is zero-filled).
//              The query tile (A operand) is loaded once and stays in shared memory when
//              the batch is small enough (<= 64 queries of width 1024); otherwise its
//              slices travel through the ring next to the bank's.  Small batches must
//              not re-read the queries per bank tile: every block would ask L2 for
//              the same few lines at the same moment.
//   warp 1     MMA issuer: one thread issues tcgen05.mma 128x256x16 (64x256x16 when at most
//              64 queries are resident) per 16 columns of a slice, accumulating
//              D[query][bank row] in one of two 256-column tensor-memory buffers;
//              tcgen05.commit hands smem stages back to the producer and finished
//              accumulators to the epilogue.
//   warps 2-5  epilogue: a thread owns one query of the tile (its TMEM lane).  It reads
//              its 256 similarities of a bank tile a chunk at a time, compares them with
//              the query's running threshold held in a register, and appends the few
//              survivors to the query's private candidate list in global memory.
//              When a list fills, the warp cuts it back to its best k1 with an exact
//              radix select over registers and the threshold rises.
//   warp 6     threshold tracker (scans of two or more query tiles): re-reads the shared
//              histograms of the block's queries on a thinning schedule and posts each
//              query's current bin threshold in shared memory, so that the epilogue threads
//              do not wait on global memory between tiles.
//
// With two or more query tiles, blocks run in clusters of two (cta_group::2): a pair shares
// one 256-query x 256-row tile, each block loading its own queries and half of the bank slice.
//
// Up to 32 queries take the same pipeline with the operands' roles swapped (see kSwapN): the bank
// rows sit on the accumulator's lanes (M = 128) and the queries on its columns, padded to 16 or 32
// instead of to 64; a thread of the epilogue then owns a bank row, and what belongs to a query lives
// in shared memory (swap_epilogue).  The scan is bound by HBM in either layout; the swapped one
// spends a quarter to a half of the tensor work, which under the board's power cap is SM clock.
//
// A bank tile is 256 consecutive entries; the queries sit on the accumulator's
// lanes so that the per-query threshold test costs one register compare and no
// cross-thread traffic.  The work of a launch is a grid of jobs (query tile,
// bank split); the bank tiles of a split are interleaved (t = split, split+S, ...)
// so that blocks working on different query tiles touch the same bank tile at about
// the same time and share it through L2.
//
// The same kernel has a "dense" mode that writes every similarity of a small,
// strided sample of the bank; a value that at least k1 of a query's sampled similarities
// reach is a safe starting threshold for the full scan (at least k1 entries of the bank
// reach it).
//
// During the full scan the blocks tighten the thresholds together.  Each query has a
// small histogram in global memory over the similarity range above its starting
// threshold; every survivor is counted in it, and a threshold is raised to the highest bin
// edge that was seen with k1 survivors at or above it.  With one query tile the scan runs
// at HBM speed and each epilogue thread reads its query's counters before each of the first tiles and then
// before every fourth; with
// more, the tensor cores set the pace, the thread reads them itself only for the first
// tiles of a job and the tracker warp takes over.  Counters only grow, so whatever mix of
// old and new values a reader sees undercounts, and a threshold derived from it still has
// at least k1 real entries above it: the selection stays exact while the survivor rate
// falls from k1/sample to about k1/(rows scanned so far by all blocks).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the block's
// abort flag, every role leaves its loop, the producer waits (bounded again) for the
// copies it still has in flight, tensor memory is released and the status word
// reports EVK_ERR_DEVICE_TIMEOUT.
#include <cuda.h>

#include "evk_common.cuh"
#include "evk_kernels.cuh"

namespace evk {

namespace {

constexpr int kBlockM = 128;
constexpr int kBlockN = 256;
constexpr int kBlockK = 64;
constexpr int kUmmaK = 16;
constexpr int kMaxStages = 6;
constexpr int kResidentStages = 4;                   // ring depth used (more fit, fewer are slower)
constexpr int kThreads = 224;
constexpr uint32_t kABytes = kBlockM * kBlockK * 2;  // 16 KB: a streamed slice of the query tile
constexpr uint32_t kBBytes = kBlockN * kBlockK * 2;  // 32 KB: a slice of a bank tile
constexpr uint32_t kTmemCols = 512;                  // two accumulators of 256 fp32 columns
constexpr size_t kSmemMax = 232448;                  // 227 KB of dynamic shared memory per block
constexpr size_t kSmemFixed = 1024 + 256 + 1536;     // alignment slack + barriers + tracker mailboxes
constexpr int kHistBins = 64;
constexpr int kChunk = 32;                           // accumulator columns per tensor-memory load (pick() assumes 32)
// Self-starting histogram (scans of one query tile).  A similarity's bin is the top 13 bits of its
// order-preserving bit pattern (sign, exponent, four mantissa bits: sixteen bins to the octave), so
// every block bins alike without having seen any data; a query's 64 counters cover the window of
// bins that the first block to look at its first kBootCols rows anchors two octaves above those rows'
// largest similarity (128 rows may miss the few entries that are much closer to the query than
// the rest, as in a clustered bank).  Values above the window count in its top bin, values below it in bin 0, which never
// serves as a threshold: a counter can only under-state how many entries reach its bin's edge.
constexpr int kAbsShift = 19;
constexpr int kAbsBins = 1 << (32 - kAbsShift);
constexpr int kAbsHeadroom = 32;                     // bins between the anchoring maximum and the window's top
constexpr int kBootCols = 128;                       // rows of a job's first tile that anchor the window and are counted
constexpr int kBootBin = kHistBins - 1 - kAbsHeadroom - 16;   // ... from this window bin up (half the anchoring maximum)
                                                     // before any entry is filed
constexpr int kReadEvery = 4;                        // scans without a tracker: tiles between two looks at the counters
constexpr int kSyncTiles = 4;                        // tiles of a job whose threshold the epilogue reads itself
constexpr int kSyncAlways = 1 << 28;                 // ... or every tile: the tracker stays idle
constexpr long long kTimeoutCycles = 4000000000LL;   // about two seconds

// tcgen05 instruction descriptor, kind::f16: D=f32, A=B=bf16, both K-major, N=256, M=128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                                ((uint32_t)(kBlockM >> 4) << 24);

struct MmaParams {
    int64_t size;       // valid bank rows (filter mode) or sample rows (dense mode)
    int B, d, k1;
    int n_qt, splits, n_tiles;
    int mode;           // 0 = filter, 1 = dense
    int a_resident;     // 1: the query tile is loaded once (n_qt == 1), 0: streamed with the bank
    int a_rows;         // rows of the query TMA box (multiple of 8)
    int n_stages;       // depth of the shared-memory ring
    const float *tau0;  // [B] starting thresholds, or nullptr
    const float2 *range;  // [B] (lowest counted similarity, bins per unit) of the shared histogram
    unsigned *hist;       // [B][kHistBins] survivors counted by similarity bin
    uint64_t *cand;     // [n_qt*splits][128][kMmaCandCap]
    int *cand_cnt;      // [n_qt*splits][128]
    float *dense;       // [B][dense_ld]
    int dense_ld;
    int32_t *status;
    int sync_tiles;     // kSyncTiles, or kSyncAlways when the scan is bound by HBM and the epilogue has time
    int m64;            // 1 (single block, at most 64 resident queries): M = 64 instructions, half the tensor work
    int stall;          // test aid: the producer of the full scan issues no loads, so a bounded wait runs out
    int b3d;            // 1: bank stages are kSubRows rows x kSubSlices slices (contiguous bytes per row), see make_map3
    int abs_hist;       // 1: no sampled thresholds; the shared histogram bins by the similarity's own bits (see kAbsShift)
    int *anchor;        // [B] abs_hist: lowest bin of each query's histogram window + 1, 0 until the first block sets it
    const uint32_t *live_bits;   // entries dropped from the memory are skipped (null: none ever was)
    uint32_t *dev;      // the bank's device words: candidates filed and list cut-backs are counted there (or null)
    int wait_queries;   // the queries come out of the library's conversion kernel: wait for it before loading them
};

// ---- PTX wrappers -----------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false means the block is aborting.
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
    return true;
}

// Bounded wait that ignores the abort flag (used once the block is already backing out).
__device__ __forceinline__ bool mbar_wait_deadline(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// The same load with an L2 eviction-priority hint (see l2_evict_first_policy).
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
// A box of a three-dimensional map {64 columns, rows, 64-column slices}: `rows` x `slices` pieces of
// 128 bytes, laid down slice by slice as K-major tiles.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int row, int slice) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(row), "r"(slice)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int row, int slice,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(row), "r"(slice), "l"(policy)
        : "memory");
}
// "Evict this first": for data that is read once, so that it does not push out lines that are
// read again and again (the queries, the histograms, the candidate lists).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// M = 64: accumulator row i lands on lane 32 * (i / 16) + i % 16, sixteen rows per lane quarter.
constexpr uint32_t kInstrDescM64 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                                   ((uint32_t)(64 >> 4) << 24);

// The contiguous stage layout (resident queries): a stage holds kSubRows bank rows x kSubSlices slices,
// i.e. 256 contiguous bytes of each row, and feeds N = kSubRows instructions.  Measured over 2 GiB at
// 1 / 32 / 64 queries: 0.307 / 0.311 / 0.326 ms against 0.314 / 0.317 / 0.330 for 256 rows x 1 slice.
// 64 rows x 4 slices load faster still (7.3 TB/s) but need four times the instructions, and one
// tcgen05.mma into an accumulator that the previous one wrote takes ~110 cycles whatever its N: 0.417 ms.
constexpr int kSubRows = 128;
constexpr int kSubSlices = 2;
constexpr uint32_t kInstrDescSub = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kSubRows >> 3) << 17) |
                                   ((uint32_t)(kBlockM >> 4) << 24);
constexpr uint32_t kInstrDescSubM64 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kSubRows >> 3) << 17) |
                                      ((uint32_t)(64 >> 4) << 24);

// Swapped roles for up to kSwapMax queries: the bank rows are the M side (128 of them per instruction, one
// per accumulator lane), the queries the N side, padded to a multiple of kSwapN instead of to 64: as
// little as a quarter of the tensor work per bank row.  The scan is bound by HBM either way; under the power cap the tensor cores'
// share of the board's power is what sets the clock, and padding rows cost as much as real ones.
constexpr int kSwapN = 16;                           // queries per chunk of the epilogue, granularity of N
#ifndef EVK_SWAP_MAX
#define EVK_SWAP_MAX 32
#endif
constexpr int kSwapMax = EVK_SWAP_MAX;               // most queries this layout takes
__host__ __device__ constexpr int swap_n(int B) { return ((B + kSwapN - 1) / kSwapN) * kSwapN; }
__device__ __forceinline__ uint32_t instr_desc_swap(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kSubRows >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate,
                                          uint32_t idesc) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- two SMs on one tile (cta_group::2) ----------------------------------------------------
// A cluster of two blocks shares one 256-query x 256-row tile: each block holds its own 128
// queries (A) and HALF of the bank slice (B), the leader block issues one M=256 instruction
// that reads both halves, and each block's tensor memory receives the accumulator rows of its
// own queries.  Per block and slice 16 KB of B travel instead of 32 KB.
constexpr uint32_t kInstrDescPair = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                                    ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this block's shared memory whose bytes are counted on a barrier of the pair's leader
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int x, int y,
                                                      uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(kInstrDescPair), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at this offset in BOTH blocks of the pair once the MMAs issued so far finished.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// kChunk consecutive fp32 columns of this thread's TMEM lane: the load is asynchronous, the
// registers hold the data only after tmem_ld_wait on the same array (which waits for every
// outstanding tcgen05.ld of the thread; the registers are named as in/out operands so that no
// use of them can be scheduled ahead of the wait).
__device__ __forceinline__ void tmem_ld_issue(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
        :
        : "memory");
}

// Sixteen columns (the swapped layout: one column per query).
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16_wait(uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
        :
        : "memory");
}

// v[j] for a run-time j without spilling the array: a select tree, one level per bit of j.
__device__ __forceinline__ uint32_t pick(const uint32_t (&v)[32], int j) {
    const bool b0 = j & 1, b1 = j & 2, b2 = j & 4, b3 = j & 8, b4 = j & 16;
    uint32_t a[16], b[8], c[4];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = b0 ? v[2 * i + 1] : v[2 * i];
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = b1 ? a[2 * i + 1] : a[2 * i];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = b2 ? b[2 * i + 1] : b[2 * i];
    const uint32_t d0 = b3 ? c[1] : c[0], d1 = b3 ? c[3] : c[2];
    return b4 ? d1 : d0;
}

// Highest bin of a query's shared histogram with k1 counted survivors at or above it (0 when
// there is none yet).  All sixteen loads are issued before the first is looked at.
__device__ __forceinline__ int hist_best_bin(const unsigned *hist, int k1) {
    uint4 c[kHistBins / 4];
#pragma unroll
    for (int g = 0; g < kHistBins / 4; ++g) c[g] = __ldcg(reinterpret_cast<const uint4 *>(hist) + g);
    int acc_cnt = 0, best = 0;
    bool found = false;
#pragma unroll
    for (int g = kHistBins / 4 - 1; g >= 0; --g) {
        const unsigned cs[4] = {c[g].x, c[g].y, c[g].z, c[g].w};
#pragma unroll
        for (int e = 3; e >= 0; --e) {
            acc_cnt += (int)cs[e];
            if (!found && acc_cnt >= k1) {
                found = true;
                best = g * 4 + e;
            }
        }
    }
    return best;
}

// ---- warp-wide exact selection over one candidate list ------------------------
// The whole warp cuts the list `buf` (n <= kMmaCandCap distinct non-zero keys) back to
// its k largest and returns the k-th largest key.  Keys live in registers (32 per
// lane); the k-th largest is found 4 bits at a time from the top.
__device__ __noinline__ uint64_t warp_select_topk(uint64_t *buf, int n, int k) {
    const int lane = threadIdx.x & 31;
    constexpr int kPerLane = kMmaCandCap / 32;
    uint64_t r[kPerLane];
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        const int i = j * 32 + lane;
        r[j] = (i < n) ? buf[i] : 0;
    }
    uint64_t prefix = 0, mask = 0;
    int kk = k;
#pragma unroll 1
    for (int shift = 60; shift >= 0; shift -= 4) {
        // per-lane counts of the 16 digit values, 8 bits each (a lane holds at most 32 keys)
        uint64_t c_lo = 0, c_hi = 0;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            if ((r[j] & mask) == prefix && r[j] != 0) {
                const int dgt = (int)((r[j] >> shift) & 15);
                if (dgt < 8) c_lo += (uint64_t)1 << (8 * dgt);
                else c_hi += (uint64_t)1 << (8 * (dgt - 8));
            }
        }
        int acc = 0, digit = 0;
        bool found = false;
#pragma unroll
        for (int b = 15; b >= 0; --b) {
            const uint32_t mine = (uint32_t)(((b < 8) ? (c_lo >> (8 * b)) : (c_hi >> (8 * (b - 8)))) & 0xff);
            const int cnt = (int)__reduce_add_sync(0xffffffffu, mine);
            if (!found) {
                if (kk <= acc + cnt) {
                    digit = b;
                    found = true;
                } else {
                    acc += cnt;
                }
            }
        }
        kk -= acc;
        prefix |= (uint64_t)digit << shift;
        mask |= (uint64_t)15 << shift;
    }
    // prefix is the k-th largest key; exactly k keys are >= prefix.  Compact in place.
    int keep = 0;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) keep += (r[j] >= prefix && r[j] != 0);
    int start = keep;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, start, off);
        if (lane >= off) start += v;
    }
    start -= keep;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < kPerLane; ++j)
        if (r[j] >= prefix && r[j] != 0) buf[start++] = r[j];
    __syncwarp();
    return prefix;
}

// ---- the kernel ---------------------------------------------------------------

// kPair: clusters of two blocks on 256-query tiles.  kMode: 0 filter (the scan proper), 1 dense (every
// similarity of a small sample is written out).  kAbs: thresholds started off by the scan itself
// (scans of one query tile) instead of sampled ones.  Three shapes are built: <false, 0, true>,
// <true, 0, false> and <false, 1, false>; each carries only its own code (the epilogue's speed
// depends on how much code it has to run through).
// ---- epilogue of the swapped layout (up to kSwapN queries) ---------------------------------------
// A thread owns one bank row of each 128-row group (its accumulator lane) and holds that row's
// similarity to every query in registers; what is per query lives in shared memory, shared by the four
// epilogue warps: list length, thresholds, histogram window.  Query j is looked after by warp j % 4
// (threshold reads, cut-backs).  The warps meet at a named barrier between the phases of a tile; every
// branch around such a barrier is taken by all four alike (a failed wait is published through a flag
// that all read behind the next barrier, see `fail`).
struct SwapState {
    int cnt[kSwapMax];            // candidates in the job's list of query j (at a job's start: the first rows'
                                  // largest similarity as ordered bits, until the window is anchored)
    int tau_bin[kSwapMax];        // bin threshold from the shared histogram
    float tau_sim[kSwapMax];      // cheap first test: no larger than either exact threshold
    uint64_t tau_key[kSwapMax];   // exact key threshold (rises when the list is cut back)
    int a_base[kSwapMax];         // lowest absolute bin of the window, -1 until anchored
};
static_assert(sizeof(SwapState) <= 1536, "lives in the tracker's mailboxes, which this layout leaves unused");

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Highest bin of a histogram with k1 counted entries at or above it (0: none yet), from the 64 counters
// held two per lane.
__device__ __forceinline__ int warp_best_bin(uint2 c, int k1, int lane) {
    int own = (int)(c.x + c.y), incl = own;   // incl: this lane's counters and all higher ones
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += v;
    }
    const int above = incl - own;
    const bool here = above < k1 && k1 <= incl;
    const unsigned who = __ballot_sync(0xffffffffu, here);
    if (!who) return 0;
    const int src = __ffs(who) - 1;
    const int bin = (above + (int)c.y >= k1) ? 2 * lane + 1 : 2 * lane;
    return __shfl_sync(0xffffffffu, bin, src);
}

// Returns false when a wait ran out (the block then backs out like the other layouts).
// fail[2]: a wait ran out in a round of this parity.
__device__ __forceinline__ bool swap_epilogue(const MmaParams &p, SwapState *st, volatile int *fail, uint32_t tmem_base,
                                              uint32_t tfull0, uint32_t tempty0, volatile int *abort_flag,
                                              long long wait_limit, int warp, int lane, int worker, int n_jobs,
                                              int n_workers) {
    const int quarter = warp & 3;            // this warp's tensor-memory lanes: 32 * quarter ...
    const int tid128 = quarter * 32 + lane;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int n_pad = p.a_rows;              // accumulator columns per row group
    const int n_chunks = n_pad / kSwapN;
    uint32_t acc = 0, acc_phase = 0;
    int round = 0;
    bool ok = true;
    if (tid128 == 0) fail[0] = fail[1] = 0;
    for (int job = worker; job < n_jobs && ok; job += n_workers) {
        const int split = job % p.splits;    // one query tile: the job is the bank split
        if (tid128 < kSwapMax) {
            st->cnt[tid128] = 0;
            st->tau_bin[tid128] = 0;
            st->tau_sim[tid128] = -INFINITY;
            st->tau_key[tid128] = 0;
            st->a_base[tid128] = -1;
        }
        epi_bar();
        int n_done = 0;
        for (int t = split; t < p.n_tiles; t += p.splits, ++n_done) {
            if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag, wait_limit)) fail[round & 1] = 1;
            epi_bar();
            if (fail[round & 1]) { ok = false; break; }
            ++round;
            tc_fence_after();
            // this thread's row of group 0 and of group 1 against sixteen queries at a time
            uint32_t v0[kSwapN], v1[kSwapN];
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBlockN;
            const int64_t row_a = (int64_t)t * kBlockN + tid128, row_b = row_a + kSubRows;
            const bool live_a = row_a < p.size && entry_live(p.live_bits, row_a);
            const bool live_b = row_b < p.size && entry_live(p.live_bits, row_b);
            int skip_from = kHistBins;
            int64_t counted_end = 0;
            if (n_done == 0) {
                // The job's first 128 rows start the histogram off: their largest similarity anchors each
                // query's window (whoever comes first), and those of them from window bin kBootBin up are
                // counted before anything is filed (see the other layout's epilogue).
#pragma unroll 1
                for (int c = 0; c < n_chunks; ++c) {
                    tmem_ld16_issue(t_addr + c * kSwapN, v0);
                    tmem_ld16_wait(v0);
#pragma unroll
                    for (int j = 0; j < kSwapN; ++j) {
                        const int q = c * kSwapN + j;
                        if (q < p.B) {
                            const float x = __uint_as_float(v0[j]);
                            const unsigned ob = (row_a < p.size && fabsf(x) <= 3.0e38f) ? ordered_bits(x + 0.0f) : 0u;
                            const unsigned wm = __reduce_max_sync(0xffffffffu, ob);
                            if (lane == 0 && wm) atomicMax(reinterpret_cast<unsigned *>(&st->cnt[q]), wm);
                        }
                    }
                }
                epi_bar();
                {
                    // one lane per query of this warp's share (quarter, quarter + 4, ...)
                    const int q = quarter + 4 * lane;
                    if (q < p.B) {
                        const unsigned mx = (unsigned)st->cnt[q];
                        int enc = __ldcg(p.anchor + q);
                        if (enc == 0 && mx != 0) {
                            int prop = (int)(mx >> kAbsShift) + kAbsHeadroom - (kHistBins - 1);
                            prop = prop < 0 ? 0 : (prop > kAbsBins - kHistBins ? kAbsBins - kHistBins : prop);
                            const int got = atomicCAS(p.anchor + q, 0, prop + 1);
                            enc = got ? got : prop + 1;
                        }
                        if (enc != 0) st->a_base[q] = enc - 1;
                    }
                }
                epi_bar();
                if (tid128 < kSwapMax) st->cnt[tid128] = 0;   // from here on: the lists' lengths
#pragma unroll 1
                for (int c = 0; c < n_chunks; ++c) {
                    tmem_ld16_issue(t_addr + c * kSwapN, v0);
                    tmem_ld16_wait(v0);
#pragma unroll
                    for (int j = 0; j < kSwapN; ++j) {
                        const int q = c * kSwapN + j;
                        if (q < p.B) {
                            const int ab = st->a_base[q];
                            const float x = __uint_as_float(v0[j]);
                            if (ab >= 0 && live_a && x >= from_ordered_bits((uint32_t)(ab + kBootBin) << kAbsShift)) {
                                int bin = (int)(ordered_bits(x + 0.0f) >> kAbsShift) - ab;
                                bin = bin > kHistBins - 1 ? kHistBins - 1 : bin;
                                atomicAdd(p.hist + (size_t)q * kHistBins + bin, 1u);
                            }
                        }
                    }
                }
                skip_from = kBootBin;
                counted_end = (int64_t)t * kBlockN + kBootCols;
                epi_bar();
            }
            // the thresholds: read before each of the first tiles, then before every kReadEvery-th
            if (n_done < kReadEvery || n_done % kReadEvery == 0) {
                // this warp's queries (quarter, quarter + 4, ...): all their counters are asked for before the
                // first answer is looked at, one trip to L2 instead of one per query
                uint2 ctr[kSwapMax / 4];
#pragma unroll
                for (int i = 0; i < kSwapMax / 4; ++i) {
                    const int q = quarter + 4 * i;
                    ctr[i] = (q < p.B) ? __ldcg(reinterpret_cast<const uint2 *>(p.hist + (size_t)q * kHistBins) + lane)
                                       : make_uint2(0u, 0u);
                }
#pragma unroll
                for (int i = 0; i < kSwapMax / 4; ++i) {
                    const int q = quarter + 4 * i;
                    if (q < p.B) {
                        const int ab = st->a_base[q];
                        if (ab >= 0) {
                            const int best = warp_best_bin(ctr[i], p.k1, lane);
                            if (lane == 0 && best > st->tau_bin[q]) {
                                st->tau_bin[q] = best;
                                st->tau_sim[q] = fmaxf(key_sim(st->tau_key[q]), from_ordered_bits((uint32_t)(ab + best) << kAbsShift));
                            }
                        }
                    }
                }
                epi_bar();
            }
            // file what passes: one ballot per query and row group, the list's slots claimed per warp
            auto file_one = [&](uint32_t bits, int64_t row, bool live, int q, float cheap) {
                const float sv = __uint_as_float(bits);
                bool pass = live && sv >= cheap;
                // (nearly every ballot of the cheap test comes back empty)
                if (!__any_sync(0xffffffffu, pass)) return;
                uint64_t key = 0;
                int bin = 0;
                const int ab = st->a_base[q];
                if (pass) {
                    key = make_key(sv, (int32_t)row);
                    if (ab >= 0) {
                        bin = (int)(ordered_bits(sv + 0.0f) >> kAbsShift) - ab;
                        bin = bin < 0 ? 0 : (bin > kHistBins - 1 ? kHistBins - 1 : bin);
                    }
                    pass = key > st->tau_key[q] && bin >= st->tau_bin[q];
                }
                const unsigned m = __ballot_sync(0xffffffffu, pass);
                if (m) {
                    const int first = __ffs(m) - 1;
                    int base = 0;
                    if (lane == first) base = atomicAdd(&st->cnt[q], __popc(m));
                    base = __shfl_sync(0xffffffffu, base, first);
                    if (pass) {
                        p.cand[((size_t)split * kBlockM + q) * kMmaCandCap + base + __popc(m & lt_mask)] = key;
                        // (entries of the counted first rows from kBootBin up are in the counters already)
                        if (ab >= 0 && (bin < skip_from || row >= counted_end))
                            atomicAdd(p.hist + (size_t)q * kHistBins + bin, 1u);
                    }
                }
            };
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c) {
                tmem_ld16_issue(t_addr + c * kSwapN, v0);
                tmem_ld16_issue(t_addr + n_pad + c * kSwapN, v1);
                tmem_ld16_wait(v0);
                tmem_ld16_wait(v1);
                if (c == n_chunks - 1) {
                    // the whole accumulator has been read: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
                }
                // the chunk's sixteen cheap thresholds in one trip to shared memory
                float cheap[kSwapN];
#pragma unroll
                for (int j4 = 0; j4 < kSwapN / 4; ++j4) {
                    const float4 f = *reinterpret_cast<const float4 *>(&st->tau_sim[c * kSwapN + 4 * j4]);
                    cheap[4 * j4] = f.x; cheap[4 * j4 + 1] = f.y; cheap[4 * j4 + 2] = f.z; cheap[4 * j4 + 3] = f.w;
                }
#pragma unroll
                for (int j = 0; j < kSwapN; ++j) {
                    const int q = c * kSwapN + j;
                    if (q < p.B) {
                        file_one(v0[j], row_a, live_a, q, cheap[j]);
                        file_one(v1[j], row_b, live_b, q, cheap[j]);
                    }
                }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            // a list that the next tile could overflow (256 rows may all pass) is cut back to its best k1
            epi_bar();
            for (int q = quarter; q < p.B; q += 4) {
                const int n = st->cnt[q];
                if (n > kMmaCandCap - kBlockN) {
                    const uint64_t kth = warp_select_topk(p.cand + ((size_t)split * kBlockM + q) * kMmaCandCap, n, p.k1);
                    if (lane == 0) {
                        if (p.dev) atomicAdd(p.dev + kDevCutbacks, 1u);
                        st->cnt[q] = p.k1;
                        st->tau_key[q] = kth;
                        st->tau_sim[q] = fmaxf(st->tau_sim[q], key_sim(kth));
                    }
                }
            }
            epi_bar();
        }
        epi_bar();
        if (tid128 < p.B) p.cand_cnt[(size_t)split * kBlockM + tid128] = ok ? st->cnt[tid128] : 0;
        if (p.dev && ok && tid128 == 0) {
            unsigned long long left = 0;
            for (int j = 0; j < p.B; ++j) left += (unsigned long long)st->cnt[j];
            if (left) atomicAdd(reinterpret_cast<unsigned long long *>(p.dev + kDevFiledLo), left);
        }
        epi_bar();
    }
    if (!ok) {
        // backing out: whatever this block was to deliver counts as empty, so the merge reads nothing stale
        for (int job = worker; job < n_jobs; job += n_workers)
            if (tid128 < p.B) p.cand_cnt[(size_t)(job % p.splits) * kBlockM + tid128] = 0;
    }
    return ok;
}

template <bool kPair, int kMode, bool kAbs, bool kSwap = false>
__global__ void __launch_bounds__(kThreads, 1)
score_mma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_bank,
                 const MmaParams p) {
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzled tiles
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    unsigned char *tiles_ptr = smem_raw + (tiles - raw);
    // kPair: blocks come in clusters of two; `rank` is the block's place in its pair, a "worker" is
    // a pair.  Otherwise every block is a worker of its own.
    const uint32_t rank = kPair ? cluster_ctarank() : 0u;
    const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int n_jobs = (kPair ? (p.n_qt + 1) / 2 : p.n_qt) * p.splits;
    // a width that is no multiple of 64 ends in a partial slice: TMA fills the columns beyond d with
    // zeros, which add nothing to a similarity
    const int k_chunks = (p.d + kBlockK - 1) / kBlockK;
    // ring stages per bank tile: one per slice, or (contiguous layout) one per (row group, slice group)
    const int n_sg = (k_chunks + kSubSlices - 1) / kSubSlices;
    const int n_sub = (!kPair && p.b3d) ? (kBlockN / kSubRows) * n_sg : k_chunks;
    // [resident query tile: k_chunks slices of a_rows x 128 B] [ring of n_stages stages] [barriers]
    const uint32_t a_slice = (uint32_t)p.a_rows * 128u;
    const uint32_t a_region = p.a_resident ? (uint32_t)k_chunks * a_slice : 0u;
    const uint32_t b_bytes = kPair ? kBBytes / 2 : kBBytes;   // this block's share of a bank slice
    const uint32_t stage_bytes = p.a_resident ? b_bytes : (kABytes + b_bytes);
    const uint32_t b_off = p.a_resident ? 0u : kABytes;   // the bank slice inside a stage
    const uint32_t ring = tiles + a_region;
    const int kStages = p.n_stages;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tiles_ptr + a_region + (size_t)kStages * stage_bytes);
    // bars[0..6) full, [6..12) empty, [12..14) tmem_full, [14..16) tmem_empty, [16] queries resident
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 5);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    // tracker mailboxes, one per epilogue thread: the query it serves now (-1: none) going in,
    // (query << 32 | bin threshold) coming back; epi_done counts epilogue warps that have finished
    volatile int *epi_done = reinterpret_cast<volatile int *>(tmem_slot + 2);
    volatile int *tile_seq = reinterpret_cast<volatile int *>(tmem_slot + 3);   // accumulators examined so far
    // written by the partner block of a pair at teardown: slices its producer issued, its abort flag
    volatile int *peer_issued = reinterpret_cast<volatile int *>(tmem_slot + 4);
    volatile int *peer_abort = reinterpret_cast<volatile int *>(tmem_slot + 5);
    volatile int *slot_q = reinterpret_cast<volatile int *>(reinterpret_cast<unsigned char *>(bars) + 256);
    volatile unsigned long long *slot_tau =
        reinterpret_cast<volatile unsigned long long *>(reinterpret_cast<unsigned char *>(bars) + 256 + 512);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool abs_mode = kAbs;
    const long long wait_limit = p.stall ? kTimeoutCycles / 16 : kTimeoutCycles;
    pdl_trigger();
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kMaxStages;
    const uint32_t tfull0 = empty0 + 8 * kMaxStages, tempty0 = tfull0 + 16, afull = tempty0 + 16;

    if (threadIdx.x == 0) {
        mbar_init(afull, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull0 + 8 * b, 1);
            mbar_init(tempty0 + 8 * b, kPair ? 8 : 4);  // one arrival per epilogue warp of every block on the tile
        }
        *abort_flag = 0;
        *epi_done = 0;
        *tile_seq = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x >= 64 && threadIdx.x < 64 + kBlockM) {
        slot_q[threadIdx.x - 64] = -1;
        slot_tau[threadIdx.x - 64] = ~0ull;
    }
    if (warp == 0) {
        __syncwarp();
        if (kPair) {
            tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(tmem_slot), kTmemCols);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (kPair) cluster_sync_all();  // the partner's barriers exist before anything is signalled across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // the producer's record of what it has put in flight (thread 0 only), for the teardown
    int n_issued = 0;        // ring slices armed and issued so far
    bool a_armed = false;    // the resident query tile was requested

    if (warp == 0) {
        // ===== TMA producer =====
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = !(p.stall && kMode == 0);
            // one query tile (or one pair of them): every bank tile is read exactly once.  With more,
            // the blocks that share a tile read it within a few tiles of one another, and the hint
            // would let it go in between (4,096 queries over 6 GiB: 22.7 against 19.5 ms).
            const bool stream_once = kMode == 0 && (kPair ? p.n_qt <= 2 : p.n_qt == 1);
            const uint64_t bank_policy = l2_evict_first_policy();
            // This kernel may have been started while the kernels before it still run: their blocks have said
            // that dependents may be scheduled, not that they are done, and the same holds for the kernels
            // before those.  Rows appended by an insert - even two calls ago - may not be in memory yet (seen on
            // a bank of one tile: a third of 400 rounds of insert -> retrieve returned stale rows).  So a tile is
            // loaded only once the bank's rows-ready word, which every insert publishes behind its last row,
            // covers it: nearly all tiles at once (the scan streams while the merge, the update and the insert
            // before it finish), the last one when that insert is done.  Without the word, and for queries that
            // the library's own conversion kernel writes, no load is issued before griddepcontrol.wait.
            if (p.wait_queries || !p.dev) pdl_wait();
            int64_t rows_ready = p.dev ? (int64_t)ld_acquire_u32(p.dev + kDevRowsReady) : p.size;
            // (the rows were written with ordinary stores and are read by bulk tensor copies: order the two proxies)
            asm volatile("fence.proxy.async.global;" ::: "memory");
            if (kMode == 1) rows_ready = INT64_MAX;   // the sample pass is launched in plain stream order
            if (ok && p.a_resident && worker < n_jobs) {
                a_armed = true;
                mbar_arrive_expect_tx(afull, a_region);
                for (int kc = 0; kc < k_chunks; ++kc) tma_load_2d(tiles + kc * a_slice, &map_q, afull, kc * kBlockK, 0);
            }
            for (int job = worker; job < n_jobs && ok; job += n_workers) {
                const int qt = kPair ? (job / p.splits) * 2 + (int)rank : job / p.splits;
                const int split = job % p.splits;
                for (int t = split; t < p.n_tiles && ok; t += p.splits) {
                    {
                        const int64_t tile_end = (int64_t)(t + 1) * kBlockN;
                        const int64_t need = tile_end < p.size ? tile_end : p.size;
                        if (rows_ready < need) {
                            const long long t0 = clock64();
                            while ((rows_ready = (int64_t)ld_acquire_u32(p.dev + kDevRowsReady)) < need) {
                                if (*abort_flag || clock64() - t0 > wait_limit) {
                                    *abort_flag = 1;
                                    ok = false;
                                    break;
                                }
                                __nanosleep(200);
                            }
                            if (!ok) break;
                            asm volatile("fence.proxy.async.global;" ::: "memory");
                        }
                    }
                    for (int u = 0; u < n_sub; ++u) {
                        if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit)) { ok = false; break; }
                        const uint32_t s_dst = ring + stage * stage_bytes;
                        if (!kPair && p.b3d) {
                            // kSubRows rows x kSubSlices slices: each row contributes one contiguous piece
                            const int row = t * kBlockN + (u / n_sg) * kSubRows, slice = (u % n_sg) * kSubSlices;
                            mbar_arrive_expect_tx(full0 + 8 * stage, stage_bytes);
                            if (stream_once)
                                tma_load_3d_hint(s_dst, &map_bank, full0 + 8 * stage, row, slice, bank_policy);
                            else
                                tma_load_3d(s_dst, &map_bank, full0 + 8 * stage, row, slice);
                        } else if (kPair) {
                            const int kc = u;
                            // both blocks' bytes are counted on the leader's barrier, which the MMA waits on
                            const uint32_t leader_full = mapa_u32(full0 + 8 * stage, 0);
                            if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * stage, 2 * stage_bytes);
                            tma_load_2d_pair(s_dst, &map_q, leader_full, kc * kBlockK, qt * kBlockM);
                            if (stream_once)
                                tma_load_2d_pair_hint(s_dst + b_off, &map_bank, leader_full, kc * kBlockK,
                                                      t * kBlockN + (int)rank * (kBlockN / 2), bank_policy);
                            else
                                tma_load_2d_pair(s_dst + b_off, &map_bank, leader_full, kc * kBlockK,
                                                 t * kBlockN + (int)rank * (kBlockN / 2));
                        } else {
                            const int kc = u;
                            mbar_arrive_expect_tx(full0 + 8 * stage, stage_bytes);
                            if (!p.a_resident) tma_load_2d(s_dst, &map_q, full0 + 8 * stage, kc * kBlockK, qt * kBlockM);
                            if (stream_once)
                                tma_load_2d_hint(s_dst + b_off, &map_bank, full0 + 8 * stage, kc * kBlockK, t * kBlockN, bank_policy);
                            else
                                tma_load_2d(s_dst + b_off, &map_bank, full0 + 8 * stage, kc * kBlockK, t * kBlockN);
                        }
                        ++n_issued;
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer =====
        if (lane == 0 && rank == 0) {  // in a pair only the leader issues
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            if (p.a_resident && worker < n_jobs) ok = mbar_wait(afull, 0, abort_flag, wait_limit);
            for (int job = worker; job < n_jobs && ok; job += n_workers) {
                const int split = job % p.splits;
                for (int t = split; t < p.n_tiles && ok; t += p.splits) {
                    if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag, wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kBlockN;
                    for (int u = 0; u < n_sub; ++u) {
                        if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, wait_limit)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t s_addr = ring + stage * stage_bytes;
                        if (!kPair && p.b3d) {
                            // this stage: row group g of the tile, slice group sg -> accumulator columns of group g
                            const int g = u / n_sg, sg = u % n_sg;
                            const uint32_t idesc = p.m64 ? kInstrDescSubM64 : kInstrDescSub;
#pragma unroll
                            for (int sl = 0; sl < kSubSlices; ++sl) {
                                const int kc = sg * kSubSlices + sl;
                                if (kc < k_chunks) {
                                    const uint64_t a_desc = smem_desc(tiles + kc * a_slice);
                                    const uint64_t b_desc = smem_desc(s_addr + sl * (kSubRows * 128));
#pragma unroll
                                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                                        if (kSwap)   // bank rows on the lanes, row group g in columns [N g, N g + N), N = a_rows
                                            umma_bf16(d_tmem + g * p.a_rows, b_desc + (uint64_t)(2 * k), a_desc + (uint64_t)(2 * k),
                                                      (kc > 0 || k > 0) ? 1u : 0u, instr_desc_swap(p.a_rows));
                                        else
                                            umma_bf16(d_tmem + g * kSubRows, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k),
                                                      (kc > 0 || k > 0) ? 1u : 0u, idesc);
                                    }
                                }
                            }
                            umma_commit(empty0 + 8 * stage);
                            if (++stage == kStages) { stage = 0; phase ^= 1; }
                            continue;
                        }
                        const int kc = u;
                        // a resident query tile narrower than 128 rows is read past its end: the
                        // surplus accumulator rows belong to no query and are never looked at
                        const uint64_t a_desc = smem_desc(p.a_resident ? tiles + kc * a_slice : s_addr);
                        const uint64_t b_desc = smem_desc(s_addr + b_off);
#pragma unroll
                        for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                            // advancing 16 bf16 = 32 bytes inside the swizzle row: +2 in the address field
                            if (kPair)
                                umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k),
                                               (kc > 0 || k > 0) ? 1u : 0u);
                            else
                                umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k),
                                          (kc > 0 || k > 0) ? 1u : 0u, p.m64 ? kInstrDescM64 : kInstrDesc);
                        }
                        if (kPair) umma_commit_pair(empty0 + 8 * stage); else umma_commit(empty0 + 8 * stage);
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    if (kPair) umma_commit_pair(tfull0 + 8 * acc); else umma_commit(tfull0 + 8 * acc);
                    if (++acc == 2) { acc = 0; acc_phase ^= 1; }
                }
            }
        }
    } else if (warp < 6) {
        // ===== epilogue: thread = one query of the tile = one TMEM lane =====
        // The thresholds, the histogram and the candidate lists belong to the kernels before this one.
        pdl_wait();
        if constexpr (kSwap) {
            SwapState *st = reinterpret_cast<SwapState *>(reinterpret_cast<unsigned char *>(bars) + 256);
            swap_epilogue(p, st, reinterpret_cast<volatile int *>(tmem_slot + 6), tmem_base, tfull0, tempty0, abort_flag,
                          wait_limit, warp, lane, worker, n_jobs, n_workers);
            __syncwarp();
            if (lane == 0) atomicAdd(const_cast<int *>(epi_done), 1);
        } else {
        const int quarter = warp & 3;              // warps 2,3,4,5 -> lane quarters 2,3,0,1
        const int m = quarter * 32 + lane;
        // the tile's row on this lane: m itself, or with M = 64 sixteen rows per quarter (none on lanes 16-31)
        const int row = p.m64 ? (lane < 16 ? quarter * 16 + lane : -1) : m;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int job = worker; job < n_jobs && ok; job += n_workers) {
            const int qt = kPair ? (job / p.splits) * 2 + (int)rank : job / p.splits;
            const int split = job % p.splits;
            const int list_job = qt * p.splits + split;   // candidate lists are per (query tile, split)
            const int q = qt * kBlockM + row;
            const bool q_valid = row >= 0 && q < p.B;
            // Two filters, both lower bounds of the query's final k1-th key: the key threshold of this
            // list (exact, rises when the list is cut back) and the bin threshold shared through
            // the histogram.  tau_sim is a float no larger than either, for the cheap first test.
            float tau_sim = INFINITY, key_sim_floor = INFINITY;
            uint64_t tau_key = ~(uint64_t)0;
            float h_lo = 0.0f, h_scale = 0.0f;
            int tau_bin = 0;
            unsigned *my_hist = nullptr;
            // self-starting histogram: window base (in absolute bins), whether this thread has one yet, and
            // the window bin from which this tile's entries were already counted ahead of filing
            int a_base = 0, skip_from = kHistBins;
            int64_t counted_end = 0;   // first tile of a job: its rows below this were counted from bin skip_from up before filing
            bool anchored = false;
            if (q_valid) {
                if (abs_mode) {
                    key_sim_floor = -INFINITY;
                    tau_key = 0;
                    my_hist = p.hist + (size_t)q * kHistBins;
                } else if (p.tau0) {
                    // every entry whose similarity reaches the sampled threshold passes
                    key_sim_floor = p.tau0[q];
                    tau_key = (uint64_t)ordered_bits(key_sim_floor + 0.0f) << 32;
                    const float2 r = p.range[q];
                    h_lo = r.x;
                    h_scale = r.y;
                    if (h_scale > 0.0f) my_hist = p.hist + (size_t)q * kHistBins;
                } else {
                    key_sim_floor = -INFINITY;
                    tau_key = 0;
                }
                tau_sim = key_sim_floor;
            }
            slot_q[m] = my_hist ? q : -1;   // the tracker follows this query from now on
            int cnt = 0;
            uint64_t *my_buf = p.cand + ((size_t)list_job * kBlockM + (row < 0 ? 0 : row)) * kMmaCandCap;
            // Files one similarity that reached tau_sim.
            auto file = [&](float s, int64_t row) {
                if (row < p.size && entry_live(p.live_bits, row)) {
                    const uint64_t key = make_key(s, (int32_t)row);
                    int bin = 0;
                    if (my_hist) {
                        if (abs_mode)
                            bin = anchored ? (int)(ordered_bits(s + 0.0f) >> kAbsShift) - a_base : 0;
                        else   // truncation and the clamp at 0 together equal floor and the clamp
                            bin = __float2int_rz((s - h_lo) * h_scale);
                        bin = bin < 0 ? 0 : (bin > kHistBins - 1 ? kHistBins - 1 : bin);
                    }
                    if (key > tau_key && bin >= tau_bin) {
                        my_buf[cnt++] = key;
                        if (my_hist && (bin < skip_from || row >= counted_end) && (anchored || !abs_mode)) atomicAdd(my_hist + bin, 1u);
                    }
                }
            };
            // One chunk of columns: store it (dense mode) or file the entries that pass the filters.
            auto process = [&](uint32_t (&v)[kChunk], int64_t row0, int c0) {
                if (kMode == 1) {
                    if (q_valid) {
                        float4 *dst = reinterpret_cast<float4 *>(p.dense + (size_t)q * p.dense_ld + row0 + c0);
#pragma unroll
                        for (int j = 0; j < kChunk / 4; ++j)
                            dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                 __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    }
                    return;
                }
                // The epilogue warps run one to a scheduler, so every dependent instruction costs its full
                // latency: the code below is written as short trees, not chains.  First the chunk's maximum
                // (nearly every chunk fails the test as a whole), four strands of eight.
                float mx[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    mx[g] = __uint_as_float(v[g]);
#pragma unroll
                    for (int j = g + 4; j < kChunk; j += 4) mx[g] = fmaxf(mx[g], __uint_as_float(v[j]));
                }
                if (fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) >= tau_sim) {
                    // one bit per column that passes, gathered by a tree of ORs
                    uint32_t bits[kChunk];
#pragma unroll
                    for (int j = 0; j < kChunk; ++j) bits[j] = __uint_as_float(v[j]) >= tau_sim ? (1u << j) : 0u;
#pragma unroll
                    for (int w = kChunk / 2; w >= 1; w >>= 1) {
#pragma unroll
                        for (int j = 0; j < w; ++j) bits[j] |= bits[j + w];
                    }
                    uint32_t pass = bits[0];
                    while (pass) {
                        const int j = __ffs(pass) - 1;
                        pass &= pass - 1;
                        file(__uint_as_float(pick(v, j)), row0 + c0 + j);
                    }
                }
                // lists that could overflow on the next chunk are cut back to their best k1
                uint32_t need = __ballot_sync(0xffffffffu, cnt > kMmaCandCap - kChunk);
                while (need) {
                    const int owner = __ffs(need) - 1;
                    need &= need - 1;
                    const int n = __shfl_sync(0xffffffffu, cnt, owner);
                    uint64_t *buf = reinterpret_cast<uint64_t *>(
                        __shfl_sync(0xffffffffu, (unsigned long long)my_buf, owner));
                    __syncwarp();
                    const uint64_t kth = warp_select_topk(buf, n, p.k1);
                    if (lane == owner) {
                        if (p.dev) atomicAdd(p.dev + kDevCutbacks, 1u);
                        cnt = p.k1;
                        tau_key = kth;
                        key_sim_floor = key_sim(kth);
                        tau_sim = fmaxf(tau_sim, key_sim_floor);
                    }
                }
            };
            auto raise_bin = [&](int best) {
                if (best > tau_bin) {
                    tau_bin = best;
                    // self-starting: the smallest value of that bin, exactly.  Sampled range: a similarity in
                    // bin b is at least h_lo + b / h_scale up to rounding; stay a hundredth of a bin below that
                    // and let the bin test decide
                    tau_sim = fmaxf(key_sim_floor,
                                    abs_mode ? from_ordered_bits((uint32_t)(a_base + tau_bin) << kAbsShift)
                                             : h_lo + ((float)tau_bin - 0.01f) / h_scale);
                }
            };
            // Takes the tracker's latest word for this query.
            auto refresh = [&]() {
                if (my_hist && (anchored || !abs_mode)) {
                    const unsigned long long word = slot_tau[m];
                    if ((int)(word >> 32) == q) raise_bin((int)(uint32_t)word);
                }
            };
            int sync_left = p.sync_tiles;
            int n_done = 0;   // tiles of this job examined so far
            for (int t = split; t < p.n_tiles && ok; t += p.splits, ++n_done) {
                if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag, wait_limit)) { ok = false; break; }
                tc_fence_after();
                if (warp == 2 && lane == 0) *tile_seq = *tile_seq + 1;   // paces the tracker
                uint32_t va[kChunk], vb[kChunk];
                const int64_t row0 = (int64_t)t * kBlockN;
                const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBlockN;
                skip_from = kHistBins;
                counted_end = 0;
                if (abs_mode && kMode == 0 && n_done == 0) {
                    // The job's first tile starts the histogram off (every lane of the warp walks through this,
                    // the tensor-memory loads being warp-wide).  Its first kBootCols rows anchor the window
                    // (whoever comes first) and are counted from window bin kBootBin up; then the tile is filed
                    // like any other.  All blocks start together, so by the time this one reads the counters
                    // most of the others have counted their first rows too, and the counters give a threshold
                    // that a few hundred of the 18,944 rows counted pass, where one block's own rows could
                    // justify none (a threshold from fewer counts is lower, never wrong).
                    int enc = my_hist ? __ldcg(p.anchor + q) : 1;
                    if (__any_sync(0xffffffffu, enc == 0)) {
                        // nobody has anchored this query's window yet: these rows' largest similarity does
                        float mx = -INFINITY;
#pragma unroll 1
                        for (int c0 = 0; c0 < kBootCols; c0 += kChunk) {
                            tmem_ld_issue(t_addr + c0, va);
                            tmem_ld_wait(va);
#pragma unroll
                            for (int j = 0; j < kChunk; ++j) {
                                const float x = __uint_as_float(va[j]);
                                if (row0 + c0 + j < p.size && fabsf(x) <= 3.0e38f) mx = fmaxf(mx, x);
                            }
                        }
                        if (my_hist && enc == 0 && mx > -INFINITY) {
                            int prop = (int)(ordered_bits(mx + 0.0f) >> kAbsShift) + kAbsHeadroom - (kHistBins - 1);
                            prop = prop < 0 ? 0 : (prop > kAbsBins - kHistBins ? kAbsBins - kHistBins : prop);
                            const int got = atomicCAS(p.anchor + q, 0, prop + 1);
                            enc = got ? got : prop + 1;
                        }
                    }
                    if (my_hist && enc != 0) {
                        a_base = enc - 1;
                        anchored = true;
                    }
                    const float cnt_edge = anchored ? from_ordered_bits((uint32_t)(a_base + kBootBin) << kAbsShift) : INFINITY;
#pragma unroll 1
                    for (int c0 = 0; c0 < kBootCols; c0 += kChunk) {
                        tmem_ld_issue(t_addr + c0, va);
                        tmem_ld_wait(va);
                        uint32_t bits[kChunk];
#pragma unroll
                        for (int j = 0; j < kChunk; ++j) bits[j] = __uint_as_float(va[j]) >= cnt_edge ? (1u << j) : 0u;
#pragma unroll
                        for (int w = kChunk / 2; w >= 1; w >>= 1) {
#pragma unroll
                            for (int j = 0; j < w; ++j) bits[j] |= bits[j + w];
                        }
                        uint32_t pass = bits[0];
                        while (pass) {
                            const int j = __ffs(pass) - 1;
                            pass &= pass - 1;
                            if (anchored && row0 + c0 + j < p.size && entry_live(p.live_bits, row0 + c0 + j)) {
                                int bin = (int)(ordered_bits(__uint_as_float(pick(va, j)) + 0.0f) >> kAbsShift) - a_base;
                                bin = bin > kHistBins - 1 ? kHistBins - 1 : bin;
                                atomicAdd(my_hist + bin, 1u);
                            }
                        }
                    }
                    // the counted rows' entries from kBootBin up are in the counters already
                    if (anchored) {
                        skip_from = kBootBin;
                        counted_end = row0 + kBootCols;
                    }
                }
                // At the start of a job a threshold moves with every tile and the tracker's word comes
                // a tile late: there the thread reads its counters itself, later it takes the word.  A scan
                // without a tracker keeps reading them, every tile at first and every kReadEvery-th after that:
                // all blocks read the same one or two L2 lines per query, the very lines the survivors' atomic
                // updates go to, and reading them for every tile slowed the whole scan (2 GiB, 128 queries:
                // 0.38-0.39 against 0.357 ms; 64 queries: 5-10 us; the lists grow by 2 %).
                if (sync_left > 0 && (n_done < kReadEvery || n_done % kReadEvery == 0)) {
                    --sync_left;
                    // (sampled thresholds: nothing to read before the block's very first tile, every block
                    // starts at once and the counters are still empty)
                    if (my_hist && (abs_mode ? anchored : !(job == worker && n_done == 0)))
                        raise_bin(hist_best_bin(my_hist, p.k1));
                } else {
                    refresh();
                }
                // two register buffers: the next chunk's load is in flight while one is examined
                tmem_ld_issue(t_addr, va);
                tmem_ld_wait(va);
#pragma unroll 1
                for (int c0 = 0; c0 < kBlockN - 2 * kChunk; c0 += 2 * kChunk) {
                    tmem_ld_issue(t_addr + c0 + kChunk, vb);
                    process(va, row0, c0);
                    tmem_ld_wait(vb);
                    tmem_ld_issue(t_addr + c0 + 2 * kChunk, va);
                    refresh();
                    process(vb, row0, c0 + kChunk);
                    tmem_ld_wait(va);
                }
                tmem_ld_issue(t_addr + kBlockN - kChunk, vb);
                process(va, row0, kBlockN - 2 * kChunk);
                tmem_ld_wait(vb);
                // every column of this accumulator is in registers: hand it back before the last look
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (kPair) mbar_arrive_cluster(mapa_u32(tempty0 + 8 * acc, 0)); else mbar_arrive(tempty0 + 8 * acc);
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
                process(vb, row0, kBlockN - kChunk);
            }
            if (kMode == 0 && ok && qt < p.n_qt && row >= 0) p.cand_cnt[(size_t)list_job * kBlockM + row] = cnt;
            if (kMode == 0 && p.dev) {
                // candidates this warp leaves behind for the merge (one atomic per warp and job)
                const unsigned left = __reduce_add_sync(0xffffffffu, (unsigned)((ok && q_valid) ? cnt : 0));
                if (lane == 0 && left)
                    atomicAdd(reinterpret_cast<unsigned long long *>(p.dev + kDevFiledLo), (unsigned long long)left);
            }
        }
        slot_q[m] = -1;
        if (!ok && kMode == 0) {
            // aborting: whatever this block was to deliver counts as empty, so the merge reads nothing stale
            for (int job = worker; job < n_jobs; job += n_workers) {
                const int qt = kPair ? (job / p.splits) * 2 + (int)rank : job / p.splits;
                if (qt < p.n_qt && row >= 0) p.cand_cnt[((size_t)qt * p.splits + job % p.splits) * kBlockM + row] = 0;
            }
        }
        __syncwarp();
        if (lane == 0) atomicAdd(const_cast<int *>(epi_done), 1);
        }
    } else {
        // ===== threshold tracker: lane l looks after epilogue threads l, l+32, l+64, l+96 =====
        // The counters are read on a thinning schedule: after every tile at the start of a job,
        // where a threshold still moves with each tile, then about every eighth of the tiles done
        // so far (the survivor rate falls like 1 / rows scanned, so a threshold that is an eighth
        // of the scan old lets through an eighth more).  Reading them after every tile throughout
        // costs a tenth of the kernel's time: the reads of all blocks meet the survivors' atomic
        // updates on the same L2 lines.
        if (kMode == 0 && (p.tau0 != nullptr || abs_mode) && p.sync_tiles != kSyncAlways) {
            pdl_wait();
            const long long t0 = clock64();
            int seen = -1, job_start = 0, next_poll = 0, q_first = -2;
            auto running = [&]() { return *epi_done < 4 && !*abort_flag && clock64() - t0 < 2 * wait_limit; };
            while (running()) {
                while (*tile_seq == seen && running()) __nanosleep(100);
                seen = *tile_seq;
                // a new job (other queries on the mailboxes) starts the schedule afresh
                const int q_now = __shfl_sync(0xffffffffu, slot_q[lane], 0);
                if (q_now != q_first) {
                    q_first = q_now;
                    job_start = seen;
                    next_poll = seen + p.sync_tiles - 1;   // until then the epilogue reads the counters itself
                }
                if (seen < next_poll) continue;
                next_poll = seen + 1 + (seen - job_start) / 8;
#pragma unroll 1
                for (int r = 0; r < kBlockM / 32; r += 2) {
                    const int m0 = r * 32 + lane, m1 = m0 + 32;
                    const int q0 = slot_q[m0], q1 = slot_q[m1];
                    // two queries at a time, so that their loads overlap
                    const int b0 = hist_best_bin(p.hist + (size_t)(q0 < 0 ? 0 : q0) * kHistBins, p.k1);
                    const int b1 = hist_best_bin(p.hist + (size_t)(q1 < 0 ? 0 : q1) * kHistBins, p.k1);
                    if (q0 >= 0) slot_tau[m0] = ((unsigned long long)(uint32_t)q0 << 32) | (uint32_t)b0;
                    if (q1 >= 0) slot_tau[m1] = ((unsigned long long)(uint32_t)q1 << 32) | (uint32_t)b1;
                }
            }
        }
    }

    // ===== teardown =====
    tc_fence_before();
    __syncthreads();
    const int aborted = *abort_flag;
    if (kPair) {
        // each block tells its partner how far its producer got and whether it is backing out
        if (threadIdx.x == 0) {
            st_cluster_u32(mapa_u32(smem_u32(const_cast<int *>(peer_issued)), rank ^ 1u), (uint32_t)n_issued);
            st_cluster_u32(mapa_u32(smem_u32(const_cast<int *>(peer_abort)), rank ^ 1u), (uint32_t)aborted);
        }
        cluster_sync_all();
    }
    if (aborted || (kPair && *peer_abort)) {
        // Backing out: no copy may still be on its way into this block's shared memory when the block
        // ends.  Both producers have left their loops, so nothing new is issued except the stand-ins
        // below; then the thread that armed the full barriers waits, bounded, for every phase it or
        // its partner counted bytes on.
        if (threadIdx.x == 0) {
            int n_all = n_issued;
            if (kPair) {
                // The two producers of a pair are never more than a ring apart (a slice is issued only
                // after the MMA that consumed the slice one ring earlier, which needed both halves).
                // The one that stopped first issues stand-in loads (tile 0) for the slices its partner
                // still issued, so that every such phase of the leader's barriers completes.
                const int n_peer = *peer_issued;
                for (int i = n_issued; i < n_peer; ++i) {
                    const int s = i % kStages;
                    const uint32_t s_dst = ring + s * stage_bytes;
                    const uint32_t leader_full = mapa_u32(full0 + 8 * s, 0);
                    if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * s, 2 * stage_bytes);
                    tma_load_2d_pair(s_dst, &map_q, leader_full, 0, 0);
                    tma_load_2d_pair(s_dst + b_off, &map_bank, leader_full, 0, 0);
                }
                if (n_peer > n_all) n_all = n_peer;
            }
            if (rank == 0) {   // the bytes of both blocks of a pair are counted on the leader's barriers
                if (a_armed) mbar_wait_deadline(afull, 0, wait_limit);
                for (int s = 0; s < kStages; ++s) {
                    if (n_all <= s) break;
                    const int last = s + kStages * ((n_all - 1 - s) / kStages);   // last slice that used stage s
                    mbar_wait_deadline(full0 + 8 * s, (uint32_t)(last / kStages) & 1u, wait_limit);
                }
            }
            if (aborted) atomicCAS(p.status, 0, (int)EVK_ERR_DEVICE_TIMEOUT);
        }
        __syncthreads();
    }
    if (kPair) cluster_sync_all();  // neither block frees tensor memory or leaves while the other may touch it
    if (warp == 0) {
        tc_fence_after();
        if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Clears the shared histograms and window anchors of a scan that starts them off itself.
__global__ void __launch_bounds__(256)
hist_reset_kernel(unsigned *__restrict__ hist, int *__restrict__ anchor, int n_queries) {
    pdl_trigger();
    pdl_wait();   // the previous user of this workspace may still be reading them
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i < n_queries * kHistBins) hist[i] = 0;
    if (i < n_queries) anchor[i] = 0;
}

// A starting threshold per query from its sample similarities: any value that at least k1 of
// the sampled entries reach is a lower bound of the query's final k1-th similarity.  The exact
// k1-th largest is not needed, so one pass over a fine histogram of the sample's range picks
// the highest bin edge with k1 samples at or above it, and the threshold is the smallest
// sample in those bins (exact whatever the rounding of the bin arithmetic).
constexpr int kSelThreads = 256;
constexpr int kSelPerThread = kMmaSample / kSelThreads;
constexpr int kSelBins = 1024;

// (The samples are kept in shared memory, not in registers: at 64 registers a thread only four blocks fit
// an SM and 1,024 queries took two waves.)
__global__ void __launch_bounds__(kSelThreads, 8)
sample_threshold_kernel(const float *__restrict__ dense, int ld, int n_sample, int k1, float *__restrict__ tau0,
                        float2 *__restrict__ range, unsigned *__restrict__ hist_out,
                        const uint32_t *__restrict__ live_bits, int64_t sample_stride) {
    __shared__ int bins[kSelBins];
    __shared__ float sv[kMmaSample];
    __shared__ float red_lo[kSelThreads / 32], red_hi[kSelThreads / 32];
    __shared__ int red_cnt[kSelThreads / 32];
    __shared__ int chosen;
    const int q = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_trigger();
    pdl_wait();
    for (int i = tid; i < kHistBins; i += kSelThreads) hist_out[(size_t)q * kHistBins + i] = 0;
    for (int i = tid; i < kSelBins; i += kSelThreads) bins[i] = 0;
    if (tid == 0) chosen = 0;
    // this thread's samples; a non-finite similarity counts as the lowest value
    float lo = INFINITY, hi = -INFINITY;
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j) {
        const int i = tid + j * kSelThreads;
        float x = (i < n_sample) ? dense[(size_t)q * ld + i] : -INFINITY;
        // a non-finite similarity, or a sampled entry that has been dropped from the memory, counts as
        // the lowest value: it cannot vouch for a threshold
        if (i < n_sample && (!(fabsf(x) <= 3.0e38f) || !entry_live(live_bits, (int64_t)i * sample_stride))) x = -3.0e38f;
        sv[tid + j * kSelThreads] = x;   // read back by this thread alone
        if (i < n_sample) {
            lo = fminf(lo, x);
            hi = fmaxf(hi, x);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
    }
    if (lane == 0) {
        red_lo[warp] = lo;
        red_hi[warp] = hi;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kSelThreads / 32; ++i) {
        lo = fminf(lo, red_lo[i]);
        hi = fmaxf(hi, red_hi[i]);
    }
    float scale = (float)kSelBins / (hi - lo);
    if (!(scale > 0.0f) || !(scale < 3.0e38f)) scale = 0.0f;   // no spread: everything in bin 0
    auto bin_of = [&](float x) {
        const int b = (int)((x - lo) * scale);
        return b < 0 ? 0 : (b > kSelBins - 1 ? kSelBins - 1 : b);
    };
#pragma unroll 4
    for (int j = 0; j < kSelPerThread; ++j)
        if (tid + j * kSelThreads < n_sample) atomicAdd(&bins[bin_of(sv[tid + j * kSelThreads])], 1);
    __syncthreads();
    // thread t owns bins [4t, 4t+4); count of samples in its bins and in all higher ones
    int mine[4], sum = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        mine[j] = bins[4 * tid + j];
        sum += mine[j];
    }
    int incl = sum;   // this lane and the higher lanes of the warp
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int u = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += u;
    }
    if (lane == 0) red_cnt[warp] = incl;
    __syncthreads();
    int above = incl - sum;   // samples in bins higher than this thread's
    for (int i = warp + 1; i < kSelThreads / 32; ++i) above += red_cnt[i];
    if (above < k1 && k1 <= above + sum) {   // exactly one thread: the k1-th largest lies in its bins
        int c = above, b = 4 * tid;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            if (k1 <= c + mine[j]) {
                b = 4 * tid + j;
                break;
            }
            c += mine[j];
        }
        chosen = b;
    }
    __syncthreads();
    const int b_min = chosen;
    float t = INFINITY;
#pragma unroll 4
    for (int j = 0; j < kSelPerThread; ++j) {
        const float x = sv[tid + j * kSelThreads];
        if (tid + j * kSelThreads < n_sample && bin_of(x) >= b_min) t = fminf(t, x);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t = fminf(t, __shfl_xor_sync(0xffffffffu, t, off));
    if (lane == 0) red_lo[warp] = t;   // last read of red_lo was before two barriers
    __syncthreads();
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < kSelThreads / 32; ++i) t = fminf(t, red_lo[i]);
        // the shared histogram spans from the starting threshold to half a range above the sample's
        // best similarity; whatever lies higher is counted in the last bin
        const float start = t, best = hi;
        const float top = best + 0.5f * (best - start);
        float h_scale = 0.0f;  // 0 switches the histogram off (a sample without spread)
        if (top - start > 1e-2f * fmaxf(fabsf(start), fabsf(top)) && top - start > 1e-30f)
            h_scale = (float)kHistBins / (top - start);
        if (!(h_scale > 0.0f) || !(h_scale < 3.0e38f)) h_scale = 0.0f;
        tau0[q] = start;
        range[q] = make_float2(start, h_scale);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// A [rows][d] bf16 matrix whose consecutive rows are row_stride_elems apart, boxed 64 x box_rows.
bool make_map(CUtensorMap *map, const void *base, int d, int64_t rows, int64_t row_stride_elems, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)row_stride_elems * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix seen as {64 columns, rows, slices of 64 columns}, boxed 64 x kSubRows x kSubSlices: one
// copy brings kSubSlices * 128 contiguous bytes of each row and lays them down as kSubSlices K-major
// tiles.  (Plain copies into shared memory, measured on B200 over 2 GiB: 7.2 TB/s with 256 contiguous
// bytes per row, 7.3 with 512, against 6.9-7.0 TB/s for boxes of 256 rows x 128 bytes.)
// Needs a width that is a multiple of 64: the innermost extent is a fixed 64 columns.
bool make_map3(CUtensorMap *map, const void *base, int d, int64_t rows, int64_t row_stride_elems) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || d % kBlockK != 0) return false;
    const cuuint64_t gdim[3] = {(cuuint64_t)kBlockK, (cuuint64_t)rows, (cuuint64_t)(d / kBlockK)};
    const cuuint64_t gstride[2] = {(cuuint64_t)row_stride_elems * 2, (cuuint64_t)kBlockK * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kSubRows, (cuuint32_t)kSubSlices};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shared-memory plan for a batch: does the query tile stay resident, how deep is the ring.
struct SmemPlan {
    int a_resident, a_rows, n_stages;
    size_t bytes;
};

SmemPlan smem_plan(int B, int d) {
    SmemPlan sp;
    // up to kSwapMax queries of whole slices go to the swapped layout, whose query tile is padded to 16 rows
    const int rows = (B <= kSwapMax && d % kBlockK == 0) ? swap_n(B) : (B < kBlockM ? ((B + 7) / 8) * 8 : kBlockM);
    const size_t a_bytes = (size_t)rows * ((d + kBlockK - 1) / kBlockK * kBlockK) * 2;
    const size_t budget = kSmemMax - kSmemFixed;
    if (B <= kBlockM && a_bytes + 3 * (size_t)kBBytes <= budget) {
        sp.a_resident = 1;
        sp.a_rows = rows;
        size_t st = (budget - a_bytes) / kBBytes;
        // four stages, even where six would fit: measured 3 % faster over 2 GiB at 1-32 queries
        // (0.318 against 0.328 ms at one query; two stages: 0.372)
        sp.n_stages = (int)(st > (size_t)kResidentStages ? kResidentStages : st);
        sp.bytes = kSmemFixed + a_bytes + (size_t)sp.n_stages * kBBytes;
    } else {
        sp.a_resident = 0;
        sp.a_rows = kBlockM;
        sp.n_stages = 4;
        sp.bytes = kSmemFixed + (size_t)sp.n_stages * (kABytes + kBBytes);
    }
    return sp;
}

// overlap = true: programmatic dependent launch behind the kernel enqueued just before.
// pair = true: clusters of two blocks (grid must be even), the cta_group::2 variant.
cudaError_t launch_kernel(const CUtensorMap &mq, const CUtensorMap &mb, const MmaParams &p, int grid,
                          size_t smem_bytes, bool overlap, bool pair, cudaStream_t stream, bool swap = false) {
    auto kern = pair ? score_mma_kernel<true, 0, false>
                     : (p.mode == 1 ? score_mma_kernel<false, 1, false>
                                    : (swap ? score_mma_kernel<false, 0, true, true> : score_mma_kernel<false, 0, true>));
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (overlap) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    if (pair) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 2;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    return cudaLaunchKernelEx(&cfg, kern, mq, mb, p);
}

// Two SMs share a tile when there are at least two query tiles to pair up.
bool use_pairs(int n_qt) { return n_qt >= 2; }

// Bank splits per query tile.  Jobs (query tile, split) are dealt round-robin to the
// blocks, one block per SM; the split count is the smallest one from 148 / n_qt upwards whose
// job count fills whole rounds of 148 blocks to 97 % or better.  Fewer splits keep more query
// tiles side by side on the same bank tiles (they share them through L2).
int splits_for(int n_qt, int n_tiles) {
    if (n_qt <= 0) n_qt = 1;
    // workers: single blocks, or pairs of blocks that take two query tiles at a time
    const int n_work = use_pairs(n_qt) ? num_sms() / 2 : num_sms();
    const int n_units = use_pairs(n_qt) ? (n_qt + 1) / 2 : n_qt;
    int base = n_work / n_units;
    if (base < 1) base = 1;
    int splits = base;
    if (n_units < n_work) {
        for (int s = base; s <= 4 * base && s <= n_work; ++s) {
            const int jobs = n_units * s;
            const int rounds = (jobs + n_work - 1) / n_work;
            if (jobs * 100 >= 97 * rounds * n_work) {
                splits = s;
                break;
            }
        }
    }
    if (splits > n_tiles) splits = n_tiles > 0 ? n_tiles : 1;
    return splits;
}

struct MmaLayout {
    size_t cand, cand_cnt, dense, tau0, range, hist, total;
};

MmaLayout mma_layout(int B) {
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t n_qt = (size_t)((B + kBlockM - 1) / kBlockM);
    // one candidate list per (job, query of the tile); the split count can only shrink for small banks
    const size_t lists = n_qt * (size_t)splits_for((int)n_qt, 1 << 30) * kBlockM;
    MmaLayout l;
    l.cand = 0;
    l.cand_cnt = l.cand + align(lists * kMmaCandCap * sizeof(uint64_t));
    l.dense = l.cand_cnt + align(lists * sizeof(int));
    l.tau0 = l.dense + align(n_qt * kBlockM * kMmaSample * sizeof(float));
    l.range = l.tau0 + align(n_qt * kBlockM * sizeof(float));
    l.hist = l.range + align(n_qt * kBlockM * sizeof(float2));
    l.total = l.hist + align(n_qt * kBlockM * kHistBins * sizeof(unsigned));
    return l;
}

}  // namespace

bool mma_supported(int d, int k1) {
    // rows must start on 16-byte boundaries for TMA (d % 8 == 0) and span at least one 64-column slice
    return d % 8 == 0 && d >= kBlockK && k1 <= kMmaCandCap / 2 && encode_fn() != nullptr;
}

MmaPlan mma_plan(int64_t size, int B, int k1) {
    MmaPlan pl;
    pl.n_qt = (B + kBlockM - 1) / kBlockM;
    pl.n_tiles = (int)((size + kBlockN - 1) / kBlockN);
    pl.splits = splits_for(pl.n_qt, pl.n_tiles);
    pl.pair = use_pairs(pl.n_qt) ? 1 : 0;
    if (pl.pair) {
        const int jobs = ((pl.n_qt + 1) / 2) * pl.splits;
        pl.grid = 2 * (jobs < num_sms() / 2 ? jobs : num_sms() / 2);
    } else {
        const int jobs = pl.n_qt * pl.splits;
        pl.grid = jobs < num_sms() ? jobs : num_sms();
    }
    if (pl.grid < 1) pl.grid = 1;
    // a strided sample of the bank gives each query a starting threshold
    // Paired scans (two or more query tiles) take their starting thresholds from a strided sample of the
    // bank; scans of one query tile start theirs off themselves (see kAbsShift).  Measured with the
    // self-starting histogram in paired scans too: 0.54 against 0.48 ms per retrieval for 1,024 queries over
    // the clustered bank (a first tile without a row of the query's own cluster anchors the window too
    // low), 21.9 against 21.5 ms for 4,096 queries over 6 GiB.
    pl.n_sample = (pl.pair && size >= 4 * (int64_t)kMmaSample && k1 < kMmaSample) ? kMmaSample : 0;
    pl.sample_stride = pl.n_sample ? size / pl.n_sample : 0;
    pl.stall = 0;
    pl.live_bits = nullptr;
    pl.dev = nullptr;
    pl.wait_queries = 1;
    return pl;
}

size_t mma_workspace_bytes(int B) { return mma_layout(B).total; }

cudaError_t launch_score_mma(const __nv_bfloat16 *bank, int64_t size, int64_t capacity, int d,
                             const __nv_bfloat16 *queries, int B, int k1, const MmaPlan &pl, void *workspace,
                             int32_t *status, uint64_t **cand_out, int **cand_cnt_out,
                             cudaEvent_t ev_start, cudaEvent_t ev_stop, cudaStream_t stream, int *launches) {
    const MmaLayout l = mma_layout(B);
    char *ws = static_cast<char *>(workspace);
    uint64_t *cand = reinterpret_cast<uint64_t *>(ws + l.cand);
    int *cand_cnt = reinterpret_cast<int *>(ws + l.cand_cnt);
    float *dense = reinterpret_cast<float *>(ws + l.dense);
    float *tau0 = reinterpret_cast<float *>(ws + l.tau0);
    float2 *range = reinterpret_cast<float2 *>(ws + l.range);
    unsigned *hist = reinterpret_cast<unsigned *>(ws + l.hist);
    *cand_out = cand;
    *cand_cnt_out = cand_cnt;

    const SmemPlan sp = smem_plan(B, d);
    CUtensorMap map_q, map_bank;
    if (!make_map(&map_q, queries, d, B, d, sp.a_rows)) return cudaErrorInvalidValue;

    MmaParams p;
    p.B = B;
    p.d = d;
    p.k1 = k1;
    p.n_qt = pl.n_qt;
    p.cand = cand;
    p.cand_cnt = cand_cnt;
    p.dense = dense;
    p.dense_ld = kMmaSample;
    p.status = status;
    p.stall = pl.stall;
    p.tau0 = nullptr;
    p.range = range;
    p.hist = hist;
    p.live_bits = pl.live_bits;
    p.dev = pl.dev;
    p.wait_queries = pl.wait_queries;
    p.abs_hist = pl.pair ? 0 : 1;
    p.anchor = reinterpret_cast<int *>(tau0);   // the sampled thresholds' array, unused by such a scan
    // One query tile: the scan runs at HBM speed, a bank tile arrives every ~11 us and the epilogue
    // idles most of that, so it reads its counters itself before every tile (freshest thresholds).
    // More tiles: the tensor cores set the pace and the reads move to the tracker warp.
    p.sync_tiles = pl.pair ? kSyncTiles : kSyncAlways;
    p.a_resident = sp.a_resident;
    // Up to 64 resident queries: M = 64 instructions.  The scan is bound by HBM either way, but the
    // tensor cores then do half the work on padding rows, and under the power cap that is worth
    // 250 MHz of SM clock and 4-5 % of a step (0.398 against 0.420 ms at 64 queries over 2 GiB).
    p.m64 = (sp.a_resident && sp.a_rows <= 64) ? 1 : 0;   // (the swapped layout has its own instruction shape)
    p.a_rows = sp.a_rows;
    p.n_stages = sp.n_stages;
    // resident queries and a width of whole slices: bank stages of 64 rows x 4 slices
    p.b3d = (sp.a_resident && d % kBlockK == 0) ? 1 : 0;

    if (pl.n_sample) {
        // dense pass over every sample_stride-th row
        CUtensorMap map_sample;
        if (!(p.b3d ? make_map3(&map_sample, bank, d, pl.n_sample, pl.sample_stride * d)
                    : make_map(&map_sample, bank, d, pl.n_sample, pl.sample_stride * d, kBlockN)))
            return cudaErrorInvalidValue;
        p.size = pl.n_sample;
        p.mode = 1;
        p.n_tiles = pl.n_sample / kBlockN;
        // the sample pass is small: single blocks, as many splits as fit next to the query tiles
        int s_splits = num_sms() / p.n_qt;
        if (s_splits < 1) s_splits = 1;
        if (s_splits > p.n_tiles) s_splits = p.n_tiles;
        p.splits = s_splits;
        const int jobs = p.n_qt * p.splits;
        cudaError_t err = launch_kernel(map_q, map_sample, p, jobs < num_sms() ? jobs : num_sms(), sp.bytes, false, false, stream);
        if (err != cudaSuccess) return err;
        ++*launches;
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(B);
            cfg.blockDim = dim3(kSelThreads);
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            err = cudaLaunchKernelEx(&cfg, sample_threshold_kernel, (const float *)dense, (int)kMmaSample,
                                     (int)pl.n_sample, (int)k1, tau0, range, hist, pl.live_bits, (int64_t)pl.sample_stride);
        }
        if (err != cudaSuccess) return err;
        ++*launches;
        p.tau0 = tau0;
    }

    // in a pair every block loads its half of a bank slice (128 rows) and its own query slice
    if (pl.pair) p.b3d = 0;
    if (!(p.b3d ? make_map3(&map_bank, bank, d, capacity, d)
                : make_map(&map_bank, bank, d, capacity, d, pl.pair ? kBlockN / 2 : kBlockN)))
        return cudaErrorInvalidValue;
    size_t smem_bytes = sp.bytes;
    if (pl.pair) {
        p.m64 = 0;
        p.a_resident = 0;
        p.a_rows = kBlockM;
        // four stages here too: the same speed as six on short scans, 5 % faster on the long
        // power-capped one (19.7 against 20.7 ms for 4,096 queries over 6 GiB).  One pair of query tiles
        // is bound by HBM instead, and four stages of 16 KB of bank rows keep too few bytes in flight:
        // six there (129-256 queries over 2 GiB: 0.433-0.493 -> 0.410-0.472 ms)
        p.n_stages = pl.n_qt <= 2 ? kMaxStages : kResidentStages;
        smem_bytes = kSmemFixed + (size_t)p.n_stages * (kABytes + kBBytes / 2);
    }
    p.size = size;
    p.mode = 0;
    p.n_tiles = pl.n_tiles;
    p.splits = pl.splits;
    cudaError_t err = cudaSuccess;
    if (p.abs_hist) {
        const int n = B * kHistBins;
        err = launch_overlapped(hist_reset_kernel, dim3((n + 255) / 256), dim3(256), 0, stream, hist, p.anchor, B);
        if (err != cudaSuccess) return err;
        ++*launches;
    }
    if (ev_start) err = cudaEventRecord(ev_start, stream);
    // behind the threshold (or reset) kernel the scan may start early; its epilogue waits for that kernel
    if (err == cudaSuccess)
        // (Only a scan of single blocks starts early.  A kernel launched as a cluster with the programmatic
        // attribute was seen, on B200 with driver 580, to run past its griddepcontrol.wait while its
        // predecessor was still running, so the paired scan is launched in plain stream order.)
        err = launch_kernel(map_q, map_bank, p, pl.grid, smem_bytes, p.abs_hist && !pl.pair && !ev_start,
                            pl.pair != 0, stream, !pl.pair && p.b3d && B <= kSwapMax);
    if (err != cudaSuccess) return err;
    ++*launches;
    if (ev_stop) err = cudaEventRecord(ev_stop, stream);
    return err;
}

}  // namespace evk
