// Host-side launchers of the kernels, one per step of the hot path.  Each returns a
// cudaError_t from the launch; none synchronises.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace evk {

// ---- insert (Eq. 1) ---------------------------------------------------------
// live_bits: one bit per entry, set for the new entries; dev: the bank's device words (live count).
cudaError_t launch_insert(__nv_bfloat16 *bank, float *q_tables, uint32_t *visits, uint32_t *live_bits, uint32_t *dev,
                          int64_t capacity,
                          int d, int n_stages, int64_t first, int64_t n, const void *emb, int emb_dtype,
                          int stage, const float *q_init, float q_default, int32_t *ids_out,
                          cudaStream_t stream, int *launches);

// fp32 -> bf16 (nearest even) conversion of a query batch.
cudaError_t launch_convert_queries(const float *src, __nv_bfloat16 *dst, int64_t n_elems,
                                   cudaStream_t stream, int *launches);

// ---- phase 1, streaming kernel ---------------------------------------------
// Candidate lists: for query q and part p, part_counts[q*nparts+p] keys at
// part_keys[(q*nparts+p)*part_stride ...].
struct StreamPlan {
    int qb;        // queries per pass over the bank
    int nparts;    // thread blocks per pass (= candidate lists per query)
    int cap;       // shared-memory candidate capacity per query
    size_t smem;   // dynamic shared memory per block
    const uint32_t *live_bits;   // entries dropped from the memory are skipped (null: none ever was)
};
bool stream_supported(int d);
StreamPlan stream_plan(int64_t size, int d, int B, int k1);
cudaError_t launch_score_stream(const __nv_bfloat16 *bank, int64_t size, int d,
                                const __nv_bfloat16 *queries, int B, int k1, const StreamPlan &plan,
                                uint64_t *part_keys, int *part_counts, cudaStream_t stream, int *launches);

// ---- phase 1, tensor-core kernel ---------------------------------------------
// Candidate lists: job = query_tile * splits + split; list = job * 128 + (query % 128);
// cand_cnt[list] keys at cand[list * kMmaCandCap ...].
constexpr int kMmaCandCap = 1024;  // keys per candidate list
constexpr int kMmaSample = 4096;   // bank rows sampled for the starting thresholds
struct MmaPlan {
    int n_qt;               // query tiles of 128
    int n_tiles;            // bank tiles of 256 rows
    int splits;             // bank splits per query tile (= candidate lists per query)
    int grid;               // thread blocks
    int pair;               // 1: clusters of two blocks share 256-query tiles (cta_group::2)
    int n_sample;           // 0: no sampling pass
    int64_t sample_stride;  // rows between sampled entries
    int stall;              // test aid, see evk_mem_inject_stall
    const uint32_t *live_bits;   // entries dropped from the memory are skipped (null: none ever was)
    uint32_t *dev;               // the bank's device words (counters), or null
    int wait_queries;            // the query matrix comes out of the library's own conversion kernel, which may
                                 // still be running when the scan starts (mma_plan sets 1, the cautious value)
};
bool mma_supported(int d, int k1);
MmaPlan mma_plan(int64_t size, int B, int k1);
size_t mma_workspace_bytes(int B);
// ev_start / ev_stop (may be null) are recorded around the full-bank launch only.
cudaError_t launch_score_mma(const __nv_bfloat16 *bank, int64_t size, int64_t capacity, int d,
                             const __nv_bfloat16 *queries, int B, int k1, const MmaPlan &plan, void *workspace,
                             int32_t *status, uint64_t **cand_out, int **cand_cnt_out,
                             cudaEvent_t ev_start, cudaEvent_t ev_stop, cudaStream_t stream, int *launches);

// ---- pool merge + phase 2 ------------------------------------------------------
// List of (query q, part p): (q / qt_size) * (nparts * qt_size) + p * qt_size + q % qt_size.
// expect: entries every query must at least have (min(k1, size)); fewer sets EVK_ERR_INCOMPLETE.
constexpr int kMergeMaxParts = 2048;
// Merges each query's lists into its pool (optionally written to pool_*_user, [B][k1]) and
// runs phase 2 on it: ids_out / scores_out [B][k2].  norm: 0 raw mix, 1 pool z-scores.
// live_count (may be null): device word with the number of live entries; expect is capped by it.
cudaError_t launch_merge_rerank(const uint64_t *part_keys, const int *part_counts, int nparts,
                                int part_stride, int qt_size, int B, int k1, int expect, const uint32_t *live_count,
                                int32_t *status,
                                int32_t *pool_ids_user, float *pool_sims_user,
                                int k2, const float *q_stage, float w, int norm, int32_t *ids_out, float *scores_out,
                                cudaStream_t stream, int *launches);

// ---- Eq. 4 update -----------------------------------------------------------
size_t q_update_workspace_bytes(int64_t m);
// visits == nullptr: constant step size alpha.  Otherwise alpha_t = 1 / visits[id] after counting
// the update (decreasing step size), and the counts are advanced.
// longest_run (may be null): device word raised to the longest run of one id seen in a batch.
cudaError_t launch_q_update(float *q_stage, int64_t size, const int32_t *ids, const float *rewards,
                            int64_t m, float alpha, uint32_t *visits, int32_t *status, void *workspace,
                            cudaStream_t stream, int *launches, uint32_t *longest_run = nullptr);

// Eq. 4 update with scratch held in a static device array (no caller workspace).
int64_t q_update_static_max();
cudaError_t launch_q_update_static(float *q_stage, int64_t size, const int32_t *ids, const float *rewards,
                                   int64_t m, float alpha, int32_t *status, cudaStream_t stream, int *launches);

// ---- epsilon-greedy exploration over the pool -----------------------------------------
cudaError_t launch_explore(const int32_t *pool_ids, const float *pool_sims, int B, int k1, int k2,
                           const float *q_stage, float w, int norm, float epsilon, uint64_t seed, uint64_t step,
                           int32_t *ids_out, float *scores_out, uint8_t *explored_out, cudaStream_t stream,
                           int *launches);

// ---- start points by value (Section 3.4) -----------------------------------------------
cudaError_t launch_select_by_value(const int32_t *cand_ids, const int32_t *offsets, int n_tasks, int64_t size,
                                   const uint32_t *live_bits, const float *q_stage, int k, int32_t *ids_out, float *q_out, int32_t *status,
                                   cudaStream_t stream, int *launches);

// ---- a bank split by rows over several GPUs ---------------------------------------------
cudaError_t launch_tag_pool(const int32_t *pool_ids, int64_t n, int32_t id_offset, const float *q_stage,
                            int32_t *gids_out, float *q_out, cudaStream_t stream, int *launches);
cudaError_t launch_merge_shards(const int32_t *gids, const float *sims, const float *qs, int n_shards, int B, int k1,
                                int k2, float w, int32_t *ids_out, float *scores_out, int32_t *pool_gids_out,
                                float *pool_sims_out, cudaStream_t stream);

// ---- dropping entries, export and import ---------------------------------------------------------
// Clears the live bit of every id (the whole call is refused, through `status`, if one is out of range).
cudaError_t launch_tombstone(const int32_t *ids, int64_t n, int64_t size, uint32_t *live_bits, uint32_t *dev,
                             int32_t *status, cudaStream_t stream, int *launches);
// live bits [first, first + n) as one byte per entry (1 = live).
cudaError_t launch_live_export(const uint32_t *live_bits, int64_t first, int64_t n, uint8_t *out, cudaStream_t stream,
                               int *launches);
// entries [first, first + n), all live so far: those whose byte is 0 are dropped.
cudaError_t launch_live_import(const uint8_t *live, int64_t first, int64_t n, uint32_t *live_bits, uint32_t *dev,
                               cudaStream_t stream, int *launches);

// ---- read-only bandwidth calibration ---------------------------------------------------------------
// Streams `bytes` (rounded down to whole 32 KB pieces) of device memory into shared memory once.
cudaError_t launch_read_probe(const void *src, size_t bytes, int32_t *status, cudaStream_t stream);

// ---- rewards (Eq. 5, Eq. 6, running normalisation) ---------------------------------
cudaError_t launch_reward_draft(const uint8_t *feasible, int64_t n, float *out, cudaStream_t stream);
cudaError_t launch_reward_refine(const float *best, const float *latency, const uint8_t *feasible, int64_t n,
                                 float *out, cudaStream_t stream);
cudaError_t launch_reward_normalize(double *state, const float *raw, int64_t n, float sigma_min, float clip,
                                    float *out, cudaStream_t stream);

}  // namespace evk
