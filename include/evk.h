/*
 * evk.h — C ABI of the value-driven experience memory (CUDA, sm_100a).
 *
 * The library keeps a bank of embeddings with one value estimate per entry and
 * stage, and runs the two operations of the method on it:
 *   - value-driven retrieval (Section 3.2): dense retrieval of a top-k1 candidate
 *     pool by inner-product similarity, then a cut to k2 items using the
 *     stage-specific value table Q_stage;
 *   - the unified value update (Eq. 4; Eq. 8 in Appendix A):
 *     Q <- Q + alpha * (r - Q) for every retrieved item once a reward is seen.
 * New experiences are appended as the memory grows (Eq. 1).
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless its name ends in `_host`.
 *     The caller owns all device memory (bank arena, workspaces, inputs,
 *     outputs); the library allocates none and frees none.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *     return; work is ordered by the stream, so an insert or update enqueued
 *     before a retrieve on the same stream is visible to it.  Calls on one handle
 *     from several streams or threads at once are not synchronised.
 *   - Every function returning int returns EVK_OK (0) or a negative evk_status.
 *     Errors detectable on the host are returned before anything is enqueued.
 *     Errors only the device can see (an id out of range, a non-finite reward, a
 *     wait that ran out) are recorded in a device status word by a checking pass
 *     that runs before any mutation; the mutating kernels of that call then do
 *     nothing.  evk_last_status() reads the word.
 *   - No function throws, aborts or traps.
 */
#ifndef EVK_H_
#define EVK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum evk_status {
    EVK_OK = 0,
    EVK_ERR_INVALID = -1,        /* bad argument (null pointer, stage, k, alpha, w, dtype, alignment) */
    EVK_ERR_CAPACITY = -2,       /* insert beyond the capacity given at create                       */
    EVK_ERR_WORKSPACE = -3,      /* workspace or arena smaller than the *_bytes query says            */
    EVK_ERR_RANGE = -4,          /* device check: an entry id outside [0, size)                       */
    EVK_ERR_NONFINITE = -5,      /* device check: a reward that is NaN or infinite                    */
    EVK_ERR_DEVICE_TIMEOUT = -6, /* device: a bounded wait inside a kernel ran out                    */
    EVK_ERR_CUDA = -7,           /* a CUDA runtime or driver call failed                              */
    EVK_ERR_UNSUPPORTED = -8,    /* shape outside what the kernels support (see each call)            */
    EVK_ERR_INCOMPLETE = -9      /* device check: a query found fewer candidates than min(k1, size),
                                    which only non-finite similarities (NaN embeddings) can cause      */
} evk_status;

enum { EVK_DTYPE_F32 = 0, EVK_DTYPE_BF16 = 1 };
enum { EVK_STAGE_DRAFT = 0, EVK_STAGE_REFINE = 1, EVK_STAGE_ALL = -1 };
/* Which phase-1 kernel evk_retrieve uses. */
enum { EVK_SCORING_AUTO = 0, EVK_SCORING_STREAM = 1, EVK_SCORING_TENSOR = 2 };
/* How phase 2 mixes similarity and value (evk_mem_set_score_norm). */
enum { EVK_NORM_NONE = 0, EVK_NORM_POOL_ZSCORE = 1 };

enum { EVK_MAX_K1 = 1024, EVK_MAX_D = 2048, EVK_MAX_STAGES = 8 };

typedef struct evk_mem evk_mem; /* opaque; host-side state only */

typedef struct evk_config {
    int32_t d;          /* embedding width; multiple of 8, <= EVK_MAX_D                    */
    int32_t n_stages;   /* value tables per entry; 2 = {draft, refine} (Appendix A)          */
    int64_t capacity;   /* most entries the bank will ever hold, < 2^31                      */
    float q_default;    /* value given to stages an insert does not name                     */
    int32_t reserved;   /* must be 0                                                         */
    void *arena;        /* device memory, 256-byte aligned, evk_mem_bytes_required() bytes   */
    size_t arena_bytes;
} evk_config;

/* Bytes of device memory a bank of this shape needs (embeddings as bf16 rows
 * [capacity][d], value tables fp32 and update counts uint32 [n_stages][capacity], one live bit per
 * entry, a block of status and counter words).  0 if the config is invalid.  `arena` and `arena_bytes`
 * are ignored. */
size_t evk_mem_bytes_required(const evk_config *cfg);

/* Create an empty memory M_0 over the caller's arena (Eq. 1 starts from a seed
 * bank; seed entries are inserted like any other).  The arena is not cleared
 * except for the status word (one small async memset on the default stream,
 * followed by a synchronise).  The handle is host memory owned by the library
 * until evk_mem_destroy. */
int evk_mem_create(const evk_config *cfg, evk_mem **out);

/* Free the host-side handle.  Device memory stays the caller's. */
int evk_mem_destroy(evk_mem *mem);

/* Entries currently stored (host-side count, already including inserts that are
 * enqueued but not yet executed). */
int64_t evk_mem_size(const evk_mem *mem);

/* Choose the phase-1 kernel: AUTO (default) picks by batch size and shape,
 * STREAM forces the streaming kernel, TENSOR the tcgen05 kernel (retrieve then
 * returns EVK_ERR_UNSUPPORTED for shapes that kernel cannot take). */
int evk_mem_set_scoring(evk_mem *mem, int mode);

/* Choose how phase 2 mixes the two terms of its score.  The method ranks the pool by
 * Q_stage alone (Section 3.2) and normalises rewards only (Section 3.4), so neither mode
 * has a counterpart in the paper beyond w = 1 and w = 0:
 *   EVK_NORM_NONE (default)   score = (1-w)*sim + w*Q_stage[id];
 *   EVK_NORM_POOL_ZSCORE      each term is first replaced, per query, by its z-score over
 *                             the query's pool: z(x) = (x - mean) / std with the population
 *                             standard deviation of the pool's valid entries, and z = 0 for
 *                             a column whose std is <= 1e-6.  score = (1-w)*z(sim) + w*z(Q).
 *                             Statistics are taken in fp64, the score is rounded to fp32.
 * The order of the result is unchanged for w = 0 and w = 1 and under any positive affine
 * change of the value table.  Applies to evk_retrieve, evk_retrieve_host and
 * evk_retrieve_explore; evk_merge_shards always mixes raw terms.
 * Errors: EVK_ERR_INVALID for an unknown mode. */
int evk_mem_set_score_norm(evk_mem *mem, int mode);

/* Append n entries: M <- M ∪ {new items} (Eq. 1).  `emb` is [n][d] row-major,
 * fp32 (rounded to bf16, nearest-even) or bf16 (copied).  Entry ids are the
 * insertion indices size, size+1, ...; they are written to ids_out [n] if it is
 * not NULL.  `q_init` [n] (or NULL for q_default) seeds the value table of
 * `stage`, or of every stage with EVK_STAGE_ALL; other stages get q_default.
 * Embeddings are stored as given: the library does not normalise them.
 * Errors: EVK_ERR_CAPACITY (nothing is inserted), EVK_ERR_INVALID. */
int evk_mem_insert(evk_mem *mem, const void *emb, int emb_dtype, int64_t n, int stage,
                   const float *q_init, int32_t *ids_out, void *stream);

/* Workspace bytes evk_retrieve needs for a batch of B queries and pool size k1
 * at the bank's capacity (an upper bound for every size up to capacity). */
size_t evk_retrieve_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1);

/* Value-driven retrieval (Section 3.2) for B queries at one stage.
 *   phase 1: sim[b][i] = <query_b, e_i> (bf16 operands, fp32 accumulation) over
 *            all stored entries; the pool is the k1 entries of largest sim,
 *            ordered (sim descending, id ascending);
 *   phase 2: score = (1-w)*sim + w*Q_stage[id] over the pool; the result is the k2
 *            entries of largest score, ordered (score desc, sim desc, id asc).
 *            w = 1 ranks the pool by Q_stage alone, which is the rule the method
 *            states; w = 0 is similarity-only retrieval.
 * queries: [B][d] row-major, fp32 (rounded to bf16 first) or bf16.
 * ids_out [B][k2] int32, scores_out [B][k2] fp32; pool_ids_out / pool_sims_out
 * [B][k1] may be NULL.  If fewer than k1 (k2) entries exist, the pool (result) is
 * padded with id -1 and score -inf; an empty bank is not an error.
 * Limits: 1 <= k2 <= k1 <= EVK_MAX_K1, 0 <= w <= 1, B >= 0.
 * The workspace must hold evk_retrieve_workspace_bytes(mem, B, k1) bytes, 256-byte
 * aligned; its contents are scratch and calls sharing one workspace must not
 * overlap on the device. */
int evk_retrieve(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage,
                 int32_t k1, int32_t k2, float w,
                 int32_t *ids_out, float *scores_out,
                 int32_t *pool_ids_out, float *pool_sims_out,
                 void *workspace, size_t workspace_bytes, void *stream);

/* Workspace bytes evk_q_update needs for a batch of M updates. */
size_t evk_q_update_workspace_bytes(const evk_mem *mem, int64_t M);

/* Unified value update (Eq. 4): for t = 0..M-1 in array order,
 *   Q_stage[ids[t]] <- Q + alpha * (rewards[t] - Q)
 * in binary32 as a subtraction, a multiplication and an addition, each rounded to
 * nearest on its own (no fused multiply-add).  An id that occurs several times
 * receives its updates one after another in array order, so the stored bits equal
 * those of the sequential loop and do not depend on how the batch is split across
 * calls.  0 < alpha <= 1.  Ids outside [0, size) or non-finite rewards make the
 * whole call a no-op and set the status word (EVK_ERR_RANGE / EVK_ERR_NONFINITE).
 * The workspace must hold evk_q_update_workspace_bytes(mem, M) bytes. */
int evk_q_update(evk_mem *mem, const int32_t *ids, int64_t M, int stage,
                 const float *rewards, float alpha,
                 void *workspace, size_t workspace_bytes, void *stream);

/* evk_q_update for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of the library.)
 *
 * Some hosts of this library cannot call cudaMalloc or grow a memory pool while
 * they work: a serving loop whose device memory was carved up once at start-up and
 * is fully spoken for, a plug-in running inside another framework's memory budget,
 * a latency-critical section where an allocation (which may synchronise the device
 * or fail) is not acceptable.  For them the scratch that the update's sort needs
 * lives in a fixed array inside the library image instead of a caller workspace.
 *
 * Same arithmetic, order and error behaviour as evk_q_update; results are
 * bit-identical.  Differences:
 *   - M <= EVK_Q_UPDATE_STATIC_MAX; a larger batch returns EVK_ERR_UNSUPPORTED and
 *     does nothing (split it: consecutive calls give the same bits as one call).
 *   - About 1.06 MB of device memory is reserved on every GPU that loads the
 *     library, for the life of the process, whether or not this call is used.
 *   - The first call on each device looks up the array's device address (with that
 *     device current, which it must be at every call); make that first call before
 *     any stream capture begins.  The call itself allocates and frees nothing.  The address is
 *     remembered per device ordinal (ordinals 0..63; a higher one returns EVK_ERR_CUDA) for the
 *     life of the process: after cudaDeviceReset, or anything else that destroys the device's
 *     primary context, it is stale and this call must not be used again in that process.
 *   - Every call on a device shares the one array.  Calls are safe one after
 *     another on one stream; two calls whose kernels can overlap on the GPU
 *     (different streams without ordering) race on the scratch and corrupt each
 *     other.  The array keeps the previous call's contents; the kernels clear or
 *     overwrite everything they read.
 * `ids` and `rewards` are device arrays as in evk_q_update. */
enum { EVK_Q_UPDATE_STATIC_MAX = 65536 };
int evk_q_update_static(evk_mem *mem, const int32_t *ids, int64_t M, int stage,
                        const float *rewards, float alpha, void *stream);

/* The value update with a decreasing step size (Appendix A, Eq. 8 with alpha_t under the
 * Robbins-Monro conditions): alpha_t = 1 / (number of decay updates the entry has received at
 * this stage, this one included), so the stored value is the running mean of those rewards and
 * the first such update replaces the initial value.  Same ordering, arithmetic (alpha_t by
 * IEEE division in binary32, then subtract / multiply / add), checks and workspace as
 * evk_q_update.  The per-entry counts live in the arena, start at 0 at insert, are advanced
 * only by this call, and can be read with evk_visits_read (uint32 [n]). */
int evk_q_update_decay(evk_mem *mem, const int32_t *ids, int64_t M, int stage, const float *rewards,
                       void *workspace, size_t workspace_bytes, void *stream);
int evk_visits_read(evk_mem *mem, int stage, int64_t first, int64_t n, uint32_t *out, void *stream);
int evk_visits_write(evk_mem *mem, int stage, int64_t first, int64_t n, const uint32_t *values, void *stream);

/* Copy Q_stage[first .. first+n) to / from a device array. */
int evk_q_read(evk_mem *mem, int stage, int64_t first, int64_t n, float *out, void *stream);
int evk_q_write(evk_mem *mem, int stage, int64_t first, int64_t n, const float *values, void *stream);

/* Copy the stored bf16 rows [first .. first+n) to a device array [n][d] of uint16. */
int evk_bank_read(evk_mem *mem, int64_t first, int64_t n, void *out_bf16, void *stream);

/* Dropping entries from a live memory.  The memory of Eq. 1 only grows, but the method also hands
 * a FILTERED bank on (Experiment section, transfer across backbones: a bank from which entries were
 * removed initialises another generator's run), so entries can be taken out without rebuilding the
 * bank.  Every id in ids [n] (device) loses its place: no retrieval on this stream after this call
 * returns it, it takes no slot of a pool, and evk_select_by_value skips it.  The other entries keep
 * their ids; the dropped entry's row and values stay in the arena (an update that names it is
 * applied and never seen).  Naming an id twice, or one that was dropped before, is harmless.  If
 * any id is outside [0, size) the whole call does nothing and the status word becomes EVK_ERR_RANGE.
 * A pool is then as long as min(k1, live entries).  There is no way to bring an entry back. */
int evk_mem_tombstone(evk_mem *mem, const int32_t *ids, int64_t n, void *stream);

/* Carrying a memory from one run into the next (Experiment section: the bank learned on one level
 * of tasks initialises the run on the next; a bank is handed to other generators).
 * evk_mem_export copies entries [first, first + n) out to caller buffers on the device, any of
 * which may be NULL: rows_bf16 [n][d] (uint16 bit patterns), q [n_stages][n], visits
 * [n_stages][n] (the counts of evk_q_update_decay), live [n] (1 = in the memory, 0 = dropped).
 * evk_mem_import appends n entries from such buffers: rows are required; NULL q / visits / live
 * mean q_default / 0 / all live.  Entries marked 0 in `live` keep their place (ids are positions)
 * but are dropped at once; a caller that wants a compact bank leaves them out of the buffers.
 * ids_out [n] (may be NULL) receives the new ids.  Errors: EVK_ERR_INVALID (range, null rows),
 * EVK_ERR_CAPACITY (nothing is imported). */
int evk_mem_export(evk_mem *mem, int64_t first, int64_t n, void *rows_bf16, float *q, uint32_t *visits,
                   uint8_t *live, void *stream);
int evk_mem_import(evk_mem *mem, int64_t n, const void *rows_bf16, const float *q, const uint32_t *visits,
                   const uint8_t *live, int32_t *ids_out, void *stream);

/* Counters of one bank (no counterpart in the paper: they explain a slow batch in the field).
 * Synchronises `stream`.  candidates_filed: (similarity, id) pairs the tensor-core scans left in
 * their candidate lists for the merge, summed over all retrievals (k1 per query is the least
 * possible); list_cutbacks: times such a list filled up and was cut back to its best k1 (only
 * adversarial row orders cause it); longest_update_run: the most updates one entry received in a
 * single batch (runs of more than 8), which one thread or warp has to apply one after another. */
typedef struct evk_stats {
    int64_t entries, live_entries, dropped_entries;
    int64_t retrieve_calls, update_calls, insert_calls, kernel_launches;
    int64_t candidates_filed, list_cutbacks, longest_update_run;
} evk_stats;
int evk_mem_stats(evk_mem *mem, evk_stats *out, void *stream);

/* Host-buffer forms of the three hot calls, for callers whose data lives in host memory (the
 * loop of Section 3.2 is driven from the host: queries, rewards and new entries arrive there).
 * They copy the inputs to the device and run the same kernels.  Every host-side check of the
 * device-pointer form is made before anything is copied.  `workspace` is DEVICE memory of the
 * *_host_workspace_bytes amount (staging plus the kernel workspace), 256-byte aligned.
 *
 * Without a staging buffer each call synchronises the stream before it returns (the caller's
 * arrays may be pageable; they are the caller's again on return whatever the outcome).
 *
 * evk_mem_set_host_staging hands the library a page-locked, device-visible host buffer
 * (cudaHostAlloc / cudaHostRegister memory; 256-byte aligned, at least 16 KB; it stays the
 * caller's and must outlive the handle or be withdrawn with pinned_host = NULL, which waits for
 * the work that still reads it).  It is cut into four slots used in turn.  Then, for inputs that
 * fit one slot:
 *   - evk_q_update_host and evk_mem_insert_host copy the caller's arrays into a slot (host
 *     memcpy), enqueue the transfer and the kernels, and return WITHOUT waiting for the device:
 *     the caller's arrays are free on return, and what the device finds (an id out of range)
 *     reaches the status word exactly as with evk_q_update;
 *   - evk_retrieve_host lets the merge kernel write ids and scores straight into a slot, waits
 *     for the stream, and copies them to ids_out_host / scores_out_host.
 * Larger inputs take the path without staging.  EVK_ERR_INVALID if the buffer is not page-locked
 * host memory the device can address.  evk_mem_insert_host assigns ids like evk_mem_insert (the
 * next n ids in row order) and does not return them. */
int evk_mem_set_host_staging(evk_mem *mem, void *pinned_host, size_t bytes);
size_t evk_retrieve_host_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1, int32_t k2);
int evk_retrieve_host(evk_mem *mem, const void *queries_host, int q_dtype, int32_t B, int stage,
                      int32_t k1, int32_t k2, float w,
                      int32_t *ids_out_host, float *scores_out_host,
                      void *workspace, size_t workspace_bytes, void *stream);
size_t evk_q_update_host_workspace_bytes(const evk_mem *mem, int64_t M);
int evk_q_update_host(evk_mem *mem, const int32_t *ids_host, int64_t M, int stage,
                      const float *rewards_host, float alpha,
                      void *workspace, size_t workspace_bytes, void *stream);
size_t evk_mem_insert_host_workspace_bytes(const evk_mem *mem, int64_t n);
int evk_mem_insert_host(evk_mem *mem, const void *emb_host, int emb_dtype, int64_t n, int stage,
                        const float *q_init_host, void *workspace, size_t workspace_bytes, void *stream);

/* evk_retrieve with epsilon-greedy exploration (Section 3.3: the context is drawn from the
 * pool with an epsilon-greedy policy over the stage's values).  Per query, word 0 of a
 * Philox4x32-10 stream keyed by (seed; counter = query index, step, block) gives
 * u = (word >> 8) * 2^-24; if u < epsilon the query explores: its result is min(k2, n) entries
 * of its pool (n = pool length) drawn uniformly without replacement — a partial Fisher-Yates
 * shuffle of the pool positions in (sim desc, id asc) order, position i swapped with
 * i + floor(word_{i+1} * (n - i) / 2^32) — written in draw order with their mixed scores.
 * Other queries get the greedy result of evk_retrieve.  The draw depends only on (seed,
 * step, query index): pass a new `step` for every call of an episode.  explored_out [B]
 * (may be NULL) receives 1 for queries that explored.  epsilon in [0, 1]; epsilon = 0 is
 * evk_retrieve.  Workspace: evk_retrieve_explore_workspace_bytes(mem, B, k1). */
size_t evk_retrieve_explore_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1);
int evk_retrieve_explore(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage,
                         int32_t k1, int32_t k2, float w, float epsilon, uint64_t seed, uint64_t step,
                         int32_t *ids_out, float *scores_out, uint8_t *explored_out,
                         int32_t *pool_ids_out, float *pool_sims_out,
                         void *workspace, size_t workspace_bytes, void *stream);

/* Start-point selection by value (Section 3.4: among the feasible kernels P(x) of a task,
 * the next start point is chosen with Q_2).  Task t owns the candidate entry ids
 * cand_ids[offsets[t] .. offsets[t+1]) (device arrays; offsets has n_tasks + 1 elements; ids
 * distinct within a task, at most 4096 per task).  For every task the k candidates of largest
 * Q_stage are written to ids_out / q_out [n_tasks][k], ordered (Q descending, id ascending),
 * padded with id -1 / -inf.  1 <= k <= EVK_MAX_K1.  An id outside [0, size) sets
 * EVK_ERR_RANGE, a task longer than 4096 EVK_ERR_UNSUPPORTED (status word; that task's row is
 * all padding). */
int evk_select_by_value(evk_mem *mem, const int32_t *cand_ids, const int32_t *offsets, int32_t n_tasks, int stage,
                        int32_t k, int32_t *ids_out, float *q_out, void *stream);

/* A bank split by rows over several GPUs (one process and one evk_mem per GPU).  Shard g
 * stores the entries with global ids [id_offset_g, id_offset_g + size_g) and their values.
 *
 * evk_retrieve_local: phase 1 on this shard for all B queries, each candidate tagged with its
 *   global id (local id + id_offset) and its Q_stage: gids_out / sims_out / q_out [B][k1],
 *   ordered (sim desc, id asc), padded with gid -1, sim -inf, q 0.
 * evk_merge_shards: gids / sims / qs are the gathered outputs of all shards, [n_shards][B][k1],
 *   shards in ascending id-range order (the caller gathers them, e.g. with an all-gather; the
 *   arrays are in this GPU's own memory).  Per query: the k1 best of the n_shards * k1
 *   candidates (sim desc, global id asc) — the pool one unsplit bank would give — then phase 2
 *   with the values that came along: ids_out (global ids) / scores_out [B][k2], and optionally
 *   the merged pool [B][k1].  Needs no handle and no workspace.
 * Updates: each shard applies, in array order, the (id, reward) pairs whose id it owns. */
size_t evk_retrieve_local_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1);
int evk_retrieve_local(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage, int32_t k1,
                       int32_t id_offset, int32_t *gids_out, float *sims_out, float *q_out,
                       void *workspace, size_t workspace_bytes, void *stream);
int evk_merge_shards(const int32_t *gids, const float *sims, const float *qs, int32_t n_shards, int32_t B,
                     int32_t k1, int32_t k2, float w, int32_t *ids_out, float *scores_out,
                     int32_t *pool_gids_out, float *pool_sims_out, void *stream);

/* Rewards for evk_q_update.  All arrays are device arrays of n elements.
 *
 * evk_reward_draft (Eq. 5): +1 where feasible[i] != 0, else -1.
 * evk_reward_refine (Eq. 6): -1 where infeasible, else tanh(log best_latency[i] - log latency[i])
 *   (best_latency = the best latency seen before this attempt; latencies must be > 0).
 * evk_reward_normalize (Appendix A, running normalisation): replaces raw reward r_t by
 *   (r_t - mu_{t-1}) / max(sigma_{t-1}, sigma_min), clipped to [-clip, clip] if clip > 0, where
 *   mu and sigma are the mean and population standard deviation of every raw reward that went
 *   through `state` before r_t (earlier calls and earlier elements of this call, in array
 *   order).  The first two rewards ever seen pass through unchanged.  Stored values are not
 *   rescaled when the statistics move.  `state` is evk_reward_norm_state_bytes() bytes of
 *   device memory, 8-byte aligned, owned by the caller, zeroed by evk_reward_norm_reset; calls
 *   sharing a state must be ordered on one stream.  sigma_min > 0, clip >= 0 (0 = no clipping). */
int evk_reward_draft(const uint8_t *feasible, int64_t n, float *rewards_out, void *stream);
int evk_reward_refine(const float *best_latency, const float *latency, const uint8_t *feasible, int64_t n,
                      float *rewards_out, void *stream);
size_t evk_reward_norm_state_bytes(void);
int evk_reward_norm_reset(void *state, void *stream);
int evk_reward_normalize(void *state, const float *raw, int64_t n, float sigma_min, float clip,
                         float *rewards_out, void *stream);

/* What evk_retrieve would run for a batch of B queries at the current size: the
 * phase-1 kernel (EVK_SCORING_STREAM or EVK_SCORING_TENSOR) and how many times it
 * is launched (each launch scans the whole bank once). */
int evk_retrieve_plan(const evk_mem *mem, int32_t B, int32_t k1, int32_t *kind_out, int32_t *launches_out);

/* Timing aid: the next evk_retrieve on this handle records `start_event` right
 * before its phase-1 scoring launches and `stop_event` right after them, on that
 * call's stream.  Both are cudaEvent_t owned by the caller, passed as void*.  The
 * setting is used by one call and then cleared; NULLs clear it. */
int evk_mem_profile_scoring(evk_mem *mem, void *start_event, void *stop_event);

/* Measurement aid (no counterpart in the paper): reads the stored rows once, 32 KB at a time, into
 * shared memory with the copy engine the scans use, and drops them: one kernel on `stream`.  Timed
 * by the caller, bytes = size * d * 2 over its duration is the read-only bandwidth of this GPU, the
 * ceiling of a scan (a copy's measured bandwidth counts reads and writes and lies below it). */
int evk_mem_read_probe(evk_mem *mem, void *stream);

/* Failure-detection test aid.  The next evk_retrieve that runs the tensor kernel starves its
 * own pipeline: the producer warp issues no loads, so the consumer's bounded wait (shortened to
 * about a tenth of a second for this call) runs out.  Nothing faults or hangs: every block
 * raises its abort flag, releases tensor memory and returns, the status word becomes
 * EVK_ERR_DEVICE_TIMEOUT, that call's outputs are padding, and the handle stays usable. */
int evk_mem_inject_stall(evk_mem *mem);

/* Synchronise `stream`, return the device status word (EVK_OK or the first
 * device-detected error since the last read) and clear it. */
int evk_last_status(evk_mem *mem, void *stream);

/* Number of kernels this handle has launched so far (host-side counter). */
int64_t evk_launch_count(const evk_mem *mem);

/* A static, human-readable name for a status code. */
const char *evk_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* EVK_H_ */
