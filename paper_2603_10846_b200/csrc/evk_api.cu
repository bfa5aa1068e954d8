// The C ABI (include/evk.h): argument checks, memory layout, kernel dispatch.
#include <math.h>
#include <mutex>
#include <new>
#include <string.h>

#include "evk_common.cuh"
#include "evk_kernels.cuh"

using namespace evk;

namespace evk {
int num_sms() {
    constexpr int kFallback = 148, kMaxDev = 64;
    static std::mutex mu;
    static int cache[kMaxDev];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) {
        (void)cudaGetLastError();
        return kFallback;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 2) n = kFallback;
        cache[dev] = n;
    }
    return cache[dev];
}
}  // namespace evk

struct evk_mem {
    evk_config cfg;
    int64_t size;
    __nv_bfloat16 *bank;  // [capacity][d]
    float *q_tables;      // [n_stages][capacity]
    uint32_t *visits;     // [n_stages][capacity] updates received (decreasing step size)
    uint32_t *live_bits;  // [ceil(capacity / 32)] one bit per entry: 1 = in the memory, 0 = dropped
    int32_t *status;      // device status word (word 0 of the device block)
    uint32_t *dev;        // the device block as words: live count, counters (see DevWord)
    int any_dropped;      // an entry may have been dropped: the scans consult the live bits
    int64_t n_retrieve, n_update, n_insert;   // calls that enqueued work
    int scoring;
    int score_norm;       // EVK_NORM_*: how phase 2 mixes similarity and value
    int stall_next;       // evk_mem_inject_stall: the next tensor-path retrieve starves its consumer
    int64_t launches;
    cudaEvent_t prof_start, prof_stop;  // armed by evk_mem_profile_scoring for one retrieve
    // the caller's page-locked staging buffer (evk_mem_set_host_staging), cut into slots used in turn;
    // a slot's event marks the end of the device work that reads it
    char *stage_host;     // host address of slot 0, nullptr = none
    char *stage_dev;      // the same memory as the device sees it
    size_t slot_bytes;
    int slot_next;
    bool slot_busy[4];
    cudaEvent_t slot_ev[4];
};

namespace {

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct ArenaLayout {
    size_t bank, q_tables, visits, live_bits, status, total;
};

bool config_ok(const evk_config *c) {
    return c && c->d > 0 && c->d % 8 == 0 && c->d <= EVK_MAX_D && c->n_stages >= 1 &&
           c->n_stages <= EVK_MAX_STAGES && c->capacity >= 1 && c->capacity < ((int64_t)1 << 31) &&
           c->reserved == 0 && isfinite(c->q_default);
}

ArenaLayout arena_layout(const evk_config *c) {
    ArenaLayout l;
    l.bank = 0;
    l.q_tables = align256((size_t)c->capacity * c->d * sizeof(__nv_bfloat16));
    l.visits = l.q_tables + align256((size_t)c->n_stages * c->capacity * sizeof(float));
    l.live_bits = l.visits + align256((size_t)c->n_stages * c->capacity * sizeof(uint32_t));
    l.status = l.live_bits + align256((size_t)((c->capacity + 31) / 32) * sizeof(uint32_t));
    l.total = l.status + 256;
    return l;
}

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Which phase-1 kernel a batch goes to: EVK_SCORING_STREAM, EVK_SCORING_TENSOR, or 0 if the
// forced kernel cannot take the shape.
int pick_kind(const evk_mem *m, int32_t B, int32_t k1) {
    const bool tensor_ok = mma_supported(m->cfg.d, k1);
    const bool stream_ok = stream_supported(m->cfg.d);
    if (m->scoring == EVK_SCORING_STREAM) return stream_ok ? EVK_SCORING_STREAM : 0;
    if (m->scoring == EVK_SCORING_TENSOR) return tensor_ok ? EVK_SCORING_TENSOR : 0;
    // measured on B200: the tensor kernel scans at the same speed as the streaming kernel for one
    // query and its candidate lists are far shorter, so it takes every batch it supports
    if (tensor_ok) return EVK_SCORING_TENSOR;
    return stream_ok ? EVK_SCORING_STREAM : (tensor_ok ? EVK_SCORING_TENSOR : 0);
}

struct RetrieveLayout {
    size_t q_bf16, scratch, total;
    size_t part_counts, part_keys;  // streaming kernel only, inside scratch
    int nparts_max;
};

RetrieveLayout retrieve_layout(const evk_mem *m, int32_t B, int32_t k1, int kind) {
    RetrieveLayout l;
    const size_t b = (size_t)(B > 0 ? B : 0);
    l.q_bf16 = 0;
    l.scratch = l.q_bf16 + align256(b * m->cfg.d * sizeof(__nv_bfloat16));
    l.part_counts = l.part_keys = 0;
    l.nparts_max = 0;
    size_t scratch_bytes = 256;
    if (kind == EVK_SCORING_TENSOR) {
        scratch_bytes = mma_workspace_bytes(B);
    } else if (kind == EVK_SCORING_STREAM) {
        const StreamPlan plan = stream_plan(m->cfg.capacity, m->cfg.d, B, k1);
        l.nparts_max = plan.nparts;
        l.part_counts = l.scratch;
        l.part_keys = l.part_counts + align256(b * l.nparts_max * sizeof(int));
        scratch_bytes = (l.part_keys - l.scratch) + align256(b * l.nparts_max * (size_t)k1 * sizeof(uint64_t));
    }
    l.total = l.scratch + scratch_bytes;
    return l;
}

bool stage_ok(const evk_mem *m, int stage) { return stage >= 0 && stage < m->cfg.n_stages; }

int cuda_status(cudaError_t e) { return e == cudaSuccess ? EVK_OK : EVK_ERR_CUDA; }

constexpr int kHostSlots = 4;

// The next staging slot, once the device work that read it last has ended.  -1 if that wait fails.
int acquire_slot(evk_mem *m) {
    const int s = m->slot_next;
    m->slot_next = (s + 1) % kHostSlots;
    if (m->slot_busy[s]) {
        if (cudaEventSynchronize(m->slot_ev[s]) != cudaSuccess) return -1;
        m->slot_busy[s] = false;
    }
    return s;
}

// Marks the slot as read by everything enqueued on `stream` so far.
bool release_slot_after(evk_mem *m, int s, cudaStream_t stream) {
    if (cudaEventRecord(m->slot_ev[s], stream) != cudaSuccess) return false;
    m->slot_busy[s] = true;
    return true;
}

void drop_staging(evk_mem *m) {
    if (!m->stage_host) return;
    for (int s = 0; s < kHostSlots; ++s) {
        if (m->slot_busy[s]) (void)cudaEventSynchronize(m->slot_ev[s]);
        (void)cudaEventDestroy(m->slot_ev[s]);
        m->slot_busy[s] = false;
    }
    m->stage_host = m->stage_dev = nullptr;
    m->slot_bytes = 0;
}

}  // namespace

extern "C" {

size_t evk_mem_bytes_required(const evk_config *cfg) {
    if (!config_ok(cfg)) return 0;
    return arena_layout(cfg).total;
}

int evk_mem_create(const evk_config *cfg, evk_mem **out) {
    if (!out) return EVK_ERR_INVALID;
    *out = nullptr;
    if (!config_ok(cfg) || !cfg->arena || !aligned(cfg->arena, 256)) return EVK_ERR_INVALID;
    const ArenaLayout l = arena_layout(cfg);
    if (cfg->arena_bytes < l.total) return EVK_ERR_WORKSPACE;
    evk_mem *m = new (std::nothrow) evk_mem;
    if (!m) return EVK_ERR_INVALID;
    m->cfg = *cfg;
    m->size = 0;
    char *base = static_cast<char *>(cfg->arena);
    m->bank = reinterpret_cast<__nv_bfloat16 *>(base + l.bank);
    m->q_tables = reinterpret_cast<float *>(base + l.q_tables);
    m->visits = reinterpret_cast<uint32_t *>(base + l.visits);
    m->live_bits = reinterpret_cast<uint32_t *>(base + l.live_bits);
    m->status = reinterpret_cast<int32_t *>(base + l.status);
    m->dev = reinterpret_cast<uint32_t *>(base + l.status);
    m->any_dropped = 0;
    m->n_retrieve = m->n_update = m->n_insert = 0;
    m->scoring = EVK_SCORING_AUTO;
    m->score_norm = EVK_NORM_NONE;
    m->stall_next = 0;
    m->launches = 0;
    m->prof_start = m->prof_stop = nullptr;
    m->stage_host = m->stage_dev = nullptr;
    m->slot_bytes = 0;
    m->slot_next = 0;
    for (int s = 0; s < kHostSlots; ++s) m->slot_busy[s] = false;
    cudaError_t err = cudaMemsetAsync(m->status, 0, 256, 0);
    if (err == cudaSuccess) err = cudaStreamSynchronize(0);
    if (err != cudaSuccess) {
        delete m;
        return EVK_ERR_CUDA;
    }
    *out = m;
    return EVK_OK;
}

int evk_mem_destroy(evk_mem *mem) {
    if (mem) drop_staging(mem);
    delete mem;
    return EVK_OK;
}

int evk_mem_set_host_staging(evk_mem *mem, void *pinned_host, size_t bytes) {
    if (!mem) return EVK_ERR_INVALID;
    if (!pinned_host) {
        drop_staging(mem);
        return EVK_OK;
    }
    if (!aligned(pinned_host, 256) || bytes / kHostSlots < 4096) return EVK_ERR_INVALID;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, pinned_host) != cudaSuccess) {
        (void)cudaGetLastError();
        return EVK_ERR_INVALID;
    }
    // page-locked and visible to the device: the result of a retrieval is written straight into it
    if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) return EVK_ERR_INVALID;
    drop_staging(mem);
    for (int s = 0; s < kHostSlots; ++s) {
        if (cudaEventCreateWithFlags(&mem->slot_ev[s], cudaEventDisableTiming) != cudaSuccess) {
            for (int t = 0; t < s; ++t) (void)cudaEventDestroy(mem->slot_ev[t]);
            return EVK_ERR_CUDA;
        }
    }
    mem->stage_host = static_cast<char *>(pinned_host);
    mem->stage_dev = static_cast<char *>(attr.devicePointer);
    mem->slot_bytes = (bytes / kHostSlots) & ~(size_t)255;
    mem->slot_next = 0;
    return EVK_OK;
}

int64_t evk_mem_size(const evk_mem *mem) { return mem ? mem->size : 0; }

int64_t evk_launch_count(const evk_mem *mem) { return mem ? mem->launches : 0; }

int evk_mem_inject_stall(evk_mem *mem) {
    if (!mem) return EVK_ERR_INVALID;
    mem->stall_next = 1;
    return EVK_OK;
}

int evk_mem_set_score_norm(evk_mem *mem, int mode) {
    if (!mem || (mode != EVK_NORM_NONE && mode != EVK_NORM_POOL_ZSCORE)) return EVK_ERR_INVALID;
    mem->score_norm = mode;
    return EVK_OK;
}

int evk_mem_set_scoring(evk_mem *mem, int mode) {
    if (!mem || mode < EVK_SCORING_AUTO || mode > EVK_SCORING_TENSOR) return EVK_ERR_INVALID;
    mem->scoring = mode;
    return EVK_OK;
}

int evk_mem_insert(evk_mem *mem, const void *emb, int emb_dtype, int64_t n, int stage,
                   const float *q_init, int32_t *ids_out, void *stream) {
    if (!mem || n < 0 || (emb_dtype != EVK_DTYPE_F32 && emb_dtype != EVK_DTYPE_BF16)) return EVK_ERR_INVALID;
    if (stage != EVK_STAGE_ALL && !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!emb || !aligned(emb, 16)) return EVK_ERR_INVALID;
    if (mem->size + n > mem->cfg.capacity) return EVK_ERR_CAPACITY;
    int launches = 0;
    cudaError_t err = launch_insert(mem->bank, mem->q_tables, mem->visits, mem->live_bits, mem->dev, mem->cfg.capacity, mem->cfg.d,
                                    mem->cfg.n_stages, mem->size, n, emb, emb_dtype, stage, q_init,
                                    mem->cfg.q_default, ids_out, static_cast<cudaStream_t>(stream), &launches);
    mem->launches += launches;
    if (err != cudaSuccess) return EVK_ERR_CUDA;
    mem->size += n;
    ++mem->n_insert;
    return EVK_OK;
}

size_t evk_retrieve_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1) {
    if (!mem || B < 0 || k1 < 1 || k1 > EVK_MAX_K1) return 0;
    return retrieve_layout(mem, B, k1, pick_kind(mem, B, k1)).total + 256;
}

int evk_retrieve(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage,
                 int32_t k1, int32_t k2, float w,
                 int32_t *ids_out, float *scores_out,
                 int32_t *pool_ids_out, float *pool_sims_out,
                 void *workspace, size_t workspace_bytes, void *stream_v) {
    if (!mem || B < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (k1 < 1 || k1 > EVK_MAX_K1 || k2 < 1 || k2 > k1) return EVK_ERR_INVALID;
    if (!(w >= 0.0f && w <= 1.0f)) return EVK_ERR_INVALID;
    if (q_dtype != EVK_DTYPE_F32 && q_dtype != EVK_DTYPE_BF16) return EVK_ERR_INVALID;
    if (B == 0) return EVK_OK;
    if (!queries || !aligned(queries, 16) || !ids_out || !scores_out) return EVK_ERR_INVALID;
    if (!workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    const int kind = pick_kind(mem, B, k1);
    if (kind == 0) return EVK_ERR_UNSUPPORTED;
    const RetrieveLayout l = retrieve_layout(mem, B, k1, kind);
    if (workspace_bytes < l.total) return EVK_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    char *ws = static_cast<char *>(workspace);
    int launches = 0;
    cudaError_t err = cudaSuccess;

    const __nv_bfloat16 *q_bf16 = static_cast<const __nv_bfloat16 *>(queries);
    if (q_dtype == EVK_DTYPE_F32) {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(ws + l.q_bf16);
        err = launch_convert_queries(static_cast<const float *>(queries), dst, (int64_t)B * mem->cfg.d, stream, &launches);
        q_bf16 = dst;
    }

    cudaEvent_t ev_start = mem->prof_start, ev_stop = mem->prof_stop;
    mem->prof_start = mem->prof_stop = nullptr;

    // phase 1: per-(query, part) candidate lists, then one merge per query
    const uint64_t *part_keys = nullptr;
    const int *part_counts = nullptr;
    int nparts = 0, part_stride = k1, qt_size = 1;
    if (err == cudaSuccess && mem->size > 0) {
        if (kind == EVK_SCORING_TENSOR) {
            MmaPlan plan = mma_plan(mem->size, B, k1);
            plan.stall = mem->stall_next;
            mem->stall_next = 0;
            plan.live_bits = mem->any_dropped ? mem->live_bits : nullptr;
            plan.dev = mem->dev;
            plan.wait_queries = q_dtype == EVK_DTYPE_F32 ? 1 : 0;
            uint64_t *cand = nullptr;
            int *cand_cnt = nullptr;
            err = launch_score_mma(mem->bank, mem->size, mem->cfg.capacity, mem->cfg.d, q_bf16, B, k1, plan,
                                   ws + l.scratch, mem->status, &cand, &cand_cnt, ev_start, ev_stop, stream, &launches);
            part_keys = cand;
            part_counts = cand_cnt;
            nparts = plan.splits;
            part_stride = kMmaCandCap;
            qt_size = 128;
        } else {
            StreamPlan plan = stream_plan(mem->size, mem->cfg.d, B, k1);
            plan.live_bits = mem->any_dropped ? mem->live_bits : nullptr;
            uint64_t *keys = reinterpret_cast<uint64_t *>(ws + l.part_keys);
            int *counts = reinterpret_cast<int *>(ws + l.part_counts);
            if (ev_start) err = cudaEventRecord(ev_start, stream);
            if (err == cudaSuccess)
                err = launch_score_stream(mem->bank, mem->size, mem->cfg.d, q_bf16, B, k1, plan, keys, counts,
                                          stream, &launches);
            if (err == cudaSuccess && ev_stop) err = cudaEventRecord(ev_stop, stream);
            part_keys = keys;
            part_counts = counts;
            nparts = plan.nparts;
        }
    }
    const int expect = (int)(mem->size < k1 ? mem->size : k1);
    if (err == cudaSuccess)
        err = launch_merge_rerank(part_keys, part_counts, nparts, part_stride, qt_size, B, k1, expect,
                                  mem->any_dropped ? mem->dev + kDevLive : nullptr, mem->status,
                                  pool_ids_out, pool_sims_out, k2,
                                  mem->q_tables + (size_t)stage * mem->cfg.capacity, w, mem->score_norm, ids_out,
                                  scores_out, stream, &launches);
    mem->launches += launches;
    ++mem->n_retrieve;
    return cuda_status(err);
}

int evk_retrieve_plan(const evk_mem *mem, int32_t B, int32_t k1, int32_t *kind_out, int32_t *launches_out) {
    if (!mem || B < 0 || k1 < 1 || k1 > EVK_MAX_K1 || !kind_out || !launches_out) return EVK_ERR_INVALID;
    const int kind = pick_kind(mem, B, k1);
    if (kind == 0) return EVK_ERR_UNSUPPORTED;
    *kind_out = kind;
    if (mem->size <= 0 || B <= 0) {
        *launches_out = 0;
    } else if (kind == EVK_SCORING_TENSOR) {
        *launches_out = 1;
    } else {
        const StreamPlan plan = stream_plan(mem->size, mem->cfg.d, B, k1);
        *launches_out = (B + plan.qb - 1) / plan.qb;
    }
    return EVK_OK;
}

int evk_mem_profile_scoring(evk_mem *mem, void *start_event, void *stop_event) {
    if (!mem) return EVK_ERR_INVALID;
    mem->prof_start = static_cast<cudaEvent_t>(start_event);
    mem->prof_stop = static_cast<cudaEvent_t>(stop_event);
    return EVK_OK;
}

size_t evk_q_update_workspace_bytes(const evk_mem *mem, int64_t M) {
    if (!mem || M < 0) return 0;
    return q_update_workspace_bytes(M) + 256;
}

int evk_q_update(evk_mem *mem, const int32_t *ids, int64_t M, int stage,
                 const float *rewards, float alpha,
                 void *workspace, size_t workspace_bytes, void *stream) {
    if (!mem || M < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (!(alpha > 0.0f && alpha <= 1.0f)) return EVK_ERR_INVALID;
    if (M == 0) return EVK_OK;
    if (M >= ((int64_t)1 << 31)) return EVK_ERR_UNSUPPORTED;
    if (!ids || !rewards || !workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (workspace_bytes < q_update_workspace_bytes(M)) return EVK_ERR_WORKSPACE;
    int launches = 0;
    cudaError_t err = launch_q_update(mem->q_tables + (size_t)stage * mem->cfg.capacity, mem->size, ids, rewards,
                                      M, alpha, nullptr, mem->status, workspace, static_cast<cudaStream_t>(stream),
                                      &launches, mem->dev + kDevLongestRun);
    mem->launches += launches;
    ++mem->n_update;
    return cuda_status(err);
}

int evk_q_update_decay(evk_mem *mem, const int32_t *ids, int64_t M, int stage, const float *rewards,
                       void *workspace, size_t workspace_bytes, void *stream) {
    if (!mem || M < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (M == 0) return EVK_OK;
    if (M >= ((int64_t)1 << 31)) return EVK_ERR_UNSUPPORTED;
    if (!ids || !rewards || !workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (workspace_bytes < q_update_workspace_bytes(M)) return EVK_ERR_WORKSPACE;
    int launches = 0;
    const size_t off = (size_t)stage * mem->cfg.capacity;
    cudaError_t err = launch_q_update(mem->q_tables + off, mem->size, ids, rewards, M, 1.0f, mem->visits + off,
                                      mem->status, workspace, static_cast<cudaStream_t>(stream), &launches,
                                      mem->dev + kDevLongestRun);
    mem->launches += launches;
    ++mem->n_update;
    return cuda_status(err);
}

int evk_visits_write(evk_mem *mem, int stage, int64_t first, int64_t n, const uint32_t *values, void *stream) {
    if (!mem || !stage_ok(mem, stage) || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!values) return EVK_ERR_INVALID;
    return cuda_status(cudaMemcpyAsync(mem->visits + (size_t)stage * mem->cfg.capacity + first, values,
                                       (size_t)n * sizeof(uint32_t), cudaMemcpyDeviceToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

int evk_visits_read(evk_mem *mem, int stage, int64_t first, int64_t n, uint32_t *out, void *stream) {
    if (!mem || !stage_ok(mem, stage) || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!out) return EVK_ERR_INVALID;
    return cuda_status(cudaMemcpyAsync(out, mem->visits + (size_t)stage * mem->cfg.capacity + first,
                                       (size_t)n * sizeof(uint32_t), cudaMemcpyDeviceToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

int evk_q_update_static(evk_mem *mem, const int32_t *ids, int64_t M, int stage,
                        const float *rewards, float alpha, void *stream) {
    if (!mem || M < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (!(alpha > 0.0f && alpha <= 1.0f)) return EVK_ERR_INVALID;
    if (M == 0) return EVK_OK;
    if (M > q_update_static_max()) return EVK_ERR_UNSUPPORTED;
    if (!ids || !rewards) return EVK_ERR_INVALID;
    int launches = 0;
    cudaError_t err = launch_q_update_static(mem->q_tables + (size_t)stage * mem->cfg.capacity, mem->size, ids,
                                             rewards, M, alpha, mem->status, static_cast<cudaStream_t>(stream),
                                             &launches);
    mem->launches += launches;
    return cuda_status(err);
}

int evk_q_read(evk_mem *mem, int stage, int64_t first, int64_t n, float *out, void *stream) {
    if (!mem || !stage_ok(mem, stage) || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!out) return EVK_ERR_INVALID;
    return cuda_status(cudaMemcpyAsync(out, mem->q_tables + (size_t)stage * mem->cfg.capacity + first,
                                       (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

int evk_q_write(evk_mem *mem, int stage, int64_t first, int64_t n, const float *values, void *stream) {
    if (!mem || !stage_ok(mem, stage) || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!values) return EVK_ERR_INVALID;
    return cuda_status(cudaMemcpyAsync(mem->q_tables + (size_t)stage * mem->cfg.capacity + first, values,
                                       (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

int evk_bank_read(evk_mem *mem, int64_t first, int64_t n, void *out_bf16, void *stream) {
    if (!mem || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!out_bf16) return EVK_ERR_INVALID;
    return cuda_status(cudaMemcpyAsync(out_bf16, mem->bank + (size_t)first * mem->cfg.d,
                                       (size_t)n * mem->cfg.d * sizeof(__nv_bfloat16), cudaMemcpyDeviceToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

// ---- dropping entries, export, import, counters ------------------------------------------------

int evk_mem_tombstone(evk_mem *mem, const int32_t *ids, int64_t n, void *stream) {
    if (!mem || n < 0) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!ids) return EVK_ERR_INVALID;
    int launches = 0;
    cudaError_t err = launch_tombstone(ids, n, mem->size, mem->live_bits, mem->dev, mem->status,
                                       static_cast<cudaStream_t>(stream), &launches);
    mem->launches += launches;
    mem->any_dropped = 1;
    return cuda_status(err);
}

int evk_mem_export(evk_mem *mem, int64_t first, int64_t n, void *rows_bf16, float *q, uint32_t *visits,
                   uint8_t *live, void *stream_v) {
    if (!mem || first < 0 || n < 0 || first + n > mem->size) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t err = cudaSuccess;
    if (rows_bf16)
        err = cudaMemcpyAsync(rows_bf16, mem->bank + (size_t)first * mem->cfg.d,
                              (size_t)n * mem->cfg.d * sizeof(__nv_bfloat16), cudaMemcpyDeviceToDevice, stream);
    for (int s = 0; s < mem->cfg.n_stages && err == cudaSuccess; ++s) {
        const size_t off = (size_t)s * mem->cfg.capacity + first;
        if (q)
            err = cudaMemcpyAsync(q + (size_t)s * n, mem->q_tables + off, (size_t)n * sizeof(float),
                                  cudaMemcpyDeviceToDevice, stream);
        if (visits && err == cudaSuccess)
            err = cudaMemcpyAsync(visits + (size_t)s * n, mem->visits + off, (size_t)n * sizeof(uint32_t),
                                  cudaMemcpyDeviceToDevice, stream);
    }
    int launches = 0;
    if (live && err == cudaSuccess) err = launch_live_export(mem->live_bits, first, n, live, stream, &launches);
    mem->launches += launches;
    return cuda_status(err);
}

int evk_mem_import(evk_mem *mem, int64_t n, const void *rows_bf16, const float *q, const uint32_t *visits,
                   const uint8_t *live, int32_t *ids_out, void *stream_v) {
    if (!mem || n < 0) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!rows_bf16 || !aligned(rows_bf16, 16)) return EVK_ERR_INVALID;
    if (mem->size + n > mem->cfg.capacity) return EVK_ERR_CAPACITY;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int64_t first = mem->size;
    // the rows go in like any insert (every stage at q_default, counts at 0, live) ...
    int rc = evk_mem_insert(mem, rows_bf16, EVK_DTYPE_BF16, n, EVK_STAGE_ALL, nullptr, ids_out, stream_v);
    if (rc != EVK_OK) return rc;
    // ... then the saved values, update counts and dropped marks are laid over them
    cudaError_t err = cudaSuccess;
    for (int s = 0; s < mem->cfg.n_stages && err == cudaSuccess; ++s) {
        const size_t off = (size_t)s * mem->cfg.capacity + first;
        if (q)
            err = cudaMemcpyAsync(mem->q_tables + off, q + (size_t)s * n, (size_t)n * sizeof(float),
                                  cudaMemcpyDeviceToDevice, stream);
        if (visits && err == cudaSuccess)
            err = cudaMemcpyAsync(mem->visits + off, visits + (size_t)s * n, (size_t)n * sizeof(uint32_t),
                                  cudaMemcpyDeviceToDevice, stream);
    }
    int launches = 0;
    if (live && err == cudaSuccess) {
        err = launch_live_import(live, first, n, mem->live_bits, mem->dev, stream, &launches);
        mem->any_dropped = 1;
    }
    mem->launches += launches;
    return cuda_status(err);
}

int evk_mem_read_probe(evk_mem *mem, void *stream) {
    if (!mem) return EVK_ERR_INVALID;
    if (mem->size <= 0) return EVK_OK;
    const cudaError_t err = launch_read_probe(mem->bank, (size_t)mem->size * mem->cfg.d * sizeof(__nv_bfloat16),
                                              mem->status, static_cast<cudaStream_t>(stream));
    ++mem->launches;
    return cuda_status(err);
}

int evk_mem_stats(evk_mem *mem, evk_stats *out, void *stream_v) {
    if (!mem || !out) return EVK_ERR_INVALID;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (cudaMemcpyAsync(w, mem->dev, sizeof(w), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return EVK_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return EVK_ERR_CUDA;
    out->entries = mem->size;
    out->live_entries = (int64_t)w[kDevLive];
    out->dropped_entries = (int64_t)w[kDevDropped];
    out->retrieve_calls = mem->n_retrieve;
    out->update_calls = mem->n_update;
    out->insert_calls = mem->n_insert;
    out->kernel_launches = mem->launches;
    out->candidates_filed = (int64_t)(((uint64_t)w[kDevFiledHi] << 32) | w[kDevFiledLo]);
    out->list_cutbacks = (int64_t)w[kDevCutbacks];
    out->longest_update_run = (int64_t)w[kDevLongestRun];
    return EVK_OK;
}

// ---- host-buffer forms -------------------------------------------------------

size_t evk_retrieve_host_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1, int32_t k2) {
    if (!mem || B < 0 || k1 < 1 || k1 > EVK_MAX_K1 || k2 < 1 || k2 > k1) return 0;
    const size_t b = (size_t)B;
    return align256(b * mem->cfg.d * sizeof(float)) + 2 * align256(b * k2 * sizeof(float)) +
           evk_retrieve_workspace_bytes(mem, B, k1);
}

int evk_retrieve_host(evk_mem *mem, const void *queries_host, int q_dtype, int32_t B, int stage,
                      int32_t k1, int32_t k2, float w,
                      int32_t *ids_out_host, float *scores_out_host,
                      void *workspace, size_t workspace_bytes, void *stream_v) {
    // every check evk_retrieve makes on the host is made here first: nothing is copied for a call
    // that would be refused
    if (!mem || B < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (k1 < 1 || k1 > EVK_MAX_K1 || k2 < 1 || k2 > k1) return EVK_ERR_INVALID;
    if (!(w >= 0.0f && w <= 1.0f)) return EVK_ERR_INVALID;
    if (q_dtype != EVK_DTYPE_F32 && q_dtype != EVK_DTYPE_BF16) return EVK_ERR_INVALID;
    if (B == 0) return EVK_OK;
    if (!queries_host || !ids_out_host || !scores_out_host || !workspace || !aligned(workspace, 256))
        return EVK_ERR_INVALID;
    if (pick_kind(mem, B, k1) == 0) return EVK_ERR_UNSUPPORTED;
    if (workspace_bytes < evk_retrieve_host_workspace_bytes(mem, B, k1, k2)) return EVK_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t b = (size_t)B;
    const size_t q_bytes = b * mem->cfg.d * (q_dtype == EVK_DTYPE_F32 ? sizeof(float) : sizeof(__nv_bfloat16));
    char *ws = static_cast<char *>(workspace);
    void *q_dev = ws;
    int32_t *ids_dev = reinterpret_cast<int32_t *>(ws + align256(b * mem->cfg.d * sizeof(float)));
    float *scores_dev = reinterpret_cast<float *>(reinterpret_cast<char *>(ids_dev) + align256(b * k2 * sizeof(float)));
    char *inner = reinterpret_cast<char *>(scores_dev) + align256(b * k2 * sizeof(float));
    const size_t inner_bytes = workspace_bytes - (size_t)(inner - ws);
    // with a staging buffer the result is written into it by the merge kernel itself and handed over
    // after the synchronise; without one it is copied back from the workspace
    const size_t res_bytes = align256(b * k2 * sizeof(int32_t)) + b * k2 * sizeof(float);
    int slot = -1;
    if (mem->stage_host && res_bytes <= mem->slot_bytes) {
        slot = acquire_slot(mem);
        if (slot < 0) return EVK_ERR_CUDA;
    }
    if (cudaMemcpyAsync(q_dev, queries_host, q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return EVK_ERR_CUDA;
    // from here on a copy may be in flight: every return synchronises, so that the caller's host
    // buffers are its own again whatever the outcome
    int rc;
    if (slot >= 0) {
        char *res_dev = mem->stage_dev + (size_t)slot * mem->slot_bytes;
        rc = evk_retrieve(mem, q_dev, q_dtype, B, stage, k1, k2, w, reinterpret_cast<int32_t *>(res_dev),
                          reinterpret_cast<float *>(res_dev + align256(b * k2 * sizeof(int32_t))), nullptr, nullptr,
                          inner, inner_bytes, stream_v);
    } else {
        rc = evk_retrieve(mem, q_dev, q_dtype, B, stage, k1, k2, w, ids_dev, scores_dev, nullptr, nullptr,
                          inner, inner_bytes, stream_v);
        if (rc == EVK_OK &&
            (cudaMemcpyAsync(ids_out_host, ids_dev, b * k2 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
             cudaMemcpyAsync(scores_out_host, scores_dev, b * k2 * sizeof(float), cudaMemcpyDeviceToHost, stream) != cudaSuccess))
            rc = EVK_ERR_CUDA;
    }
    const cudaError_t sync = cudaStreamSynchronize(stream);
    if (rc == EVK_OK && sync != cudaSuccess) rc = EVK_ERR_CUDA;
    if (rc == EVK_OK && slot >= 0) {
        const char *res = mem->stage_host + (size_t)slot * mem->slot_bytes;
        memcpy(ids_out_host, res, b * k2 * sizeof(int32_t));
        memcpy(scores_out_host, res + align256(b * k2 * sizeof(int32_t)), b * k2 * sizeof(float));
    }
    return rc;
}

size_t evk_q_update_host_workspace_bytes(const evk_mem *mem, int64_t M) {
    if (!mem || M < 0) return 0;
    return 2 * align256((size_t)M * 4) + evk_q_update_workspace_bytes(mem, M);
}

int evk_q_update_host(evk_mem *mem, const int32_t *ids_host, int64_t M, int stage,
                      const float *rewards_host, float alpha,
                      void *workspace, size_t workspace_bytes, void *stream_v) {
    // the host-side checks of evk_q_update, before anything is copied
    if (!mem || M < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (!(alpha > 0.0f && alpha <= 1.0f)) return EVK_ERR_INVALID;
    if (M == 0) return EVK_OK;
    if (M >= ((int64_t)1 << 31)) return EVK_ERR_UNSUPPORTED;
    if (!ids_host || !rewards_host || !workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (workspace_bytes < evk_q_update_host_workspace_bytes(mem, M)) return EVK_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    char *ws = static_cast<char *>(workspace);
    int32_t *ids_dev = reinterpret_cast<int32_t *>(ws);
    float *r_dev = reinterpret_cast<float *>(ws + align256((size_t)M * 4));
    char *inner = ws + 2 * align256((size_t)M * 4);
    const size_t r_off = align256((size_t)M * 4);
    if (mem->stage_host && r_off + (size_t)M * 4 <= mem->slot_bytes) {
        // staged: the batch is copied into the page-locked slot here and travels from there, so the
        // caller's arrays are its own again on return and nothing waits for the device
        const int slot = acquire_slot(mem);
        if (slot < 0) return EVK_ERR_CUDA;
        char *h = mem->stage_host + (size_t)slot * mem->slot_bytes;
        memcpy(h, ids_host, (size_t)M * 4);
        memcpy(h + r_off, rewards_host, (size_t)M * 4);
        if (cudaMemcpyAsync(ids_dev, h, r_off + (size_t)M * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return EVK_ERR_CUDA;
        if (!release_slot_after(mem, slot, stream)) {
            (void)cudaStreamSynchronize(stream);
            return EVK_ERR_CUDA;
        }
        return evk_q_update(mem, ids_dev, M, stage, r_dev, alpha, inner, workspace_bytes - (size_t)(inner - ws), stream_v);
    }
    int rc = EVK_OK;
    if (cudaMemcpyAsync(ids_dev, ids_host, (size_t)M * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return EVK_ERR_CUDA;
    // a copy may be in flight from here on: every return synchronises first
    if (cudaMemcpyAsync(r_dev, rewards_host, (size_t)M * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        rc = EVK_ERR_CUDA;
    if (rc == EVK_OK)
        rc = evk_q_update(mem, ids_dev, M, stage, r_dev, alpha, inner, workspace_bytes - (size_t)(inner - ws), stream_v);
    const cudaError_t sync = cudaStreamSynchronize(stream);
    if (rc == EVK_OK && sync != cudaSuccess) rc = EVK_ERR_CUDA;
    return rc;
}

size_t evk_mem_insert_host_workspace_bytes(const evk_mem *mem, int64_t n) {
    if (!mem || n < 0) return 0;
    return align256((size_t)n * mem->cfg.d * sizeof(float)) + align256((size_t)n * sizeof(float)) + 256;
}

int evk_mem_insert_host(evk_mem *mem, const void *emb_host, int emb_dtype, int64_t n, int stage,
                        const float *q_init_host, void *workspace, size_t workspace_bytes, void *stream_v) {
    // the host-side checks of evk_mem_insert, before anything is copied
    if (!mem || n < 0 || (emb_dtype != EVK_DTYPE_F32 && emb_dtype != EVK_DTYPE_BF16)) return EVK_ERR_INVALID;
    if (stage != EVK_STAGE_ALL && !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!emb_host || !workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (mem->size + n > mem->cfg.capacity) return EVK_ERR_CAPACITY;
    if (workspace_bytes < evk_mem_insert_host_workspace_bytes(mem, n)) return EVK_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t e_bytes = (size_t)n * mem->cfg.d * (emb_dtype == EVK_DTYPE_F32 ? sizeof(float) : sizeof(__nv_bfloat16));
    const size_t q_off = align256((size_t)n * mem->cfg.d * sizeof(float));
    const size_t q_bytes = q_init_host ? (size_t)n * sizeof(float) : 0;
    char *ws = static_cast<char *>(workspace);
    const float *q_dev = q_init_host ? reinterpret_cast<const float *>(ws + q_off) : nullptr;
    if (mem->stage_host && align256(e_bytes) + q_bytes <= mem->slot_bytes) {
        // staged like evk_q_update_host: rows and start values leave through the page-locked slot
        const int slot = acquire_slot(mem);
        if (slot < 0) return EVK_ERR_CUDA;
        char *h = mem->stage_host + (size_t)slot * mem->slot_bytes;
        memcpy(h, emb_host, e_bytes);
        if (q_bytes) memcpy(h + align256(e_bytes), q_init_host, q_bytes);
        cudaError_t err = cudaMemcpyAsync(ws, h, e_bytes, cudaMemcpyHostToDevice, stream);
        if (err == cudaSuccess && q_bytes)
            err = cudaMemcpyAsync(ws + q_off, h + align256(e_bytes), q_bytes, cudaMemcpyHostToDevice, stream);
        if (err != cudaSuccess || !release_slot_after(mem, slot, stream)) {
            (void)cudaStreamSynchronize(stream);
            return EVK_ERR_CUDA;
        }
        return evk_mem_insert(mem, ws, emb_dtype, n, stage, q_dev, nullptr, stream_v);
    }
    int rc = EVK_OK;
    if (cudaMemcpyAsync(ws, emb_host, e_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return EVK_ERR_CUDA;
    // a copy may be in flight from here on: every return synchronises first
    if (q_bytes && cudaMemcpyAsync(ws + q_off, q_init_host, q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        rc = EVK_ERR_CUDA;
    if (rc == EVK_OK) rc = evk_mem_insert(mem, ws, emb_dtype, n, stage, q_dev, nullptr, stream_v);
    const cudaError_t sync = cudaStreamSynchronize(stream);
    if (rc == EVK_OK && sync != cudaSuccess) rc = EVK_ERR_CUDA;
    return rc;
}

// ---- exploration -----------------------------------------------------------------

size_t evk_retrieve_explore_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1) {
    const size_t inner = evk_retrieve_workspace_bytes(mem, B, k1);
    if (inner == 0) return 0;
    return inner + 2 * align256((size_t)B * k1 * sizeof(float));
}

int evk_retrieve_explore(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage,
                         int32_t k1, int32_t k2, float w, float epsilon, uint64_t seed, uint64_t step,
                         int32_t *ids_out, float *scores_out, uint8_t *explored_out,
                         int32_t *pool_ids_out, float *pool_sims_out,
                         void *workspace, size_t workspace_bytes, void *stream) {
    if (!(epsilon >= 0.0f && epsilon <= 1.0f)) return EVK_ERR_INVALID;
    if (!mem || B < 0 || k1 < 1 || k1 > EVK_MAX_K1) return EVK_ERR_INVALID;
    if (B == 0) return EVK_OK;
    if (!workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (workspace_bytes < evk_retrieve_explore_workspace_bytes(mem, B, k1)) return EVK_ERR_WORKSPACE;
    // the pool is needed in its canonical order: use the caller's arrays or scratch of our own
    char *ws = static_cast<char *>(workspace);
    const size_t pool_bytes = align256((size_t)B * k1 * sizeof(float));
    int32_t *pool_ids = pool_ids_out ? pool_ids_out : reinterpret_cast<int32_t *>(ws);
    float *pool_sims = pool_sims_out ? pool_sims_out : reinterpret_cast<float *>(ws + pool_bytes);
    int rc = evk_retrieve(mem, queries, q_dtype, B, stage, k1, k2, w, ids_out, scores_out, pool_ids, pool_sims,
                          ws + 2 * pool_bytes, workspace_bytes - 2 * pool_bytes, stream);
    if (rc != EVK_OK) return rc;
    int launches = 0;
    cudaError_t err = launch_explore(pool_ids, pool_sims, B, k1, k2, mem->q_tables + (size_t)stage * mem->cfg.capacity,
                                     w, mem->score_norm, epsilon, seed, step, ids_out, scores_out, explored_out,
                                     static_cast<cudaStream_t>(stream), &launches);
    mem->launches += launches;
    return cuda_status(err);
}

// ---- start points ------------------------------------------------------------------

int evk_select_by_value(evk_mem *mem, const int32_t *cand_ids, const int32_t *offsets, int32_t n_tasks, int stage,
                        int32_t k, int32_t *ids_out, float *q_out, void *stream) {
    if (!mem || n_tasks < 0 || !stage_ok(mem, stage) || k < 1 || k > EVK_MAX_K1) return EVK_ERR_INVALID;
    if (n_tasks == 0) return EVK_OK;
    if (!cand_ids || !offsets || !ids_out || !q_out) return EVK_ERR_INVALID;
    int launches = 0;
    cudaError_t err = launch_select_by_value(cand_ids, offsets, n_tasks, mem->size,
                                             mem->any_dropped ? mem->live_bits : nullptr, mem->q_tables + (size_t)stage * mem->cfg.capacity, k, ids_out, q_out,
                                             mem->status, static_cast<cudaStream_t>(stream), &launches);
    mem->launches += launches;
    return cuda_status(err);
}

// ---- row-sharded banks -------------------------------------------------------------

size_t evk_retrieve_local_workspace_bytes(const evk_mem *mem, int32_t B, int32_t k1) {
    const size_t inner = evk_retrieve_workspace_bytes(mem, B, k1);
    if (inner == 0) return 0;
    return inner + align256((size_t)B * k1 * sizeof(int32_t)) + 2 * align256((size_t)B * sizeof(float));
}

int evk_retrieve_local(evk_mem *mem, const void *queries, int q_dtype, int32_t B, int stage, int32_t k1,
                       int32_t id_offset, int32_t *gids_out, float *sims_out, float *q_out,
                       void *workspace, size_t workspace_bytes, void *stream) {
    if (!mem || B < 0 || k1 < 1 || k1 > EVK_MAX_K1 || id_offset < 0 || !stage_ok(mem, stage)) return EVK_ERR_INVALID;
    if (B == 0) return EVK_OK;
    if (!gids_out || !sims_out || !q_out || !workspace || !aligned(workspace, 256)) return EVK_ERR_INVALID;
    if (workspace_bytes < evk_retrieve_local_workspace_bytes(mem, B, k1)) return EVK_ERR_WORKSPACE;
    char *ws = static_cast<char *>(workspace);
    int32_t *pool_ids = reinterpret_cast<int32_t *>(ws);
    size_t off = align256((size_t)B * k1 * sizeof(int32_t));
    int32_t *top_ids = reinterpret_cast<int32_t *>(ws + off);
    off += align256((size_t)B * sizeof(float));
    float *top_scores = reinterpret_cast<float *>(ws + off);
    off += align256((size_t)B * sizeof(float));
    // phase 1 on this shard's rows (the k2 = 1 result is not used)
    int rc = evk_retrieve(mem, queries, q_dtype, B, stage, k1, 1, 0.0f, top_ids, top_scores, pool_ids, sims_out,
                          ws + off, workspace_bytes - off, stream);
    if (rc != EVK_OK) return rc;
    int launches = 0;
    cudaError_t err = launch_tag_pool(pool_ids, (int64_t)B * k1, id_offset,
                                      mem->q_tables + (size_t)stage * mem->cfg.capacity, gids_out, q_out,
                                      static_cast<cudaStream_t>(stream), &launches);
    mem->launches += launches;
    return cuda_status(err);
}

int evk_merge_shards(const int32_t *gids, const float *sims, const float *qs, int32_t n_shards, int32_t B,
                     int32_t k1, int32_t k2, float w, int32_t *ids_out, float *scores_out,
                     int32_t *pool_gids_out, float *pool_sims_out, void *stream) {
    if (n_shards < 1 || B < 0 || k1 < 1 || k1 > EVK_MAX_K1 || k2 < 1 || k2 > k1) return EVK_ERR_INVALID;
    if (!(w >= 0.0f && w <= 1.0f)) return EVK_ERR_INVALID;
    if ((int64_t)n_shards * k1 >= ((int64_t)1 << 31)) return EVK_ERR_UNSUPPORTED;
    if (B == 0) return EVK_OK;
    if (!gids || !sims || !qs || !ids_out || !scores_out) return EVK_ERR_INVALID;
    return cuda_status(launch_merge_shards(gids, sims, qs, n_shards, B, k1, k2, w, ids_out, scores_out,
                                           pool_gids_out, pool_sims_out, static_cast<cudaStream_t>(stream)));
}

// ---- rewards -------------------------------------------------------------------

int evk_reward_draft(const uint8_t *feasible, int64_t n, float *rewards_out, void *stream) {
    if (n < 0) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!feasible || !rewards_out) return EVK_ERR_INVALID;
    return cuda_status(launch_reward_draft(feasible, n, rewards_out, static_cast<cudaStream_t>(stream)));
}

int evk_reward_refine(const float *best_latency, const float *latency, const uint8_t *feasible, int64_t n,
                      float *rewards_out, void *stream) {
    if (n < 0) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!best_latency || !latency || !feasible || !rewards_out) return EVK_ERR_INVALID;
    return cuda_status(launch_reward_refine(best_latency, latency, feasible, n, rewards_out,
                                            static_cast<cudaStream_t>(stream)));
}

size_t evk_reward_norm_state_bytes(void) { return 4 * sizeof(double); }

int evk_reward_norm_reset(void *state, void *stream) {
    if (!state || !aligned(state, 8)) return EVK_ERR_INVALID;
    return cuda_status(cudaMemsetAsync(state, 0, evk_reward_norm_state_bytes(), static_cast<cudaStream_t>(stream)));
}

int evk_reward_normalize(void *state, const float *raw, int64_t n, float sigma_min, float clip,
                         float *rewards_out, void *stream) {
    if (!state || !aligned(state, 8) || n < 0 || !(sigma_min > 0.0f) || !(clip >= 0.0f)) return EVK_ERR_INVALID;
    if (n == 0) return EVK_OK;
    if (!raw || !rewards_out) return EVK_ERR_INVALID;
    return cuda_status(launch_reward_normalize(static_cast<double *>(state), raw, n, sigma_min, clip, rewards_out,
                                               static_cast<cudaStream_t>(stream)));
}

int evk_last_status(evk_mem *mem, void *stream_v) {
    if (!mem) return EVK_ERR_INVALID;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, mem->status, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return EVK_ERR_CUDA;
    if (cudaMemsetAsync(mem->status, 0, sizeof(word), stream) != cudaSuccess) return EVK_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return EVK_ERR_CUDA;
    return word;
}

const char *evk_strerror(int status) {
    switch (status) {
        case EVK_OK: return "ok";
        case EVK_ERR_INVALID: return "invalid argument";
        case EVK_ERR_CAPACITY: return "bank capacity exceeded";
        case EVK_ERR_WORKSPACE: return "workspace or arena too small";
        case EVK_ERR_RANGE: return "entry id out of range";
        case EVK_ERR_NONFINITE: return "non-finite reward";
        case EVK_ERR_DEVICE_TIMEOUT: return "bounded wait in a kernel ran out";
        case EVK_ERR_CUDA: return "CUDA call failed";
        case EVK_ERR_UNSUPPORTED: return "unsupported shape";
        case EVK_ERR_INCOMPLETE: return "fewer candidates than min(k1, size): non-finite similarities";
        default: return "unknown status";
    }
}

}  // extern "C"
