// C-ABI entry points of libgoodserve: argument checks, context lifetime, kernel sequencing.
#include <new>
#include <stdint.h>
#include <string.h>

#include "gs_internal.cuh"

namespace {

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

int cuda_fail(gs_ctx *ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    return GS_ERR_CUDA;
}

// Makes the context's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int check_pool(const gs_ctx *ctx, const gs_instances *inst, const gs_types *types, bool device_ptrs) {
    if (!ctx || !inst || !types) return GS_ERR_INVALID_ARG;
    if (inst->n_instances < 1 || types->n_types < 1) return GS_ERR_INVALID_ARG;
    if (inst->n_instances > ctx->max_instances || types->n_types > ctx->max_types) return GS_ERR_CAPACITY;
    const void *ptrs[] = {inst->type_id, inst->queued_prefill_tokens, inst->decode_batch,
                          inst->free_kv_tokens, inst->q_ema_ms, types->prefill_ms_per_tok,
                          types->tpot_a_ms, types->tpot_b_ms};
    for (const void *p : ptrs) if (!p) return GS_ERR_INVALID_ARG;
    if (device_ptrs)
        for (int k = 0; k < 5; ++k) if (misaligned(ptrs[k])) return GS_ERR_ALIGN;
    return GS_OK;
}

// Grows one of the context's staging buffers.  (cudaFree waits for everything the device still
// has to do, so a buffer that copies enqueued earlier still use is never pulled from under them.)
int ensure_stage(gs_ctx *ctx, char **stage, size_t *stage_bytes, size_t bytes) {
    if (bytes <= *stage_bytes) return GS_OK;
    if (*stage) { cudaFree(*stage); *stage = nullptr; *stage_bytes = 0; }
    const size_t want = bytes + bytes / 8 + 4096;
    cudaError_t e = cudaMalloc(stage, want);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    *stage_bytes = want;
    return GS_OK;
}

inline size_t pad256(size_t b) { return (b + 255) & ~(size_t)255; }

// Bump allocator over the staging buffer.
struct Carver {
    char *base; size_t off = 0;
    template <typename T> T *take(size_t count) {
        T *p = reinterpret_cast<T *>(base + off);
        off += pad256(count * sizeof(T));
        return p;
    }
};

// Device copies of a host-side pool description; returns bytes needed when base == nullptr.
struct PoolStage {
    gs_instances inst;
    gs_types types;
};

size_t pool_stage_bytes(int M, int Tn) { return 5 * pad256((size_t)M * 4) + 3 * pad256((size_t)Tn * 4); }

// The eight small arrays are first put together in a pinned image laid out like their device
// copies and then sent as one copy (a copy costs some 20 us beside its bytes).
cudaError_t stage_pool(Carver &c, const gs_instances *h_inst, const gs_types *h_types,
                       PoolStage *out, char *pinned_image, cudaStream_t st) {
    const int M = h_inst->n_instances, Tn = h_types->n_types;
    char *const first = c.base + c.off;
    int32_t *type_id = c.take<int32_t>(M), *queued = c.take<int32_t>(M), *batch = c.take<int32_t>(M),
            *kv = c.take<int32_t>(M);
    float *qe = c.take<float>(M), *p = c.take<float>(Tn), *a = c.take<float>(Tn), *b = c.take<float>(Tn);
    const void *src[] = {h_inst->type_id, h_inst->queued_prefill_tokens, h_inst->decode_batch,
                         h_inst->free_kv_tokens, h_inst->q_ema_ms, h_types->prefill_ms_per_tok,
                         h_types->tpot_a_ms, h_types->tpot_b_ms};
    void *dst[] = {type_id, queued, batch, kv, qe, p, a, b};
    for (int k = 0; k < 8; ++k)
        memcpy(pinned_image + ((char *)dst[k] - first), src[k], (size_t)(k < 5 ? M : Tn) * 4);
    const cudaError_t e = cudaMemcpyAsync(first, pinned_image, (size_t)(c.base + c.off - first), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return e;
    out->inst = gs_instances{type_id, queued, batch, kv, qe, M};
    out->types = gs_types{p, a, b, Tn};
    return cudaSuccess;
}

}  // namespace

namespace gs {

LaunchTimer::LaunchTimer(gs_ctx *c, int k, cudaStream_t s) : ctx(c), st(s), kernel(k) {
    if (!ctx) return;
    ctx->launches += 1;
    if (!ctx->timing) return;
    for (cudaEvent_t *ev : {&start, &stop}) {
        if (!ctx->free_events->empty()) { *ev = ctx->free_events->back(); ctx->free_events->pop_back(); }
        else if (cudaEventCreate(ev) != cudaSuccess) { *ev = nullptr; }
    }
    if (start && stop) cudaEventRecord(start, st);
}

LaunchTimer::~LaunchTimer() {
    if (!ctx || !ctx->timing || !start || !stop) return;
    cudaEventRecord(stop, st);
    ctx->pending->push_back({kernel, start, stop});
}

}  // namespace gs

extern "C" {

GS_API const char *gs_strerror(int code) {
    switch (code) {
        case GS_OK: return "ok";
        case GS_ERR_INVALID_ARG: return "invalid argument (null pointer, negative size or empty pool)";
        case GS_ERR_CAPACITY: return "pool larger than the context was created for";
        case GS_ERR_CUDA: return "a CUDA runtime call failed (see gs_last_cuda_error)";
        case GS_ERR_ALIGN: return "array pointer is not 16-byte aligned";
        case GS_ERR_NO_DEVICE: return "no usable CUDA device";
        case GS_ERR_TOO_LARGE: return "n_active exceeds GS_NOALLOC_MAX_ACTIVE, the fixed scratch of the no-allocation scan";
        default: return "unknown error code";
    }
}

GS_API int gs_create(gs_ctx **out, int device, int max_instances, int max_types) {
    if (!out) return GS_ERR_INVALID_ARG;
    *out = nullptr;
    if (max_instances < 1 || max_types < 1) return GS_ERR_INVALID_ARG;
    if (max_instances > GS_MAX_INSTANCES || max_types > GS_MAX_TYPES) return GS_ERR_CAPACITY;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1 || device < 0 || device >= n_dev)
        return GS_ERR_NO_DEVICE;
    DeviceGuard guard(device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;

    gs_ctx *ctx = new (std::nothrow) gs_ctx();
    if (!ctx) return GS_ERR_INVALID_ARG;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->max_instances = max_instances;
    ctx->max_types = max_types;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { delete ctx->pending; delete ctx->free_events; delete ctx; return GS_ERR_CUDA; }
    ctx->n_sm = prop.multiProcessorCount;
    ctx->pending = new (std::nothrow) std::vector<gs_ctx::TimedLaunch>();
    ctx->free_events = new (std::nothrow) std::vector<cudaEvent_t>();
    if (!ctx->pending || !ctx->free_events) { delete ctx->pending; delete ctx->free_events; delete ctx; return GS_ERR_INVALID_ARG; }

    const size_t Mx = GS_MAX_INSTANCES;
    gs::Scratch &s = ctx->s;
    struct { void **p; size_t bytes; } allocs[] = {
        {(void **)&s.rows, Mx * sizeof(gs::Row)},
        {(void **)&s.row_bounds, gs::kMaxPaddedRows * sizeof(uint2)},
        {(void **)&s.group_bounds, gs::kMaxPaddedRows / 8 * sizeof(float2)},
        {(void **)&s.row_p, gs::kMaxPaddedRows * sizeof(float)},
        {(void **)&s.start_table, (size_t)GS_MAX_TYPES * gs::kStartBuckets * gs::kStartSlots},
        {(void **)&s.headers, GS_MAX_TYPES * sizeof(gs::TypeHeader)},
        {(void **)&s.table_info, 64},
        {(void **)&s.cand_table, gs::kCandSlots * sizeof(unsigned short)},
        {(void **)&s.pool, gs::kPoolEntries * sizeof(uint2)},
        {(void **)&s.bucket_list, (size_t)GS_MAX_TYPES * gs::kStartBuckets * sizeof(unsigned short)},
        {(void **)&s.start_list, (size_t)GS_MAX_TYPES * gs::kStartBuckets * gs::kStartSlots},
        {(void **)&s.chord, (size_t)GS_MAX_TYPES * gs::kStartBuckets * sizeof(float4)},
        {(void **)&s.q_by_g, Mx * sizeof(float)},
        {(void **)&s.deltas, 3 * Mx * sizeof(unsigned long long)},
        {(void **)&s.scan_counts, gs::kMaxScanCtas * sizeof(unsigned)},
        {(void **)&s.status, 256},
    };
    for (auto &a : allocs) {
        e = cudaMalloc(a.p, a.bytes);
        if (e == cudaSuccess) e = cudaMemset(*a.p, 0, a.bytes);
        if (e != cudaSuccess) { gs_destroy(ctx); return GS_ERR_CUDA; }
    }
    if (gs::configure_route(ctx) != cudaSuccess || gs::configure_prologue() != cudaSuccess) {
        gs_destroy(ctx);
        return GS_ERR_CUDA;
    }
    *out = ctx;
    return GS_OK;
}

GS_API int gs_destroy(gs_ctx *ctx) {
    if (!ctx) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    gs::Scratch &s = ctx->s;
    void *ptrs[] = {s.rows, s.row_bounds, s.group_bounds, s.row_p, s.start_table, s.headers, s.table_info, s.cand_table, s.pool, s.bucket_list, s.start_list, s.chord, s.q_by_g, s.deltas, s.scan_counts, s.status, ctx->stage, ctx->scan_stage};
    for (void *p : ptrs) if (p) cudaFree(p);
    if (ctx->pending) for (auto &t : *ctx->pending) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
    if (ctx->free_events) for (cudaEvent_t ev : *ctx->free_events) cudaEventDestroy(ev);
    if (ctx->host_pipe_ready) {
        cudaStreamDestroy(ctx->host_out_stream);
        for (cudaEvent_t ev : ctx->host_events) cudaEventDestroy(ev);
        cudaFreeHost(ctx->host_counts);
        for (char *image : ctx->host_pool_image) cudaFreeHost(image);
    }
    delete ctx->pending;
    delete ctx->free_events;
    delete ctx;
    return GS_OK;
}

GS_API int gs_timing_enable(gs_ctx *ctx, int on) {
    if (!ctx) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    for (auto &t : *ctx->pending) { ctx->free_events->push_back(t.start); ctx->free_events->push_back(t.stop); }
    ctx->pending->clear();
    for (int k = 0; k < GS_K_COUNT; ++k) { ctx->time_ms[k] = 0.0; ctx->time_launches[k] = 0; }
    ctx->timing = on != 0;
    return GS_OK;
}

GS_API int gs_timing_read(gs_ctx *ctx, int kernel, double *total_ms, int64_t *launches) {
    if (!ctx || kernel < 0 || kernel >= GS_K_COUNT || !total_ms || !launches) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    for (auto &t : *ctx->pending) {
        cudaError_t e = cudaEventSynchronize(t.stop);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.start, t.stop);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->time_ms[t.kernel] += (double)ms;
        ctx->time_launches[t.kernel] += 1;
        ctx->free_events->push_back(t.start);
        ctx->free_events->push_back(t.stop);
    }
    ctx->pending->clear();
    *total_ms = ctx->time_ms[kernel];
    *launches = ctx->time_launches[kernel];
    return GS_OK;
}

GS_API int gs_last_cuda_error(const gs_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

GS_API int gs_eval_counters(gs_ctx *ctx, void *cuda_stream, uint64_t *out, int clear) {
    if (!ctx || !out) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
    unsigned long long v[gs::kCountN];
    if (e == cudaSuccess) e = gs::read_eval_counters(v, clear != 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    for (int k = 0; k < gs::kCountN; ++k) out[k] = v[k];
    return GS_OK;
}

GS_API int64_t gs_launch_count(const gs_ctx *ctx) { return ctx ? ctx->launches : 0; }

GS_API int gs_device_status(gs_ctx *ctx, void *cuda_stream, unsigned *out_bits) {
    if (!ctx || !out_bits) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e == cudaSuccess) e = cudaMemcpy(out_bits, ctx->s.status, sizeof(unsigned), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemset(ctx->s.status, 0, sizeof(unsigned));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    // (the checking build's index tests; always 0 in the regular build)
    if (gs::route_index_errors(true) | gs::prologue_index_errors(true)) *out_bits |= (unsigned)GS_DEV_INTERNAL;
    return GS_OK;
}

GS_API int gs_route_batch(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms, int64_t n_requests,
                   const gs_instances *inst, const gs_types *types, float ema_alpha,
                   int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                   uint8_t *out_tier, unsigned flags, void *cuda_stream)
{
    int rc = check_pool(ctx, inst, types, true);
    if (rc != GS_OK) return rc;
    if (n_requests < 0 || n_requests > gs::kMaxRouteRequests || (flags & ~GS_ROUTE_ACCUMULATE)) return GS_ERR_INVALID_ARG;
    if (n_requests > 0) {
        const void *ptrs[] = {prompt_len, pred_decode_len, slo_ms, out_instance_idx, out_est_e2e_ms, out_slack_ms};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
        if (out_tier && misaligned(out_tier)) return GS_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (n_requests == 0 && !(flags & GS_ROUTE_ACCUMULATE)) return GS_OK;
    cudaError_t e = gs::launch_prologue(ctx, *inst, *types, ema_alpha, (flags & GS_ROUTE_ACCUMULATE) != 0, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    e = gs::launch_route(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, nullptr, inst->n_instances, types->n_types,
                         out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier,
                         (flags & GS_ROUTE_ACCUMULATE) != 0, false, st);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_route_batch_prefix(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                          const float *slo_ms, int64_t n_requests,
                          const int32_t *prefix_inst, const int32_t *prefix_hit_len, int n_slots,
                          int64_t slot_stride,
                          const gs_instances *inst, const gs_types *types, float ema_alpha,
                          int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                          uint8_t *out_tier, void *cuda_stream)
{
    int rc = check_pool(ctx, inst, types, true);
    if (rc != GS_OK) return rc;
    if (n_requests < 0 || n_requests > gs::kMaxRouteRequests || n_slots < 0 || n_slots > GS_MAX_PREFIX_SLOTS)
        return GS_ERR_INVALID_ARG;
    if (n_slots > 0 && n_requests > 0) {
        if (!prefix_inst || !prefix_hit_len || slot_stride < n_requests) return GS_ERR_INVALID_ARG;
        if (misaligned(prefix_inst) || misaligned(prefix_hit_len) || (slot_stride & 3)) return GS_ERR_ALIGN;
    }
    if (n_requests > 0) {
        const void *ptrs[] = {prompt_len, pred_decode_len, slo_ms, out_instance_idx, out_est_e2e_ms, out_slack_ms};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
        if (out_tier && misaligned(out_tier)) return GS_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (n_requests == 0) return GS_OK;
    cudaError_t e = gs::launch_prologue(ctx, *inst, *types, ema_alpha, false, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const gs::PrefixHits hits = {prefix_inst, prefix_hit_len, n_slots, slot_stride};
    e = gs::launch_route(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, &hits, inst->n_instances, types->n_types,
                         out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier, false, false, st);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_ema_update(gs_ctx *ctx, float alpha, int32_t n_instances,
                  const float *obs_q_ms, const float *obs_p_ms_per_tok, const float *obs_d_ms_per_tok,
                  float *q_ms, float *p_ms_per_tok, float *d_ms_per_tok, void *cuda_stream)
{
    if (!ctx || n_instances < 1) return GS_ERR_INVALID_ARG;
    if (n_instances > ctx->max_instances) return GS_ERR_CAPACITY;
    const float *obs[3] = {obs_q_ms, obs_p_ms_per_tok, obs_d_ms_per_tok};
    float *col[3] = {q_ms, p_ms_per_tok, d_ms_per_tok};
    for (int c = 0; c < 3; ++c) {
        if (!obs[c]) continue;
        if (!col[c]) return GS_ERR_INVALID_ARG;
        if (misaligned(obs[c]) || misaligned(col[c])) return GS_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    const cudaError_t e = gs::launch_ema(ctx, alpha, n_instances, obs_q_ms, obs_p_ms_per_tok, obs_d_ms_per_tok,
                                         q_ms, p_ms_per_tok, d_ms_per_tok, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_route_batch_direct(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                          const float *slo_ms, int64_t n_requests, const gs_instance_table *table,
                          int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                          uint8_t *out_tier, void *cuda_stream)
{
    if (!ctx || !table || n_requests < 0 || n_requests > gs::kMaxRouteRequests || table->n_instances < 1)
        return GS_ERR_INVALID_ARG;
    if (table->n_instances > ctx->max_instances) return GS_ERR_CAPACITY;
    const void *cols[] = {table->q_ms, table->p_ms_per_tok, table->d_ms_per_tok, table->free_kv_tokens};
    for (const void *p : cols) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
    if (n_requests > 0) {
        const void *ptrs[] = {prompt_len, pred_decode_len, slo_ms, out_instance_idx, out_est_e2e_ms, out_slack_ms};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
        if (out_tier && misaligned(out_tier)) return GS_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (n_requests == 0) return GS_OK;
    cudaError_t e = gs::launch_prologue_direct(ctx, *table, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    e = gs::launch_route(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, nullptr, table->n_instances, gs::kDirectGroups,
                         out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier, false, true, st);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_route_sequential(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                        const float *slo_ms, int64_t n_requests,
                        const int32_t *type_id, const gs_instances_mut *state, const gs_types *types,
                        float ema_alpha,
                        int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                        uint8_t *out_tier, void *cuda_stream)
{
    if (!ctx || !state || !types || !type_id || n_requests < 0) return GS_ERR_INVALID_ARG;
    if (state->n_instances < 1 || types->n_types < 1) return GS_ERR_INVALID_ARG;
    if (state->n_instances > ctx->max_instances || types->n_types > ctx->max_types) return GS_ERR_CAPACITY;
    const void *pool[] = {type_id, state->queued_prefill_tokens, state->decode_batch, state->free_kv_tokens,
                          state->q_ema_ms, types->prefill_ms_per_tok, types->tpot_a_ms, types->tpot_b_ms};
    for (const void *p : pool) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
    if (n_requests > 0) {
        const void *ptrs[] = {prompt_len, pred_decode_len, slo_ms, out_instance_idx, out_est_e2e_ms, out_slack_ms};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
        if (out_tier && misaligned(out_tier)) return GS_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    const cudaError_t e = gs::launch_sequential(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, type_id, *state,
                                                *types, ema_alpha, out_instance_idx, out_est_e2e_ms, out_slack_ms,
                                                out_tier, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_advance_state(gs_ctx *ctx, const gs_instances_mut *inst, void *cuda_stream) {
    if (!ctx || !inst) return GS_ERR_INVALID_ARG;
    if (inst->n_instances < 1) return GS_ERR_INVALID_ARG;
    if (inst->n_instances > ctx->max_instances) return GS_ERR_CAPACITY;
    const void *ptrs[] = {inst->queued_prefill_tokens, inst->decode_batch, inst->free_kv_tokens, inst->q_ema_ms};
    for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaError_t e = gs::launch_advance(ctx, *inst, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_risk_scan(gs_ctx *ctx, const int32_t *assigned_inst, const int32_t *generated_tokens,
                 const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                 int64_t n_active, const gs_instances *inst, const gs_types *types,
                 uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
                 int64_t *out_cand_count, void *cuda_stream)
{
    int rc = check_pool(ctx, inst, types, true);
    if (rc != GS_OK) return rc;
    if (n_active < 0 || n_active > gs::kMaxActive || cand_capacity < 0 || !out_cand_count)
        return GS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(out_cand_count) & 7u) return GS_ERR_ALIGN;
    if (cand_capacity > 0 && !out_cand_idx) return GS_ERR_INVALID_ARG;
    if (out_cand_idx && misaligned(out_cand_idx)) return GS_ERR_ALIGN;
    if (n_active > 0) {
        const void *ptrs[] = {assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, out_flag_bits};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const cudaError_t e = gs::launch_risk(ctx, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
                                          n_active, *inst, *types, out_flag_bits, out_cand_idx, cand_capacity,
                                          out_cand_count, st);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_reroute_candidates(gs_ctx *ctx, const int32_t *cand_idx, const int64_t *cand_count,
                                 int64_t cand_capacity,
                                 const int32_t *assigned_inst, const int32_t *generated_tokens,
                                 const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                                 const int32_t *prompt_len, int64_t n_active,
                                 const gs_instances *inst, const gs_types *types, float ema_alpha,
                                 int32_t *out_new_instance, float *out_est_ms, float *out_slack_ms,
                                 uint8_t *out_tier, void *cuda_stream)
{
    int rc = check_pool(ctx, inst, types, true);
    if (rc != GS_OK) return rc;
    if (cand_capacity < 0 || n_active < 0 || n_active > gs::kMaxActive || !cand_count) return GS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(cand_count) & 7u) return GS_ERR_ALIGN;
    if (cand_capacity > 0) {
        if (n_active == 0) return GS_ERR_INVALID_ARG;
        const void *ptrs[] = {cand_idx, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, prompt_len,
                              out_new_instance, out_est_ms, out_slack_ms};
        for (const void *p : ptrs) { if (!p) return GS_ERR_INVALID_ARG; if (misaligned(p)) return GS_ERR_ALIGN; }
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cand_capacity == 0) return GS_OK;
    cudaError_t e = gs::launch_prologue(ctx, *inst, *types, ema_alpha, false, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    e = gs::launch_reroute(ctx, cand_idx, cand_count, cand_capacity, assigned_inst, generated_tokens, pred_len,
                           elapsed_ms, slo_ms, prompt_len, n_active, inst->n_instances, types->n_types,
                           out_new_instance, out_est_ms, out_slack_ms, out_tier, st);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

// The *_host entry points work through their input in pieces: while the kernels of piece k run
// and its results travel back on a second stream, the inputs of piece k + 1 are already on
// their way -- the link to the host carries traffic in both directions at once.
static int ensure_host_pipe(gs_ctx *ctx) {
    if (ctx->host_pipe_ready) return GS_OK;
    cudaError_t e = cudaStreamCreateWithFlags(&ctx->host_out_stream, cudaStreamNonBlocking);
    for (int k = 0; k < GS_HOST_PIECES && e == cudaSuccess; ++k)
        e = cudaEventCreateWithFlags(&ctx->host_events[k], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&ctx->host_counts, GS_HOST_PIECES * sizeof(int64_t), cudaHostAllocDefault);
    for (int k = 0; k < 2 && e == cudaSuccess; ++k)
        e = cudaHostAlloc((void **)&ctx->host_pool_image[k], pool_stage_bytes(ctx->max_instances, ctx->max_types), cudaHostAllocDefault);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->host_pipe_ready = true;
    return GS_OK;
}

// Requests per piece: a multiple of 1024 (pieces start 16-byte aligned and on whole flag words).
static int64_t host_piece(int64_t n) {
    int64_t piece = (n + GS_HOST_PIECES - 1) / GS_HOST_PIECES;
    if (piece < gs::kHostPieceMin) piece = gs::kHostPieceMin;
    return (piece + 1023) & ~(int64_t)1023;
}

static int route_batch_host(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                            const float *slo_ms, int64_t n_requests,
                            const gs_instances *inst, const gs_types *types, float ema_alpha,
                            int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                            uint8_t *out_tier, void *cuda_stream, bool wait)
{
    int rc = check_pool(ctx, inst, types, false);
    if (rc != GS_OK) return rc;
    if (n_requests < 0 || n_requests > gs::kMaxRouteRequests) return GS_ERR_INVALID_ARG;
    if (n_requests > 0 && (!prompt_len || !pred_decode_len || !slo_ms || !out_instance_idx ||
                           !out_est_e2e_ms || !out_slack_ms)) return GS_ERR_INVALID_ARG;
    if (n_requests == 0) return GS_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    if ((rc = ensure_host_pipe(ctx)) != GS_OK) return rc;
    const size_t n = (size_t)n_requests;
    const size_t bytes = pool_stage_bytes(inst->n_instances, types->n_types) + 6 * pad256(n * 4) + pad256(n);
    cudaStream_t st = (cudaStream_t)cuda_stream, out = ctx->host_out_stream;
    // (an earlier deferred round may still be sending results back from the same buffers)
    if (cudaStreamSynchronize(out) != cudaSuccess) return cuda_fail(ctx, cudaGetLastError());
    rc = ensure_stage(ctx, &ctx->stage, &ctx->stage_bytes, bytes);
    if (rc != GS_OK) return rc;
    Carver c{ctx->stage};
    PoolStage pool;
    cudaError_t e = stage_pool(c, inst, types, &pool, ctx->host_pool_image[0], st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    int32_t *dx = c.take<int32_t>(n), *dy = c.take<int32_t>(n);
    float *dD = c.take<float>(n);
    int32_t *didx = c.take<int32_t>(n);
    float *dest = c.take<float>(n), *dslack = c.take<float>(n);
    uint8_t *dtier = out_tier ? c.take<uint8_t>(n) : nullptr;
    if ((e = gs::launch_prologue(ctx, pool.inst, pool.types, ema_alpha, false, st)) != cudaSuccess) return cuda_fail(ctx, e);
    const int64_t piece = host_piece(n_requests);
    int k = 0;
    for (int64_t off = 0; off < n_requests; off += piece, ++k) {
        const size_t len = (size_t)(n_requests - off < piece ? n_requests - off : piece);
        if ((e = cudaMemcpyAsync(dx + off, prompt_len + off, len * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(dy + off, pred_decode_len + off, len * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(dD + off, slo_ms + off, len * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess)
            break;
        if ((e = gs::launch_route(ctx, dx + off, dy + off, dD + off, (int64_t)len, nullptr, inst->n_instances,
                                  types->n_types, didx + off, dest + off, dslack + off, dtier ? dtier + off : nullptr,
                                  false, false, st)) != cudaSuccess) break;
        // the piece's results go back on the second stream as soon as they exist
        if ((e = cudaEventRecord(ctx->host_events[k], st)) != cudaSuccess ||
            (e = cudaStreamWaitEvent(out, ctx->host_events[k], 0)) != cudaSuccess ||
            (e = cudaMemcpyAsync(out_instance_idx + off, didx + off, len * 4, cudaMemcpyDeviceToHost, out)) != cudaSuccess ||
            (e = cudaMemcpyAsync(out_est_e2e_ms + off, dest + off, len * 4, cudaMemcpyDeviceToHost, out)) != cudaSuccess ||
            (e = cudaMemcpyAsync(out_slack_ms + off, dslack + off, len * 4, cudaMemcpyDeviceToHost, out)) != cudaSuccess)
            break;
        if (out_tier && (e = cudaMemcpyAsync(out_tier + off, dtier + off, len, cudaMemcpyDeviceToHost, out)) != cudaSuccess)
            break;
    }
    // (after an error always: nothing may still be using the staging buffers when the call returns)
    if (wait || e != cudaSuccess) {
        const cudaError_t e1 = cudaStreamSynchronize(st), e2 = cudaStreamSynchronize(out);
        if (e == cudaSuccess) e = e1 != cudaSuccess ? e1 : e2;
    }
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_route_batch_host(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                        const float *slo_ms, int64_t n_requests,
                        const gs_instances *inst, const gs_types *types, float ema_alpha,
                        int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                        uint8_t *out_tier, void *cuda_stream)
{
    return route_batch_host(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, inst, types, ema_alpha,
                            out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier, cuda_stream, true);
}

GS_API int gs_route_batch_host_deferred(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                        const float *slo_ms, int64_t n_requests,
                        const gs_instances *inst, const gs_types *types, float ema_alpha,
                        int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                        uint8_t *out_tier, void *cuda_stream)
{
    return route_batch_host(ctx, prompt_len, pred_decode_len, slo_ms, n_requests, inst, types, ema_alpha,
                            out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier, cuda_stream, false);
}

GS_API int gs_host_wait(gs_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return GS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
    if (e == cudaSuccess && ctx->host_pipe_ready) e = cudaStreamSynchronize(ctx->host_out_stream);
    return e == cudaSuccess ? GS_OK : cuda_fail(ctx, e);
}

GS_API int gs_risk_scan_host(gs_ctx *ctx, const int32_t *assigned_inst, const int32_t *generated_tokens,
                      const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                      int64_t n_active, const gs_instances *inst, const gs_types *types,
                      uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
                      int64_t *out_cand_count, void *cuda_stream)
{
    int rc = check_pool(ctx, inst, types, false);
    if (rc != GS_OK) return rc;
    if (n_active < 0 || n_active > gs::kMaxActive || cand_capacity < 0 || !out_cand_count)
        return GS_ERR_INVALID_ARG;
    if (cand_capacity > 0 && !out_cand_idx) return GS_ERR_INVALID_ARG;
    if (n_active > 0 && (!assigned_inst || !generated_tokens || !pred_len || !elapsed_ms || !slo_ms ||
                         !out_flag_bits)) return GS_ERR_INVALID_ARG;
    if (n_active == 0) { *out_cand_count = 0; return GS_OK; }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GS_ERR_NO_DEVICE;
    if ((rc = ensure_host_pipe(ctx)) != GS_OK) return rc;
    const size_t n = (size_t)n_active;
    const size_t words = (n + 31) / 32;
    const size_t cap = (size_t)(cand_capacity < n_active ? cand_capacity : n_active);
    const size_t bytes = pool_stage_bytes(inst->n_instances, types->n_types) + 5 * pad256(n * 4) +
                         pad256(words * 4) + pad256(cap * 4) + 256;
    rc = ensure_stage(ctx, &ctx->scan_stage, &ctx->scan_stage_bytes, bytes);
    if (rc != GS_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream, out = ctx->host_out_stream;
    Carver c{ctx->scan_stage};
    PoolStage pool;
    cudaError_t e = stage_pool(c, inst, types, &pool, ctx->host_pool_image[1], st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    int32_t *dg = c.take<int32_t>(n), *dgen = c.take<int32_t>(n), *dtot = c.take<int32_t>(n);
    float *del = c.take<float>(n), *dslo = c.take<float>(n);
    uint32_t *dbits = c.take<uint32_t>(words);
    int32_t *dcand = c.take<int32_t>(cap);
    int64_t *dcount = c.take<int64_t>(2);           // running totals, two slots taken in turn
    const void *src[] = {assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms};
    void *dst[] = {dg, dgen, dtot, del, dslo};
    // every piece's copies and kernels are enqueued first: piece k scans its own requests, lists
    // its candidates behind those of the pieces before it and leaves the running total
    const int64_t piece = host_piece(n_active);
    int n_pieces = 0;
    for (int64_t off = 0; off < n_active && e == cudaSuccess; off += piece, ++n_pieces) {
        const int k = n_pieces;
        const size_t len = (size_t)(n_active - off < piece ? n_active - off : piece);
        for (int col = 0; col < 5 && e == cudaSuccess; ++col)
            e = cudaMemcpyAsync((char *)dst[col] + off * 4, (const char *)src[col] + off * 4, len * 4, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) break;
        e = gs::launch_risk(ctx, dg + off, dgen + off, dtot + off, del + off, dslo + off, (int64_t)len, pool.inst, pool.types,
                            dbits + off / 32, cap ? dcand : nullptr, (int64_t)cap, dcount + (k & 1), st,
                            k ? dcount + ((k - 1) & 1) : nullptr, (int32_t)off);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->host_counts + k, dcount + (k & 1), sizeof(int64_t), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->host_events[k], st);
    }
    // then, piece by piece as the totals arrive: its flag words and its stretch of the list go back
    // on the second stream while later pieces are still being copied in and scanned
    int64_t before = 0;
    for (int k = 0; k < n_pieces && e == cudaSuccess; ++k) {
        const int64_t off = (int64_t)k * piece;
        const size_t len = (size_t)(n_active - off < piece ? n_active - off : piece);
        if ((e = cudaEventSynchronize(ctx->host_events[k])) != cudaSuccess) break;
        const int64_t total = ctx->host_counts[k];
        e = cudaMemcpyAsync(out_flag_bits + off / 32, dbits + off / 32, ((len + 31) / 32) * 4, cudaMemcpyDeviceToHost, out);
        const int64_t lo = before < (int64_t)cap ? before : (int64_t)cap, hi = total < (int64_t)cap ? total : (int64_t)cap;
        if (e == cudaSuccess && hi > lo)
            e = cudaMemcpyAsync(out_cand_idx + lo, dcand + lo, (size_t)(hi - lo) * 4, cudaMemcpyDeviceToHost, out);
        before = total;
    }
    const cudaError_t e1 = cudaStreamSynchronize(st), e2 = cudaStreamSynchronize(out);
    if (e == cudaSuccess) e = e1 != cudaSuccess ? e1 : e2;
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    *out_cand_count = before;
    return GS_OK;
}

}  // extern "C"
