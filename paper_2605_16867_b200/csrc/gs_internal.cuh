// Internal declarations shared by the translation units of libgoodserve.
// Nothing here is part of the C ABI (see include/goodserve.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "goodserve.h"

namespace gs {

// Exact per-instance coefficients of Eq. 2 for the current round, in caller order.
struct __align__(16) Row {
    float q, p, d;
    int kv;
};

// The per-round search structure (built by the prologue, walked by the route kernel) is an
// array of 8-byte nodes in depth-first order, one subtree per GPU type.  Node words:
//   x: lower bound of q over the rows below, low 11 bits = target node index (where the walk
//      continues when this node's bound fails; for a leaf, the end of its type's subtree)
//   y: lower bound of d over the rows below, low 11 bits = 0 for a block,
//      kNodeLeafFlag | instance index for a leaf (one instance).
constexpr unsigned kNodeTagMask = 0x7FFu;
constexpr unsigned kNodeLeafFlag = 0x400u;
constexpr int kMaxNodes = 1536;         // 1024 leaves + every block of 4/16/64/256 rows, any type mix

// One GPU type's entry point: bound over all its rows, and its node range.
struct __align__(16) TypeHeader {
    float p_lo, q_lo, d_lo, d_max;
    int begin, end, pad0, pad1;
};

constexpr int kRiskChunk = 1024;        // requests per warp-chunk of the risk scan (32 flag words)
constexpr int kMaxActive = 2147483647;  // n_active < 2^31 (indices are int32)

// Device scratch owned by a context.
struct Scratch {
    Row *rows;                // [max_instances] exact coefficients, caller order
    uint2 *nodes;             // [kMaxNodes] search structure of the current round
    TypeHeader *headers;      // [GS_MAX_TYPES] in walk order (largest d first)
    int *table_info;          // {n_nodes, unsafe, n_instances, n_active_types}
    float *d_by_g;            // [max_instances] d_g in caller order (risk scan gather)
    float *q_by_g;            // [max_instances] q_g in caller order (carried by advance)
    unsigned long long *deltas;   // [3 * max_instances] pending sums: L_in, count, L_in + L_out
    unsigned *chunk_counts;   // [chunk_cap + 1] flagged requests per risk chunk, then offsets
    unsigned *status;         // device status word
};

}  // namespace gs

struct gs_ctx {
    int device;
    int max_instances;
    int max_types;
    int n_sm;
    int route_ctas_per_sm;
    gs::Scratch s;
    size_t chunk_cap;
    int64_t launches;
    int last_cuda_error;
    // staging for the *_host entry points (device memory, grown on demand)
    char *stage;
    size_t stage_bytes;
    // optional per-kernel timing (gs_timing_enable)
    bool timing;
    struct TimedLaunch { int kernel; cudaEvent_t start, stop; };
    std::vector<TimedLaunch> *pending;       // recorded, not yet resolved
    std::vector<cudaEvent_t> *free_events;   // recycled events
    double time_ms[GS_K_COUNT];
    int64_t time_launches[GS_K_COUNT];
};

namespace gs {

// Brackets one kernel launch with events when timing is enabled; counts the launch.
struct LaunchTimer {
    gs_ctx *ctx; cudaStream_t st; int kernel; cudaEvent_t start = nullptr, stop = nullptr;
    LaunchTimer(gs_ctx *c, int k, cudaStream_t s);
    ~LaunchTimer();
};

// launchers (each returns the cudaError_t of its launch)
cudaError_t launch_prologue(gs_ctx *ctx, const gs_instances &inst, const gs_types &types,
                            float ema_alpha, cudaStream_t st);
cudaError_t launch_route(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                         const float *slo_ms, int64_t n, int n_instances,
                         int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                         bool accumulate, cudaStream_t st);
cudaError_t configure_route(gs_ctx *ctx);
cudaError_t launch_advance(gs_ctx *ctx, const gs_instances_mut &inst, cudaStream_t st);
cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n_active, int n_instances,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st);

}  // namespace gs
