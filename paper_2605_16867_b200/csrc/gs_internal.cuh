// Internal declarations shared by the translation units of libgoodserve.
// Nothing here is part of the C ABI (see include/goodserve.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "goodserve.h"

namespace gs {

// Work counters of the routing kernels, only in a library built with -DGS_COUNT_EVALS (the
// benchmark's second build; one global atomic per event, far too slow for anything else).
enum EvalCounter {
    kCountExact = 0,        // pairs (request, instance) scored exactly, T of Eq. 2 in full
    kCountBound = 1,        // row bounds tested (a lower bound of T for one pair)
    kCountTypeTest = 2,     // whole-type bounds tested
    kCountQueued = 3,       // requests that the first attempt left to the full search
    kCountFallback = 4,     // requests that ran the per-lane fallback (no feasible instance)
    kCountExhaustive = 5,   // requests scored against every instance by a whole warp
    kCountN = 8
};
cudaError_t read_eval_counters(unsigned long long *out, bool clear);     // zeros unless GS_COUNT_EVALS

// Checking build (-DGS_DEBUG), in place of a memory checker: every index into a shared-memory
// table that the search computes from table contents, and every position the prologue writes a
// table entry to, is tested against the table's size first.  A failed test is counted in a
// per-file device counter and the index pulled to 0, so the access that follows stays legal;
// nothing traps.  gs_device_status then reports GS_DEV_INTERNAL.  (GS_CHECKED compiles to the
// bare index in the regular build.)
#ifdef GS_DEBUG
#define GS_DEBUG_COUNTER(name) __device__ unsigned name
#define GS_CHECKED(counter, idx, limit) gs::checked_index(&(counter), (int)(idx), (int)(limit))
__device__ __forceinline__ int checked_index(unsigned *counter, int idx, int limit) {
    if ((unsigned)idx >= (unsigned)limit) { atomicAdd(counter, 1u); return 0; }
    return idx;
}
#else
#define GS_CHECKED(counter, idx, limit) (idx)
#endif
unsigned route_index_errors(bool clear);       // failed index checks since the last clear (0 unless GS_DEBUG)
unsigned prologue_index_errors(bool clear);

// Exact per-instance coefficients of Eq. 2 for the current round, in caller order.
struct __align__(16) Row {
    float q, p, d;
    int kv;
};

// Per-round search tables (built by the prologue, read by the route kernel).  Rows are
// grouped by GPU type and, inside a type, kept in preference order (d descending, index
// ascending); each type's rows are padded to a multiple of 16.
//   row_bounds[i]   = {bits of q_lo | instance index, bits of d_lo}   (one row)
//   start_table[(t * kStartBuckets + b) * kStartSlots + s] = first group of 8 rows of type t
//                     worth looking at when L_out falls in bucket b and the largest d that can
//                     still meet the deadline falls in slot s
// Storage slot of padded row i.  Eight consecutive rows (64 bytes) are read together as four
// 16-byte chunks; which chunk sits where is XOR-swizzled with the group number so that lanes
// reading different groups in the same instruction spread over all shared-memory banks.
__host__ __device__ __forceinline__ int row_slot(int i) {
    const int group = i >> 3, pair = (i >> 1) & 3;
    return (group << 3) | (((pair ^ ((group >> 1) & 3)) << 1) | (i & 1));
}

// Where the exact coefficients of instance g sit in the table `rows` (in global memory and in its
// shared-memory copies).  Lanes often ask for instances a fixed stride apart (all of one GPU type
// when types are dealt round robin); the low bits are mixed with the next ones so that such lanes
// spread over the shared-memory banks.  A permutation inside every aligned block of eight.
__host__ __device__ __forceinline__ int row_pos(int g) { return g ^ (((g >> 3) ^ (g >> 6)) & 7); }

constexpr unsigned kRowTagMask = 0x3FFu;            // instance index in the low bits of a q word
// groups of consecutive rank (d descending) that stand in for GPU types when the coefficients
// are given per instance
#ifndef GS_DIRECT_GROUPS
#define GS_DIRECT_GROUPS 8
#endif
constexpr int kDirectGroups = GS_DIRECT_GROUPS;
constexpr int kMaxPaddedRows = GS_MAX_INSTANCES + GS_MAX_TYPES * 16;
#ifndef GS_START_MB
#define GS_START_MB 1
#endif
#ifndef GS_START_SLOTS
#define GS_START_SLOTS 64
#endif
#ifndef GS_SLOT_WIDEN
#define GS_SLOT_WIDEN 1.0625f
#endif
constexpr int kStartSlots = GS_START_SLOTS;
constexpr int kBucketBits = GS_START_MB;  // mantissa bits of L_out that pick the bucket: 2^bits buckets per octave
constexpr int kStartBuckets = 16 << kBucketBits;   // sixteen octaves of L_out; the last bucket is open-ended

// One GPU type's entry: bound over all its rows, where its rows are, start-table geometry.
struct __align__(16) TypeHeader {
    float p_lo, q_lo, d_lo, d_max;
    int base;           // first padded row (multiple of 16)
    int n_padded;       // rows including padding (multiple of 16)
    float inv_w;        // slots per unit of d; 0 = no start table, begin at group 0
    float d0;           // d at the low edge of slot 0
};

// Candidate table: which GPU types (bit = position in the search order) can hold a feasible
// instance at all, by the slot of D / L_out among the types' least d (a type needs
// d_lo * L_out <= D).  The top slot and a pool whose types all have about the same least d
// name every type.
constexpr int kCandSlots = 64;

// Record lists (typed pools).  For every GPU type and bucket of L_out the rows that can be the
// first of their type to pass a bound test (see the prologue), as {q word, d_lo} entries in one
// pool; a list ends in kListWindow entries that never pass, so a window of that many entries
// read from any start inside the list stays inside it.
#ifndef GS_POOL_ENTRIES
#define GS_POOL_ENTRIES 8192
#endif
constexpr int kPoolEntries = GS_POOL_ENTRIES;
constexpr int kListWindow = 8;             // entries the first attempt may test (four, then four more)
constexpr int kListMax = 510;              // longer lists are not stored (start_list counts pairs of entries in a byte)
constexpr unsigned short kNoList = 0xFFFFu;
constexpr unsigned kPadQ = 0x7FC00000u;    // q word of a padding entry (a NaN: its bound test is false); no row has it

constexpr int64_t kMaxRouteRequests = (int64_t)1 << 36;   // per routing call (the kernel's queues hold a request's
                                                          // index within its CTA's run of requests in 32 bits)
#ifndef GS_HOST_PIECES
#define GS_HOST_PIECES 4                 // the *_host entry points work through their input in up to this many pieces
#endif
constexpr int64_t kHostPieceMin = 1 << 18;   // ... of at least this many requests
constexpr int kMaxScanCtas = 4096;      // CTAs of one risk scan (a few per SM), one flag count each
constexpr int kMaxActive = 2147483647;  // n_active < 2^31 (indices are int32)

// Device scratch owned by a context.
struct Scratch {
    Row *rows;                // [GS_MAX_INSTANCES] exact coefficients, instance g at row_pos(g)
    uint2 *row_bounds;        // [kMaxPaddedRows]
    float2 *group_bounds;     // [kMaxPaddedRows / 8] per eight rows: {least q word as a float, d_lo of the last row}; +inf, 0 = padding only
    float *row_p;             // [kMaxPaddedRows] lower bound of each row's p, in row order (unswizzled)
    unsigned char *start_table;   // [GS_MAX_TYPES * kStartBuckets * kStartSlots]
    TypeHeader *headers;      // [GS_MAX_TYPES] in search order (largest d first)
    int *table_info;          // {padded rows, unsafe, n_instances, n_active_types, bits of the candidate
                              //  table's origin (least d_lo of any type), bits of its slots per unit of d,
                              //  pool entries handed out to the types, 1 = q_by_g holds a round to carry,
                              //  the most free KV of any instance}
    unsigned short *cand_table;   // [kCandSlots] candidate types by slot of D / L_out
    uint2 *pool;              // [kPoolEntries] record lists
    unsigned short *bucket_list;  // [GS_MAX_TYPES * kStartBuckets] first pool entry of the list, halved; kNoList = none
    unsigned char *start_list;    // [GS_MAX_TYPES * kStartBuckets * kStartSlots] like start_table, in pairs of list entries
    float4 *chord;            // [GS_MAX_TYPES * kStartBuckets] {a, s, p_lo, -}: a + s * L_out is below every row bound of
                              //  the type for L_out in the bucket (typed pools; see the prologue)
    float *q_by_g;            // [max_instances] q_g of the latest ACCUMULATE round, caller order (carried by advance)
    unsigned long long *deltas;   // [3 * max_instances] pending sums: L_in, count, L_in + L_out
    unsigned *scan_counts;    // [kMaxScanCtas] risk scan: requests flagged by each CTA of pass 1
    unsigned *status;         // device status word
};

}  // namespace gs

struct gs_ctx {
    int device;
    int max_instances;
    int max_types;
    int n_sm;
    gs::Scratch s;
    int64_t launches;
    int last_cuda_error;
    // staging for the *_host entry points (device memory, grown on demand), and what their
    // pipeline of copies and kernels needs (created by the first such call)
    char *stage;                             // ... of gs_route_batch_host
    size_t stage_bytes;
    char *scan_stage;                        // ... of gs_risk_scan_host (its own: a routing round's results may still be
    size_t scan_stage_bytes;                 //     on their way back when the scan's inputs arrive)
    cudaStream_t host_out_stream;            // results travel back on it while the next piece's inputs arrive
    cudaEvent_t host_events[GS_HOST_PIECES]; // piece k computed
    int64_t *host_counts;                    // pinned: candidates up to and including piece k
    char *host_pool_image[2];                // pinned: the pool description as it is laid out on the device, one copy
                                             //  each for the routing and the scan entry point (they may overlap)
    bool host_pipe_ready;
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
// (ctx may be null: then nothing is counted or timed)
struct LaunchTimer {
    gs_ctx *ctx; cudaStream_t st; int kernel; cudaEvent_t start = nullptr, stop = nullptr;
    LaunchTimer(gs_ctx *c, int k, cudaStream_t s);
    ~LaunchTimer();
};

// Sparse prefix-cache state of a batch (Eq. 2's H): n_slots (instance, hit length) pairs per
// request, slot k of request r at k * slot_stride + r.
struct PrefixHits {
    const int32_t *inst;
    const int32_t *hit_len;
    int n_slots;
    int64_t slot_stride;
};

// Launches `kernel` as a programmatic dependent of the kernel before it in the stream: the launch
// may be set up, and the CTAs placed, while that kernel still runs (once all its CTAs have said so
// with griddepcontrol.launch_dependents, or have ended).  Every kernel launched this way waits
// (griddepcontrol.wait: the whole earlier grid done, its stores visible) before it reads or
// writes anything an earlier kernel of the stream may touch.  Hides a launch latency per kernel.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// launchers (each returns the cudaError_t of its launch)
cudaError_t launch_prologue(gs_ctx *ctx, const gs_instances &inst, const gs_types &types,
                            float ema_alpha, bool carry_q, cudaStream_t st);
cudaError_t launch_sequential(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                              const float *slo_ms, int64_t n, const int32_t *type_id,
                              const gs_instances_mut &state, const gs_types &types, float alpha,
                              int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                              cudaStream_t st);
cudaError_t launch_ema(gs_ctx *ctx, float alpha, int M, const float *obs_q, const float *obs_p, const float *obs_d,
                       float *q, float *p, float *d, cudaStream_t st);
cudaError_t launch_prologue_direct(gs_ctx *ctx, const gs_instance_table &tab, cudaStream_t st);
cudaError_t launch_route(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                         const float *slo_ms, int64_t n, const PrefixHits *hits, int n_instances, int n_types,
                         int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                         bool accumulate, bool row_p, cudaStream_t st);
cudaError_t launch_reroute(gs_ctx *ctx, const int32_t *cand_idx, const int64_t *cand_count, int64_t cand_capacity,
                           const int32_t *assigned, const int32_t *generated, const int32_t *pred_len,
                           const float *elapsed, const float *slo, const int32_t *prompt_len, int64_t n_active,
                           int n_instances, int n_types, int32_t *out_inst, float *out_est, float *out_slack, uint8_t *out_tier,
                           cudaStream_t st);
cudaError_t configure_route(gs_ctx *ctx);
cudaError_t configure_prologue();
cudaError_t launch_advance(gs_ctx *ctx, const gs_instances_mut &inst, cudaStream_t st);
cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n_active, const gs_instances &inst, const gs_types &types,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st,
                        const int64_t *prev_count = nullptr, int32_t index_base = 0);   // a scan in pieces: see risk.cu

}  // namespace gs
