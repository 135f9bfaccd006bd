/*
 * goodserve.h -- C ABI of the GoodServe routing hot path on one NVIDIA B200 (sm_100a).
 *
 * Two operations of the paper's proxy router are provided as data-parallel GPU passes:
 *
 *   gs_route_batch   for every pending request r and every serving instance g, the
 *                    end-to-end latency estimate  T(r,g) = q_g + p_g * L_in_r + d_g * L_out_r
 *                    (Eq. 2 with no prefix-cache hit), the feasible set {g : T(r,g) <= D_r}
 *                    restricted to instances with KV room, the "just-enough" choice
 *                    argmax d_g over that set, and the fallback argmin T when the set is
 *                    empty (Algorithm 1; Sec. 3.4).
 *   gs_route_batch_prefix  the same round with Eq. 2's prefix-cache term: per request a
 *                    few (instance, cached prefix length) pairs lower T on those instances.
 *   gs_route_batch_direct / gs_ema_update   the same round against per-instance q, p, d given
 *                    directly (black-box estimates smoothed by an EMA, Sec. 3.3).
 *   gs_route_sequential  Algorithm 1 one request at a time, each seeing the state left by the
 *                    ones before it (the literal reading; a single dependent chain).
 *   gs_risk_scan     for every active request, the SLO-violation risk test of Sec. 3.4
 *                    (expected finish time under the latest estimates exceeds the SLO) and
 *                    the ascending list of flagged requests (migration candidates).
 *   gs_advance_state between the rounds of a stream, folds one round's assignments back
 *                    into the per-instance queue / batch / KV state and carries the smoothed
 *                    queue delay of the EMA step (Algorithm 1) to the next round.
 *
 * Conventions that hold for every call unless its comment says otherwise
 *   - Units: times in milliseconds (float), token counts int32.
 *   - All array arguments of the device entry points are DEVICE pointers owned by the
 *     caller; arrays must be 16-byte aligned (else GS_ERR_ALIGN).  The *_host variants take
 *     HOST pointers (pinned memory makes their copies asynchronous) and stage through
 *     buffers owned by the context.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Device entry points only enqueue work on it and return; they do not synchronise.
 *   - Return value: GS_OK or a negative gs_error.  Every error but GS_ERR_CUDA is found in the
 *     arguments before anything is enqueued; GS_ERR_CUDA (a launch or copy that the CUDA runtime
 *     refused) can leave the part of the call that came before it on the stream.
 *   - Invalid DATA never faults or traps: negative token counts and negative/NaN q_ema are
 *     read as 0, a type id outside [0, n_types) as type 0, an assigned instance outside
 *     [0, n_instances) is clamped into range; a bit of the device status word records it
 *     (gs_device_status).  A NaN deadline is never met, so such a request takes the fallback.
 *   - Calls of the same kind on one context must not overlap on the GPU (they share the
 *     context's scratch memory).  gs_route_batch / gs_advance_state on one stream and
 *     gs_risk_scan on another may overlap each other: they use separate scratch.
 */
#ifndef GOODSERVE_H_
#define GOODSERVE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define GS_API __attribute__((visibility("default")))
#else
#define GS_API
#endif

#define GS_MAX_INSTANCES 1024   /* instance table is staged whole in shared memory */
#define GS_MAX_TYPES 16

typedef struct gs_ctx gs_ctx;   /* opaque; owns only scratch memory and a status word */

enum gs_error {
    GS_OK = 0,
    GS_ERR_INVALID_ARG = -1,    /* NULL pointer, negative size, n_instances < 1, ... */
    GS_ERR_CAPACITY = -2,       /* n_instances or n_types above what the context was created for */
    GS_ERR_CUDA = -3,           /* a CUDA runtime call failed; see gs_last_cuda_error */
    GS_ERR_ALIGN = -4,          /* an array pointer is not 16-byte aligned */
    GS_ERR_NO_DEVICE = -5,      /* no usable CUDA device */
    GS_ERR_TOO_LARGE = -6       /* gs_risk_scan_noalloc: n_active above GS_NOALLOC_MAX_ACTIVE */
};

/* bits of the device status word */
enum gs_dev_status {
    GS_DEV_BAD_INSTANCE = 1,    /* assigned_inst outside [0, n_instances) was clamped */
    GS_DEV_BAD_TYPE = 2,        /* type_id outside [0, n_types) was read as 0 */
    GS_DEV_BAD_VALUE = 4,       /* negative count or negative/NaN q_ema was read as 0 */
    GS_DEV_TIMEOUT = 8,         /* a bounded device-side wait expired (the route kernel's wait for its table
                                   copies); the outputs of that call are invalid */
    GS_DEV_CAND_TRUNCATED = 16, /* more flagged requests than cand_capacity; list was cut */
    GS_DEV_INTERNAL = 32        /* only from a library built with -DGS_DEBUG: one of its index checks failed
                                   (a table index computed by the search fell outside its table) */
};

/* gs_route_batch flags */
#define GS_ROUTE_ACCUMULATE 1u  /* also add this round's assignments to the context's pending
                                   per-instance deltas, to be applied by gs_advance_state */

/* Per-instance serving state, structure of arrays, n_instances entries each.
 * Together with the type table these give the coefficients of Eq. 2:
 *   p_g = prefill_ms_per_tok[type_id[g]]
 *   d_g = tpot_a_ms[t] + tpot_b_ms[t] * decode_batch[g]       (per-token decode latency under load)
 *   w_g = queued_prefill_tokens[g] * p_g                      (stand-in for the observed wait)
 *   q_g = alpha * w_g + (1 - alpha) * q_ema_ms[g]             (EMA step of Algorithm 1)
 * free_kv_tokens[g] bounds L_in + L_out of a request placed on g (the memory constraint). */
typedef struct gs_instances {
    const int32_t *type_id;
    const int32_t *queued_prefill_tokens;
    const int32_t *decode_batch;
    const int32_t *free_kv_tokens;
    const float   *q_ema_ms;
    int32_t        n_instances;      /* 1 .. GS_MAX_INSTANCES */
} gs_instances;

/* Per-GPU-type constants, n_types entries each (1 .. GS_MAX_TYPES). */
typedef struct gs_types {
    const float *prefill_ms_per_tok;
    const float *tpot_a_ms;
    const float *tpot_b_ms;
    int32_t      n_types;
} gs_types;

/* Mutable view of the same instance state for gs_advance_state. */
typedef struct gs_instances_mut {
    int32_t *queued_prefill_tokens;
    int32_t *decode_batch;
    int32_t *free_kv_tokens;
    float   *q_ema_ms;
    int32_t  n_instances;
} gs_instances_mut;

/* Create a context on CUDA device `device` for pools of up to `max_instances` instances and
 * `max_types` types.  Allocates the context's scratch memory (a few MB) with cudaMalloc.
 * `*out` receives the context; destroy it with gs_destroy. */
GS_API int gs_create(gs_ctx **out, int device, int max_instances, int max_types);

/* Frees everything the context owns.  The caller makes sure no call is still running. */
GS_API int gs_destroy(gs_ctx *ctx);

/* Static, never-NULL description of a gs_error code. */
GS_API const char *gs_strerror(int code);

/* cudaError_t of the last failed CUDA call of this context (0 if none), as int. */
GS_API int gs_last_cuda_error(const gs_ctx *ctx);

/* Synchronises `cuda_stream`, then reads and clears the device status word. */
GS_API int gs_device_status(gs_ctx *ctx, void *cuda_stream, unsigned *out_bits);

/* Number of kernels this context has launched since it was created. */
GS_API int64_t gs_launch_count(const gs_ctx *ctx);

/* Work counters of the routing kernels, for benchmarks.  Synchronises `cuda_stream`, copies the
 * GS_EVAL_COUNT counters to `out` (host) and clears them if `clear` != 0.  They count, since they
 * were last cleared: [0] request-instance pairs scored exactly (T of Eq. 2 evaluated in full),
 * [1] per-instance lower bounds of T tested, [2] whole-type lower bounds tested, [3] requests that
 * the straight-line first attempt left to the full search, [4] requests that ran the fallback
 * (Algorithm 1's else branch), [5] requests scored against every instance by a whole warp.
 * Only a library built with -DGS_COUNT_EVALS counts (one global atomic per event: a measuring
 * build, many times slower); the regular build returns zeros. */
#define GS_EVAL_COUNT 8
GS_API int gs_eval_counters(gs_ctx *ctx, void *cuda_stream, uint64_t *out, int clear);

/* Kernels of the library, for gs_timing_read. */
enum gs_kernel {
    GS_K_PROLOGUE = 0,       /* instance coefficients + preference order (per round) */
    GS_K_ROUTE = 1,          /* pair scoring + selection */
    GS_K_ADVANCE = 2,        /* state advance */
    GS_K_RISK_FLAGS = 3,     /* risk test + flag words + per-chunk flag counts */
    GS_K_RISK_SCATTER = 4,   /* ordered candidate list */
    GS_K_REROUTE = 5,        /* re-routing of the candidates */
    GS_K_EMA = 6,            /* EMA step of directly given coefficients */
    GS_K_SEQUENTIAL = 7,     /* one-request-at-a-time routing */
    GS_K_COUNT = 8
};

/* Optional per-kernel timing for benchmarks.  While enabled (on != 0) every kernel launch of
 * this context is bracketed by a pair of CUDA events on the launching stream.
 * gs_timing_read waits for the recorded events, adds their durations to per-kernel totals,
 * and returns the total milliseconds and number of launches of `kernel` since timing was
 * last enabled.  Off by default; enabling it resets the totals. */
GS_API int gs_timing_enable(gs_ctx *ctx, int on);
GS_API int gs_timing_read(gs_ctx *ctx, int kernel, double *total_ms, int64_t *launches);

/*
 * One routing round (Algorithm 1 applied to every pending request against one snapshot of
 * the instance state; the EMA step is taken once per round).
 *
 * Inputs, n_requests entries each:  prompt_len = L_in, pred_decode_len = predicted L_out,
 * slo_ms = D_r.   Outputs, n_requests entries each:
 *   out_instance_idx  g*            (index into the caller's instance arrays)
 *   out_est_e2e_ms    T(r, g*)      computed as fma(d, L_out, fma(p, L_in, q)) in float
 *   out_slack_ms      D_r - T(r, g*)
 *   out_tier          (may be NULL) 1 = just-enough pick among feasible instances,
 *                     2 = no feasible instance: minimum T among instances with KV room,
 *                     3 = no instance has KV room: minimum T among all.
 * Ties (equal d_g, or equal T in the fallback) go to the smallest instance index.
 * Feasibility is T <= D (a request whose estimate equals its deadline is feasible).
 * n_requests == 0 is valid; more than 2^36 requests in one call is refused (GS_ERR_INVALID_ARG,
 * nothing enqueued).  Never writes the instance state.
 */
GS_API int gs_route_batch(gs_ctx *ctx,
                   const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms, int64_t n_requests,
                   const gs_instances *inst, const gs_types *types, float ema_alpha,
                   int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                   uint8_t *out_tier, unsigned flags, void *cuda_stream);

/*
 * One routing round with the prefix-cache term of Eq. 2,
 *   T(r,g) = q_g + p_g * (L_in_r - H_{r,g}) + d_g * L_out_r,
 * where H_{r,g} (Algorithm 1's ReusePrefix) is the number of prompt tokens of r already cached
 * on g.  H is given in sparse form: n_slots (instance, hit length) pairs per request; every
 * pair not named has H = 0.
 *
 * prefix_inst, prefix_hit_len: device arrays of n_slots * slot_stride int32 entries; slot k
 * of request r is at index k * slot_stride + r.  slot_stride >= n_requests and a multiple of
 * 4 (each slot's column starts 16-byte aligned, else GS_ERR_ALIGN).  0 <= n_slots <=
 * GS_MAX_PREFIX_SLOTS; with n_slots == 0 the two pointers are not read and the result is that
 * of gs_route_batch.
 *   - a slot whose instance is negative is empty;
 *   - an instance >= n_instances names nothing: the slot is ignored and GS_DEV_BAD_INSTANCE set;
 *   - a hit length is clamped into [0, L_in]; one outside sets GS_DEV_BAD_VALUE;
 *   - an instance named by several slots keeps its longest hit.
 * The estimate is computed as fma(d, L_out, fma(p, L_in - H, q)) in float.  The memory
 * constraint is the one of gs_route_batch (L_in + L_out <= free_kv_tokens): a cached prefix
 * does not lower it.  Outputs, tiers, ties and feasibility as for gs_route_batch.  Does not
 * touch the context's pending per-instance deltas.
 */
#define GS_MAX_PREFIX_SLOTS 8
GS_API int gs_route_batch_prefix(gs_ctx *ctx,
                   const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms, int64_t n_requests,
                   const int32_t *prefix_inst, const int32_t *prefix_hit_len, int n_slots,
                   int64_t slot_stride,
                   const gs_instances *inst, const gs_types *types, float ema_alpha,
                   int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                   uint8_t *out_tier, void *cuda_stream);

/*
 * Black-box instance coefficients (Sec. 3.3): q_g, p_g and d_g of Eq. 2 estimated directly from
 * their recent observed values and smoothed by an exponential moving average, with no
 * reference to GPU type, batch size or queue content.
 *
 * Per-instance table, structure of arrays, n_instances entries each, DEVICE pointers:
 *   q_ms            smoothed queueing delay q_g
 *   p_ms_per_tok    smoothed per-token prefill latency p_g
 *   d_ms_per_tok    smoothed per-token decode latency d_g
 *   free_kv_tokens  bounds L_in + L_out of a request placed on g
 */
typedef struct gs_instance_table {
    const float *q_ms;
    const float *p_ms_per_tok;
    const float *d_ms_per_tok;
    const int32_t *free_kv_tokens;
    int32_t n_instances;
} gs_instance_table;

/*
 * One EMA step per instance for up to three coefficient columns, in place:
 *   c[g] <- fma(alpha, obs[g], (1 - alpha) * c[g])                 for c in {q, p, d}.
 * obs_* are device arrays of n_instances fresh observations; a NULL obs pointer skips that
 * column (its state pointer is then not read and may be NULL too).  An observation that is
 * negative or NaN is no observation: that entry keeps its value and GS_DEV_BAD_VALUE is set.
 * 1 <= n_instances <= the context's max_instances.  Only enqueues work on the stream.
 */
GS_API int gs_ema_update(gs_ctx *ctx, float alpha, int32_t n_instances,
                  const float *obs_q_ms, const float *obs_p_ms_per_tok, const float *obs_d_ms_per_tok,
                  float *q_ms, float *p_ms_per_tok, float *d_ms_per_tok, void *cuda_stream);

/*
 * One routing round (as gs_route_batch) against coefficients given directly.  The table is
 * used as it is: no EMA step is taken inside the round (gs_ema_update is that step).  A
 * negative or NaN coefficient is read as 0 and a negative free_kv_tokens as 0, with
 * GS_DEV_BAD_VALUE set; an infinite coefficient also sets it and makes every request of the
 * round take the exhaustive (still exact) path.  Outputs, tiers, ties and feasibility as for
 * gs_route_batch; the estimate is fma(d, L_out, fma(p, L_in, q)) in float.  Does not touch the
 * context's pending per-instance deltas.
 */
GS_API int gs_route_batch_direct(gs_ctx *ctx,
                   const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms, int64_t n_requests, const gs_instance_table *table,
                   int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                   uint8_t *out_tier, void *cuda_stream);

/*
 * Algorithm 1 one request at a time (its literal reading): the requests are taken in array
 * order and each one sees the instance state left by the ones before it.  For every request
 *   1. every instance takes the EMA step on the current state (w_g = queued_g * p_g,
 *      q_g <- alpha * w_g + (1 - alpha) * q_g) and d_g = a_t + b_t * batch_g is read from the
 *      current batch,
 *   2. T(r,g), the feasible set, the just-enough pick and the fallback are those of
 *      gs_route_batch,
 *   3. the chosen instance takes the request (queued += L_in, batch += 1,
 *      free KV -= L_in + L_out, saturating as in gs_advance_state) and the smoothed q_g of
 *      step 1 becomes the carried state of every instance.
 * This equals n_requests rounds of gs_route_batch(ACCUMULATE) + gs_advance_state with one
 * request each.  `type_id` (n_instances entries) is read; `state` is advanced IN PLACE and is
 * the pool's state after the last request when the stream reaches the end of the call.
 * The requests form one dependent chain, so a single thread block does the work, one thread
 * for up to four instances: about 1.5 million requests per second at 1,024 instances, whatever
 * the GPU's size (every request updates and scores every instance: the chain is bound by the
 * instructions one SM can issue per request).
 * It exists to measure what the snapshot reading of gs_route_batch changes (the herd onto
 * one instance within a round), not as the fast path.  Outputs and error behaviour as for
 * gs_route_batch; n_requests == 0 enqueues nothing and leaves the state as it is.
 */
GS_API int gs_route_sequential(gs_ctx *ctx,
                   const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms, int64_t n_requests,
                   const int32_t *type_id, const gs_instances_mut *state, const gs_types *types,
                   float ema_alpha,
                   int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                   uint8_t *out_tier, void *cuda_stream);

/*
 * Applies the deltas accumulated by gs_route_batch(..., GS_ROUTE_ACCUMULATE) since the last
 * advance: per instance g,  queued_prefill_tokens += sum of L_in routed to g  (saturating at
 * INT32_MAX), decode_batch += number of requests routed to g (saturating),
 * free_kv_tokens = max(free_kv_tokens - sum of (L_in + L_out), 0), and q_ema_ms = q_g of the
 * latest GS_ROUTE_ACCUMULATE round (other routing calls in between do not disturb it; without
 * such a round since the last advance q_ema_ms is left as it is).  Clears the pending deltas.  Integer sums, so the result does not depend on
 * the order in which requests were processed.
 */
GS_API int gs_advance_state(gs_ctx *ctx, const gs_instances_mut *inst, void *cuda_stream);

/*
 * SLO-violation risk scan over n_active ongoing requests (Sec. 3.4).  Per request i:
 *   rem    = max(pred_len[i] - generated_tokens[i], 0)      (pred_len is the re-estimated TOTAL)
 *   finish = fma(d_{assigned_inst[i]}, rem, elapsed_ms[i])
 *   flag   = finish > slo_ms[i]                              (strict: "exceeds")
 * Outputs: out_flag_bits, ceil(n_active / 32) words, request i is bit (i % 32) of word
 * (i / 32), unused high bits zero; out_cand_idx, the ascending indices of flagged requests,
 * at most cand_capacity of them (may be NULL when cand_capacity == 0); out_cand_count, ONE
 * int64 on the device that receives the TRUE number of flagged requests even when it exceeds
 * cand_capacity (then GS_DEV_CAND_TRUNCATED is set).  n_active must be < 2^31.
 */
GS_API int gs_risk_scan(gs_ctx *ctx,
                 const int32_t *assigned_inst, const int32_t *generated_tokens,
                 const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                 int64_t n_active,
                 const gs_instances *inst, const gs_types *types,
                 uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
                 int64_t *out_cand_count, void *cuda_stream);

/*
 * Re-routing of the scan's candidates (Sec. 3.4: a request whose expected finish exceeds its
 * SLO is re-routed to another instance with stronger processing capability, still by the
 * just-enough rule; the migration moves token IDs, so the target re-prefills the context).
 *
 * cand_idx / cand_count are gs_risk_scan's outputs (device; at most cand_capacity entries are
 * read); the five active columns are those given to the scan, prompt_len[n_active] is the
 * requests' L_in.  For candidate j = request i = cand_idx[j] on instance c = assigned_inst[i]:
 *   x' = prompt_len[i] + generated_tokens[i]      tokens the target has to prefill again
 *   y' = max(pred_len[i] - generated_tokens[i], 0) tokens left to decode
 *   D' = slo_ms[i] - elapsed_ms[i]                 time left
 *   eligible instances: d_g < d_c  (strictly lower per-token decode latency than where it runs)
 * and Algorithm 1 is applied to (x', y', D') over the eligible instances only.  Outputs, one
 * entry per candidate (cand_capacity entries each): out_new_instance (-1: no eligible instance,
 * the request is already on the fastest one), out_est_ms = T(x', y', g*), out_slack_ms = D' - T,
 * out_tier (may be NULL): 0 no move, 1 just-enough pick, 2 / 3 fallback among eligible
 * instances with / without KV room.  Uses the instance snapshot given here (EMA step included).
 */
GS_API int gs_reroute_candidates(gs_ctx *ctx,
                                 const int32_t *cand_idx, const int64_t *cand_count, int64_t cand_capacity,
                                 const int32_t *assigned_inst, const int32_t *generated_tokens,
                                 const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                                 const int32_t *prompt_len, int64_t n_active,
                                 const gs_instances *inst, const gs_types *types, float ema_alpha,
                                 int32_t *out_new_instance, float *out_est_ms, float *out_slack_ms,
                                 uint8_t *out_tier, void *cuda_stream);

/*
 * Host-buffer variants: every pointer (including those inside `inst` and `types`) is a HOST
 * pointer.  The call copies the inputs to context-owned device buffers (grown with
 * cudaMalloc when a larger size is first seen), runs the same kernels, copies the results
 * back and synchronises `cuda_stream` before returning.  No alignment requirement.
 * gs_risk_scan_host writes the true count to *out_cand_count (host) and returns at most
 * cand_capacity indices.
 */
GS_API int gs_route_batch_host(gs_ctx *ctx,
                        const int32_t *prompt_len, const int32_t *pred_decode_len,
                        const float *slo_ms, int64_t n_requests,
                        const gs_instances *inst, const gs_types *types, float ema_alpha,
                        int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                        uint8_t *out_tier, void *cuda_stream);

GS_API int gs_risk_scan_host(gs_ctx *ctx,
                      const int32_t *assigned_inst, const int32_t *generated_tokens,
                      const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                      int64_t n_active,
                      const gs_instances *inst, const gs_types *types,
                      uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
                      int64_t *out_cand_count, void *cuda_stream);

/*
 * gs_route_batch_host that returns as soon as all its copies and kernels are enqueued, so that
 * the results of the routing round (Algorithm 1) travel back to the host while the caller's
 * next call -- typically gs_risk_scan_host for the same scheduling tick (Sec. 3.4) -- already
 * sends its inputs the other way.  Same arguments, same results.  The input and output buffers
 * must stay untouched, and the outputs are not valid, until gs_host_wait, or any later
 * gs_route_batch_host / gs_risk_scan_host call on this context, has returned GS_OK.  With
 * pageable (not pinned) host memory the copies, and so the call, block as usual.
 * Errors: as gs_route_batch_host; what fails on the device later is reported by the call that
 * waits.
 */
GS_API int gs_route_batch_host_deferred(gs_ctx *ctx,
                        const int32_t *prompt_len, const int32_t *pred_decode_len,
                        const float *slo_ms, int64_t n_requests,
                        const gs_instances *inst, const gs_types *types, float ema_alpha,
                        int32_t *out_instance_idx, float *out_est_e2e_ms, float *out_slack_ms,
                        uint8_t *out_tier, void *cuda_stream);

/* Waits for everything the *_host calls of this context have enqueued on `cuda_stream` and on
 * the context's own copy stream.  GS_ERR_CUDA if any of it failed. */
GS_API int gs_host_wait(gs_ctx *ctx, void *cuda_stream);

/*
 * Risk scan without any allocation.  (The paper has no counterpart: this entry point exists
 * only because of how some callers must run, not because of the method.)
 *
 * Who needs it: code that may not call cudaMalloc / cudaFree or anything that might -- a
 * serving process that handed all device memory to its KV-cache allocator at start-up, a
 * plugin running inside someone else's memory pool, a latency-critical loop where an
 * allocation's implicit device synchronisation is unacceptable.  Such callers cannot create
 * a gs_ctx (gs_create allocates), so this call takes none: the scratch that gs_risk_scan
 * keeps in its context (the per-CTA flag counts its two passes exchange) lives instead
 * in a fixed array inside the library image, 16 KB that every GPU loading the library
 * holds until the process exits.  It computes exactly what gs_risk_scan computes, with the
 * same kernels; inputs, outputs and their layout are the same and still belong to the caller.
 *
 *   - Runs on the CURRENT device (cudaGetDevice) and enqueues on `cuda_stream`, which must
 *     belong to it.  No cudaMalloc, cudaFree or allocating library routine is called.
 *   - n_active may not exceed GS_NOALLOC_MAX_ACTIVE (the stated limit of this entry point); a
 *     larger value returns GS_ERR_TOO_LARGE and enqueues nothing.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress).  Make that first call outside any stream capture.
 *   - All calls on one GPU share the one array, and it keeps the previous call's contents;
 *     the call rewrites every word it later reads, so results never depend on earlier calls.
 *     But two calls that overlap on the GPU (different streams, or different host threads)
 *     race on the array and give wrong results: serialise them.
 *   - out_status_bits (device pointer to one word, may be NULL) is OR-ed with gs_dev_status
 *     bits; the caller zeroes it beforehand.  With NULL the bits are dropped.
 */
#define GS_NOALLOC_MAX_ACTIVE 16777216

GS_API int gs_risk_scan_noalloc(const int32_t *assigned_inst, const int32_t *generated_tokens,
                                const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                                int64_t n_active,
                                const gs_instances *inst, const gs_types *types,
                                uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
                                int64_t *out_cand_count, unsigned *out_status_bits, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* GOODSERVE_H_ */
