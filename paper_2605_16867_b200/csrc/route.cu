// gs_route_batch kernels: pair scoring (Eq. 2), feasibility, just-enough pick and fallback
// (Algorithm 1) for every pending request of a round.
//
// One thread owns four consecutive requests (128-bit column loads and stores).  The per-round
// tables built by the prologue are staged once per CTA in shared memory.  For each request and
// each GPU type in turn (types with the largest d first):
//   1. the type is tested against a lower bound of T over all its instances (the same
//      shared-memory address for all lanes: a broadcast) and dropped if it cannot meet the
//      deadline or cannot beat the best d found so far;
//   2. a start table turns the largest d that could still meet the deadline into the first
//      group of 16 rows worth looking at;
//   3. from there, four block bounds (4 rows each) are tested per step until one passes, the
//      four rows of that block are tested against their own bounds, and a row that passes is
//      scored exactly as the definition says, T = fma(d, y, fma(p, x, q)), and checked against
//      the deadline and the instance's free KV.
// Rows of a type are in preference order (d descending, index ascending), so the first
// feasible row of a type is that type's best.  Every bound is a true lower bound in the
// kernel's own arithmetic, so nothing feasible is ever skipped and the result is exactly
// argmax d_g over the feasible set, ties to the smallest index.
//
// A request for which this finds nothing (no feasible instance: the fallback of Algorithm 1)
// is queued in shared memory and finished by a whole warp that scores every instance, lanes
// across instances, with shuffle reductions for the argmin.
#include "gs_internal.cuh"

namespace gs {

constexpr int kRouteThreads = 256;
constexpr int kReqPerThread = 4;
constexpr int kRouteTile = kRouteThreads * kReqPerThread;

// T(r,g) of Eq. 2 with H = 0, each step rounded once.
__device__ __forceinline__ float latency(const Row &r, float x, float y) {
    return __fmaf_rn(r.d, y, __fmaf_rn(r.p, x, r.q));
}

__device__ __forceinline__ unsigned orderable_bits(float f) {
    const unsigned b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_orderable_bits(unsigned o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
}

// Adds one routed request to the CTA's pending-delta histogram.  Lanes of the warp that
// chose the same instance are combined first, so a herd onto one instance costs three
// shared-memory atomics per warp instead of 96.  Called by all 32 lanes; g < 0 = no request.
__device__ __forceinline__ void accumulate_choice(unsigned long long *hist, int M, int g,
                                                  unsigned x, unsigned need)
{
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, g);
    const unsigned x_lo = __reduce_add_sync(peers, x & 0xFFFFu);
    const unsigned x_hi = __reduce_add_sync(peers, x >> 16);
    const unsigned n_lo = __reduce_add_sync(peers, need & 0xFFFFu);
    const unsigned n_hi = __reduce_add_sync(peers, need >> 16);
    const int lane = threadIdx.x & 31;
    if (g >= 0 && lane == __ffs(peers) - 1) {
        atomicAdd(&hist[g], ((unsigned long long)x_hi << 16) + x_lo);
        atomicAdd(&hist[M + g], (unsigned long long)__popc(peers));
        atomicAdd(&hist[2 * M + g], ((unsigned long long)n_hi << 16) + n_lo);
    }
}

// Shared-memory image of the round's tables.
struct Tables {
    const TypeHeader *headers;
    const float2 *block_bounds;
    const uint2 *row_bounds;
    const unsigned short *start_table;
    const Row *rows;
    int n_types;
};

__device__ __forceinline__ bool bound_passes(float q_lo, float d_lo, float y, float R) {
    return __fmaf_rn(d_lo, y, q_lo) <= R;
}

// Just-enough pick for one request; called by all 32 lanes of the warp together.
// Returns the chosen instance or -1 (no feasible one, or a request this search does not take).
__device__ __forceinline__ int pick_instance(const Tables &tb, float x, float y, float D, unsigned need,
                                             float &T_out)
{
    int g_best = -1;
    float d_best = -1.0f, T_best = 0.f;
    const float ry = __frcp_rn(y);            // y == 0 never gets here with a live type (see caller)
    for (int t = 0; t < tb.n_types; ++t) {
        const float4 h = *reinterpret_cast<const float4 *>(&tb.headers[t]);   // p_lo, q_lo, d_lo, d_max
        const float R = __fmaf_rn(-h.x, x, D) + 1e-30f;
        const bool live = bound_passes(h.y, h.z, y, R) && !(h.w < d_best);
        if (!__any_sync(0xFFFFFFFFu, live)) continue;
        if (live) {
            const int4 g4 = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);  // base, n_groups, inv_w, d0
            const int n_groups = g4.y;
            const float inv_w = __int_as_float(g4.z);
            int grp = 0;
            if (inv_w > 0.f) {
                // largest d that can still meet the deadline -> slot -> first group worth a look
                const float z = (R - h.y) * ry;
                const float sf = fminf(fmaxf((z - __int_as_float(g4.w)) * inv_w, 0.f), (float)(kStartSlots - 1));
                grp = tb.start_table[t * kStartSlots + __float2int_rd(sf)];
            }
            const float2 *blocks = tb.block_bounds + (g4.x >> 2);
            const uint2 *rowb = tb.row_bounds + g4.x;
            bool done = false;
            while (!done) {
                unsigned m = 0;
                for (; grp < n_groups; ++grp) {
                    const float4 a = *reinterpret_cast<const float4 *>(blocks + 4 * grp);
                    const float4 b = *reinterpret_cast<const float4 *>(blocks + 4 * grp + 2);
                    m = (bound_passes(a.x, a.y, y, R) ? 1u : 0u) | (bound_passes(a.z, a.w, y, R) ? 2u : 0u) |
                        (bound_passes(b.x, b.y, y, R) ? 4u : 0u) | (bound_passes(b.z, b.w, y, R) ? 8u : 0u);
                    if (m) break;
                }
                if (!m) break;                                   // type exhausted
                do {
                    const int blk = __ffs(m) - 1;
                    m &= m - 1;
                    const uint4 *rp = reinterpret_cast<const uint4 *>(rowb + 16 * grp + 4 * blk);
                    const uint4 r0 = rp[0], r1 = rp[1];
                    unsigned rm =
                        (bound_passes(__uint_as_float(r0.x), __uint_as_float(r0.y), y, R) ? 1u : 0u) |
                        (bound_passes(__uint_as_float(r0.z), __uint_as_float(r0.w), y, R) ? 2u : 0u) |
                        (bound_passes(__uint_as_float(r1.x), __uint_as_float(r1.y), y, R) ? 4u : 0u) |
                        (bound_passes(__uint_as_float(r1.z), __uint_as_float(r1.w), y, R) ? 8u : 0u);
                    while (rm) {
                        const int rr = __ffs(rm) - 1;
                        rm &= rm - 1;
                        const unsigned dw = rr == 0 ? r0.y : rr == 1 ? r0.w : rr == 2 ? r1.y : r1.w;
                        const int inst = (int)(dw & kRowTagMask);
                        const Row row = tb.rows[inst];
                        const float T = latency(row, x, y);
                        const bool feasible = (T <= D) && (need <= (unsigned)row.kv);
                        const bool worse = row.d < d_best;
                        if (feasible && !worse && (g_best < 0 || row.d > d_best || inst < g_best)) {
                            d_best = row.d; g_best = inst; T_best = T;
                        }
                        // feasible: the rest of this type ranks lower.  worse: so does all that follows.
                        if (feasible || worse) { done = true; rm = 0; m = 0; }
                    }
                } while (m);
                ++grp;
            }
        }
    }
    T_out = T_best;
    return g_best;
}

template <bool kAccumulate>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const int32_t *__restrict__ prompt_len, const int32_t *__restrict__ pred_decode_len,
             const float *__restrict__ slo_ms, int64_t n,
             const Row *__restrict__ g_rows, const uint2 *__restrict__ g_row_bounds,
             const float2 *__restrict__ g_block_bounds, const unsigned short *__restrict__ g_start_table,
             const TypeHeader *__restrict__ g_headers, const int *__restrict__ table_info,
             int32_t *__restrict__ out_idx, float *__restrict__ out_est,
             float *__restrict__ out_slack, uint8_t *__restrict__ out_tier,
             unsigned long long *__restrict__ deltas, unsigned *__restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int n_padded = table_info[0];
    const bool unsafe = table_info[1] != 0;
    const int M = table_info[2];
    const int n_act = table_info[3];
    Row *sh_rows = reinterpret_cast<Row *>(smem);
    TypeHeader *sh_headers = reinterpret_cast<TypeHeader *>(sh_rows + GS_MAX_INSTANCES);
    uint2 *sh_row_bounds = reinterpret_cast<uint2 *>(sh_headers + GS_MAX_TYPES);
    float2 *sh_block_bounds = reinterpret_cast<float2 *>(sh_row_bounds + kMaxPaddedRows);
    unsigned short *sh_start = reinterpret_cast<unsigned short *>(sh_block_bounds + kMaxBlocks);
    int *sh_queue = reinterpret_cast<int *>(sh_start + GS_MAX_TYPES * kStartSlots);
    int *sh_qcount = sh_queue + kRouteTile;
    unsigned long long *hist = reinterpret_cast<unsigned long long *>(sh_qcount + 4);

    for (int k = threadIdx.x; k < M; k += blockDim.x) sh_rows[k] = g_rows[k];
    for (int k = threadIdx.x; k < n_padded; k += blockDim.x) sh_row_bounds[k] = g_row_bounds[k];
    for (int k = threadIdx.x; k < (n_padded >> 2); k += blockDim.x) sh_block_bounds[k] = g_block_bounds[k];
    for (int k = threadIdx.x; k < n_act * kStartSlots; k += blockDim.x) sh_start[k] = g_start_table[k];
    if (threadIdx.x < n_act) sh_headers[threadIdx.x] = g_headers[threadIdx.x];
    if (threadIdx.x == 0) *sh_qcount = 0;
    if (kAccumulate)
        for (int k = threadIdx.x; k < 3 * M; k += blockDim.x) hist[k] = 0ull;
    __syncthreads();

    Tables tb;
    tb.headers = sh_headers; tb.block_bounds = sh_block_bounds; tb.row_bounds = sh_row_bounds;
    tb.start_table = sh_start; tb.rows = sh_rows;
    tb.n_types = unsafe ? 0 : n_act;          // unusable bounds: every request takes the exhaustive path

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned bad = 0;
    const int64_t n_tiles = (n + kRouteTile - 1) / kRouteTile;
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t first = tile * kRouteTile + (int64_t)threadIdx.x * kReqPerThread;
        int xi[kReqPerThread], yi[kReqPerThread];
        float D[kReqPerThread];
        if (first + kReqPerThread <= n) {
            const int4 xv = __ldcs(reinterpret_cast<const int4 *>(prompt_len + first));
            const int4 yv = __ldcs(reinterpret_cast<const int4 *>(pred_decode_len + first));
            const float4 dv = __ldcs(reinterpret_cast<const float4 *>(slo_ms + first));
            xi[0] = xv.x; xi[1] = xv.y; xi[2] = xv.z; xi[3] = xv.w;
            yi[0] = yv.x; yi[1] = yv.y; yi[2] = yv.z; yi[3] = yv.w;
            D[0] = dv.x; D[1] = dv.y; D[2] = dv.z; D[3] = dv.w;
        } else {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j) {
                const bool v = first + j < n;
                xi[j] = v ? prompt_len[first + j] : 0;
                yi[j] = v ? pred_decode_len[first + j] : 0;
                D[j] = v ? slo_ms[first + j] : -1.0f;
            }
        }
        int g_out[kReqPerThread];
        float T_out[kReqPerThread];
#pragma unroll
        for (int j = 0; j < kReqPerThread; ++j) {
            if (xi[j] < 0) { xi[j] = 0; bad |= GS_DEV_BAD_VALUE; }
            if (yi[j] < 0) { yi[j] = 0; bad |= GS_DEV_BAD_VALUE; }
            const unsigned need = (unsigned)xi[j] + (unsigned)yi[j];      // < 2^32, no overflow
            const bool valid = first + j < n;
            // an empty slot, or L_out == 0 (the start table divides by it), skips the search;
            // a real request that comes back empty-handed goes to the exhaustive path below
            const float Dj = (valid && yi[j] > 0) ? D[j] : -1.0f;
            g_out[j] = pick_instance(tb, __int2float_rn(xi[j]), __int2float_rn(yi[j]), Dj, need, T_out[j]);
            if (valid && g_out[j] < 0) sh_queue[atomicAdd(sh_qcount, 1)] = threadIdx.x * kReqPerThread + j;
            if (kAccumulate) accumulate_choice(hist, M, valid ? g_out[j] : -1, (unsigned)xi[j], need);
        }
        if (first + kReqPerThread <= n) {
            __stcs(reinterpret_cast<int4 *>(out_idx + first), make_int4(g_out[0], g_out[1], g_out[2], g_out[3]));
            __stcs(reinterpret_cast<float4 *>(out_est + first), make_float4(T_out[0], T_out[1], T_out[2], T_out[3]));
            __stcs(reinterpret_cast<float4 *>(out_slack + first),
                   make_float4(__fsub_rn(D[0], T_out[0]), __fsub_rn(D[1], T_out[1]),
                               __fsub_rn(D[2], T_out[2]), __fsub_rn(D[3], T_out[3])));
            if (out_tier) *reinterpret_cast<uchar4 *>(out_tier + first) = make_uchar4(1, 1, 1, 1);
        } else {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j)
                if (first + j < n) {
                    out_idx[first + j] = g_out[j];
                    out_est[first + j] = T_out[j];
                    out_slack[first + j] = __fsub_rn(D[j], T_out[j]);
                    if (out_tier) out_tier[first + j] = 1;
                }
        }
        __syncthreads();

        // ---- requests with no feasible instance: one warp each, lanes across instances ----
        const int n_queued = *sh_qcount;
        for (int e = warp; e < n_queued; e += kRouteThreads / 32) {
            const int64_t r = tile * kRouteTile + sh_queue[e];
            int xr = prompt_len[r], yr = pred_decode_len[r];
            if (xr < 0) xr = 0;
            if (yr < 0) yr = 0;
            const float Dr = slo_ms[r];
            const float x = __int2float_rn(xr), y = __int2float_rn(yr);
            const unsigned need = (unsigned)xr + (unsigned)yr;
            unsigned long long k_feas = 0ull;                    // max over feasible: (d, smallest index)
            unsigned long long k_room = ~0ull, k_all = ~0ull;    // min over KV-ok / all: (T, index)
            float T_feas = 0.f;
            for (int inst = lane; inst < M; inst += 32) {
                const Row row = sh_rows[inst];
                const float T = latency(row, x, y);
                const bool room = need <= (unsigned)row.kv;
                const unsigned long long kt = ((unsigned long long)orderable_bits(T) << 32) | (unsigned)inst;
                if (kt < k_all) k_all = kt;
                if (room && kt < k_room) k_room = kt;
                if (room && T <= Dr) {
                    const unsigned long long kd =
                        ((unsigned long long)orderable_bits(row.d) << 32) | (0xFFFFu - (unsigned)inst);
                    if (kd > k_feas) { k_feas = kd; T_feas = T; }
                }
            }
            unsigned long long w_feas = k_feas, w_room = k_room, w_all = k_all;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const unsigned long long a = __shfl_xor_sync(0xFFFFFFFFu, w_feas, off);
                const unsigned long long b = __shfl_xor_sync(0xFFFFFFFFu, w_room, off);
                const unsigned long long c = __shfl_xor_sync(0xFFFFFFFFu, w_all, off);
                if (a > w_feas) w_feas = a;
                if (b < w_room) w_room = b;
                if (c < w_all) w_all = c;
            }
            int g; float T; uint8_t tier;
            if (w_feas != 0ull) {
                const unsigned owner = __ballot_sync(0xFFFFFFFFu, k_feas == w_feas);
                T = __shfl_sync(0xFFFFFFFFu, T_feas, __ffs(owner) - 1);
                g = (int)(0xFFFFu - (unsigned)(w_feas & 0xFFFFu)); tier = 1;
            } else if (w_room != ~0ull) {
                g = (int)(w_room & 0xFFFFFFFFull); T = from_orderable_bits((unsigned)(w_room >> 32)); tier = 2;
            } else {
                g = (int)(w_all & 0xFFFFFFFFull); T = from_orderable_bits((unsigned)(w_all >> 32)); tier = 3;
            }
            if (lane == 0) {
                out_idx[r] = g;
                out_est[r] = T;
                out_slack[r] = __fsub_rn(Dr, T);
                if (out_tier) out_tier[r] = tier;
                if (kAccumulate) {
                    atomicAdd(&hist[g], (unsigned long long)(unsigned)xr);
                    atomicAdd(&hist[M + g], 1ull);
                    atomicAdd(&hist[2 * M + g], (unsigned long long)need);
                }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) *sh_qcount = 0;
        __syncthreads();
    }
    if (bad) atomicOr(status, bad);

    if (kAccumulate) {
        __syncthreads();
        for (int k = threadIdx.x; k < 3 * M; k += blockDim.x) {
            const unsigned long long v = hist[k];
            if (v) atomicAdd(&deltas[(k / M) * GS_MAX_INSTANCES + (k % M)], v);
        }
    }
}

constexpr size_t kRouteSmemBase = (size_t)GS_MAX_INSTANCES * sizeof(Row) + GS_MAX_TYPES * sizeof(TypeHeader) +
                                  (size_t)kMaxPaddedRows * sizeof(uint2) + (size_t)kMaxBlocks * sizeof(float2) +
                                  (size_t)GS_MAX_TYPES * kStartSlots * sizeof(unsigned short) +
                                  (kRouteTile + 4) * sizeof(int);
constexpr size_t kRouteSmemHist = (size_t)3 * GS_MAX_INSTANCES * sizeof(unsigned long long);

cudaError_t launch_route(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                         const float *slo_ms, int64_t n, int M,
                         int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                         bool accumulate, cudaStream_t st)
{
    (void)M;
    if (n == 0) return cudaSuccess;
    const size_t smem = kRouteSmemBase + (accumulate ? kRouteSmemHist : 0);
    const int64_t n_tiles = (n + kRouteTile - 1) / kRouteTile;
    int64_t blocks = n_tiles;
    const int64_t cap = (int64_t)ctx->n_sm * ctx->route_ctas_per_sm;
    if (blocks > cap) blocks = cap;
    LaunchTimer timer(ctx, GS_K_ROUTE, st);
    if (accumulate)
        route_kernel<true><<<(unsigned)blocks, kRouteThreads, smem, st>>>(
            prompt_len, pred_decode_len, slo_ms, n, ctx->s.rows, ctx->s.row_bounds, ctx->s.block_bounds,
            ctx->s.start_table, ctx->s.headers,
            ctx->s.table_info, out_idx, out_est, out_slack, out_tier, ctx->s.deltas, ctx->s.status);
    else
        route_kernel<false><<<(unsigned)blocks, kRouteThreads, smem, st>>>(
            prompt_len, pred_decode_len, slo_ms, n, ctx->s.rows, ctx->s.row_bounds, ctx->s.block_bounds,
            ctx->s.start_table, ctx->s.headers,
            ctx->s.table_info, out_idx, out_est, out_slack, out_tier, ctx->s.deltas, ctx->s.status);
    return cudaGetLastError();
}

// Raises the dynamic shared-memory limit of the route kernels (called once per context).
cudaError_t configure_route(gs_ctx *ctx)
{
    cudaError_t e = cudaFuncSetAttribute(route_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kRouteSmemBase + kRouteSmemHist));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(route_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRouteSmemBase);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, route_kernel<false>, kRouteThreads, kRouteSmemBase);
    if (e != cudaSuccess) return e;
    ctx->route_ctas_per_sm = occ > 0 ? occ : 1;
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------
// state advance between rounds of a stream
// ---------------------------------------------------------------------------------------

__global__ void advance_kernel(int32_t *__restrict__ queued, int32_t *__restrict__ batch,
                               int32_t *__restrict__ free_kv, float *__restrict__ q_ema, int M,
                               unsigned long long *__restrict__ deltas,
                               const float *__restrict__ q_by_g)
{
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= M) return;
    const long long kMax = 2147483647ll;
    const long long dq = (long long)deltas[g];
    const long long db = (long long)deltas[GS_MAX_INSTANCES + g];
    const long long dk = (long long)deltas[2 * GS_MAX_INSTANCES + g];
    deltas[g] = 0ull; deltas[GS_MAX_INSTANCES + g] = 0ull; deltas[2 * GS_MAX_INSTANCES + g] = 0ull;
    long long Q = max(queued[g], 0), B = max(batch[g], 0), K = max(free_kv[g], 0);
    Q = min(Q + dq, kMax);
    B = min(B + db, kMax);
    K = max(K - dk, 0ll);
    queued[g] = (int32_t)Q;
    batch[g] = (int32_t)B;
    free_kv[g] = (int32_t)K;
    q_ema[g] = q_by_g[g];
}

cudaError_t launch_advance(gs_ctx *ctx, const gs_instances_mut &inst, cudaStream_t st)
{
    const int M = inst.n_instances;
    LaunchTimer timer(ctx, GS_K_ADVANCE, st);
    advance_kernel<<<(M + 255) / 256, 256, 0, st>>>(inst.queued_prefill_tokens, inst.decode_batch,
                                                    inst.free_kv_tokens, inst.q_ema_ms, M,
                                                    ctx->s.deltas, ctx->s.q_by_g);
    return cudaGetLastError();
}

}  // namespace gs
