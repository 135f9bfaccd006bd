// gs_route_batch kernels: pair scoring (Eq. 2), feasibility, just-enough pick and fallback
// (Algorithm 1) for every pending request of a round.
//
// One thread owns one request.  The per-round instance table (rows in preference order:
// d descending, index ascending) is staged once per CTA in shared memory; every lane of a
// warp walks the same rows, so each shared-memory read is a broadcast.  Because the
// preference order does not depend on the request, argmax d_g over the feasible set is the
// FIRST feasible row, and a lane stops scanning as soon as it has found one.
#include "gs_internal.cuh"

namespace gs {

constexpr int kRouteThreads = 256;

// T(r,g) of Eq. 2 with H = 0, each step rounded once.
__device__ __forceinline__ float latency(const InstRow &r, float x, float y) {
    return __fmaf_rn(r.d, y, __fmaf_rn(r.p, x, r.q));
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

template <bool kAccumulate>
__global__ void __launch_bounds__(kRouteThreads)
route_scan_kernel(const int32_t *__restrict__ prompt_len, const int32_t *__restrict__ pred_decode_len,
                  const float *__restrict__ slo_ms, int64_t n, int M,
                  const InstRow *__restrict__ rows, const int *__restrict__ row_g,
                  int32_t *__restrict__ out_idx, float *__restrict__ out_est,
                  float *__restrict__ out_slack, uint8_t *__restrict__ out_tier,
                  unsigned long long *__restrict__ deltas, unsigned *__restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    InstRow *sh_rows = reinterpret_cast<InstRow *>(smem);
    int *sh_g = reinterpret_cast<int *>(sh_rows + M);
    unsigned long long *hist = reinterpret_cast<unsigned long long *>(
        smem + (((size_t)M * (sizeof(InstRow) + sizeof(int)) + 15) & ~(size_t)15));

    for (int k = threadIdx.x; k < M; k += blockDim.x) {
        sh_rows[k] = rows[k];
        sh_g[k] = row_g[k];
    }
    if (kAccumulate)
        for (int k = threadIdx.x; k < 3 * M; k += blockDim.x) hist[k] = 0ull;
    __syncthreads();

    unsigned bad = 0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int lane = threadIdx.x & 31;
    // `base` is the warp's first request, so the trip count is uniform across the warp
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31); base < n; base += stride) {
        const int64_t i = base + lane;
        const bool valid = i < n;
        int xi = valid ? prompt_len[i] : 0, yi = valid ? pred_decode_len[i] : 0;
        if (xi < 0) { xi = 0; bad |= GS_DEV_BAD_VALUE; }
        if (yi < 0) { yi = 0; bad |= GS_DEV_BAD_VALUE; }
        const float D = valid ? slo_ms[i] : 0.f;
        const float x = __int2float_rn(xi), y = __int2float_rn(yi);
        const unsigned need = (unsigned)xi + (unsigned)yi;    // < 2^32, no overflow

        int pick = -1;                         // row of the just-enough pick
        float T_pick = 0.f;
        int row_k = -1, row_a = -1;            // fallback rows: min T among KV-ok / among all
        int g_k = 0, g_a = 0;
        float T_k = 0.f, T_a = 0.f;
        for (int k = 0; k < M; ++k) {
            const InstRow r = sh_rows[k];
            const float T = latency(r, x, y);
            const bool kv_ok = need <= (unsigned)r.kv;
            if (kv_ok && T <= D) { pick = k; T_pick = T; break; }
            const int g = sh_g[k];
            if (kv_ok && (row_k < 0 || T < T_k || (T == T_k && g < g_k))) { row_k = k; T_k = T; g_k = g; }
            if (row_a < 0 || T < T_a || (T == T_a && g < g_a)) { row_a = k; T_a = T; g_a = g; }
        }
        int row; float T; uint8_t tier;
        if (pick >= 0)       { row = pick;  T = T_pick; tier = 1; }
        else if (row_k >= 0) { row = row_k; T = T_k;    tier = 2; }
        else                 { row = row_a; T = T_a;    tier = 3; }
        const int g = sh_g[row];
        if (valid) {
            out_idx[i] = g;
            out_est[i] = T;
            out_slack[i] = __fsub_rn(D, T);
            if (out_tier) out_tier[i] = tier;
        }
        if (kAccumulate) accumulate_choice(hist, M, valid ? g : -1, (unsigned)xi, need);
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

cudaError_t launch_route(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                         const float *slo_ms, int64_t n, int M,
                         int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                         bool accumulate, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    size_t smem = (((size_t)M * (sizeof(InstRow) + sizeof(int)) + 15) & ~(size_t)15);
    if (accumulate) smem += (size_t)3 * M * sizeof(unsigned long long);
    int64_t blocks = (n + kRouteThreads - 1) / kRouteThreads;
    const int64_t cap = (int64_t)ctx->n_sm * 8;
    if (blocks > cap) blocks = cap;
    LaunchTimer timer(ctx, GS_K_ROUTE, st);
    if (accumulate)
        route_scan_kernel<true><<<(unsigned)blocks, kRouteThreads, smem, st>>>(
            prompt_len, pred_decode_len, slo_ms, n, M, ctx->s.rows, ctx->s.row_g,
            out_idx, out_est, out_slack, out_tier, ctx->s.deltas, ctx->s.status);
    else
        route_scan_kernel<false><<<(unsigned)blocks, kRouteThreads, smem, st>>>(
            prompt_len, pred_decode_len, slo_ms, n, M, ctx->s.rows, ctx->s.row_g,
            out_idx, out_est, out_slack, out_tier, ctx->s.deltas, ctx->s.status);
    return cudaGetLastError();
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
