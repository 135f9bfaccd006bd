// gs_route_sequential: Algorithm 1 one request at a time.  Every request sees the instance
// state left by the requests before it, so the requests cannot be spread over the GPU; what
// is parallel is the loop over instances.  One CTA, up to four instances per thread: the thread
// keeps its instances' state (queued prefill tokens, decode batch, free KV, smoothed queue
// delay) in registers for the whole batch.  Per request every thread takes the EMA step of its
// instances, scores the pairs (Eq. 2) and enters a CTA-wide arg-max / arg-min; the thread that
// owns the chosen instance books the request on it and writes the outputs.  (Four per thread
// because the chain is bound by instructions issued per request on one SM: fewer warps repeat
// the cross-warp part of the reduction fewer times.)
//
// The reduction costs one barrier per request: a warp reduces its 32 candidates with redux
// instructions for all three tiers at once, writes three 64-bit keys to shared memory
// (double-buffered by request parity), and after the barrier every warp reduces the warp keys
// again for itself, so no second barrier is needed to publish the result.  Requests are staged through shared memory
// a tile at a time so that the per-request loop never waits on global memory.
#include "gs_internal.cuh"

namespace gs {

constexpr int kSeqTile = 256;            // requests staged per tile

__device__ __forceinline__ unsigned seq_orderable(float f) {
    const unsigned b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Warp-wide maximum of (hi, lo) pairs, lexicographic, over the lanes with `has`; lo is never 0
// for a lane that takes part, so a result with lo == 0 means that none did.
__device__ __forceinline__ unsigned long long warp_argmax(bool has, unsigned hi, unsigned lo) {
    const unsigned all = 0xFFFFFFFFu;
    const unsigned w_hi = __reduce_max_sync(all, has ? hi : 0u);
    const unsigned w_lo = __reduce_max_sync(all, (has && hi == w_hi) ? lo : 0u);
    return ((unsigned long long)w_hi << 32) | w_lo;
}

constexpr int kSeqPerThread = 4;         // instances per thread
constexpr int kSeqThreads = GS_MAX_INSTANCES / kSeqPerThread;

__global__ void __launch_bounds__(kSeqThreads)
sequential_kernel(const int32_t *__restrict__ prompt_len, const int32_t *__restrict__ pred_decode_len,
                  const float *__restrict__ slo_ms, int64_t n,
                  const int32_t *__restrict__ type_id, int32_t *__restrict__ queued, int32_t *__restrict__ batch,
                  int32_t *__restrict__ free_kv, float *__restrict__ q_ema, int M,
                  const float *__restrict__ p_type, const float *__restrict__ a_type,
                  const float *__restrict__ b_type, int n_types, float alpha,
                  int32_t *__restrict__ out_idx, float *__restrict__ out_est, float *__restrict__ out_slack,
                  uint8_t *__restrict__ out_tier, unsigned *__restrict__ status)
{
    __shared__ int sh_x[kSeqTile], sh_y[kSeqTile];
    __shared__ float sh_D[kSeqTile];
    __shared__ unsigned long long sh_keys[2][3][32];     // request parity x tier x warp
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_threads = blockDim.x;
    const int n_warps = (n_threads + 31) >> 5;
    unsigned bad = 0;

    // this thread's instances: tid, tid + n_threads, ...
    float p[kSeqPerThread], a[kSeqPerThread], b[kSeqPerThread], q[kSeqPerThread];
    int Q[kSeqPerThread], B[kSeqPerThread], K[kSeqPerThread];
    bool has[kSeqPerThread];
#pragma unroll
    for (int i = 0; i < kSeqPerThread; ++i) {
        const int g = tid + i * n_threads;
        has[i] = g < M;
        p[i] = a[i] = b[i] = q[i] = 0.f; Q[i] = B[i] = K[i] = 0;
        if (has[i]) {
            int t = type_id[g];
            if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
            p[i] = p_type[t]; a[i] = a_type[t]; b[i] = b_type[t];
            Q[i] = queued[g]; B[i] = batch[g]; K[i] = free_kv[g]; q[i] = q_ema[g];
            if (Q[i] < 0) { bad |= GS_DEV_BAD_VALUE; Q[i] = 0; }
            if (B[i] < 0) { bad |= GS_DEV_BAD_VALUE; B[i] = 0; }
            if (K[i] < 0) { bad |= GS_DEV_BAD_VALUE; K[i] = 0; }
        }
    }
    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    const long long kMax = 2147483647ll;

    for (int64_t r0 = 0; r0 < n; r0 += kSeqTile) {
        const int n_tile = (int)min((int64_t)kSeqTile, n - r0);
        __syncthreads();                                   // the previous tile has been consumed
        for (int k = tid; k < n_tile; k += n_threads) {
            int xv = prompt_len[r0 + k], yv = pred_decode_len[r0 + k];
            if (xv < 0) { xv = 0; bad |= GS_DEV_BAD_VALUE; }
            if (yv < 0) { yv = 0; bad |= GS_DEV_BAD_VALUE; }
            sh_x[k] = xv; sh_y[k] = yv; sh_D[k] = slo_ms[r0 + k];
        }
        __syncthreads();
        for (int k = 0; k < n_tile; ++k) {
            const int xi = sh_x[k], yi = sh_y[k];
            const float D = sh_D[k];
            const float x = __int2float_rn(xi), y = __int2float_rn(yi);
            const long long need = (long long)xi + (long long)yi;
            // per tier the best of this thread's instances as a 64-bit key (value bits, then
            // 2^32 - 1 - index, so that the larger key is the smaller index); 0 = none
            unsigned long long k1 = 0ull, k2 = 0ull, k3 = 0ull;
            float T[kSeqPerThread];
#pragma unroll
            for (int i = 0; i < kSeqPerThread; ++i) {
                // step 1: coefficients from the current state, EMA step
                if (has[i] && !(q[i] >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; q[i] = 0.0f; }
                const float d = __fmaf_rn(b[i], __int2float_rn(B[i]), a[i]);
                const float w = __fmul_rn(__int2float_rn(Q[i]), p[i]);
                q[i] = __fmaf_rn(alpha, w, __fmul_rn(one_minus_alpha, q[i]));
                // step 2: Eq. 2 and the three candidate sets
                T[i] = __fmaf_rn(d, y, __fmaf_rn(p[i], x, q[i]));
                const bool room = has[i] && need <= (long long)K[i];
                const bool feasible = room && T[i] <= D;
                const unsigned idx_key = 0xFFFFFFFFu - (unsigned)(tid + i * n_threads);
                const unsigned long long kd = ((unsigned long long)seq_orderable(d) << 32) | idx_key;
                const unsigned long long kt = ((unsigned long long)(~seq_orderable(T[i])) << 32) | idx_key;
                if (feasible && kd > k1) k1 = kd;
                if (room && kt > k2) k2 = kt;
                if (has[i] && kt > k3) k3 = kt;
            }
            // one key per warp and tier, one barrier, then every warp finishes the reduction
            // over the warp keys for itself
            unsigned long long (*slots)[32] = sh_keys[k & 1];
            k1 = warp_argmax((unsigned)k1 != 0u, (unsigned)(k1 >> 32), (unsigned)k1);
            k2 = warp_argmax((unsigned)k2 != 0u, (unsigned)(k2 >> 32), (unsigned)k2);
            k3 = warp_argmax((unsigned)k3 != 0u, (unsigned)(k3 >> 32), (unsigned)k3);
            if (lane == 0) { slots[0][warp] = k1; slots[1][warp] = k2; slots[2][warp] = k3; }
            __syncthreads();
            unsigned tier = 1;
            unsigned long long kw = lane < n_warps ? slots[0][lane] : 0ull;
            unsigned long long win = warp_argmax((unsigned)kw != 0u, (unsigned)(kw >> 32), (unsigned)kw);
            if ((unsigned)win == 0u) {
                tier = 2;
                kw = lane < n_warps ? slots[1][lane] : 0ull;
                win = warp_argmax((unsigned)kw != 0u, (unsigned)(kw >> 32), (unsigned)kw);
            }
            if ((unsigned)win == 0u) {
                tier = 3;
                kw = lane < n_warps ? slots[2][lane] : 0ull;
                win = warp_argmax((unsigned)kw != 0u, (unsigned)(kw >> 32), (unsigned)kw);
            }
            // step 3: the owner of the chosen instance books the request
            const int g_star = (int)(0xFFFFFFFFu - (unsigned)win);
#pragma unroll
            for (int i = 0; i < kSeqPerThread; ++i) {
                if (g_star == tid + i * n_threads) {
                    Q[i] = (int)min((long long)Q[i] + (long long)xi, kMax);
                    B[i] = (int)min((long long)B[i] + 1ll, kMax);
                    K[i] = (int)max((long long)K[i] - need, 0ll);
                    const int64_t r = r0 + k;
                    out_idx[r] = g_star;
                    out_est[r] = T[i];
                    out_slack[r] = __fsub_rn(D, T[i]);
                    if (out_tier) out_tier[r] = (uint8_t)tier;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kSeqPerThread; ++i) {
        const int g = tid + i * n_threads;
        if (has[i]) { queued[g] = Q[i]; batch[g] = B[i]; free_kv[g] = K[i]; q_ema[g] = q[i]; }
    }
    if (bad) atomicOr(status, bad);
}

cudaError_t launch_sequential(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                              const float *slo_ms, int64_t n, const int32_t *type_id,
                              const gs_instances_mut &state, const gs_types &types, float alpha,
                              int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                              cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    // up to kSeqPerThread instances per thread, whole warps
    const int threads = (((state.n_instances + kSeqPerThread - 1) / kSeqPerThread) + 31) & ~31;
    LaunchTimer timer(ctx, GS_K_SEQUENTIAL, st);
    sequential_kernel<<<1, threads, 0, st>>>(prompt_len, pred_decode_len, slo_ms, n, type_id,
                                             state.queued_prefill_tokens, state.decode_batch, state.free_kv_tokens,
                                             state.q_ema_ms, state.n_instances, types.prefill_ms_per_tok,
                                             types.tpot_a_ms, types.tpot_b_ms, types.n_types, alpha,
                                             out_idx, out_est, out_slack, out_tier, ctx->s.status);
    return cudaGetLastError();
}

}  // namespace gs
