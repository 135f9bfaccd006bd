// Per-round instance prologue: the coefficients of Eq. 2 for every instance, the EMA step
// of Algorithm 1, and the request-independent preference order used by the just-enough pick
// (argmax d_g over the feasible set == first feasible instance when instances are visited by
// d descending, index ascending).
#include "gs_internal.cuh"

namespace gs {

__device__ __forceinline__ int clamp_count(int v, unsigned &bad) {
    if (v < 0) { bad |= GS_DEV_BAD_VALUE; return 0; }
    return v;
}

// One CTA of GS_MAX_INSTANCES threads, thread g owns instance g.
__global__ void __launch_bounds__(GS_MAX_INSTANCES)
prologue_kernel(const int32_t *__restrict__ type_id, const int32_t *__restrict__ queued,
                const int32_t *__restrict__ batch, const int32_t *__restrict__ free_kv,
                const float *__restrict__ q_ema, int M,
                const float *__restrict__ p_type, const float *__restrict__ a_type,
                const float *__restrict__ b_type, int n_types, float alpha,
                Scratch s)
{
    __shared__ float sh_d[GS_MAX_INSTANCES];
    const int g = threadIdx.x;
    unsigned bad = 0;
    float q = 0.f, p = 0.f, d = 0.f;
    int kv = 0;
    if (g < M) {
        int t = type_id[g];
        if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
        const float Qtok = __int2float_rn(clamp_count(queued[g], bad));
        const float B = __int2float_rn(clamp_count(batch[g], bad));
        float qe = q_ema[g];
        if (!(qe >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; qe = 0.0f; }
        kv = clamp_count(free_kv[g], bad);
        p = p_type[t];
        d = __fmaf_rn(b_type[t], B, a_type[t]);             // loaded per-token decode latency
        const float w = __fmul_rn(Qtok, p);                 // time to drain the queued prefill
        const float keep = __fmul_rn(__fsub_rn(1.0f, alpha), qe);
        q = __fmaf_rn(alpha, w, keep);                      // EMA step
        sh_d[g] = d;
    }
    __syncthreads();
    if (g < M) {
        // preference rank: how many instances come before g
        int rank = 0;
        for (int h = 0; h < M; ++h) {
            const float dh = sh_d[h];
            rank += (dh > d) || (dh == d && h < g);
        }
        InstRow row; row.q = q; row.p = p; row.d = d; row.kv = kv;
        s.rows[rank] = row;
        s.row_g[rank] = g;
        s.d_by_g[g] = d;
        s.q_by_g[g] = q;
    }
    if (bad) atomicOr(s.status, bad);
}

cudaError_t launch_prologue(gs_ctx *ctx, const gs_instances &inst, const gs_types &types,
                            float ema_alpha, cudaStream_t st)
{
    LaunchTimer timer(ctx, GS_K_PROLOGUE, st);
    prologue_kernel<<<1, GS_MAX_INSTANCES, 0, st>>>(
        inst.type_id, inst.queued_prefill_tokens, inst.decode_batch, inst.free_kv_tokens,
        inst.q_ema_ms, inst.n_instances, types.prefill_ms_per_tok, types.tpot_a_ms,
        types.tpot_b_ms, types.n_types, ema_alpha, ctx->s);
    return cudaGetLastError();
}

}  // namespace gs
