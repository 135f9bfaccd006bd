// Per-round instance prologue (one CTA):
//   1. the coefficients of Eq. 2 for every instance and the EMA step of Algorithm 1
//      (rows[g] = {q_g, p_g, d_g, free KV}, exact, in caller order);
//   2. the search tables of the route kernel.  Instances are grouped by GPU type (types
//      ordered by their largest d first) and, inside a type, put in preference order
//      (d descending, index ascending).  Per type the tables hold
//        - a lower bound (q_lo, d_lo) for every row, tagged with the instance index,
//        - a header with the bound over the whole type, and
//        - a start table: for a threshold on d, the first group of 8 rows that can matter.
//      A type's rows are padded to a multiple of 16 with entries that never pass a test.
//
// Bounds: q_lo <= q (1 - 2^-19), d_lo <= d (1 - 2^-19), p_lo = p (1 - 2^-19).  With all
// coefficients non-negative and each fused step of T = fma(d, y, fma(p, x, q)) rounding by at
// most 2^-24 relative, the single-precision test  fma(d_lo, y, q_lo) > fma(-p_lo, x, D)
// implies  T(r,g) > D  for every row the bound covers.  The low bits of a row's d word
// carry the instance index; the bound is lowered by one unit of the remaining mantissa
// first, so it stays a lower bound.
#include "gs_internal.cuh"

namespace gs {

__device__ __forceinline__ int clamp_count(int v, unsigned &bad) {
    if (v < 0) { bad |= GS_DEV_BAD_VALUE; return 0; }
    return v;
}

// Monotone map float -> unsigned (total order of all non-NaN floats).
__device__ __forceinline__ unsigned orderable(float f) {
    const unsigned b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

constexpr float kShrink = 1.0f - 1.9073486328125e-6f;   // 1 - 2^-19
constexpr unsigned kPadQ = 0x7FC00000u;                 // NaN: compares false with everything

// Bit pattern of a lower bound of v >= 0 whose low tag bits are zero and may be overwritten.
__device__ __forceinline__ unsigned lower_bound_bits(float v) {
    const unsigned b = __float_as_uint(__fmul_rn(v, kShrink)) & ~kRowTagMask;
    return b >= (kRowTagMask + 1u) ? b - (kRowTagMask + 1u) : 0u;
}

__global__ void __launch_bounds__(GS_MAX_INSTANCES)
prologue_kernel(const int32_t *__restrict__ type_id, const int32_t *__restrict__ queued,
                const int32_t *__restrict__ batch, const int32_t *__restrict__ free_kv,
                const float *__restrict__ q_ema, int M,
                const float *__restrict__ p_type, const float *__restrict__ a_type,
                const float *__restrict__ b_type, int n_types, float alpha,
                Scratch s)
{
    __shared__ unsigned long long sh_key[GS_MAX_INSTANCES];
    __shared__ unsigned long long sh_key2[2][GS_MAX_INSTANCES];      // exchange buffers of the sort
    __shared__ float sh_q[GS_MAX_INSTANCES], sh_d[GS_MAX_INSTANCES];       // by instance index
    __shared__ float sh_row_d[kMaxPaddedRows];                             // row d_lo as float (untagged)
    __shared__ int sh_cnt[GS_MAX_TYPES], sh_rank[GS_MAX_TYPES], sh_row0[GS_MAX_TYPES + 1];
    __shared__ unsigned sh_dmax[GS_MAX_TYPES], sh_qmin[GS_MAX_TYPES];
    __shared__ int sh_base[GS_MAX_TYPES + 1];                              // padded row offset per type
    __shared__ float sh_inv_w[GS_MAX_TYPES], sh_d0[GS_MAX_TYPES];
    __shared__ int sh_unsafe, sh_n_act;

    const int g = threadIdx.x;
    unsigned bad = 0;
    float d = 0.f;
    int t = 0;
    if (g < GS_MAX_TYPES) { sh_cnt[g] = 0; sh_dmax[g] = 0u; sh_qmin[g] = 0xFFFFFFFFu; }
    if (g == 0) sh_unsafe = 0;
    // every table entry starts as padding
    for (int i = g; i < kMaxPaddedRows; i += blockDim.x) s.row_bounds[i] = make_uint2(kPadQ, 0u);
    __syncthreads();

    // ---- 1. coefficients ----------------------------------------------------------------
    if (g < M) {
        t = type_id[g];
        if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
        const float Qtok = __int2float_rn(clamp_count(queued[g], bad));
        const float B = __int2float_rn(clamp_count(batch[g], bad));
        float qe = q_ema[g];
        if (!(qe >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; qe = 0.0f; }
        const int kv = clamp_count(free_kv[g], bad);
        const float p = p_type[t];
        d = __fmaf_rn(b_type[t], B, a_type[t]);             // loaded per-token decode latency
        const float w = __fmul_rn(Qtok, p);                 // time to drain the queued prefill
        const float keep = __fmul_rn(__fsub_rn(1.0f, alpha), qe);
        const float q = __fmaf_rn(alpha, w, keep);          // EMA step
        sh_q[g] = q; sh_d[g] = d;
        Row row; row.q = q; row.p = p; row.d = d; row.kv = kv;
        s.rows[g] = row;
        s.d_by_g[g] = d;
        s.q_by_g[g] = q;
        // the bounds of the search tables need finite, non-negative coefficients
        const float big = 3.0e38f;
        if (!(q >= 0.f && q < big && p >= 0.f && p < big && d >= 0.f && d < big)) atomicOr(&sh_unsafe, 1);
        atomicAdd(&sh_cnt[t], 1);
        atomicMax(&sh_dmax[t], orderable(d));
    }
    __syncthreads();

    // ---- 2. order of the types (largest d first; ties: smaller type id), row offsets ------
    if (g < GS_MAX_TYPES) {
        int rank = GS_MAX_TYPES;           // unused types sort last
        if (sh_cnt[g] > 0) {
            rank = 0;
            for (int o = 0; o < GS_MAX_TYPES; ++o)
                if (sh_cnt[o] > 0 && (sh_dmax[o] > sh_dmax[g] || (sh_dmax[o] == sh_dmax[g] && o < g))) ++rank;
        }
        sh_rank[g] = rank;
    }
    __syncthreads();
    if (g < GS_MAX_TYPES) {
        // thread g handles the type at order position g
        int n_act = 0, row0 = 0, base = 0, my_n = -1;
        for (int o = 0; o < GS_MAX_TYPES; ++o) {
            const int r = sh_rank[o], n = sh_cnt[o];
            if (n == 0) continue;
            ++n_act;
            if (r == g) my_n = n;
            if (r < g) { row0 += n; base += (n + 15) & ~15; }
        }
        if (my_n >= 0) {
            sh_row0[g] = row0; sh_base[g] = base;
            if (g == n_act - 1) {
                sh_row0[n_act] = row0 + my_n;
                sh_base[n_act] = base + ((my_n + 15) & ~15);
                sh_n_act = n_act;
            }
        }
    }

    // ---- 3. sort rows by (type order, d descending, index ascending) ---------------------
    // bitonic network, one key per thread: partners closer than a warp exchange by shuffle,
    // farther ones through shared memory (two buffers, so one barrier per exchange)
    int n_sort = 32;
    while (n_sort < M) n_sort <<= 1;
    unsigned long long key = ~0ull;
    if (g < M)
        key = ((unsigned long long)sh_rank[t] << 48) | ((unsigned long long)(~orderable(d)) << 16) |
              (unsigned long long)g;
    {
        int buf = 0;
        for (int k = 2; k <= n_sort; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                unsigned long long other;
                if (j >= 32) {
                    sh_key2[buf][g] = key;
                    __syncthreads();
                    other = sh_key2[buf][g ^ j];
                    buf ^= 1;
                } else {
                    other = __shfl_xor_sync(0xFFFFFFFFu, key, j);
                }
                const bool keep_min = ((g & k) == 0) == ((g & j) == 0);
                key = (keep_min == (other < key)) ? other : key;
            }
        }
    }
    sh_key[g] = key;
    __syncthreads();

    // ---- 4. row bounds, per-type minimum of q -------------------------------------------------
    const int n_act = sh_n_act;
    if (g < M) {
        const unsigned long long key = sh_key[g];
        const int inst = (int)(key & 0xFFFFull);
        const int tr = (int)(key >> 48);
        const int k = g - sh_row0[tr];
        const int base = sh_base[tr];
        const float rq = sh_q[inst];
        const unsigned d_bits = lower_bound_bits(sh_d[inst]);
        s.row_bounds[row_slot(base + k)] = make_uint2(lower_bound_bits(rq), d_bits | (unsigned)inst);
        sh_row_d[base + k] = __uint_as_float(d_bits);
        // one shared-memory atomic per run of equal types inside the warp
        const unsigned peers = __match_any_sync(__activemask(), tr);
        const unsigned qmin = __reduce_min_sync(peers, orderable(rq));
        if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicMin(&sh_qmin[tr], qmin);
    }
    __syncthreads();

    // ---- 5. headers --------------------------------------------------------------------------
    if (g < n_act) {
        const int tr = g;
        const int n_t = sh_row0[tr + 1] - sh_row0[tr];
        const int base = sh_base[tr];
        const int first_inst = (int)(sh_key[sh_row0[tr]] & 0xFFFFull);
        const unsigned qo = sh_qmin[tr];                    // undo the monotone map
        const float qmin = __uint_as_float((qo & 0x80000000u) ? (qo & 0x7FFFFFFFu) : ~qo);
        // start table geometry: kStartSlots slots between the least and the largest row bound of d
        const float d_hi = sh_row_d[base], d_low = sh_row_d[base + n_t - 1];
        float inv_w = 0.f;
        if (n_t > 16 && (d_hi - d_low) > d_hi * (1.0f / 1024.0f))
            inv_w = (float)kStartSlots / (d_hi - d_low);
        sh_inv_w[tr] = inv_w; sh_d0[tr] = d_low;
        TypeHeader h;
        h.p_lo = __fmul_rn(s.rows[first_inst].p, kShrink);   // written in step 1 by this CTA
        h.q_lo = __uint_as_float(lower_bound_bits(qmin));
        h.d_lo = d_low;
        h.d_max = sh_d[first_inst];
        h.base = base;
        h.n_padded = (n_t + 15) & ~15;
        h.inv_w = inv_w;
        h.d0 = d_low;
        s.headers[tr] = h;
    }
    __syncthreads();

    // ---- 6. start tables: slot -> first row (multiple of 8) not certainly above the slot -------
    for (int e = g; e < n_act * kStartSlots; e += blockDim.x) {
        const int tr = e / kStartSlots, slot = e % kStartSlots;
        {
            int start_row = 0;
            const float inv_w = sh_inv_w[tr];
            if (inv_w > 0.f) {
                // two slots of margin absorb the rounding of the kernel's slot computation
                const float edge = sh_d0[tr] + (float)(slot + 2) / inv_w;
                const int b0 = sh_base[tr];
                int lo = 0, hi = sh_row0[tr + 1] - sh_row0[tr];     // rows [0, lo) have d_lo > edge
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sh_row_d[b0 + mid] > edge) lo = mid + 1; else hi = mid;
                }
                start_row = lo & ~7;
            }
            s.start_table[tr * kStartSlots + slot] = (unsigned short)start_row;
        }
    }

    if (g == 0) {
        s.table_info[0] = sh_base[n_act];      // padded rows in use
        s.table_info[1] = sh_unsafe;
        s.table_info[2] = M;
        s.table_info[3] = n_act;
    }
    if (bad) atomicOr(s.status, bad);
    if (g == 0 && sh_unsafe) atomicOr(s.status, (unsigned)GS_DEV_BAD_VALUE);
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
