// Per-round instance prologue (one CTA):
//   1. the coefficients of Eq. 2 for every instance and the EMA step of Algorithm 1
//      (rows[g] = {q_g, p_g, d_g, free KV}, exact, in caller order);
//   2. the search structure of the route kernel.  Instances are grouped by GPU type (types
//      ordered by their largest d first) and, inside a type, put in preference order
//      (d descending, index ascending).  Over the rows of a type sits a 4-ary hierarchy of
//      blocks of 4, 16, 64, 256 consecutive rows; every block and every row becomes an
//      8-byte node holding a lower bound (q_lo, d_lo) of the q and d of the rows below it.
//      Nodes are stored in depth-first order with a skip target: "if nothing below this node
//      can meet the deadline, continue at node X".
//
// Bounds: q_lo <= q (1 - 2^-19) and d_lo <= d (1 - 2^-19), and the header keeps
// p_lo = p (1 - 2^-19).  With all coefficients non-negative and each fused step of
// T = fma(d, y, fma(p, x, q)) rounding by at most 2^-24 relative, the single-precision test
// fma(d_lo, y, q_lo) > fma(-p_lo, x, D)  then implies  T(r,g) > D  for every row below.
// The low 11 mantissa bits of the two words carry the skip target and the instance index;
// the bound is lowered by one unit of the remaining mantissa first, so it stays a lower bound.
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

// Number of nodes, inside a type's subtree, that precede every node of row s: s leaves and,
// per level l = 1 .. levels-1, the blocks of 4^l rows that start before s.
__device__ __forceinline__ int first_pos(int s, int levels) {
    int pos = s;
    for (int l = 1; l < levels; ++l) pos += (s + (1 << (2 * l)) - 1) >> (2 * l);
    return pos;
}

// Position of the block of level `level` (0 = single row) that starts at row s: after every
// higher-level block starting at the same row.
__device__ __forceinline__ int node_pos(int level, int s, int levels) {
    int pos = first_pos(s, levels);
    for (int l = level + 1; l < levels; ++l) pos += (s & ((1 << (2 * l)) - 1)) == 0;
    return pos;
}

constexpr float kShrink = 1.0f - 1.9073486328125e-6f;   // 1 - 2^-19

// Bit pattern of a lower bound of v >= 0 whose low kNodeTagBits bits are free for a tag.
__device__ __forceinline__ unsigned lower_bound_bits(float v) {
    const unsigned b = __float_as_uint(__fmul_rn(v, kShrink)) & ~kNodeTagMask;
    return b >= (kNodeTagMask + 1u) ? b - (kNodeTagMask + 1u) : 0u;
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
    __shared__ float sh_q[GS_MAX_INSTANCES], sh_d[GS_MAX_INSTANCES];       // by instance index
    __shared__ float sh_nq[kMaxNodes];                                     // exact min q per node
    __shared__ int sh_cnt[GS_MAX_TYPES], sh_rank[GS_MAX_TYPES], sh_row0[GS_MAX_TYPES + 1];
    __shared__ unsigned sh_dmax[GS_MAX_TYPES];
    __shared__ int sh_base[GS_MAX_TYPES + 1], sh_levels[GS_MAX_TYPES];
    __shared__ int sh_unsafe, sh_n_act;

    const int g = threadIdx.x;
    unsigned bad = 0;
    float d = 0.f;
    int t = 0;
    if (g < GS_MAX_TYPES) { sh_cnt[g] = 0; sh_dmax[g] = 0u; }
    if (g == 0) sh_unsafe = 0;
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
        // the bounds of the search structure need finite, non-negative coefficients
        const float big = 3.0e38f;
        if (!(q >= 0.f && q < big && p >= 0.f && p < big && d >= 0.f && d < big)) atomicOr(&sh_unsafe, 1);
        atomicAdd(&sh_cnt[t], 1);
        atomicMax(&sh_dmax[t], orderable(d));
    }
    __syncthreads();

    // ---- 2. order of the types (largest d first; ties: smaller type id) and their geometry --
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
        // thread g handles the type at order position g: rows and nodes of the types before it
        int n_act = 0, row0 = 0, base = 0, my_n = 0, my_type = -1;
        for (int o = 0; o < GS_MAX_TYPES; ++o) {
            const int r = sh_rank[o], n = sh_cnt[o];
            if (n == 0) continue;
            ++n_act;
            if (r == g) { my_n = n; my_type = o; }
            if (r < g) {
                int levels = 1;
                while ((1 << (2 * levels)) < n) ++levels;
                row0 += n;
                base += first_pos(n, levels);
            }
        }
        if (my_type >= 0) {
            int levels = 1;
            while ((1 << (2 * levels)) < my_n) ++levels;      // smallest L >= 1 with 4^L >= n
            sh_row0[g] = row0; sh_base[g] = base; sh_levels[g] = levels;
            if (g == n_act - 1) {
                sh_row0[n_act] = row0 + my_n;
                sh_base[n_act] = base + first_pos(my_n, levels);
                sh_n_act = n_act;
            }
        }
    }

    // ---- 3. sort rows by (type order, d descending, index ascending) ---------------------
    int n_sort = 32;
    while (n_sort < M) n_sort <<= 1;
    {
        unsigned long long key = ~0ull;
        if (g < M)
            key = ((unsigned long long)sh_rank[t] << 48) | ((unsigned long long)(~orderable(d)) << 16) |
                  (unsigned long long)g;
        sh_key[g] = key;
    }
    __syncthreads();
    for (int k = 2; k <= n_sort; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int partner = g ^ j;
            if (g < n_sort && partner > g) {
                const unsigned long long a = sh_key[g], b = sh_key[partner];
                const bool ascending = (g & k) == 0;
                if ((a > b) == ascending) { sh_key[g] = b; sh_key[partner] = a; }
            }
            __syncthreads();
        }
    }

    // ---- 4. leaves ------------------------------------------------------------------------
    const int n_act = sh_n_act;
    int tr = 0, k = 0, levels = 0, n_t = 0, base = 0;
    const bool is_row = g < M;
    if (is_row) {
        const unsigned long long key = sh_key[g];
        const int inst = (int)(key & 0xFFFFull);
        tr = (int)(key >> 48);
        k = g - sh_row0[tr];
        n_t = sh_row0[tr + 1] - sh_row0[tr];
        levels = sh_levels[tr];
        base = sh_base[tr];
        const int pos = base + node_pos(0, k, levels);
        const float rq = sh_q[inst];
        sh_nq[pos] = rq;
        s.nodes[pos] = make_uint2(lower_bound_bits(rq) | (unsigned)sh_base[tr + 1],
                                  lower_bound_bits(sh_d[inst]) | kNodeLeafFlag | (unsigned)inst);
    }
    __syncthreads();

    // ---- 5. blocks, bottom-up; the thread of a block's first row builds the block ----------
    for (int l = 1; l <= 5; ++l) {
        const int w = 1 << (2 * l);
        const bool type_level = (l == levels);              // covers the whole type: goes to the header
        if (is_row && l <= levels && (k & (w - 1)) == 0 && (!type_level || k == 0)) {
            const int hi = min(k + w, n_t);                 // rows [k, hi)
            float bq = 3.4e38f;
            for (int c = k; c < hi; c += (w >> 2)) bq = fminf(bq, sh_nq[base + node_pos(l - 1, c, levels)]);
            const int last_inst = (int)(sh_key[sh_row0[tr] + hi - 1] & 0xFFFFull);   // smallest d
            const float bd = sh_d[last_inst];
            if (!type_level) {
                const int pos = base + node_pos(l, k, levels);
                sh_nq[pos] = bq;
                const int skip = base + first_pos(hi, levels);
                s.nodes[pos] = make_uint2(lower_bound_bits(bq) | (unsigned)skip, lower_bound_bits(bd));
            } else {
                const int first_inst = (int)(sh_key[sh_row0[tr]] & 0xFFFFull);
                TypeHeader h;
                h.p_lo = __fmul_rn(s.rows[first_inst].p, kShrink);
                h.q_lo = __uint_as_float(lower_bound_bits(bq));
                h.d_lo = __uint_as_float(lower_bound_bits(bd));
                h.d_max = sh_d[first_inst];
                h.begin = base;
                h.end = sh_base[tr + 1];
                h.pad0 = 0; h.pad1 = 0;
                s.headers[tr] = h;
            }
        }
        __syncthreads();
    }

    if (g == 0) {
        s.table_info[0] = sh_base[n_act];      // number of nodes
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
