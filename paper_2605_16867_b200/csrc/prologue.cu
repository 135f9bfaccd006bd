// Per-round instance prologue (one CTA):
//   1. the coefficients of Eq. 2 for every instance and the EMA step of Algorithm 1;
//   2. the search structure of the route kernel: instances grouped by GPU type (types by
//      their largest d first), each group in preference order (d descending, index
//      ascending), with a 4-ary hierarchy of lower bounds over consecutive rows, laid out in
//      depth-first order with skip links ("if nothing below this node can meet the deadline,
//      continue at node X").
//
// The bound of an inner node is (min q, p, min d, max kv) over the rows below it, with the
// three real coefficients shrunk by 2^-19 so that, in the kernel's own single-precision
// arithmetic,  bound > D  implies  T(r,g) > D  for every row below (all terms are
// non-negative; each of the two fused steps of T rounds by at most 2^-24 relative).
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

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Position, inside its type's subtree, of the first node that belongs to row s
// (the highest-level block starting at s, or the subtree's end when s == n).
__device__ __forceinline__ int first_pos(int s, int levels) {
    int pos = 1 + s;
    for (int l = 1, w = 4; l < levels; ++l, w <<= 2) pos += (s + w - 1) / w;
    return pos;
}

// Position, inside its type's subtree, of the block of level `level` (0 = leaf row) that
// starts at row s: after every higher-level block that starts at the same row.
__device__ __forceinline__ int node_pos(int level, int s, int levels) {
    int pos = first_pos(s, levels);
    int w = 4;
    for (int l = 1; l <= level; ++l) w <<= 2;
    for (int l = level + 1; l < levels; ++l, w <<= 2) pos += (s % w) == 0;
    return pos;
}

constexpr float kShrink = 1.0f - 1.9073486328125e-6f;   // 1 - 2^-19

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
    __shared__ int sh_kv[GS_MAX_INSTANCES];
    __shared__ float sh_nq[kMaxNodes];                                     // node q / kv while building
    __shared__ int sh_nkv[kMaxNodes];
    __shared__ int sh_cnt[GS_MAX_TYPES], sh_rank[GS_MAX_TYPES], sh_row0[GS_MAX_TYPES + 1];
    __shared__ unsigned sh_dmax[GS_MAX_TYPES];
    __shared__ int sh_base[GS_MAX_TYPES], sh_end[GS_MAX_TYPES], sh_levels[GS_MAX_TYPES];
    __shared__ float sh_p[GS_MAX_TYPES];
    __shared__ int sh_n_nodes, sh_unsafe, sh_n_act;
    // top-level nodes over types: position, first/last type (in order), skip target
    __shared__ int sh_sup_pos[GS_MAX_TYPES], sh_sup_a[GS_MAX_TYPES], sh_sup_b[GS_MAX_TYPES],
        sh_sup_skip[GS_MAX_TYPES], sh_n_sup;

    const int g = threadIdx.x;
    unsigned bad = 0;
    float q = 0.f, p = 0.f, d = 0.f;
    int kv = 0, t = 0;
    if (g < GS_MAX_TYPES) { sh_cnt[g] = 0; sh_dmax[g] = 0u; }
    if (g == 0) { sh_unsafe = 0; sh_n_sup = 0; }
    __syncthreads();

    // ---- 1. coefficients ----------------------------------------------------------------
    if (g < M) {
        t = type_id[g];
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
        sh_q[g] = q; sh_d[g] = d; sh_kv[g] = kv;
        s.d_by_g[g] = d;
        s.q_by_g[g] = q;
        // the bounds of the search structure need finite, non-negative coefficients
        const float big = 3.0e38f;
        if (!(q >= 0.f && q < big && p >= 0.f && p < big && d >= 0.f && d < big)) atomicOr(&sh_unsafe, 1);
        atomicAdd(&sh_cnt[t], 1);
        atomicMax(&sh_dmax[t], orderable(d));
    }
    __syncthreads();

    // ---- 2. order of the types: largest d first (ties: smaller type id) ------------------
    if (g < GS_MAX_TYPES) {
        int rank = 0;
        if (sh_cnt[g] > 0) {
            for (int o = 0; o < GS_MAX_TYPES; ++o)
                if (sh_cnt[o] > 0 && (sh_dmax[o] > sh_dmax[g] || (sh_dmax[o] == sh_dmax[g] && o < g))) ++rank;
        } else {
            rank = GS_MAX_TYPES;       // unused types sort last
        }
        sh_rank[g] = rank;
    }
    __syncthreads();

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

    // ---- 4. per-type geometry of the hierarchy (one thread; at most 16 types) ------------
    if (g == 0) {
        int order[GS_MAX_TYPES], n_act = 0;
        for (int r = 0; r < GS_MAX_TYPES; ++r)
            for (int o = 0; o < GS_MAX_TYPES; ++o)
                if (sh_rank[o] == r && sh_cnt[o] > 0) order[n_act++] = o;
        int row = 0;
        int nodes_of[GS_MAX_TYPES];
        for (int r = 0; r < n_act; ++r) {
            const int n = sh_cnt[order[r]];
            sh_row0[r] = row; row += n;
            int levels = 1;
            for (int w = 4; w < n; w <<= 2) ++levels;       // smallest L >= 1 with 4^L >= n
            sh_levels[r] = levels;
            nodes_of[r] = first_pos(n, levels);
            // sh_p is indexed by order position from here on
        }
        sh_row0[n_act] = row;
        float p_by_order[GS_MAX_TYPES];
        for (int r = 0; r < n_act; ++r) p_by_order[r] = p_type[order[r]];
        for (int r = 0; r < n_act; ++r) sh_p[r] = p_by_order[r];
        // binary tree over the types, depth-first, with an explicit stack
        int stack_a[2 * GS_MAX_TYPES], stack_b[2 * GS_MAX_TYPES], stack_sup[2 * GS_MAX_TYPES], sp = 0;
        int pos = 0, n_sup = 0;
        stack_a[sp] = 0; stack_b[sp] = n_act; stack_sup[sp] = -1; ++sp;
        // entries with stack_sup >= 0 are "close this super node" markers
        while (sp > 0) {
            --sp;
            const int a = stack_a[sp], b = stack_b[sp], mark = stack_sup[sp];
            if (mark >= 0) { sh_sup_skip[mark] = pos; continue; }
            if (b - a == 1) {
                sh_base[a] = pos; pos += nodes_of[a]; sh_end[a] = pos;
            } else if (b - a > 1) {
                const int id = n_sup++;
                sh_sup_pos[id] = pos++; sh_sup_a[id] = a; sh_sup_b[id] = b;
                const int mid = (a + b + 1) / 2;
                stack_a[sp] = 0; stack_b[sp] = 0; stack_sup[sp] = id; ++sp;        // close marker
                stack_a[sp] = mid; stack_b[sp] = b; stack_sup[sp] = -1; ++sp;      // right half
                stack_a[sp] = a; stack_b[sp] = mid; stack_sup[sp] = -1; ++sp;      // left half first
            }
        }
        sh_n_nodes = pos; sh_n_sup = n_sup; sh_n_act = n_act;
    }
    __syncthreads();

    // ---- 5. leaves ------------------------------------------------------------------------
    const int n_act = sh_n_act;
    int tr = 0, k = 0, levels = 0, n_t = 0, base = 0, inst = 0;
    const bool is_row = g < M;
    if (is_row) {
        const unsigned long long key = sh_key[g];
        inst = (int)(key & 0xFFFFull);
        tr = (int)(key >> 48);
        k = g - sh_row0[tr];
        n_t = sh_row0[tr + 1] - sh_row0[tr];
        levels = sh_levels[tr];
        base = sh_base[tr];
        const int pos = node_pos(0, k, levels);
        const float rq = sh_q[inst], rd = sh_d[inst];
        const int rkv = sh_kv[inst];
        Node nd; nd.q = rq; nd.p = sh_p[tr]; nd.d = rd; nd.kv = rkv;
        s.nodes[base + pos] = nd;
        s.meta[base + pos] = ((unsigned)inst << 16) | (unsigned)sh_end[tr];
        sh_nq[base + pos] = rq;
        sh_nkv[base + pos] = rkv;
    }
    __syncthreads();

    // ---- 6. inner nodes, bottom-up; the thread of a block's first row builds the block ----
    for (int l = 1, w = 4; l <= 5; ++l, w <<= 2) {
        if (is_row && l <= levels && (k % w) == 0 && (l < levels || k == 0)) {
            const bool root = (l == levels);
            const int pos = root ? 0 : node_pos(l, k, levels);
            const int hi = min(k + w, n_t);                 // rows [k, hi)
            // children: blocks (or leaves) of width w/4 starting inside [k, hi)
            float bq = 3.4e38f; int bkv = 0;
            const int cw = w >> 2;
            for (int c = k; c < hi; c += cw) {
                const int cpos = node_pos(l - 1, c, levels);
                bq = fminf(bq, sh_nq[base + cpos]);
                bkv = max(bkv, sh_nkv[base + cpos]);
            }
            const int last_inst = (int)(sh_key[sh_row0[tr] + hi - 1] & 0xFFFFull);
            sh_nq[base + pos] = bq;
            sh_nkv[base + pos] = bkv;
            Node nd;
            nd.q = __fmul_rn(bq, kShrink);
            nd.p = __fmul_rn(sh_p[tr], kShrink);
            nd.d = __fmul_rn(sh_d[last_inst], kShrink);     // rows are d-descending: last is smallest
            nd.kv = bkv;
            s.nodes[base + pos] = nd;
            const int skip = root ? sh_end[tr] : base + first_pos(hi, levels);
            s.meta[base + pos] = (0xFFFFu << 16) | (unsigned)skip;
        }
        __syncthreads();
    }

    // ---- 7. nodes over groups of types ------------------------------------------------------
    // built from the type roots; deeper (later-numbered) ones first is not needed because each
    // reads only type roots
    if (g < sh_n_sup) {
        const int a = sh_sup_a[g], b = sh_sup_b[g];
        float bq = 3.4e38f, bp = 3.4e38f, bd = 3.4e38f; int bkv = 0;
        for (int r = a; r < b; ++r) {
            const int root = sh_base[r];
            bq = fminf(bq, sh_nq[root]);
            bkv = max(bkv, sh_nkv[root]);
            bp = fminf(bp, sh_p[r]);
            const int last_inst = (int)(sh_key[sh_row0[r + 1] - 1] & 0xFFFFull);
            bd = fminf(bd, sh_d[last_inst]);
        }
        Node nd;
        nd.q = __fmul_rn(bq, kShrink); nd.p = __fmul_rn(bp, kShrink); nd.d = __fmul_rn(bd, kShrink);
        nd.kv = bkv;
        s.nodes[sh_sup_pos[g]] = nd;
        s.meta[sh_sup_pos[g]] = (0xFFFFu << 16) | (unsigned)sh_sup_skip[g];
    }
    if (g == 0) {
        s.table_info[0] = sh_n_nodes;
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
