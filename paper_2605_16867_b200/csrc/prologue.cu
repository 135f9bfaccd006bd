// Per-round instance prologue, one CTA per GPU type:
//   1. the coefficients of Eq. 2 for every instance and the EMA step of Algorithm 1
//      (rows[g] = {q_g, p_g, d_g, free KV}, exact, in caller order);
//   2. the search tables of the route kernel.  Instances are grouped by GPU type (types
//      ordered by their largest d first) and, inside a type, put in preference order
//      (d descending, index ascending).  Per type the tables hold
//        - a lower bound (q_lo, d_lo) for every row, tagged with the instance index,
//        - a header with the bound over the whole type, and
//        - a start table: for a range of L_out and a threshold on d, the first group of 8
//          rows that can hold a feasible row at all.
//      A type's rows are padded to a multiple of 16 with entries that never pass a test.
// Every CTA derives all coefficients and the order of the types (cheap, and it keeps the
// CTAs independent); the CTA at order position r then builds the tables of that type.
//
// Bounds: q_lo <= q (1 - 2^-19), d_lo <= d (1 - 2^-19), p_lo = p (1 - 2^-19).  With all
// coefficients non-negative and each fused step of T = fma(d, y, fma(p, x, q)) rounding by at
// most 2^-24 relative, the single-precision test  fma(d_lo, y, q_lo) > fma(-p_lo, x, D)
// implies  T(r,g) > D  for every row the bound covers.  The low bits of a row's q word
// carry the instance index; that bound is lowered by one unit of the remaining mantissa
// first, so it stays a lower bound.
//
// Start table.  Write R for fma(-p_lo, x, D), q0 for the type's least q_lo, y for L_out and
// z = (R - q0) / y.  A row can pass its bound test only if  q_lo - q0 <= (z - d_lo) * y.
// For all requests with y <= y_hi and z < z_edge the right side is at most
// max(z_edge - d_lo, 0) * y_hi, so a row whose q_lo - q0 exceeds that is out for all of them,
// and the search may begin at the first row that is not out.  The table is indexed by the
// bucket of y (upper edge y_hi) and the slot of z (upper edge z_edge, widened by a sixteenth of
// a slot against the rounding of the kernel's own slot computation, which stays below 0.03
// slots because a table is only built where the type's range of d exceeds d / 1024).
#include "gs_internal.cuh"

namespace gs {

#ifdef GS_DEBUG
GS_DEBUG_COUNTER(g_prologue_index_errors);
#endif
unsigned prologue_index_errors(bool clear)
{
    unsigned v = 0;
#ifdef GS_DEBUG
    if (cudaMemcpyFromSymbol(&v, g_prologue_index_errors, sizeof(v)) != cudaSuccess) return ~0u;
    if (clear) { const unsigned zero = 0; cudaMemcpyToSymbol(g_prologue_index_errors, &zero, sizeof(zero)); }
#else
    (void)clear;
#endif
    return v;
}

constexpr int kPrologueThreads = GS_MAX_INSTANCES;      // one thread per instance
constexpr int kPmFloats = 8192;                         // shared-memory floats for the running minima
constexpr int kCountSortMax = 256;                      // a group of up to this many rows is ranked by counting
// CTAs per group.  Every one of them works out the group's order, bounds and running minima
// (the same on every SM it runs on: nothing to exchange); the start cells and record lists, a
// third of the kernel's time on one SM, are then shared out by bucket of L_out.
#ifndef GS_PROLOGUE_SPLIT
#define GS_PROLOGUE_SPLIT 8
#endif
constexpr int kPrologueSplit = GS_PROLOGUE_SPLIT;
static_assert(kStartBuckets % kPrologueSplit == 0, "the buckets are dealt out evenly");

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

// Least value of a warp's lanes (non-negative floats: they order like their bits).
__device__ __forceinline__ float warp_min_nonneg(float v) {
    return __uint_as_float(__reduce_min_sync(0xFFFFFFFFu, __float_as_uint(v)));
}

// Upper edge of bucket b of L_out: buckets split every octave at 1.5, b = 2 * exponent + (mantissa >= 1.5).
__device__ __forceinline__ float bucket_upper_edge(int b) {
    const unsigned e = 127u + (unsigned)(b >> kBucketBits);
    const unsigned m = ((unsigned)b & ((1u << kBucketBits) - 1u)) + 1u;
    return __uint_as_float((m >> kBucketBits) ? ((e + 1u) << 23) : ((e << 23) | (m << (23 - kBucketBits))));
}

// Entries of the record-list pool that a type with n of the pool's M instances may use.
// (kPoolEntries * n <= 2^23: plain 32-bit arithmetic)
__device__ __forceinline__ int pool_share_of(int n, int M) { return (int)((unsigned)(kPoolEntries * n) / (unsigned)M) & ~3; }

// Bit pattern of a lower bound of v >= 0 whose low tag bits are zero and may be overwritten.
__device__ __forceinline__ unsigned lower_bound_bits(float v) {
    const unsigned b = __float_as_uint(__fmul_rn(v, kShrink)) & ~kRowTagMask;
    return b >= (kRowTagMask + 1u) ? b - (kRowTagMask + 1u) : 0u;
}

// Lower bound of v >= 0 at full precision (no tag).
__device__ __forceinline__ float lower_bound(float v) { return __fmul_rn(v, kShrink); }

// Bitonic sort of one 64-bit key per thread over the first n_sort threads' keys (n_sort a power
// of two >= 32; all kPrologueThreads threads call it, the warps beyond n_sort only meet the
// barriers).  Partners closer than a warp exchange by shuffle, farther ones through shared
// memory (two buffers, so one barrier per exchange).  Returns the key of rank tid (tid < n_sort).
__device__ __forceinline__ unsigned long long bitonic_sort(unsigned long long key, int n_sort, int tid,
                                                           unsigned long long (*sh_xchg)[GS_MAX_INSTANCES])
{
    int buf = 0;
    const bool works = tid < n_sort;            // whole warps: n_sort is a multiple of 32
    for (int k = 2; k <= n_sort; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            unsigned long long other = key;
            if (j >= 32) {
                if (works) sh_xchg[buf][tid] = key;
                __syncthreads();
                if (works) other = sh_xchg[buf][tid ^ j];
                buf ^= 1;
            } else if (works) {
                other = __shfl_xor_sync(0xFFFFFFFFu, key, j);
            }
            const bool keep_min = ((tid & k) == 0) == ((tid & j) == 0);
            key = (keep_min == (other < key)) ? other : key;
        }
    }
    __syncthreads();
    return key;
}

// kDirect = false: the coefficients come from the typed description of the pool (type
// constants, batch, queue, carried EMA state) and the groups of the search are the GPU types.
// kDirect = true: q, p, d are given per instance (black-box estimates, Sec. 3.3; the first
// three pointers are then q, p, d reinterpreted, see launch_prologue_direct).  There are no
// types to lean on, so the pool is cut into n_types groups of consecutive rank in the
// preference order (d descending, index ascending): the groups are disjoint in d, so the first
// group that yields a feasible row ends a request's search.  Inside a group p varies; the
// header and the start table use the group's least p, and every row carries its own bound of p
// (row_p) for the row tests.
template <bool kDirect>
__global__ void __launch_bounds__(kPrologueThreads)
prologue_kernel(const int32_t *__restrict__ type_id, const int32_t *__restrict__ queued,
                const int32_t *__restrict__ batch, const int32_t *__restrict__ free_kv,
                const float *__restrict__ q_ema, int M,
                const float *__restrict__ p_type, const float *__restrict__ a_type,
                const float *__restrict__ b_type, int n_types, float alpha, int carry_q,
                Scratch s)
{
    __shared__ unsigned long long sh_key[GS_MAX_INSTANCES];                // my group's rows as collected
    __shared__ unsigned long long sh_sorted[GS_MAX_INSTANCES];             // ... in preference order
    extern __shared__ unsigned long long sh_dyn[];                        // sort exchange buffers, then running minima
    unsigned long long (*sh_xchg)[GS_MAX_INSTANCES] = reinterpret_cast<unsigned long long (*)[GS_MAX_INSTANCES]>(sh_dyn);
    __shared__ float sh_q[GS_MAX_INSTANCES], sh_d[GS_MAX_INSTANCES];       // by instance index
    __shared__ float sh_p[kDirect ? GS_MAX_INSTANCES : 1];                 // kDirect: p by instance index
    __shared__ unsigned char sh_t[kDirect ? 1 : GS_MAX_INSTANCES];
    __shared__ float sh_rq[GS_MAX_INSTANCES], sh_rd[GS_MAX_INSTANCES];     // my rows: q_lo (tagged), d_lo
    __shared__ int sh_cnt[GS_MAX_TYPES], sh_plan[8];
    __shared__ unsigned sh_dmax[GS_MAX_TYPES], sh_dmin[GS_MAX_TYPES];      // by type: largest / least d
    __shared__ unsigned sh_dlow_pos[GS_MAX_TYPES];                         // least d by position in the search order
    __shared__ unsigned sh_qmin, sh_pmin;
    __shared__ int sh_kvmax;                                               // most free KV of any instance
    __shared__ float sh_tp[GS_MAX_TYPES], sh_ta[GS_MAX_TYPES], sh_tb[GS_MAX_TYPES];   // type constants
    __shared__ int sh_unsafe, sh_fill;
    __shared__ int sh_len[kPrologueThreads / 32], sh_off[kPrologueThreads / 32], sh_pool_used;

    // the kernel that follows in the stream (the routing round) may be set up from now on; it
    // waits for this whole grid before it reads a table.  This kernel itself is launched the same
    // way: the kernel before it may still be running, and may be the one that writes the pool's state.
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const bool writer = blockIdx.x == 0;       // one CTA writes what does not depend on the group
    const int tr = blockIdx.x / kPrologueSplit;    // position of this CTA's group in the search order
    const int part = blockIdx.x % kPrologueSplit;  // which of the group's CTAs this is: part 0 writes what the
                                                   // group has once; each part the cells and lists of its buckets
    const int b_lo = part * (kStartBuckets / kPrologueSplit), b_hi = b_lo + kStartBuckets / kPrologueSplit;
    unsigned bad = 0;
    const bool has = tid < M;
    // typed pools: all global loads are issued before anything else is done
    int r_type = 0, r_queued = 0, r_batch = 0, r_kv = 0;
    float r_qema = 0.f;
    if (!kDirect) {
        if (has) {
            r_type = type_id[tid]; r_queued = queued[tid]; r_batch = batch[tid];
            r_kv = free_kv[tid]; r_qema = q_ema[tid];
        }
        if (tid < n_types) { sh_tp[tid] = p_type[tid]; sh_ta[tid] = a_type[tid]; sh_tb[tid] = b_type[tid]; }
    }
    if (tid < GS_MAX_TYPES) { sh_cnt[tid] = 0; sh_dmax[tid] = 0u; sh_dmin[tid] = 0xFFFFFFFFu; }
    if (tid == 0) { sh_unsafe = 0; sh_fill = 0; sh_qmin = 0xFFFFFFFFu; sh_pmin = 0xFFFFFFFFu; sh_kvmax = 0; }
    __syncthreads();

    int base = 0, n_act = 0, padded_total = 0, n_t = 0;
    int pool_base = 0, pool_share = 0, pool_total = 0;     // record lists: this type's part of the pool
    float p_group = 0.f;                       // lower bound source: the least p of the group
    int my_kv = 0;                             // free KV of this thread's instance

    if (kDirect) {
        // ---- 1. the coefficients as given (thread g owns instance g) ---------------------------
        const float *q_in = reinterpret_cast<const float *>(type_id);
        const float *p_in = reinterpret_cast<const float *>(queued);
        const float *d_in = reinterpret_cast<const float *>(batch);
        float q = 0.f, pv = 0.f, d = 0.f;
        if (has) {
            q = q_in[tid]; pv = p_in[tid]; d = d_in[tid];
            const int kv = clamp_count(free_kv[tid], bad);
            my_kv = kv;
            if (!(q >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; q = 0.0f; }
            if (!(pv >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; pv = 0.0f; }
            if (!(d >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; d = 0.0f; }
            sh_q[tid] = q; sh_d[tid] = d; sh_p[tid] = pv;
            if (writer) {
                Row row; row.q = q; row.p = pv; row.d = d; row.kv = kv;
                s.rows[row_pos(tid)] = row;
            }
            const float big = 3.0e38f;           // the bounds need finite coefficients
            if (!(q < big && pv < big && d < big)) atomicOr(&sh_unsafe, 1);
        }
        {
            const int wmax = __reduce_max_sync(0xFFFFFFFFu, my_kv);
            if (lane == 0 && wmax > 0) atomicMax(&sh_kvmax, wmax);
        }
        // ---- 2. preference order of the whole pool, cut into groups of consecutive rank -------
        int n_sort = 32;
        while (n_sort < M) n_sort <<= 1;
        unsigned long long key = has ? (((unsigned long long)(~orderable(d)) << 16) | (unsigned)tid) : ~0ull;
        key = bitonic_sort(key, n_sort, tid, sh_xchg);          // (its barriers also publish sh_unsafe)
        const int group_rows = (((M + n_types - 1) / n_types) + 15) & ~15;
        n_act = (M + group_rows - 1) / group_rows;
        padded_total = (n_act - 1) * group_rows + ((M - (n_act - 1) * group_rows + 15) & ~15);
        if (tr < n_act) {
            base = tr * group_rows;
            n_t = min(group_rows, M - base);
        }
        // ---- 3. this CTA's slice of the order, and its least p ---------------------------------
        // the least d of every group: that of its last row (tid = rank here)
        if (has && (tid == M - 1 || (tid + 1) % group_rows == 0)) sh_dlow_pos[tid / group_rows] = ~(unsigned)(key >> 16);
        const bool mine = tr < n_act && tid >= base && tid < base + n_t;
        if (mine) sh_sorted[tid - base] = key;
        const unsigned pb = mine ? (__float_as_uint(sh_p[(int)(key & 0xFFFFull)]) & 0x7FFFFFFFu) : 0xFFFFFFFFu;
        const unsigned wmin = __reduce_min_sync(0xFFFFFFFFu, pb);   // non-negative floats order like their bits
        if (lane == 0 && wmin != 0xFFFFFFFFu) atomicMin(&sh_pmin, wmin);
        __syncthreads();
        p_group = __uint_as_float(sh_pmin);
    } else {
        // ---- 1. coefficients of every instance (thread g owns instance g) ----------------------
        {
            int t = r_type;
            if (has && (t < 0 || t >= n_types)) { bad |= GS_DEV_BAD_TYPE; t = 0; }
            if (!has) t = -1;
            float d = 0.f;
            if (has) {
                const float Qtok = __int2float_rn(clamp_count(r_queued, bad));
                const float B = __int2float_rn(clamp_count(r_batch, bad));
                float qe = r_qema;
                if (!(qe >= 0.0f)) { bad |= GS_DEV_BAD_VALUE; qe = 0.0f; }
                const int kv = clamp_count(r_kv, bad);
                my_kv = kv;
                const float p = sh_tp[t];
                d = __fmaf_rn(sh_tb[t], B, sh_ta[t]);               // loaded per-token decode latency
                const float w = __fmul_rn(Qtok, p);                 // time to drain the queued prefill
                const float keep = __fmul_rn(__fsub_rn(1.0f, alpha), qe);
                const float q = __fmaf_rn(alpha, w, keep);          // EMA step
                sh_q[tid] = q; sh_d[tid] = d; sh_t[tid] = (unsigned char)t;
                if (writer) {
                    Row row; row.q = q; row.p = p; row.d = d; row.kv = kv;
                    s.rows[row_pos(tid)] = row;
                    if (carry_q) s.q_by_g[tid] = q;     // the smoothed delay that gs_advance_state carries on
                }
                // the bounds of the search tables need finite, non-negative coefficients
                const float big = 3.0e38f;
                if (!(q >= 0.f && q < big && p >= 0.f && p < big && d >= 0.f && d < big)) atomicOr(&sh_unsafe, 1);
            }
            // instances per type and each type's largest and least d: the warp goes through the
            // types together (no divergence), lane o keeps type o's figures and adds them to the
            // CTA's with one shared-memory atomic each
            const unsigned od = orderable(d);
            int w_cnt = 0;
            unsigned w_max = 0u, w_min = 0xFFFFFFFFu;
            for (int o = 0; o < n_types; ++o) {
                const bool is = t == o;
                const int c = __popc(__ballot_sync(0xFFFFFFFFu, is));
                const unsigned mx = __reduce_max_sync(0xFFFFFFFFu, is ? od : 0u);
                const unsigned mn = __reduce_min_sync(0xFFFFFFFFu, is ? od : 0xFFFFFFFFu);
                if (lane == o) { w_cnt = c; w_max = mx; w_min = mn; }
            }
            const int wmax = __reduce_max_sync(0xFFFFFFFFu, my_kv);
            if (lane == 0 && wmax > 0) atomicMax(&sh_kvmax, wmax);
            if (w_cnt > 0) {
                atomicAdd(&sh_cnt[lane], w_cnt);
                atomicMax(&sh_dmax[lane], w_max);
                atomicMin(&sh_dmin[lane], w_min);
            }
        }
        __syncthreads();

        // ---- 2. order of the types (largest d first; ties: smaller type id) --------------------
        // One warp works it out, lane o for type o, and leaves the CTA's plan in shared memory.
        if (warp == 0) {
            const bool is_type = lane < GS_MAX_TYPES;
            const int cnt_o = is_type ? sh_cnt[lane] : 0;
            const unsigned dmax_o = is_type ? sh_dmax[lane] : 0u;
            int rank_o = 0;
#pragma unroll
            for (int k = 0; k < GS_MAX_TYPES; ++k) {
                const int cnt_k = __shfl_sync(0xFFFFFFFFu, cnt_o, k);
                const unsigned dmax_k = __shfl_sync(0xFFFFFFFFu, dmax_o, k);
                if (cnt_k > 0 && (dmax_k > dmax_o || (dmax_k == dmax_o && k < lane))) ++rank_o;
            }
            if (cnt_o == 0) rank_o = GS_MAX_TYPES;              // unused types sort last
            const int padded_o = cnt_o > 0 ? (cnt_o + 15) & ~15 : 0;
            const int share_o = cnt_o > 0 ? pool_share_of(cnt_o, M) : 0;
            if (cnt_o > 0) sh_dlow_pos[rank_o] = sh_dmin[lane];
            const int v_act = __popc(__ballot_sync(0xFFFFFFFFu, cnt_o > 0));
            const int v_padded = __reduce_add_sync(0xFFFFFFFFu, padded_o);
            const int v_pool = __reduce_add_sync(0xFFFFFFFFu, share_o);
            const int v_base = __reduce_add_sync(0xFFFFFFFFu, rank_o < tr ? padded_o : 0);
            const int v_pool_base = __reduce_add_sync(0xFFFFFFFFu, rank_o < tr ? share_o : 0);
            // the type this CTA builds: the one at position tr of the order
            const unsigned at_tr = __ballot_sync(0xFFFFFFFFu, cnt_o > 0 && rank_o == tr);
            const int v_type = at_tr ? __ffs(at_tr) - 1 : -1;
            const int v_nt = __shfl_sync(0xFFFFFFFFu, cnt_o, v_type < 0 ? 0 : v_type);
            const int v_share = __shfl_sync(0xFFFFFFFFu, share_o, v_type < 0 ? 0 : v_type);
            if (lane == 0) {
                sh_plan[0] = v_type; sh_plan[1] = v_type < 0 ? 0 : v_nt; sh_plan[2] = v_type < 0 ? 0 : v_share;
                sh_plan[3] = v_act; sh_plan[4] = v_padded; sh_plan[5] = v_pool; sh_plan[6] = v_base; sh_plan[7] = v_pool_base;
            }
        }
        __syncthreads();
        const int my_type = sh_plan[0];
        n_t = sh_plan[1]; pool_share = sh_plan[2]; n_act = sh_plan[3]; padded_total = sh_plan[4];
        pool_total = sh_plan[5]; base = sh_plan[6]; pool_base = sh_plan[7];
        if (my_type >= 0) {
            p_group = sh_tp[my_type];
            // ---- 3. collect this type's rows and sort them by (d descending, index ascending) ---
            // (one shared-memory atomic per warp; the order inside the list does not matter yet)
            const bool mine = has && sh_t[tid] == my_type;
            const unsigned votes = __ballot_sync(0xFFFFFFFFu, mine);
            int at = 0;
            if (lane == 0 && votes) at = atomicAdd(&sh_fill, __popc(votes));
            at = __shfl_sync(0xFFFFFFFFu, at, 0) + __popc(votes & ((1u << lane) - 1u));
            if (mine) sh_key[at] = ((unsigned long long)(~orderable(sh_d[tid])) << 16) | (unsigned)tid;
        }
        __syncthreads();
        if (my_type >= 0 && n_t <= kCountSortMax) {
            // Rank by counting: the keys are distinct (the index is part of them), so a row's place
            // is the number of keys below its own.  n_pow^2 / 1024 compares per thread, P threads
            // per row (consecutive lanes take consecutive keys: no bank conflicts), no barrier
            // until the places are known.
            int n_pow = 32;
            while (n_pow < n_t) n_pow <<= 1;
            const int P = kPrologueThreads / n_pow;             // 4 .. 32 threads per row
            const int i = tid / P, part = tid % P;
            const unsigned long long key_i = i < n_t ? sh_key[i] : 0ull;
            int below_i = 0;
            for (int j = part; j < n_t; j += P) below_i += sh_key[j] < key_i ? 1 : 0;
            for (int off = P >> 1; off > 0; off >>= 1) below_i += __shfl_xor_sync(0xFFFFFFFFu, below_i, off);
            if (part == 0 && i < n_t) sh_sorted[below_i] = key_i;    // (published by the barrier further down)
        } else if (my_type >= 0) {             // (uniform over the CTA)
            int n_sort = 32;
            while (n_sort < n_t) n_sort <<= 1;
            const unsigned long long key = bitonic_sort(tid < n_t ? sh_key[tid] : ~0ull, n_sort, tid, sh_xchg);
            sh_sorted[tid] = key;
        }
    }
    if (writer && tid == 0) {
        s.table_info[0] = padded_total;
        s.table_info[1] = sh_unsafe;
        s.table_info[2] = M;
        s.table_info[3] = n_act;
        s.table_info[6] = pool_total;
        if (carry_q) s.table_info[7] = 1;      // a round whose q_g is to be carried is pending
        s.table_info[8] = sh_kvmax;            // no instance has more free KV than this
        if (sh_unsafe) atomicOr(s.status, (unsigned)GS_DEV_BAD_VALUE);
    }
    if (writer && bad) atomicOr(s.status, bad);
    // candidate table: a type can hold a feasible instance only if its least d_lo times L_out is
    // within the deadline, so the slot of D / L_out names the types worth an entry test (slots
    // widened by a sixteenth against the rounding of the kernel's own slot computation)
    if (writer && tid < kCandSlots) {
        float z0 = 3.4e38f, z1 = 0.f;
        for (int r = 0; r < n_act; ++r) {
            const float v = lower_bound(__uint_as_float(sh_dlow_pos[r] & 0x7FFFFFFFu));
            z0 = fminf(z0, v); z1 = fmaxf(z1, v);
        }
        const bool usable = (z1 - z0) > z1 * (1.0f / 1024.0f);
        const float edge = (z0 + ((float)tid + 1.0625f) * ((z1 - z0) / (float)kCandSlots)) * 1.00002f;
        unsigned mask = 0;
        for (int r = 0; r < n_act; ++r) {
            const float v = lower_bound(__uint_as_float(sh_dlow_pos[r] & 0x7FFFFFFFu));
            if (!usable || tid == kCandSlots - 1 || v <= edge) mask |= 1u << r;
        }
        s.cand_table[tid] = (unsigned short)mask;
        if (tid == 0) {
            s.table_info[4] = __float_as_int(z0);
            s.table_info[5] = __float_as_int(usable ? (float)kCandSlots / (z1 - z0) : 0.f);
        }
    }
    if (n_t == 0) return;                      // no group at this position
    const int n_padded = (n_t + 15) & ~15;
    __syncthreads();

    // ---- 4. row bounds, least q of the type ---------------------------------------------------
    unsigned my_qmin = 0xFFFFFFFFu;
    for (int k = tid; k < n_padded; k += kPrologueThreads) {
        uint2 entry = make_uint2(kPadQ, 0u);
        if (k < n_t) {
            const int inst = (int)(sh_sorted[k] & 0xFFFFull);
            // the tag rides on q: d multiplies L_out, so its bound is kept at full precision
            const unsigned q_bits = lower_bound_bits(sh_q[inst]);
            const float d_lo = lower_bound(sh_d[inst]);
            entry = make_uint2(q_bits | (unsigned)inst, __float_as_uint(d_lo));
            sh_rq[k] = __uint_as_float(q_bits | (unsigned)inst);    // as the kernel tests it
            sh_rd[k] = d_lo;
            my_qmin = min(my_qmin, q_bits);             // non-negative floats order like their bits
        }
#ifdef GS_DEBUG
        // the order must be a strict one (a permutation of the group's rows, no key twice)
        if (k > 0 && k < n_t && !(sh_sorted[k - 1] < sh_sorted[k])) atomicAdd(&g_prologue_index_errors, 1u);
#endif
        if (part == 0) {
            s.row_bounds[GS_CHECKED(g_prologue_index_errors, row_slot(base + k), kMaxPaddedRows)] = entry;
            if (kDirect) s.row_p[base + k] = k < n_t ? lower_bound(sh_p[(int)(sh_sorted[k] & 0xFFFFull)]) : 0.f;
        }
    }
    my_qmin = __reduce_min_sync(0xFFFFFFFFu, my_qmin);
    if (lane == 0) atomicMin(&sh_qmin, my_qmin);
    __syncthreads();

    // bounds over every eight rows (the fallback's search skips a group whole with them)
    for (int g = tid - 64; g < n_padded / 8; g += kPrologueThreads - 64) {   // (warps 0 and 1 have other work below)
        if (g < 0 || part != 0) break;
        float q_least = __int_as_float(0x7F800000);         // +inf: a group of padding only
        float d_last = 0.f;
        for (int k = 8 * g; k < 8 * g + 8 && k < n_t; ++k) { q_least = fminf(q_least, sh_rq[k]); d_last = sh_rd[k]; }
        s.group_bounds[(base >> 3) + g] = make_float2(q_least, d_last);
    }

    // ---- 5. header ----------------------------------------------------------------------------
    const float q0 = __uint_as_float(sh_qmin);
    const float d_hi = sh_rd[0], d_low = sh_rd[n_t - 1];
    float inv_w = 0.f;              // slots per unit of d; 0 = no start table (search from row 0)
    if (n_t > 4 && (d_hi - d_low) > d_hi * (1.0f / 1024.0f)) inv_w = (float)kStartSlots / (d_hi - d_low);
    if (tid == 32 && part == 0) {
        const int first_inst = (int)(sh_sorted[0] & 0xFFFFull);
        TypeHeader h;
        h.p_lo = __fmul_rn(p_group, kShrink);
        h.q_lo = q0;
        h.d_lo = d_low;
        h.d_max = sh_d[first_inst];
        h.base = base;
        h.n_padded = n_padded;
        h.inv_w = inv_w;
        h.d0 = d_low;
        s.headers[tr] = h;
    }

    // ---- 6. start tables and record lists -----------------------------------------------------
    // For bucket b put  H_k = (q_k - q0) + y_hi d_lo_k  with q_k the row's tagged bound, the value
    // the kernel tests.  A row can pass only if H_k <= y_hi z_edge (see the header comment; rows
    // with d_lo above z_edge fail that too).  With P_k the running minimum of H over rows 0..k,
    // the first row that can pass is the first k with P_k <= y_hi z_edge: a binary search per
    // slot.
    // Record list.  Row k is a record of the bucket if H_k < P_(k-1).  A row that is not has an
    // earlier row j with q_j + y_hi d_lo_j <= q_k + y_hi d_lo_k and d_lo_j >= d_lo_k, hence
    // q_j + y d_lo_j <= q_k + y d_lo_k for every y <= y_hi: whenever its bound passes so does
    // that of row j, so it is never the first row to pass and the kernel's first attempt need
    // not look at it.  Each bucket's records are stored as a list of their own (while the
    // type's share of the pool lasts, shortest lists first) with a second start table that
    // counts in list entries.  Up to 32 buckets are done at a time, one warp each for the
    // running minima and record counts, then one (bucket, slot) cell per thread.
    {
        float *sh_pm = reinterpret_cast<float *>(sh_dyn);                         // [buckets per batch][n_t] running minima
        unsigned short *sh_pc = reinterpret_cast<unsigned short *>(sh_pm + kPmFloats);   // records before each row
        const float w_slot = inv_w > 0.f ? 1.0f / inv_w : 0.f;
        int per_batch = kPmFloats / n_t;                    // n_t <= 1024: at least 8
        if (per_batch > kPrologueThreads / 32) per_batch = kPrologueThreads / 32;   // one warp per bucket
        if (per_batch > kStartBuckets) per_batch = kStartBuckets;
        if (tid == 0) sh_pool_used = 0;
        if (kDirect || n_t > kCountSortMax) __syncthreads();       // the bitonic sort is done with sh_dyn
        for (int b0 = 0; b0 < kStartBuckets; b0 += per_batch) {
            const bool my_bucket = warp < per_batch && b0 + warp < kStartBuckets;
            if (my_bucket) {
                const int b = b0 + warp;
                // bucket b holds y in [2^e (1 + m/2), 2^e (1 + (m+1)/2)),  e = b >> 1, m = b & 1;
                // the last bucket has no upper edge: there only d_lo <= z_edge can be required
                const bool open_ended = b == kStartBuckets - 1;
                const float y_hi = bucket_upper_edge(b) * 1.00002f;
                float carry = 3.4e38f;
                int n_rec = 0;
                // (for the chord, below: the least row bound at either end of the bucket)
                const float y_lo = b == 0 ? 1.0f : bucket_upper_edge(b - 1) * 0.99998f;
                float f_lo = 3.4e38f, f_hi = 3.4e38f;
                for (int k0 = 0; k0 < n_t; k0 += 32) {
                    const int k = k0 + lane;
                    float own = 3.4e38f;
                    if (k < n_t) own = open_ended ? sh_rd[k] : __fmaf_rn(y_hi, sh_rd[k], sh_rq[k] - q0);
                    if (!kDirect && k < n_t) {
                        f_lo = fminf(f_lo, __fmaf_rn(y_lo, sh_rd[k], sh_rq[k]));
                        f_hi = fminf(f_hi, __fmaf_rn(y_hi, sh_rd[k], sh_rq[k]));
                    }
                    float h = own;
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const float up = __shfl_up_sync(0xFFFFFFFFu, h, off);
                        if (lane >= off) h = fminf(h, up);
                    }
                    h = fminf(h, carry);
                    float before = __shfl_up_sync(0xFFFFFFFFu, h, 1);       // minimum over the rows before k
                    if (lane == 0) before = carry;
                    // (kept unless an earlier row is below it by more than the rounding of H)
                    const bool rec = k < n_t && !(before * 1.000001f <= own);
                    const unsigned votes = __ballot_sync(0xFFFFFFFFu, rec);
                    if (k < n_t) {
                        sh_pm[warp * n_t + k] = h;
                        sh_pc[warp * n_t + k] = (unsigned short)(n_rec + __popc(votes & ((1u << lane) - 1u)));
                    }
                    n_rec += __popc(votes);
                    carry = __shfl_sync(0xFFFFFFFFu, h, 31);
                }
                if (lane == 0) sh_len[warp] = n_rec;
                if (!kDirect) {
                    // Chord.  F(y) = least row bound of the type at L_out = y, the minimum of the
                    // lines q_k + d_lo_k y, is concave: between two points it lies on or above the
                    // straight line through them.  The line through (y_lo, F(y_lo)) and
                    // (y_hi, F(y_hi)), the ends of the bucket pushed outwards a little, is therefore
                    // below every row bound for every L_out of the bucket: a request whose
                    // R = D - p_lo L_in is below that line can pass no row bound of the type.  Beyond
                    // the last bucket's lower end F grows at least as fast as the least d_lo.  Line
                    // and offset are lowered by 2^-16 of F, far more than the roundings here
                    // and in the kernel's tests add up to (a few 2^-20 of F).
                    f_lo = warp_min_nonneg(f_lo);
                    f_hi = warp_min_nonneg(f_hi);
                    float slope = open_ended ? sh_rd[n_t - 1] : (f_hi - f_lo) / (y_hi - y_lo);
                    slope = fmaxf(slope, 0.f);
                    const float offset = f_lo - slope * y_lo;
                    const float kMargin = 1.52587890625e-5f;            // 2^-16
                    if (lane == 0 && b >= b_lo && b < b_hi)
                        s.chord[tr * kStartBuckets + b] = make_float4(offset - kMargin * f_lo, slope * (1.0f - kMargin),
                                                                  __fmul_rn(p_group, kShrink), 0.f);
                }
            }
            __syncthreads();
            if (warp == 0) {                                // room in the pool, in bucket order (lane = bucket of the batch)
                const bool listed = !kDirect && lane < per_batch && b0 + lane < kStartBuckets - 1 &&
                                    sh_len[lane < per_batch ? lane : 0] <= kListMax;
                // padded: a window never leaves its list
                const int need = listed ? (sh_len[lane] + kListWindow + 1) & ~1 : 0;
                int upto = need;                            // entries wanted by this bucket and the ones before it
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int v = __shfl_up_sync(0xFFFFFFFFu, upto, off);
                    if (lane >= off) upto += v;
                }
                const int used = sh_pool_used;
                const bool fits = listed && used + upto <= pool_share;     // (lists only get longer with the bucket)
                if (lane < per_batch) sh_off[lane] = fits ? pool_base + used + upto - need : -1;
                const unsigned got = __ballot_sync(0xFFFFFFFFu, fits);
                const int last = got ? 31 - __clz(got) : -1;
                const int used_now = last >= 0 ? __shfl_sync(0xFFFFFFFFu, upto, last) : 0;
                __syncwarp();
                if (lane == 0) sh_pool_used = used + used_now;
            }
            // (the cells below need the running minima and record counts only, not the pool
            // offsets that warp 0 has just worked out: no barrier in between)
            // (this CTA's buckets among those of the batch)
            const int bw_lo = max(b_lo - b0, 0), bw_hi = min(min(b_hi, kStartBuckets) - b0, per_batch);
            for (int c = bw_lo * kStartSlots + tid - 32; c < bw_hi * kStartSlots; c += kPrologueThreads - 32) {
                if (tid < 32) break;                        // warp 0 is busy with the pool
                const int bw = c / kStartSlots, slot = c % kStartSlots, b = b0 + bw;
                int lo = 0;                                 // rows [0, lo) cannot pass
                if (inv_w > 0.f && slot != kStartSlots - 1) {   // (the top slot also takes every z beyond the table)
                    const bool open_ended = b == kStartBuckets - 1;
                    const float y_hi = bucket_upper_edge(b) * 1.00002f;
                    const float z_edge = d_low + ((float)slot + GS_SLOT_WIDEN) * w_slot;
                    const float limit = (open_ended ? z_edge : y_hi * z_edge) * 1.00002f;
                    const float *pm = sh_pm + bw * n_t;
                    int hi = n_t;
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        if (pm[mid] > limit) lo = mid + 1; else hi = mid;
                    }
                }
                // (a cell that no row can pass begins at the type's last group: searches always have eight rows to test)
                s.start_table[GS_CHECKED(g_prologue_index_errors, (tr * kStartBuckets + b) * kStartSlots + slot,
                                         GS_MAX_TYPES * kStartBuckets * kStartSlots)] = (unsigned char)min(lo >> 3, (n_padded >> 3) - 1);
                if (!kDirect) {
                    const int before = lo < n_t ? sh_pc[bw * n_t + lo] : sh_len[bw];    // records among rows [0, lo)
                    s.start_list[(tr * kStartBuckets + b) * kStartSlots + slot] = (unsigned char)min(before >> 1, 255);
                }
            }
            __syncthreads();
            if (my_bucket && !kDirect && b0 + warp >= b_lo && b0 + warp < b_hi) {
                const int off = sh_off[warp], len = sh_len[warp];
                if (off >= 0) {
                    const unsigned short *pc = sh_pc + warp * n_t;
                    for (int k = lane; k < n_t; k += 32) {
                        const int c = pc[k], c_next = k + 1 < n_t ? pc[k + 1] : len;
                        if (c_next != c)
                            s.pool[GS_CHECKED(g_prologue_index_errors, off + c, pool_base + pool_share)] =
                                make_uint2(__float_as_uint(sh_rq[k]), __float_as_uint(sh_rd[k]));
                    }
                    for (int k = len + lane; k < ((len + kListWindow + 1) & ~1); k += 32)
                        s.pool[GS_CHECKED(g_prologue_index_errors, off + k, pool_base + pool_share)] = make_uint2(kPadQ, 0u);
                }
                if (lane == 0)
                    s.bucket_list[tr * kStartBuckets + b0 + warp] = off >= 0 ? (unsigned short)(off >> 1) : kNoList;
            }
            if (b0 + per_batch < kStartBuckets) __syncthreads();     // the next batch writes the same shared arrays
        }
    }
}

size_t prologue_dynamic_smem() { return (size_t)kPmFloats * (sizeof(float) + sizeof(unsigned short)); }   // >= 2 sort buffers

cudaError_t configure_prologue()
{
    cudaError_t e = cudaFuncSetAttribute(prologue_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)prologue_dynamic_smem());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(prologue_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)prologue_dynamic_smem());
}

cudaError_t launch_prologue(gs_ctx *ctx, const gs_instances &inst, const gs_types &types,
                            float ema_alpha, bool carry_q, cudaStream_t st)
{
    LaunchTimer timer(ctx, GS_K_PROLOGUE, st);
    return launch_dependent(prologue_kernel<false>, dim3(GS_MAX_TYPES * kPrologueSplit), dim3(kPrologueThreads), prologue_dynamic_smem(), st,
                            inst.type_id, inst.queued_prefill_tokens, inst.decode_batch, inst.free_kv_tokens,
                            inst.q_ema_ms, inst.n_instances, types.prefill_ms_per_tok, types.tpot_a_ms,
                            types.tpot_b_ms, types.n_types, ema_alpha, carry_q ? 1 : 0, ctx->s);
}

// Tables of a round from coefficients given per instance; the instances are put into
// kDirectGroups groups of consecutive rank in the preference order, which take the place of the
// GPU types in the search.
cudaError_t launch_prologue_direct(gs_ctx *ctx, const gs_instance_table &tab, cudaStream_t st)
{
    LaunchTimer timer(ctx, GS_K_PROLOGUE, st);
    return launch_dependent(prologue_kernel<true>, dim3(GS_MAX_TYPES * kPrologueSplit), dim3(kPrologueThreads), prologue_dynamic_smem(), st,
                            reinterpret_cast<const int32_t *>(tab.q_ms), reinterpret_cast<const int32_t *>(tab.p_ms_per_tok),
                            reinterpret_cast<const int32_t *>(tab.d_ms_per_tok), tab.free_kv_tokens, (const float *)nullptr,
                            tab.n_instances, (const float *)nullptr, (const float *)nullptr, (const float *)nullptr,
                            kDirectGroups, 0.f, 0, ctx->s);
}

}  // namespace gs
