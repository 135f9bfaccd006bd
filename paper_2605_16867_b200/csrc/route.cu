// gs_route_batch kernels: pair scoring (Eq. 2), feasibility, just-enough pick and fallback
// (Algorithm 1) for every pending request of a round.
//
// One thread owns four consecutive requests (128-bit column loads and stores).  The per-round
// tables built by the prologue are staged once per CTA in shared memory.  For each request:
//   1. every GPU type is tested against a lower bound of T over all its instances (the same
//      shared-memory address for all lanes: a broadcast); types that cannot meet the deadline
//      are dropped;
//   2. for each surviving type (largest d first, and only while it can still beat the best d
//      found so far) a start table turns L_out and the largest d that could still meet the
//      deadline into the first row worth looking at; from there the rows' own lower bounds are tested
//      eight at a time, and the first row that passes is scored exactly as the definition
//      says, T = fma(d, y, fma(p, x, q)), and checked against the deadline and the
//      instance's free KV.
// Rows of a type are in preference order (d descending, index ascending), so the first
// feasible row of a type is that type's best.  Every bound is a true lower bound in the
// kernel's own arithmetic, so nothing feasible is ever skipped and the result is exactly
// argmax d_g over the feasible set, ties to the smallest index.
//
// A request for which this finds nothing (no feasible instance: the fallback of Algorithm 1)
// is finished by the same thread with a branch-and-bound minimum of T over the same tables.
// Only requests that the tables cannot serve (L_out == 0, or coefficients for which the bounds
// do not hold) are handed to their whole warp, which scores every instance, lanes across
// instances, with shuffle reductions.
#include "gs_internal.cuh"

namespace gs {

#ifdef GS_DEBUG
GS_DEBUG_COUNTER(g_route_index_errors);
#endif
unsigned route_index_errors(bool clear)
{
    unsigned v = 0;
#ifdef GS_DEBUG
    if (cudaMemcpyFromSymbol(&v, g_route_index_errors, sizeof(v)) != cudaSuccess) return ~0u;
    if (clear) { const unsigned zero = 0; cudaMemcpyToSymbol(g_route_index_errors, &zero, sizeof(zero)); }
#else
    (void)clear;
#endif
    return v;
}

#ifdef GS_COUNT_EVALS
__device__ unsigned long long g_eval_counts[kCountN];
#define GS_COUNT(k, v) atomicAdd(&gs::g_eval_counts[k], (unsigned long long)(v))
#else
#define GS_COUNT(k, v) ((void)0)
#endif
cudaError_t read_eval_counters(unsigned long long *out, bool clear)
{
    for (int k = 0; k < kCountN; ++k) out[k] = 0ull;
#ifdef GS_COUNT_EVALS
    cudaError_t e = cudaMemcpyFromSymbol(out, g_eval_counts, sizeof(unsigned long long) * kCountN);
    if (e != cudaSuccess) return e;
    if (clear) {
        unsigned long long zeros[kCountN] = {};
        return cudaMemcpyToSymbol(g_eval_counts, zeros, sizeof(zeros));
    }
#else
    (void)clear;
#endif
    return cudaSuccess;
}

#ifndef GS_ROUTE_THREADS
#define GS_ROUTE_THREADS 896
#endif
#ifndef GS_REROUTE_THREADS
#define GS_REROUTE_THREADS 1024
#endif
#ifndef GS_ROUTE_MIN_CTAS
#define GS_ROUTE_MIN_CTAS 1
#endif
constexpr int kRouteThreads = GS_ROUTE_THREADS;     // four requests per lane (large batches)
constexpr int kRouteThreadsSmall = 1024;            // one request per lane (small batches)
constexpr int kRouteMinCtas = GS_ROUTE_MIN_CTAS;
// Requests per lane: four (128-bit column loads) for large batches; one for small ones, where
// shorter tiles spread over more warps count for more than wide loads (fewer registers: more
// threads).  With per-row p the search holds more state: a quarter fewer threads, more
// registers each.
__host__ __device__ constexpr int route_threads(bool row_p, int req = 4) {
    return ((req == 1 ? kRouteThreadsSmall : kRouteThreads) * (row_p ? 3 : 4) / 4) & ~31;
}
constexpr int64_t kSmallBatch = 1 << 21;        // below this many requests: one per lane

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
    const uint2 *row_bounds;
    const float2 *group_bounds;   // per eight rows: {least q word, d_lo of the last row}
    const unsigned char *start_table;
    const Row *rows;
    const float *row_p;       // per-row lower bound of p, in row order (only where p differs inside a group)
    const unsigned short *cand;   // candidate types by slot of D / L_out
    const uint2 *pool;            // record lists (typed pools)
    const unsigned short *bucket_list;
    const unsigned char *start_list;
    const float4 *chord;          // per type and bucket of L_out: a line below every row bound (re-routing only)
    int n_types;
};

constexpr unsigned kNoRow = 0xFFFFFFFFu;

// Slot of the start tables for a request: z, about the largest d that can still meet the
// deadline R with the type's least q, in units of the table.  R is raised by a hair first: a row
// passes its test when its rounded bound is <= R, which lets the unrounded one exceed R by half
// an ulp, and where q dominates that half ulp can be worth whole slots of d.  (ry: 1 / L_out to
// within an ulp or two; the tables' slots are widened against what remains.)
__device__ __forceinline__ int start_slot(float R, float q_lo, float ry, float d0, float inv_w) {
    const float z = (__fmaf_rn(R, 4.76837158203125e-7f, R) - q_lo) * ry;
    return __float2int_rd(fminf(fmaxf((z - d0) * inv_w, 0.f), (float)(kStartSlots - 1)));
}
// Lanes of a warp that must need the fallback before each runs its own search; below that the
// whole warp would score every instance for each of them.  The full search only ever sees
// requests that the first attempt left open, a few to a warp at the end of the kernel, and
// there one lane's own search (about 700 instructions) is shorter than the warp's scan of all
// instances (about 800 for each such request), so the lane always searches for itself; the
// warp-wide scan remains for requests that the tables cannot serve.
#ifndef GS_THREAD_FALLBACK_MIN
#define GS_THREAD_FALLBACK_MIN 1
#endif
constexpr int kThreadFallbackMin = GS_THREAD_FALLBACK_MIN;

// Bound test of one row: false only if the row certainly cannot be chosen.  Where all rows of
// a group share p (GPU types) the prefill term is already in R = D - p_lo x; with kRowP the row
// brings its own bound of p and `R` is the deadline itself.
template <bool kCapped, bool kRowP>
__device__ __forceinline__ bool row_may_pass(unsigned q_word, unsigned d_word, float p_lo, float x, float y,
                                             float R, float d_cap) {
    GS_COUNT(kCountBound, 1);
    const float d_lo = __uint_as_float(d_word);
    const float base = kRowP ? __fmaf_rn(p_lo, x, __uint_as_float(q_word)) : __uint_as_float(q_word);
    return __fmaf_rn(d_lo, y, base) <= R && (!kCapped || d_lo < d_cap);
}

// Scores one row exactly and folds it into the running best.  Returns true when the search of
// this type is over: the row is feasible (later rows of the type rank lower) or already ranks
// below the best found (so does everything after it).
// With kCapped only instances with d < d_cap are eligible (re-routing to a faster instance).
template <bool kCapped>
__device__ __forceinline__ bool score_row(const Tables &tb, int inst, float x, float y, float D, unsigned need,
                                          float d_cap, int &g_best, float &d_best, float &T_best)
{
    GS_COUNT(kCountExact, 1);
    const Row row = tb.rows[GS_CHECKED(g_route_index_errors, row_pos(inst), GS_MAX_INSTANCES)];
    const float T = __fmaf_rn(row.d, y, __fmaf_rn(row.p, x, row.q));      // Eq. 2, H = 0
    const bool feasible = (T <= D) && (need <= (unsigned)row.kv) && (!kCapped || row.d < d_cap);
    const bool worse = row.d < d_best;
    if (feasible && !worse && (g_best < 0 || row.d > d_best || inst < g_best)) {
        d_best = row.d; g_best = inst; T_best = T;
    }
    return feasible || worse;
}

// Just-enough pick for one request.  Returns the chosen instance or -1 (no feasible one, or a
// request this search does not take).  `Dm` is the deadline plus a hair (see the caller).
template <bool kCapped, bool kRowP>
__device__ __forceinline__ int pick_instance(const Tables &tb, float x, float y, float D, float Dm,
                                             unsigned need, float d_cap, float &T_out)
{
    // 1. which types can hold a feasible instance at all
    unsigned alive = 0;
#pragma unroll 2
    for (int t = 0; t < tb.n_types; ++t) {
        const float4 h = *reinterpret_cast<const float4 *>(&tb.headers[t]);   // p_lo, q_lo, d_lo, d_max
        // (a type whose least d_lo is not below the cap has no eligible instance: d_lo <= d)
        if (D >= 0.f) GS_COUNT(kCountTypeTest, 1);
        if (__fmaf_rn(h.z, y, h.y) <= __fmaf_rn(-h.x, x, Dm) && (!kCapped || h.z < d_cap)) alive |= 1u << t;
    }
    int g_best = -1;
    float d_best = -1.0f, T_best = 0.f;
    const float ry = __frcp_rn(y);
    // bucket of L_out: exponent and top mantissa bit of y (y >= 1 here)
    const int ybucket = min((int)(__float_as_uint(y) >> (23 - kBucketBits)) - (127 << kBucketBits), kStartBuckets - 1);
    // 2. search them, largest d first
    while (alive) {
        const int t = __ffs(alive) - 1;
        alive &= alive - 1;
        const float4 h = *reinterpret_cast<const float4 *>(&tb.headers[t]);
        if (h.w < d_best) break;                                  // no later type can do better
        const int4 geo = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);   // base, n_padded, inv_w, d0
        const float Rg = __fmaf_rn(-h.x, x, Dm);           // deadline less the group's least prefill time
        const float R = kRowP ? Dm : Rg;                   // what a row's own bound is held against
        const float inv_w = __int_as_float(geo.z);
        int k = 0;
        if (inv_w > 0.f) {
            // largest d that can still meet the deadline -> slot -> first row worth a look
            k = 8 * tb.start_table[GS_CHECKED(g_route_index_errors, (t * kStartBuckets + ybucket) * kStartSlots +
                                   start_slot(Rg, h.y, ry, __int_as_float(geo.w), inv_w), tb.n_types * kStartBuckets * kStartSlots)];
        }
        const int k_end = geo.x + geo.y;
        k += geo.x;                                         // padded row index, a multiple of 8
        for (;;) {
            // tag word of the first row, from k on, whose bound passes
            unsigned first = kNoRow;
            for (; k < k_end; k += 8) {
                const char *grp = reinterpret_cast<const char *>(tb.row_bounds + GS_CHECKED(g_route_index_errors, k, kMaxPaddedRows - 7));
                const int sw = (k >> 4) & 3;                // see row_slot()
                const uint4 r0 = *reinterpret_cast<const uint4 *>(grp + ((0 ^ sw) << 4));
                const uint4 r1 = *reinterpret_cast<const uint4 *>(grp + ((1 ^ sw) << 4));
                const uint4 r2 = *reinterpret_cast<const uint4 *>(grp + ((2 ^ sw) << 4));
                const uint4 r3 = *reinterpret_cast<const uint4 *>(grp + ((3 ^ sw) << 4));
                float4 pa = make_float4(0.f, 0.f, 0.f, 0.f), pb = pa;      // rows k..k+3, k+4..k+7
                if (kRowP) {
                    pa = *reinterpret_cast<const float4 *>(tb.row_p + k);
                    pb = *reinterpret_cast<const float4 *>(tb.row_p + k + 4);
                }
                first = row_may_pass<kCapped, kRowP>(r3.z, r3.w, pb.w, x, y, R, d_cap) ? r3.z : first;
                first = row_may_pass<kCapped, kRowP>(r3.x, r3.y, pb.z, x, y, R, d_cap) ? r3.x : first;
                first = row_may_pass<kCapped, kRowP>(r2.z, r2.w, pb.y, x, y, R, d_cap) ? r2.z : first;
                first = row_may_pass<kCapped, kRowP>(r2.x, r2.y, pb.x, x, y, R, d_cap) ? r2.x : first;
                first = row_may_pass<kCapped, kRowP>(r1.z, r1.w, pa.w, x, y, R, d_cap) ? r1.z : first;
                first = row_may_pass<kCapped, kRowP>(r1.x, r1.y, pa.z, x, y, R, d_cap) ? r1.x : first;
                first = row_may_pass<kCapped, kRowP>(r0.z, r0.w, pa.y, x, y, R, d_cap) ? r0.z : first;
                first = row_may_pass<kCapped, kRowP>(r0.x, r0.y, pa.x, x, y, R, d_cap) ? r0.x : first;
                if (first != kNoRow) break;
            }
            if (first == kNoRow) break;                     // type exhausted
            // lanes meet again here, so the exact scoring runs once per warp, not once per step
            if (score_row<kCapped>(tb, (int)(first & kRowTagMask), x, y, D, need, d_cap, g_best, d_best, T_best)) break;
            // rare: the bound passed but the row is not feasible (KV, or inside the bound's
            // margin); go on row by row through the rest of these eight, then resume
            bool over = false, seen = false;
            for (int j = 0; j < 8 && !over; ++j) {
                const uint2 rb = tb.row_bounds[row_slot(k + j)];
                if (!seen) { seen = (rb.x == first); continue; }
                if (row_may_pass<kCapped, kRowP>(rb.x, rb.y, kRowP ? tb.row_p[k + j] : 0.f, x, y, R, d_cap))
                    over = score_row<kCapped>(tb, (int)(rb.x & kRowTagMask), x, y, D, need, d_cap, g_best, d_best, T_best);
            }
            if (over) break;
            k += 8;
        }
    }
    T_out = T_best;
    return g_best;
}

// Fallback of Algorithm 1 for one request, by one thread: the smallest T among instances with
// KV room (tier 2), else among all (tier 3); ties to the smallest index.  Branch and bound over
// the same tables: the best T found so far plays the deadline's part in the bound tests, so a
// row is skipped only when its exactly-rounded T is proven larger.
struct Pick { int g; float T; unsigned tier; };

// The eight rows at padded index k (a multiple of 8) of a type with least prefill coefficient
// p_lo, held against the best found so far; Rg = (T_best less the type's least prefill time).
template <bool kCapped, bool kRowP>
__device__ __forceinline__ void search_eight(const Tables &tb, int k, float x, float y, unsigned need, float d_cap,
                                             bool any_kv, float p_lo, int &g_best, float &T_best, float &Rg)
{
    const char *grp = reinterpret_cast<const char *>(tb.row_bounds + k);
    const int sw = (k >> 4) & 3;                // see row_slot()
    uint4 r[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) r[c] = *reinterpret_cast<const uint4 *>(grp + ((c ^ sw) << 4));
    // rows k .. k+7 in order: (r[0].x,y) (r[0].z,w) (r[1].x,y) ...; larger d first
    float4 pa = make_float4(0.f, 0.f, 0.f, 0.f), pb = pa;
    if (kRowP) {
        pa = *reinterpret_cast<const float4 *>(tb.row_p + k);
        pb = *reinterpret_cast<const float4 *>(tb.row_p + k + 4);
    }
    const float pl[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
#pragma unroll
    for (int c = 3; c >= 0; --c) {
#pragma unroll
        for (int e = 1; e >= 0; --e) {
            const unsigned qw = e ? r[c].z : r[c].x, dw = e ? r[c].w : r[c].y;
            const float R = kRowP ? T_best + 1e-30f : Rg;
            if (!row_may_pass<kCapped, kRowP>(qw, dw, pl[2 * c + e], x, y, R, d_cap)) continue;
            const int inst = (int)(qw & kRowTagMask);
            const Row row = tb.rows[GS_CHECKED(g_route_index_errors, row_pos(inst), GS_MAX_INSTANCES)];
            if (kCapped && !(row.d < d_cap)) continue;
            if (!any_kv && !(need <= (unsigned)row.kv)) continue;
            GS_COUNT(kCountExact, 1);
            const float T = __fmaf_rn(row.d, y, __fmaf_rn(row.p, x, row.q));   // Eq. 2, H = 0
            if (T < T_best || (T == T_best && inst < g_best) || g_best < 0) {
                T_best = T; g_best = inst;
                Rg = __fmaf_rn(-p_lo, x, T_best) + 1e-30f;
            }
        }
    }
}

// Types are visited fastest first and each type's rows from its smallest d upwards, which is
// where the minimum lives; the walk up a type stops at the first group whose smallest d alone
// already exceeds the best.  Returns -1 with tier 0 only when kCapped and no instance has
// d < d_cap.  `first_pass` = 1 skips the pass over instances with KV room (the caller knows
// there is none).
template <bool kCapped, bool kRowP>
__device__ __forceinline__ Pick fallback_pick(const Tables &tb, float x, float y, unsigned need, float d_cap,
                                              int first_pass = 0)
{
    unsigned tier_out = 0;
    int g_best = -1;
    float T_best = __int_as_float(0x7F800000);            // +inf
#pragma unroll 1
    for (int pass = first_pass; pass < 2 && g_best < 0; ++pass) {  // pass 0: instances with KV room only
        const bool any_kv = pass == 1;
#pragma unroll 1
        for (int t = tb.n_types - 1; t >= 0; --t) {
            const float4 h = *reinterpret_cast<const float4 *>(&tb.headers[t]);   // p_lo, q_lo, d_lo, d_max
            if (kCapped && !(h.z < d_cap)) continue;
            float Rg = __fmaf_rn(-h.x, x, T_best) + 1e-30f;      // best so far less the group's least prefill time
            if (!(__fmaf_rn(h.z, y, h.y) <= Rg)) continue;
            const int4 geo = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);   // base, n_padded, ..
#pragma unroll 1
            for (int k = geo.x + geo.y - 8; k >= geo.x; k -= 8) {
                // the group's rows have d_lo >= gb.y (its last row's) and q words >= gb.x: if even
                // the type's least q with that d misses the best, so does everything from here up;
                // if the group's own least q with it does, the group holds nothing better
                const float2 gb = tb.group_bounds[GS_CHECKED(g_route_index_errors, k >> 3, kMaxPaddedRows / 8)];
                if (!(__fmaf_rn(gb.y, y, h.y) <= Rg)) break;
                if (kRowP ? !(__fmaf_rn(gb.y, y, __fmaf_rn(h.x, x, gb.x)) <= T_best + 1e-30f)
                          : !(__fmaf_rn(gb.y, y, gb.x) <= Rg)) continue;
                search_eight<kCapped, kRowP>(tb, k, x, y, need, d_cap, any_kv, h.x, g_best, T_best, Rg);
            }
        }
        tier_out = any_kv ? 3u : 2u;
    }
    if (g_best < 0) { tier_out = 0u; T_best = 0.f; }
    Pick r;
    r.g = g_best; r.T = T_best; r.tier = tier_out;
    return r;
}

// The definition evaluated in full by one warp for one request (same arguments in all lanes):
// lanes across instances, shuffle reductions.  tier 1: feasible instance with the largest d
// (ties: smallest index); tier 2 / 3: smallest T among instances with KV room / among all
// (ties: smallest index); tier 0 (kCapped only): no instance with d < d_cap exists.
template <bool kCapped>
__device__ __forceinline__ void exhaustive_pick(const Row *rows, int M, float xs, float ys, float Ds,
                                                unsigned needs, float d_cap, int lane,
                                                int &g, float &T, unsigned &tier)
{
    unsigned long long k_feas = 0ull;                    // max over feasible: (d, smallest index)
    unsigned long long k_room = ~0ull, k_all = ~0ull;    // min over KV-ok / all: (T, index)
    float T_feas = 0.f;
    for (int inst = lane; inst < M; inst += 32) {
        const Row row = rows[row_pos(inst)];
        if (kCapped && !(row.d < d_cap)) continue;
        GS_COUNT(kCountExact, 1);
        const float Tr = latency(row, xs, ys);
        const bool room = needs <= (unsigned)row.kv;
        const unsigned long long kt = ((unsigned long long)orderable_bits(Tr) << 32) | (unsigned)inst;
        if (kt < k_all) k_all = kt;
        if (room && kt < k_room) k_room = kt;
        if (room && Tr <= Ds) {
            const unsigned long long kd =
                ((unsigned long long)orderable_bits(row.d) << 32) | (0xFFFFu - (unsigned)inst);
            if (kd > k_feas) { k_feas = kd; T_feas = Tr; }
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
    if (w_feas != 0ull) {
        const unsigned owner = __ballot_sync(0xFFFFFFFFu, k_feas == w_feas);
        T = __shfl_sync(0xFFFFFFFFu, T_feas, __ffs(owner) - 1);
        g = (int)(0xFFFFu - (unsigned)(w_feas & 0xFFFFu)); tier = 1;
    } else if (w_room != ~0ull) {
        g = (int)(w_room & 0xFFFFFFFFull); T = from_orderable_bits((unsigned)(w_room >> 32)); tier = 2;
    } else if (w_all != ~0ull) {
        g = (int)(w_all & 0xFFFFFFFFull); T = from_orderable_bits((unsigned)(w_all >> 32)); tier = 3;
    } else {
        g = -1; T = 0.f; tier = 0;
    }
}

// ---------------------------------------------------------------------------------------
// the routing round
// ---------------------------------------------------------------------------------------

// Bulk asynchronous copies (global -> this one CTA's shared memory, from this GPU's own memory)
// that report to an mbarrier.  Addresses and sizes are multiples of 16 bytes.
__device__ __forceinline__ unsigned shared_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_copy_to_shared(void *dst, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(shared_addr(dst)), "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(shared_addr(bar)) : "memory");
}

// Waits for phase `parity` of the barrier, at most kBarrierTries tries (each try itself gives up
// after a hardware time limit): a wait that cannot end turns into `false`, never into a hang.
constexpr int kBarrierTries = 1 << 20;
__device__ __forceinline__ bool wait_barrier(unsigned long long *bar, unsigned parity) {
    unsigned done = 0;
    for (int it = 0; it < kBarrierTries && !done; ++it)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(shared_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}

// Shared-memory image of the round's tables for the route kernel, in the order it is carved.
struct TableImage {
    Row *rows; TypeHeader *headers; uint2 *row_bounds; float2 *group_bounds; unsigned char *start_table;
    unsigned short *cand; unsigned char *start_list; unsigned short *bucket_list; uint2 *pool; float *row_p; float4 *chord;
    int *info; unsigned long long *bar; unsigned char *end;
};

template <bool kRowP, bool kChord = false>
__device__ __forceinline__ TableImage carve_tables(unsigned char *smem, int n_types_alloc) {
    TableImage im;
    im.rows = reinterpret_cast<Row *>(smem);
    im.headers = reinterpret_cast<TypeHeader *>(im.rows + GS_MAX_INSTANCES);
    im.row_bounds = reinterpret_cast<uint2 *>(im.headers + GS_MAX_TYPES);
    im.group_bounds = reinterpret_cast<float2 *>(im.row_bounds + kMaxPaddedRows);
    im.start_table = reinterpret_cast<unsigned char *>(im.group_bounds + kMaxPaddedRows / 8);
    unsigned char *at = im.start_table + (size_t)n_types_alloc * (kStartBuckets * kStartSlots);
    im.row_p = nullptr; im.start_list = nullptr; im.bucket_list = nullptr; im.pool = nullptr; im.chord = nullptr;
    if (kRowP) {
        im.row_p = reinterpret_cast<float *>(at); at += kMaxPaddedRows * sizeof(float);
    }
    im.cand = reinterpret_cast<unsigned short *>(at); at += kCandSlots * sizeof(unsigned short);
    if (!kRowP) {
        im.start_list = at; at += (size_t)n_types_alloc * kStartBuckets * kStartSlots;
        im.bucket_list = reinterpret_cast<unsigned short *>(at); at += (size_t)n_types_alloc * kStartBuckets * sizeof(unsigned short);
        im.pool = reinterpret_cast<uint2 *>(at); at += (size_t)kPoolEntries * sizeof(uint2);
    }
    if (kChord) {
        im.chord = reinterpret_cast<float4 *>(at); at += (size_t)n_types_alloc * kStartBuckets * sizeof(float4);
    }
    im.info = reinterpret_cast<int *>(at); at += 64;
    im.bar = reinterpret_cast<unsigned long long *>(at); at += 16;
    im.end = at;
    return im;
}

// Where the round's tables lie in global memory, and upper bounds, known to the host, of how much
// of each the round can use (what lies beyond the round's own entries is never looked at).
struct TableSource {
    const Row *rows; const uint2 *row_bounds; const float2 *group_bounds; const unsigned char *start_table;
    const TypeHeader *headers; const int *info; const unsigned short *cand; const uint2 *pool;
    const unsigned short *bucket_list; const unsigned char *start_list; const float *row_p; const float4 *chord;
    int n_types_alloc, m_rows, n_padded_max;
};

// Starts the bulk copies of all tables into the image, all in flight together, one barrier for
// all of them (one thread).  The few numbers that only the prologue knows are copied along (info).
template <bool kRowP, bool kChord = false>
__device__ __forceinline__ void start_table_copies(const TableImage &im, const TableSource &src)
{
    const unsigned b_rows = (unsigned)src.m_rows * sizeof(Row), b_headers = (unsigned)src.n_types_alloc * sizeof(TypeHeader);
    const unsigned b_bounds = (unsigned)src.n_padded_max * sizeof(uint2), b_groups = (unsigned)src.n_padded_max / 8 * sizeof(float2);
    const unsigned b_start = (unsigned)src.n_types_alloc * (kStartBuckets * kStartSlots);
    const unsigned b_cand = kCandSlots * sizeof(unsigned short), b_info = 64u;
    const unsigned b_rowp = kRowP ? (unsigned)src.n_padded_max * sizeof(float) : 0u;
    const unsigned b_bucket = kRowP ? 0u : (unsigned)src.n_types_alloc * kStartBuckets * sizeof(unsigned short);
    const unsigned b_pool = kRowP ? 0u : (unsigned)kPoolEntries * sizeof(uint2);
    const unsigned b_chord = kChord ? (unsigned)src.n_types_alloc * kStartBuckets * sizeof(float4) : 0u;
    const unsigned total = b_rows + b_headers + b_bounds + b_groups + b_start + b_cand + b_info + b_rowp +
                           (kRowP ? 0u : b_start) + b_bucket + b_pool + b_chord;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(shared_addr(im.bar)), "r"(total) : "memory");
    bulk_copy_to_shared(im.info, src.info, b_info, im.bar);
    bulk_copy_to_shared(im.cand, src.cand, b_cand, im.bar);
    bulk_copy_to_shared(im.headers, src.headers, b_headers, im.bar);
    bulk_copy_to_shared(im.rows, src.rows, b_rows, im.bar);
    if (kRowP) {
        bulk_copy_to_shared(im.row_p, src.row_p, b_rowp, im.bar);
    } else {
        bulk_copy_to_shared(im.bucket_list, src.bucket_list, b_bucket, im.bar);
        bulk_copy_to_shared(im.start_list, src.start_list, b_start, im.bar);
        bulk_copy_to_shared(im.pool, src.pool, b_pool, im.bar);
    }
    if (kChord) bulk_copy_to_shared(im.chord, src.chord, b_chord, im.bar);
    bulk_copy_to_shared(im.start_table, src.start_table, b_start, im.bar);
    bulk_copy_to_shared(im.row_bounds, src.row_bounds, b_bounds, im.bar);
    bulk_copy_to_shared(im.group_bounds, src.group_bounds, b_groups, im.bar);
}

// First row of the eight at padded index k (a multiple of 8) whose bound passes: its tag word
// replaces `first`; rows are tested last to first so that the earliest one wins.
template <bool kRowP>
__device__ __forceinline__ unsigned first_pass_of_eight(const Tables &tb, int k, float x, float y, float R, unsigned first)
{
    const char *grp = reinterpret_cast<const char *>(tb.row_bounds + k);
    const int sw = (k >> 4) & 3;                // see row_slot()
    const uint4 r0 = *reinterpret_cast<const uint4 *>(grp + ((0 ^ sw) << 4));
    const uint4 r1 = *reinterpret_cast<const uint4 *>(grp + ((1 ^ sw) << 4));
    const uint4 r2 = *reinterpret_cast<const uint4 *>(grp + ((2 ^ sw) << 4));
    const uint4 r3 = *reinterpret_cast<const uint4 *>(grp + ((3 ^ sw) << 4));
    float4 pa = make_float4(0.f, 0.f, 0.f, 0.f), pb = pa;      // rows k..k+3, k+4..k+7
    if (kRowP) {
        pa = *reinterpret_cast<const float4 *>(tb.row_p + k);
        pb = *reinterpret_cast<const float4 *>(tb.row_p + k + 4);
    }
    first = row_may_pass<false, kRowP>(r3.z, r3.w, pb.w, x, y, R, 0.f) ? r3.z : first;
    first = row_may_pass<false, kRowP>(r3.x, r3.y, pb.z, x, y, R, 0.f) ? r3.x : first;
    first = row_may_pass<false, kRowP>(r2.z, r2.w, pb.y, x, y, R, 0.f) ? r2.z : first;
    first = row_may_pass<false, kRowP>(r2.x, r2.y, pb.x, x, y, R, 0.f) ? r2.x : first;
    first = row_may_pass<false, kRowP>(r1.z, r1.w, pa.w, x, y, R, 0.f) ? r1.z : first;
    first = row_may_pass<false, kRowP>(r1.x, r1.y, pa.z, x, y, R, 0.f) ? r1.x : first;
    first = row_may_pass<false, kRowP>(r0.z, r0.w, pa.y, x, y, R, 0.f) ? r0.z : first;
    first = row_may_pass<false, kRowP>(r0.x, r0.y, pa.x, x, y, R, 0.f) ? r0.x : first;
    return first;
}

// The short way to the just-enough pick, taken by every request first.  Straight-line code
// but for two short loops over GPU types:
//   1. the candidate table names the types whose least d fits D / L_out at all; the first of
//      them (largest d first) that passes its entry test is searched;
//   2. the start table gives the first entry worth a look in the record list of that type and
//      bucket of L_out (the rows that can be the first of the type to pass; see the prologue);
//      four entries from there are tested (with per-row p, where there are no such lists:
//      sixteen row bounds of the full list), and the first row that passes is scored exactly
//      as the definition says and checked against the deadline and the instance's free KV;
//   3. no later type may be able to do better: its largest d is below the pick's, or even its
//      least q with the pick's d misses the deadline.
// Returns false whenever this does not settle the request (nothing passed among the entries
// tested, there is no list, the scored row is not feasible, another type may hold a better instance, no type
// passes its entry test); the request is then queued for the full search.  When it returns
// true the pick is the definition's: every row ranked before it was ruled out by a true lower
// bound of its T, and every type that could rank before it by one of its whole type.
template <bool kRowP>
__device__ __forceinline__ bool fast_pick(const Tables &tb, float cand_z0, float cand_inv, float x, float y,
                                          float D, unsigned need, int &g_out, float &T_out)
{
    const float Dm = D + 1e-30f;                 // see route_kernel
    float ry;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(ry) : "f"(y));
    const float sc = fminf(fmaxf((Dm * ry - cand_z0) * cand_inv, 0.f), (float)(kCandSlots - 1));
    unsigned mask = tb.cand[GS_CHECKED(g_route_index_errors, __float2int_rd(sc), kCandSlots)];
    int t = -1;
    float4 h = make_float4(0.f, 0.f, 0.f, 0.f);
    float Rg = 0.f;
    while (mask) {
        const int tt = __ffs(mask) - 1;
        mask &= mask - 1;
        h = *reinterpret_cast<const float4 *>(&tb.headers[tt]);               // p_lo, q_lo, d_lo, d_max
        Rg = __fmaf_rn(-h.x, x, Dm);
        GS_COUNT(kCountTypeTest, 1);
        if (__fmaf_rn(h.z, y, h.y) <= Rg) { t = tt; break; }
    }
    if (t < 0) return false;
    const int4 geo = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);   // base, n_padded, inv_w, d0
    const int ybucket = min((int)(__float_as_uint(y) >> (23 - kBucketBits)) - (127 << kBucketBits), kStartBuckets - 1);
    const int cell = GS_CHECKED(g_route_index_errors, (t * kStartBuckets + ybucket) * kStartSlots +
                     start_slot(Rg, h.y, ry, __int_as_float(geo.w), __int_as_float(geo.z)), tb.n_types * kStartBuckets * kStartSlots);
    unsigned first = kNoRow;
    if (kRowP) {
        // rows of a group differ in p: sixteen row bounds of the group's full list
        const int k = geo.x + 8 * tb.start_table[cell];
        const int k2 = min(k + 8, geo.x + geo.y - 8);    // (the last group of a type is tested twice)
        first = first_pass_of_eight<kRowP>(tb, k2, x, y, Dm, kNoRow);
        first = first_pass_of_eight<kRowP>(tb, k, x, y, Dm, first);
    } else {
        // the record list of this type and bucket of L_out: only rows that can be the first to pass
        const unsigned list = tb.bucket_list[t * kStartBuckets + ybucket];
        if (list == kNoList) return false;
        // (the window of four pairs of entries read from there must end inside the pool)
        const uint4 *w = reinterpret_cast<const uint4 *>(tb.pool) +
                         GS_CHECKED(g_route_index_errors, list + tb.start_list[cell], kPoolEntries / 2 - 3);
        const uint4 r0 = w[0], r1 = w[1];
        first = row_may_pass<false, false>(r1.z, r1.w, 0.f, x, y, Rg, 0.f) ? r1.z : first;
        first = row_may_pass<false, false>(r1.x, r1.y, 0.f, x, y, Rg, 0.f) ? r1.x : first;
        first = row_may_pass<false, false>(r0.z, r0.w, 0.f, x, y, Rg, 0.f) ? r0.z : first;
        first = row_may_pass<false, false>(r0.x, r0.y, 0.f, x, y, Rg, 0.f) ? r0.x : first;
        if (first == kNoRow) {                   // one lane in a hundred: the next four entries
            const uint4 r2 = w[2], r3 = w[3];    // (still inside the list or its padding: see below)
            first = row_may_pass<false, false>(r3.z, r3.w, 0.f, x, y, Rg, 0.f) ? r3.z : first;
            first = row_may_pass<false, false>(r3.x, r3.y, 0.f, x, y, Rg, 0.f) ? r3.x : first;
            first = row_may_pass<false, false>(r2.z, r2.w, 0.f, x, y, Rg, 0.f) ? r2.z : first;
            first = row_may_pass<false, false>(r2.x, r2.y, 0.f, x, y, Rg, 0.f) ? r2.x : first;
        }
    }
    if (first == kNoRow) return false;
    const int inst = (int)(first & kRowTagMask);
    GS_COUNT(kCountExact, 1);
    const Row row = tb.rows[GS_CHECKED(g_route_index_errors, row_pos(inst), GS_MAX_INSTANCES)];
    const float T = __fmaf_rn(row.d, y, __fmaf_rn(row.p, x, row.q));          // Eq. 2, H = 0
    if (!(T <= D && need <= (unsigned)row.kv)) return false;
    const float d_floor = __fmul_rn(row.d, 1.0f - 1.9073486328125e-6f);       // the bound every row with d >= the pick's carries
    while (mask) {
        const int tt = __ffs(mask) - 1;
        mask &= mask - 1;
        const float4 h2 = *reinterpret_cast<const float4 *>(&tb.headers[tt]);
        if (h2.w < row.d) break;                                              // nor can any type after it
        GS_COUNT(kCountTypeTest, 1);
        if (__fmaf_rn(fmaxf(h2.z, d_floor), y, h2.y) <= __fmaf_rn(-h2.x, x, Dm)) return false;
    }
    g_out = inst;
    T_out = T;
    return true;
}

// The same first attempt for pools whose types overlap in d, where a later type often may hold
// a better instance than the first one's pick: instead of giving up there it goes on to that
// type (and on a type whose record list ends inside the window without a row passing), keeping
// the best pick so far; it gives up only where a type's answer stays open (no list, nothing
// passes among the entries tested although the list goes on, the scored row is not feasible).
// Costs a few instructions more per request than fast_pick even when one type settles it, so
// the kernel for small batches (one request per lane) uses it and the one for large batches
// does not.
template <bool kRowP>
__device__ __forceinline__ bool fast_pick_several(const Tables &tb, float cand_z0, float cand_inv, float x, float y,
                                          float D, unsigned need, int &g_out, float &T_out)
{
    const float Dm = D + 1e-30f;                 // see route_kernel
    float ry;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(ry) : "f"(y));
    const float sc = fminf(fmaxf((Dm * ry - cand_z0) * cand_inv, 0.f), (float)(kCandSlots - 1));
    unsigned mask = tb.cand[GS_CHECKED(g_route_index_errors, __float2int_rd(sc), kCandSlots)];
    const int ybucket = min((int)(__float_as_uint(y) >> (23 - kBucketBits)) - (127 << kBucketBits), kStartBuckets - 1);
    int g_best = -1;
    float T_best = 0.f, d_best = -1.0f, d_floor = 0.f;
    for (;;) {
        int t = -1;
        float4 h = make_float4(0.f, 0.f, 0.f, 0.f);
        float Rg = 0.f;
        while (mask) {
            const int tt = __ffs(mask) - 1;
            mask &= mask - 1;
            h = *reinterpret_cast<const float4 *>(&tb.headers[tt]);               // p_lo, q_lo, d_lo, d_max
            if (h.w < d_best) { mask = 0; break; }                                // nor can any type after it
            Rg = __fmaf_rn(-h.x, x, Dm);
            GS_COUNT(kCountTypeTest, 1);
            if (__fmaf_rn(fmaxf(h.z, d_floor), y, h.y) <= Rg) { t = tt; break; }
        }
        if (t < 0) break;
        const int4 geo = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);   // base, n_padded, inv_w, d0
        const int cell = GS_CHECKED(g_route_index_errors, (t * kStartBuckets + ybucket) * kStartSlots +
                         start_slot(Rg, h.y, ry, __int_as_float(geo.w), __int_as_float(geo.z)), tb.n_types * kStartBuckets * kStartSlots);
        unsigned first = kNoRow;
        if (kRowP) {
            const int k = geo.x + 8 * tb.start_table[cell];
            const int k2 = min(k + 8, geo.x + geo.y - 8);
            first = first_pass_of_eight<kRowP>(tb, k2, x, y, Dm, kNoRow);
            first = first_pass_of_eight<kRowP>(tb, k, x, y, Dm, first);
            if (first == kNoRow) return false;
        } else {
            const unsigned list = tb.bucket_list[t * kStartBuckets + ybucket];
            if (list == kNoList) return false;
            const uint4 *w = reinterpret_cast<const uint4 *>(tb.pool) +
                             GS_CHECKED(g_route_index_errors, list + tb.start_list[cell], kPoolEntries / 2 - 3);
            const uint4 r0 = w[0], r1 = w[1];
            first = row_may_pass<false, false>(r1.z, r1.w, 0.f, x, y, Rg, 0.f) ? r1.z : first;
            first = row_may_pass<false, false>(r1.x, r1.y, 0.f, x, y, Rg, 0.f) ? r1.x : first;
            first = row_may_pass<false, false>(r0.z, r0.w, 0.f, x, y, Rg, 0.f) ? r0.z : first;
            first = row_may_pass<false, false>(r0.x, r0.y, 0.f, x, y, Rg, 0.f) ? r0.x : first;
            if (first == kNoRow) {
                const uint4 r2 = w[2], r3 = w[3];
                first = row_may_pass<false, false>(r3.z, r3.w, 0.f, x, y, Rg, 0.f) ? r3.z : first;
                first = row_may_pass<false, false>(r3.x, r3.y, 0.f, x, y, Rg, 0.f) ? r3.x : first;
                first = row_may_pass<false, false>(r2.z, r2.w, 0.f, x, y, Rg, 0.f) ? r2.z : first;
                first = row_may_pass<false, false>(r2.x, r2.y, 0.f, x, y, Rg, 0.f) ? r2.x : first;
                if (first == kNoRow) {
                    if (r3.z == kPadQ) continue;
                    return false;
                }
            }
        }
        const int inst = (int)(first & kRowTagMask);
        GS_COUNT(kCountExact, 1);
        const Row row = tb.rows[GS_CHECKED(g_route_index_errors, row_pos(inst), GS_MAX_INSTANCES)];
        const float T = __fmaf_rn(row.d, y, __fmaf_rn(row.p, x, row.q));          // Eq. 2, H = 0
        if (!(T <= D && need <= (unsigned)row.kv)) return false;
        if (g_best < 0 || row.d > d_best || (row.d == d_best && inst < g_best)) {
            g_best = inst; T_best = T; d_best = row.d;
            d_floor = __fmul_rn(row.d, 1.0f - 1.9073486328125e-6f);
        }
    }
    if (g_best < 0) return false;
    g_out = g_best;
    T_out = T_best;
    return true;
}

// The full search for one request per lane (lanes without a request pass active = false):
// the just-enough pick over all types, then the fallback of Algorithm 1 -- by the lane itself
// when several lanes need it, by the whole warp otherwise and for requests that the tables
// cannot serve (L_out == 0, unusable coefficients).
// A request that needs more KV than any instance has free (need > kv_max) cannot be served in
// tier 1 or 2: it goes straight to the minimum of T over all instances (tier 3).
template <bool kRowP>
__device__ __noinline__ Pick full_pick(const Tables tb, int M, unsigned kv_max, int lane, bool active, int xi, int yi, float D)
{
    const unsigned need = (unsigned)xi + (unsigned)yi;      // < 2^32, no overflow
    const bool room_somewhere = need <= kv_max;
    const float x = __int2float_rn(xi), y = __int2float_rn(yi);
    // an empty lane, or L_out == 0 (the start table divides by it), skips the search; the hair
    // added to the deadline of the bound tests keeps them safe when a bound's tag bits make a
    // zero coefficient a denormal
    const float Dj = (active && yi > 0 && room_somewhere) ? D : -1.0f;
    Pick out;
    out.T = 0.f;
    out.g = pick_instance<false, kRowP>(tb, x, y, Dj, Dj + 1e-30f, need, 0.f, out.T);
    out.tier = 1u;
    bool open = active && out.g < 0;
    const bool mine = open && yi > 0 && tb.n_types > 0;
    const int n_fall = __popc(__ballot_sync(0xFFFFFFFFu, mine));
    if (mine && n_fall >= kThreadFallbackMin) {
        GS_COUNT(kCountFallback, 1);
        out = fallback_pick<false, kRowP>(tb, x, y, need, 0.f, room_somewhere ? 0 : 1);
        open = false;
    }
    unsigned todo = __ballot_sync(0xFFFFFFFFu, open);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const float xs = __shfl_sync(0xFFFFFFFFu, x, src), ys = __shfl_sync(0xFFFFFFFFu, y, src);
        const float Ds = __shfl_sync(0xFFFFFFFFu, D, src);
        const unsigned needs = __shfl_sync(0xFFFFFFFFu, need, src);
        int gg; float TT; unsigned tt;
        if (lane == 0) GS_COUNT(kCountExhaustive, 1);
        exhaustive_pick<false>(tb.rows, M, xs, ys, Ds, needs, 0.f, lane, gg, TT, tt);
        if (lane == src) { out.g = gg; out.T = TT; out.tier = tt; }
    }
    return out;
}

// Prefix-cache term of Eq. 2 for one (instance, hit length) pair of a request whose hit-free
// pick is (g_cur, T_cur, tier): on the named instance T is lower by p * H; it is scored again
// with its hit and merged into the answer.
__device__ __forceinline__ void merge_hit(const Row *rows, int M, int g, int h, int xi, int yi, float D,
                                          int &g_cur, float &T_cur, unsigned &tier, unsigned &bad)
{
    if (g < 0) return;                                       // empty slot
    if (g >= M) { bad |= GS_DEV_BAD_INSTANCE; return; }      // names nothing
    if (h < 0 || h > xi) { bad |= GS_DEV_BAD_VALUE; h = h < 0 ? 0 : xi; }
    const Row row = rows[row_pos(g)];
    const float T = __fmaf_rn(row.d, __int2float_rn(yi), __fmaf_rn(row.p, __int2float_rn(xi - h), row.q));
    const bool room = (unsigned)xi + (unsigned)yi <= (unsigned)row.kv;
    bool take;
    if (room && T <= D) {                                    // feasible with its hit
        const float d_cur = tier == 1u ? rows[row_pos(g_cur)].d : 0.f;
        take = tier != 1u || row.d > d_cur || (row.d == d_cur && g < g_cur) || (g == g_cur && T < T_cur);
        if (take) tier = 1u;
    } else {                                                 // may still lead the fallback
        take = tier >= 2u && (room || tier == 3u) && (T < T_cur || (T == T_cur && g < g_cur));
    }
    if (take) { g_cur = g; T_cur = T; }
}

constexpr int kQueueCap = 160;          // per warp: at most 31 left over + the 128 requests of a tile

// A warp takes 128 consecutive requests at a time, four per lane (128-bit column loads and
// stores).  Every request first tries fast_pick; the ones it does not settle are put on the
// warp's queue in shared memory (by their index: the columns are read again), and whenever 32
// have gathered, between two tiles, each lane takes one of them through full_pick, so the
// long, divergent search always runs with all lanes busy.  Their results are stored one by one
// over the placeholders that the tile's vector stores left.
template <bool kAccumulate, bool kPrefix, bool kRowP, int kReqPerThread>
__global__ void __launch_bounds__(route_threads(kRowP, kReqPerThread), kRouteMinCtas)
route_kernel(const int32_t *__restrict__ prompt_len, const int32_t *__restrict__ pred_decode_len,
             const float *__restrict__ slo_ms, int64_t n, const PrefixHits hits, int n_types_alloc,
             const Row *__restrict__ g_rows, const uint2 *__restrict__ g_row_bounds,
             const float2 *__restrict__ g_group_bounds,
             const unsigned char *__restrict__ g_start_table,
             const TypeHeader *__restrict__ g_headers, const int *__restrict__ table_info,
             const unsigned short *__restrict__ g_cand, const uint2 *__restrict__ g_pool,
             const unsigned short *__restrict__ g_bucket_list, const unsigned char *__restrict__ g_start_list,
             const float *__restrict__ g_row_p, int m_rows, int n_padded_max,
             int32_t *__restrict__ out_idx, float *__restrict__ out_est,
             float *__restrict__ out_slack, uint8_t *__restrict__ out_tier,
             unsigned long long *__restrict__ deltas, unsigned *__restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    static_assert(kReqPerThread == 4 || kReqPerThread == 1, "four requests per lane (128-bit column loads) or one");
    const int lane = threadIdx.x & 31;
    constexpr int kWarpTile = 32 * kReqPerThread;
    const int64_t n_wtiles = (n + kWarpTile - 1) / kWarpTile;
    // A CTA owns a contiguous run of warp tiles; its warps take them one at a time from a shared
    // counter, so a warp that is held up by a full search simply takes fewer.
    const int64_t tiles_per_cta = (n_wtiles + gridDim.x - 1) / gridDim.x;
    const int64_t cta_first = (int64_t)blockIdx.x * tiles_per_cta;
    const int64_t cta_end = min(cta_first + tiles_per_cta, n_wtiles);
    __shared__ int sh_next_tile;
    if (threadIdx.x == 0) sh_next_tile = route_threads(kRowP, kReqPerThread) / 32;     // the first round is dealt by warp number
    const int64_t wt0 = cta_first + (threadIdx.x >> 5);
    // the request columns of a warp's tile, four requests per lane; slots past the end read as
    // requests that nothing can serve
    auto load_tile = [&](int64_t tile, int (&xs)[kReqPerThread], int (&ys)[kReqPerThread], float (&ds)[kReqPerThread]) {
        const int64_t first = tile * kWarpTile + (int64_t)lane * kReqPerThread;
        if (kReqPerThread == 4 && first + kReqPerThread <= n) {
            const int4 xv = __ldcs(reinterpret_cast<const int4 *>(prompt_len + first));
            const int4 yv = __ldcs(reinterpret_cast<const int4 *>(pred_decode_len + first));
            const float4 dv = __ldcs(reinterpret_cast<const float4 *>(slo_ms + first));
            const int xa[4] = {xv.x, xv.y, xv.z, xv.w}, ya[4] = {yv.x, yv.y, yv.z, yv.w};
            const float da[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j) { xs[j] = xa[j]; ys[j] = ya[j]; ds[j] = da[j]; }
        } else {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j) {
                const bool v = first + j < n;
                xs[j] = v ? __ldcs(prompt_len + first + j) : 0;
                ys[j] = v ? __ldcs(pred_decode_len + first + j) : 0;
                ds[j] = v ? __ldcs(slo_ms + first + j) : -1.0f;
            }
        }
    };
    int nx[kReqPerThread], ny[kReqPerThread];      // the tile on its way
    float nd[kReqPerThread];
#pragma unroll
    for (int j = 0; j < kReqPerThread; ++j) { nx[j] = 0; ny[j] = 0; nd[j] = -1.0f; }
    if (wt0 < cta_end) load_tile(wt0, nx, ny, nd);           // under way while the tables are staged
    // The kernel is launched as a programmatic dependent of the prologue: everything above ran
    // beside it; the tables may be read once that whole grid is done and its stores are visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The tables come in by bulk asynchronous copies (start_table_copies).
    const TableImage im = carve_tables<kRowP>(smem, n_types_alloc);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(shared_addr(im.bar)) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const TableSource src = {g_rows, g_row_bounds, g_group_bounds, g_start_table, g_headers, table_info, g_cand, g_pool,
                                 g_bucket_list, g_start_list, g_row_p, nullptr, n_types_alloc, m_rows, n_padded_max};
        start_table_copies<kRowP>(im, src);
    }
    unsigned char *after_tables = im.end;
    // the warps' queues: {L_in, L_out, bits of D, low word of the request index}, high word
    constexpr int kWarps = route_threads(kRowP, kReqPerThread) / 32;
    // (entries: the request's index less that of the CTA's first request; a CTA's run of requests
    // is far below 2^32)
    unsigned *queue_all = reinterpret_cast<unsigned *>(after_tables);
    unsigned *queue = queue_all + (threadIdx.x >> 5) * kQueueCap;
    after_tables += kWarps * kQueueCap * sizeof(unsigned);
    const int64_t cta_first_request = cta_first * kWarpTile;
    unsigned long long *hist = reinterpret_cast<unsigned long long *>(after_tables);
    if (kAccumulate)
        for (int k = threadIdx.x; k < 3 * GS_MAX_INSTANCES; k += blockDim.x) hist[k] = 0ull;
    // every thread waits for the tables itself (the barrier's phase is what makes them visible)
    {
        const bool arrived = wait_barrier(im.bar, 0u);
        if (!__syncthreads_and(arrived)) {
            // the copies did not complete in time: report it, give them one more chance to land
            // (nothing may still be writing this CTA's shared memory when it exits) and leave
            if (threadIdx.x == 0) atomicOr(status, (unsigned)GS_DEV_TIMEOUT);
            wait_barrier(im.bar, 0u);
            return;
        }
    }
    const int M = im.info[2];
    const unsigned kv_max = (unsigned)im.info[8];         // no instance has more free KV than this
    const float cand_z0 = __int_as_float(im.info[4]), cand_inv = __int_as_float(im.info[5]);
    Tables tb;
    tb.headers = im.headers; tb.row_bounds = im.row_bounds; tb.group_bounds = im.group_bounds;
    tb.start_table = im.start_table; tb.rows = im.rows; tb.row_p = im.row_p; tb.cand = im.cand;
    tb.pool = im.pool; tb.bucket_list = im.bucket_list; tb.start_list = im.start_list; tb.chord = nullptr;
    tb.n_types = im.info[1] != 0 ? 0 : im.info[3];       // unusable bounds: every request takes the exhaustive path

    const bool fast_on = tb.n_types > 0;          // unusable bounds: every request takes the full search
    unsigned bad = 0;
    int q_count = 0;                               // entries on this warp's queue (same in all lanes)

    // takes one queued request per lane through the full search and stores the results
    auto settle = [&](bool active, unsigned entry) {
        const int64_t r = cta_first_request + entry;
        int4 e = make_int4(0, 0, 0, 0);
        float D = -1.0f;
        if (active) { e.x = max(prompt_len[r], 0); e.y = max(pred_decode_len[r], 0); D = slo_ms[r]; }
        const Pick pk = full_pick<kRowP>(tb, M, kv_max, lane, active, e.x, e.y, D);
        int g = pk.g; float T = pk.T; unsigned tier = pk.tier;
        if (kPrefix && active)
            for (int k = 0; k < hits.n_slots; ++k)
                merge_hit(tb.rows, M, hits.inst[(int64_t)k * hits.slot_stride + r],
                          hits.hit_len[(int64_t)k * hits.slot_stride + r], e.x, e.y, D, g, T, tier, bad);
        if (kAccumulate) accumulate_choice(hist, M, active ? g : -1, (unsigned)e.x, (unsigned)e.x + (unsigned)e.y);
        if (active) {
            out_idx[r] = g;
            out_est[r] = T;
            out_slack[r] = __fsub_rn(D, T);
            if (out_tier) out_tier[r] = (uint8_t)tier;
        }
    };
    // ... the newest (up to) 32 of this warp's queue
    auto drain = [&]() {
        const int cnt = min(q_count, 32);
        q_count -= cnt;
        const bool active = lane < cnt;
        unsigned entry = 0;
        if (active) entry = queue[q_count + lane];
        __syncwarp();                              // the slots may be written again
        settle(active, entry);
    };

    int64_t wt = wt0;
    for (;;) {
    // (the full search is kept out of this loop: it runs between two tiles, further down)
    while (wt < cta_end && q_count < 32) {
        const int64_t first = wt * kWarpTile + (int64_t)lane * kReqPerThread;
        const bool full = kReqPerThread == 4 && first + kReqPerThread <= n;
        int xi[kReqPerThread], yi[kReqPerThread];
        float D[kReqPerThread];
#pragma unroll
        for (int j = 0; j < kReqPerThread; ++j) { xi[j] = nx[j]; yi[j] = ny[j]; D[j] = nd[j]; }
        {
            int t = 0;
            if (lane == 0) t = atomicAdd(&sh_next_tile, 1);
            wt = cta_first + __shfl_sync(0xFFFFFFFFu, t, 0);
        }
        if (wt < cta_end) load_tile(wt, nx, ny, nd);         // the next tile is on its way while this one is searched
        int any_sign = 0;
#pragma unroll
        for (int j = 0; j < kReqPerThread; ++j) any_sign |= xi[j] | yi[j];
        if (any_sign < 0) {                                  // negative counts read as 0
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j) { xi[j] = max(xi[j], 0); yi[j] = max(yi[j], 0); }
            bad |= GS_DEV_BAD_VALUE;
        }
        int g_out[kReqPerThread];
        float T_out[kReqPerThread];
        unsigned tiers = 0x01010101u;             // one byte per request
        unsigned slow = 0;                        // bit j: request j of this lane goes to the queue
#pragma unroll
        for (int j = 0; j < kReqPerThread; ++j) {
            const bool valid = first + j < n;
            g_out[j] = -1; T_out[j] = 0.f;
            // (an empty slot, or L_out == 0, which the start table cannot take, gets a deadline that
            // nothing meets and so ends up in the full search)
            bool settled = false;
            if (fast_on && (unsigned)xi[j] + (unsigned)yi[j] <= kv_max)
                settled = kReqPerThread == 1
                    ? fast_pick_several<kRowP>(tb, cand_z0, cand_inv, __int2float_rn(xi[j]), __int2float_rn(yi[j]),
                                               (valid && yi[j] > 0) ? D[j] : -1.0f, (unsigned)xi[j] + (unsigned)yi[j], g_out[j], T_out[j])
                    : fast_pick<kRowP>(tb, cand_z0, cand_inv, __int2float_rn(xi[j]), __int2float_rn(yi[j]),
                                       (valid && yi[j] > 0) ? D[j] : -1.0f, (unsigned)xi[j] + (unsigned)yi[j], g_out[j], T_out[j]);
            if (valid && !settled) { slow |= 1u << j; GS_COUNT(kCountQueued, 1); }
        }
        if (kPrefix) {
            for (int k = 0; k < hits.n_slots; ++k) {
                const int32_t *col_g = hits.inst + (int64_t)k * hits.slot_stride;
                const int32_t *col_h = hits.hit_len + (int64_t)k * hits.slot_stride;
                int hg[kReqPerThread], hh[kReqPerThread];
                if (full) {
                    const int4 gv = __ldcs(reinterpret_cast<const int4 *>(col_g + first));
                    const int4 hv = __ldcs(reinterpret_cast<const int4 *>(col_h + first));
                    const int ga[4] = {gv.x, gv.y, gv.z, gv.w}, ha[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                    for (int j = 0; j < kReqPerThread; ++j) { hg[j] = ga[j]; hh[j] = ha[j]; }
                } else {
#pragma unroll
                    for (int j = 0; j < kReqPerThread; ++j) {
                        const bool v = first + j < n;
                        hg[j] = v ? col_g[first + j] : -1;
                        hh[j] = v ? col_h[first + j] : 0;
                    }
                }
#pragma unroll
                for (int j = 0; j < kReqPerThread; ++j) {
                    if (g_out[j] < 0) continue;                      // queued: merged after the full search
                    unsigned tier = 1u;
                    merge_hit(tb.rows, M, hg[j], hh[j], xi[j], yi[j], D[j], g_out[j], T_out[j], tier, bad);
                }
            }
        }
        if (kAccumulate) {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j)
                accumulate_choice(hist, M, g_out[j], (unsigned)xi[j], (unsigned)xi[j] + (unsigned)yi[j]);
        }
        if (full) {
            constexpr int k1 = kReqPerThread > 1 ? 1 : 0, k2 = kReqPerThread > 2 ? 2 : 0, k3 = kReqPerThread > 3 ? 3 : 0;
            __stcs(reinterpret_cast<int4 *>(out_idx + first), make_int4(g_out[0], g_out[k1], g_out[k2], g_out[k3]));
            __stcs(reinterpret_cast<float4 *>(out_est + first), make_float4(T_out[0], T_out[k1], T_out[k2], T_out[k3]));
            __stcs(reinterpret_cast<float4 *>(out_slack + first),
                   make_float4(__fsub_rn(D[0], T_out[0]), __fsub_rn(D[k1], T_out[k1]),
                               __fsub_rn(D[k2], T_out[k2]), __fsub_rn(D[k3], T_out[k3])));
            if (out_tier) *reinterpret_cast<unsigned *>(out_tier + first) = tiers;
        } else {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j)
                if (first + j < n) {
                    __stcs(out_idx + first + j, g_out[j]);
                    __stcs(out_est + first + j, T_out[j]);
                    __stcs(out_slack + first + j, __fsub_rn(D[j], T_out[j]));
                    if (out_tier) out_tier[first + j] = (uint8_t)1;
                }
        }
        // ---- queue what is open ---------------------------------------------------------------
        if (__any_sync(0xFFFFFFFFu, slow != 0)) {
#pragma unroll
            for (int j = 0; j < kReqPerThread; ++j) {
                const bool push = (slow >> j) & 1u;
                const unsigned votes = __ballot_sync(0xFFFFFFFFu, push);
                if (push) queue[GS_CHECKED(g_route_index_errors, q_count + __popc(votes & ((1u << lane) - 1u)), kQueueCap)] =
                              (unsigned)(first + j - cta_first_request);
                q_count += __popc(votes);
            }
            __syncwarp();                          // the entries, and the stores above, come before the full search
        }
    }
    if (q_count < 32) break;                       // out of tiles
    do drain(); while (q_count >= 32);
    }
    // (the kernel after this one in the stream may be set up from now on)
    asm volatile("griddepcontrol.launch_dependents;");
    // What is left on the warp's queue (fewer than 32) it finishes itself, right after its last
    // tile: the warps of a CTA end up to a tile apart, so these searches overlap the other warps'
    // last tiles, and a handful of lanes per warp diverge far less than 32 would.
    while (q_count > 0) drain();
    if (bad) atomicOr(status, bad);

    if (kAccumulate) {
        __syncthreads();
        for (int k = threadIdx.x; k < 3 * M; k += blockDim.x) {
            const unsigned long long v = hist[k];
            if (v) atomicAdd(&deltas[(k / M) * GS_MAX_INSTANCES + (k % M)], v);
        }
    }
}

constexpr size_t kTablesSmemFixed = (size_t)GS_MAX_INSTANCES * sizeof(Row) + GS_MAX_TYPES * sizeof(TypeHeader) +
                                    (size_t)kMaxPaddedRows * sizeof(uint2) + kMaxPaddedRows / 8 * sizeof(float2);
constexpr size_t kRouteSmemFixed = kTablesSmemFixed + kCandSlots * sizeof(unsigned short) + 64 + 16 +   // info, barrier
                                   (size_t)(route_threads(false, 1) / 32) * kQueueCap * sizeof(unsigned);
constexpr size_t kRouteSmemPerType = (size_t)kStartBuckets * kStartSlots;
constexpr size_t kRouteSmemHist = (size_t)3 * GS_MAX_INSTANCES * sizeof(unsigned long long);
constexpr size_t kRouteSmemRowP = (size_t)kMaxPaddedRows * sizeof(float);
constexpr size_t kRouteSmemPerTypeLists = (size_t)kStartBuckets * kStartSlots + kStartBuckets * sizeof(unsigned short);
constexpr size_t kRouteSmemPool = (size_t)kPoolEntries * sizeof(uint2);

// Dynamic shared memory of one route CTA: the tables of n_types types (with record lists for a
// typed pool, per-row p for coefficients given per instance), the warps' queues, the histogram.
static size_t route_smem_bytes(int n_types, bool accumulate, bool row_p) {
    return kRouteSmemFixed + kRouteSmemPerType * n_types + (accumulate ? kRouteSmemHist : 0) +
           (row_p ? kRouteSmemRowP : kRouteSmemPerTypeLists * n_types + kRouteSmemPool);
}

// The context's tables as a kernel argument, with the upper bounds of what a kernel copies of
// them: the rows (position-mixed in blocks of eight) and the padded rows of all groups (each
// group adds less than 16 of padding).
static TableSource table_source(const gs_ctx *ctx, int n_instances, int n_types) {
    TableSource src;
    src.rows = ctx->s.rows; src.row_bounds = ctx->s.row_bounds; src.group_bounds = ctx->s.group_bounds;
    src.start_table = ctx->s.start_table; src.headers = ctx->s.headers; src.info = ctx->s.table_info;
    src.cand = ctx->s.cand_table; src.pool = ctx->s.pool; src.bucket_list = ctx->s.bucket_list;
    src.start_list = ctx->s.start_list; src.row_p = ctx->s.row_p; src.chord = ctx->s.chord;
    src.n_types_alloc = n_types;
    src.m_rows = (n_instances + 7) & ~7;
    src.n_padded_max = (n_instances + 16 * n_types + 15) & ~15;
    if (src.n_padded_max > kMaxPaddedRows) src.n_padded_max = kMaxPaddedRows;
    return src;
}

cudaError_t launch_route(gs_ctx *ctx, const int32_t *prompt_len, const int32_t *pred_decode_len,
                         const float *slo_ms, int64_t n, const PrefixHits *hits, int n_instances, int n_types,
                         int32_t *out_idx, float *out_est, float *out_slack, uint8_t *out_tier,
                         bool accumulate, bool row_p, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    if (n > kMaxRouteRequests) return cudaErrorInvalidValue;      // (the entry points refuse it first)
    const size_t smem = route_smem_bytes(n_types, accumulate, row_p);
    const TableSource src = table_source(ctx, n_instances, n_types);
    const int m_rows = src.m_rows, n_padded_max = src.n_padded_max;
    const int req = n < kSmallBatch ? 1 : 4;
    const int64_t tile = (int64_t)route_threads(row_p, req) * req;
    int64_t blocks = (n + tile - 1) / tile;
    if (blocks > ctx->n_sm) blocks = ctx->n_sm;   // one CTA per SM: its tables fill most of the shared memory
    LaunchTimer timer(ctx, GS_K_ROUTE, st);
    const PrefixHits none = {nullptr, nullptr, 0, 0};
    // a programmatic dependent of the kernel before it in the stream (the prologue): it may be
    // set up, and read its first requests, while that kernel still runs
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err = cudaSuccess;
#define GS_LAUNCH_ROUTE(ACC, PFX, ROWP)                                                               \
    if (req == 1) GS_LAUNCH_ROUTE_R(ACC, PFX, ROWP, 1); else GS_LAUNCH_ROUTE_R(ACC, PFX, ROWP, 4)
#define GS_LAUNCH_ROUTE_R(ACC, PFX, ROWP, REQ)                                                        \
    do {                                                                                              \
        cfg.blockDim = dim3(route_threads(ROWP, REQ));                                                \
        err = cudaLaunchKernelEx(&cfg, route_kernel<ACC, PFX, ROWP, REQ>,                             \
            prompt_len, pred_decode_len, slo_ms, n, hits ? *hits : none, n_types, (const Row *)ctx->s.rows,            \
            (const uint2 *)ctx->s.row_bounds, (const float2 *)ctx->s.group_bounds, (const unsigned char *)ctx->s.start_table, \
            (const TypeHeader *)ctx->s.headers, (const int *)ctx->s.table_info, (const unsigned short *)ctx->s.cand_table,  \
            (const uint2 *)ctx->s.pool, (const unsigned short *)ctx->s.bucket_list, (const unsigned char *)ctx->s.start_list, \
            (const float *)ctx->s.row_p, m_rows, n_padded_max,                                        \
            out_idx, out_est, out_slack, out_tier, ctx->s.deltas, ctx->s.status);                     \
    } while (0)
    // (the prefix term and per-row p are never combined with accumulate, nor with each other)
    if (row_p) GS_LAUNCH_ROUTE(false, false, true);
    else if (hits && hits->n_slots > 0) GS_LAUNCH_ROUTE(false, true, false);
    else if (accumulate) GS_LAUNCH_ROUTE(true, false, false);
    else GS_LAUNCH_ROUTE(false, false, false);
#undef GS_LAUNCH_ROUTE
#undef GS_LAUNCH_ROUTE_R
    return err;
}

// ---------------------------------------------------------------------------------------
// re-routing of the scan's candidates among strictly faster instances (Sec. 3.4)
// ---------------------------------------------------------------------------------------

// The short way for a re-routed candidate, modelled on fast_pick.  The search without the cap is
// tried: if its pick happens to be strictly faster than the current instance it is the capped
// search's pick as well (the eligible instances are a subset that holds the unrestricted
// optimum), and a request that is at risk where it runs can only be feasible on a faster
// instance, so this is the usual case.  Going through the candidate types in search order:
//   * a type that fails its entry test (R below the type's chord for this bucket of L_out: see
//     the prologue) holds no feasible instance;
//   * nor does a type whose record list, from the start cell on, ends inside the eight entries
//     tested without one of them passing (a row that is not a record passes only if a record
//     before it does, and the records before the start cell cannot pass);
//   * the first row that passes is scored exactly; if it is feasible and below the cap, and no
//     later type can rank before it, it is the answer.
// Returns 1 (settled: g_out, T_out), -1 (no instance at all is feasible, capped or not: the
// fallback decides) or 0 (not settled: the capped search in full).
__device__ __forceinline__ int capped_first_attempt(const Tables &tb, float x, float y,
                                                    float D, unsigned need, float d_cap, int &g_out, float &T_out)
{
    const float Dm = D + 1e-30f;
    float ry;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(ry) : "f"(y));
    const int ybucket = min((int)(__float_as_uint(y) >> (23 - kBucketBits)) - (127 << kBucketBits), kStartBuckets - 1);
    // which types pass their entry test: all of them at once, the same work in every lane
    unsigned mask = 0;
    for (int t = 0; t < tb.n_types; ++t) {
        const float4 line = tb.chord[t * kStartBuckets + ybucket];               // offset, slope, p_lo
        GS_COUNT(kCountTypeTest, 1);
        if (__fmaf_rn(line.y, y, line.x) <= __fmaf_rn(-line.z, x, Dm)) mask |= 1u << t;
    }
    for (;;) {
        if (!mask) return -1;
        const int t = __ffs(mask) - 1;
        mask &= mask - 1;
        const float4 h = *reinterpret_cast<const float4 *>(&tb.headers[t]);       // p_lo, q_lo, d_lo, d_max
        const float Rg = __fmaf_rn(-h.x, x, Dm);
        const int4 geo = *(reinterpret_cast<const int4 *>(&tb.headers[t]) + 1);   // base, n_padded, inv_w, d0
        const int cell = GS_CHECKED(g_route_index_errors, (t * kStartBuckets + ybucket) * kStartSlots +
                         start_slot(Rg, h.y, ry, __int_as_float(geo.w), __int_as_float(geo.z)), tb.n_types * kStartBuckets * kStartSlots);
        const unsigned list = tb.bucket_list[t * kStartBuckets + ybucket];
        if (list == kNoList) return 0;
        const uint4 *w = reinterpret_cast<const uint4 *>(tb.pool) +
                         GS_CHECKED(g_route_index_errors, list + tb.start_list[cell], kPoolEntries / 2 - 3);
        const uint4 r0 = w[0], r1 = w[1];
        unsigned first = kNoRow;
        first = row_may_pass<false, false>(r1.z, r1.w, 0.f, x, y, Rg, 0.f) ? r1.z : first;
        first = row_may_pass<false, false>(r1.x, r1.y, 0.f, x, y, Rg, 0.f) ? r1.x : first;
        first = row_may_pass<false, false>(r0.z, r0.w, 0.f, x, y, Rg, 0.f) ? r0.z : first;
        first = row_may_pass<false, false>(r0.x, r0.y, 0.f, x, y, Rg, 0.f) ? r0.x : first;
        if (first == kNoRow) {
            const uint4 r2 = w[2], r3 = w[3];
            first = row_may_pass<false, false>(r3.z, r3.w, 0.f, x, y, Rg, 0.f) ? r3.z : first;
            first = row_may_pass<false, false>(r3.x, r3.y, 0.f, x, y, Rg, 0.f) ? r3.x : first;
            first = row_may_pass<false, false>(r2.z, r2.w, 0.f, x, y, Rg, 0.f) ? r2.z : first;
            first = row_may_pass<false, false>(r2.x, r2.y, 0.f, x, y, Rg, 0.f) ? r2.x : first;
            if (first == kNoRow) {
                if (r3.z == kPadQ) continue;         // the list ended inside the window: nothing of this type
                return 0;
            }
        }
        const int inst = (int)(first & kRowTagMask);
        GS_COUNT(kCountExact, 1);
        const Row row = tb.rows[GS_CHECKED(g_route_index_errors, row_pos(inst), GS_MAX_INSTANCES)];
        const float T = __fmaf_rn(row.d, y, __fmaf_rn(row.p, x, row.q));          // Eq. 2, H = 0
        if (!(T <= D && need <= (unsigned)row.kv && row.d < d_cap)) return 0;
        const float d_floor = __fmul_rn(row.d, 1.0f - 1.9073486328125e-6f);       // the bound every row with d >= the pick's carries
        while (mask) {
            const int tt = __ffs(mask) - 1;
            mask &= mask - 1;
            const float4 h2 = *reinterpret_cast<const float4 *>(&tb.headers[tt]);
            if (h2.w < row.d) break;                                              // nor can any type after it
            GS_COUNT(kCountTypeTest, 1);
            if (__fmaf_rn(fmaxf(h2.z, d_floor), y, h2.y) <= __fmaf_rn(-h2.x, x, Dm)) return 0;
        }
        g_out = inst;
        T_out = T;
        return 1;
    }
}

// A warp takes 32 candidates at a time, one per lane: it gathers the flagged request's columns
// through cand_idx (the next step's are on their way while this one is searched), turns it into
// the request that a token-ID migration would pose to the target (re-prefill prompt + generated
// tokens, decode what is left, within the time that is left) and runs capped_first_attempt.
// What that does not settle goes on one of the warp's two queues in shared memory, by position
// in cand_idx: candidates that still need the capped search in full, and candidates for which
// no feasible instance exists (half of them at the largest configuration), which need
// Algorithm 1's fallback among the faster instances.  Whenever 32 have gathered on a queue each
// lane takes one of them, so the long, divergent searches always run with all lanes busy.
constexpr int kRerouteThreads = GS_REROUTE_THREADS;
constexpr int kRerouteQueue = 64;           // per warp and queue: at most 31 left over + the 32 of a step

struct Candidate {
    float x, y, D, d_cap;
    unsigned need, rem;
    bool valid;
};
struct RawCandidate { int cur, gen, tot, xin; float slo, elapsed; };

__global__ void __launch_bounds__(kRerouteThreads, 1)
reroute_kernel(const int32_t *__restrict__ cand_idx, const int64_t *__restrict__ cand_count, int64_t cand_capacity,
               const int32_t *__restrict__ assigned, const int32_t *__restrict__ generated,
               const int32_t *__restrict__ pred_len, const float *__restrict__ elapsed,
               const float *__restrict__ slo, const int32_t *__restrict__ prompt_len, int64_t n_active,
               const TableSource src,
               int32_t *__restrict__ out_inst, float *__restrict__ out_est,
               float *__restrict__ out_slack, uint8_t *__restrict__ out_tier, unsigned *__restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int kWarps = kRerouteThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.wait;" ::: "memory");       // (the tables are the prologue's, the candidates the scan's)
    const TableImage im = carve_tables<false, true>(smem, src.n_types_alloc);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(shared_addr(im.bar)) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) start_table_copies<false, true>(im, src);
    unsigned *queue_full = reinterpret_cast<unsigned *>(im.end) + warp * (2 * kRerouteQueue);
    unsigned *queue_fall = queue_full + kRerouteQueue;

    int64_t n = *cand_count;
    if (n > cand_capacity) n = cand_capacity;
    unsigned bad = 0;
    // position in cand_idx -> index of the active request (-1 past the end), and its columns
    auto index_at = [&](int64_t j) { return j < n ? cand_idx[j] : -1; };
    auto gather = [&](int idx, bool valid) {
        int64_t i = idx;
        if (i < 0 || i >= n_active) { i = 0; if (valid) bad |= GS_DEV_BAD_INSTANCE; }
        RawCandidate r;
        r.cur = assigned[i]; r.gen = generated[i]; r.tot = pred_len[i]; r.xin = prompt_len[i];
        r.slo = slo[i]; r.elapsed = elapsed[i];
        return r;
    };
    const int64_t n_steps = (n + 31) >> 5;
    const int64_t stride = (int64_t)gridDim.x * kWarps;
    int64_t step = (int64_t)blockIdx.x * kWarps + warp;
    // two steps ahead: the indices; one step ahead: the columns
    int idx_next = step < n_steps ? index_at(step * 32 + lane) : -1;
    RawCandidate raw_next = gather(idx_next, step < n_steps && step * 32 + lane < n);
    idx_next = step + stride < n_steps ? index_at((step + stride) * 32 + lane) : -1;

    {
        const bool arrived = wait_barrier(im.bar, 0u);
        if (!__syncthreads_and(arrived)) {         // see route_kernel
            if (threadIdx.x == 0) atomicOr(status, (unsigned)GS_DEV_TIMEOUT);
            wait_barrier(im.bar, 0u);
            return;
        }
    }
    const int M = im.info[2];
    const unsigned kv_max = (unsigned)im.info[8];         // no instance has more free KV than this
    Tables tb;
    tb.headers = im.headers; tb.row_bounds = im.row_bounds; tb.group_bounds = im.group_bounds;
    tb.start_table = im.start_table; tb.rows = im.rows; tb.row_p = nullptr; tb.cand = im.cand;
    tb.pool = im.pool; tb.bucket_list = im.bucket_list; tb.start_list = im.start_list; tb.chord = im.chord;
    tb.n_types = im.info[1] != 0 ? 0 : im.info[3];       // unusable bounds: every candidate is scored against every instance
    int n_full = 0, n_fall = 0;                           // entries on the warp's queues (same in all lanes)

    // the request that a candidate poses
    auto pose = [&](const RawCandidate &r, bool valid) {
        Candidate c;
        int cur = r.cur, gen = r.gen, tot = r.tot, xin = r.xin;
        if (cur < 0) { cur = 0; if (valid) bad |= GS_DEV_BAD_INSTANCE; }
        if (cur >= M) { cur = M - 1; if (valid) bad |= GS_DEV_BAD_INSTANCE; }
        if ((gen | tot | xin) < 0) {
            gen = max(gen, 0); tot = max(tot, 0); xin = max(xin, 0);
            if (valid) bad |= GS_DEV_BAD_VALUE;
        }
        c.rem = (unsigned)max(tot - gen, 0);
        const unsigned xu = (unsigned)xin + (unsigned)gen;                    // < 2^32
        const unsigned long long need64 = (unsigned long long)xu + c.rem;
        c.need = need64 > 0xFFFFFFFFull ? 0xFFFFFFFFu : (unsigned)need64;     // kv < 2^31 anyway
        c.x = __uint2float_rn(xu); c.y = __uint2float_rn(c.rem);
        c.D = __fsub_rn(r.slo, r.elapsed);                                    // time left
        c.d_cap = tb.rows[row_pos(cur)].d;
        c.valid = valid;
        return c;
    };
    auto store = [&](int64_t j, int g, float T, unsigned tier, float D) {
        out_inst[j] = g;
        out_est[j] = T;
        out_slack[j] = tier ? __fsub_rn(D, T) : 0.f;
        if (out_tier) out_tier[j] = (uint8_t)tier;
    };
    // appends the lanes that vote `push` to a queue
    auto append = [&](unsigned *queue, int &count, bool push, unsigned entry) {
        const unsigned votes = __ballot_sync(0xFFFFFFFFu, push);
        if (push) queue[GS_CHECKED(g_route_index_errors, count + __popc(votes & ((1u << lane) - 1u)), kRerouteQueue)] = entry;
        count += __popc(votes);
    };
    // the fallback for (up to) the newest 32 candidates of its queue, one per lane
    auto drain_fall = [&]() {
        const int cnt = min(n_fall, 32);
        n_fall -= cnt;
        const bool active = lane < cnt;
        const int64_t j = active ? (int64_t)queue_fall[n_fall + lane] : 0;
        __syncwarp();                              // the slots may be written again
        const Candidate c = pose(gather(active ? cand_idx[j] : 0, active), active);
        int g = -1; float T = 0.f; unsigned tier = 0;
        bool settled = !active;
        if (active && c.rem > 0 && tb.n_types > 0) {
            const Pick r = fallback_pick<true, false>(tb, c.x, c.y, c.need, c.d_cap, c.need <= kv_max ? 0 : 1);
            g = r.g; T = r.T; tier = r.tier;                                // may settle on "no move"
            settled = true;
        }
        // what the tables cannot serve (nothing left to decode, unusable coefficients): the whole
        // warp scores every instance
        unsigned todo = __ballot_sync(0xFFFFFFFFu, !settled);
        while (todo) {
            const int from = __ffs(todo) - 1;
            todo &= todo - 1;
            const float xs = __shfl_sync(0xFFFFFFFFu, c.x, from), ys = __shfl_sync(0xFFFFFFFFu, c.y, from);
            const float Ds = __shfl_sync(0xFFFFFFFFu, c.D, from), caps = __shfl_sync(0xFFFFFFFFu, c.d_cap, from);
            const unsigned needs = __shfl_sync(0xFFFFFFFFu, c.need, from);
            int gg; float TT; unsigned tt;
            exhaustive_pick<true>(tb.rows, M, xs, ys, Ds, needs, caps, lane, gg, TT, tt);
            if (lane == from) { g = gg; T = TT; tier = tt; }
        }
        if (active) store(j, g, T, tier, c.D);
    };
    // the capped search in full for (up to) the newest 32 candidates of its queue
    auto drain_full = [&]() {
        const int cnt = min(n_full, 32);
        n_full -= cnt;
        const bool active = lane < cnt;
        const int64_t j = active ? (int64_t)queue_full[n_full + lane] : 0;
        __syncwarp();
        const Candidate c = pose(gather(active ? cand_idx[j] : 0, active), active);
        float T = 0.f;
        const float Ds = active ? c.D : -1.0f;     // (queued here: rem > 0, need <= kv_max)
        const int g = pick_instance<true, false>(tb, c.x, c.y, Ds, Ds + 1e-30f, c.need, c.d_cap, T);
        if (active && g >= 0) store(j, g, T, 1u, c.D);
        append(queue_fall, n_fall, active && g < 0, (unsigned)j);
        __syncwarp();
    };

    for (; step < n_steps; step += stride) {
        const int64_t j = step * 32 + lane;
        const RawCandidate raw = raw_next;
        const bool valid = j < n;
        // the columns of the next step, the indices of the one after it
        raw_next = gather(idx_next, step + stride < n_steps && (step + stride) * 32 + lane < n);
        idx_next = step + 2 * stride < n_steps ? index_at((step + 2 * stride) * 32 + lane) : -1;
        const Candidate c = pose(raw, valid);
        int g = -1; float T = 0.f;
        int outcome = -1;          // nothing left to decode, more KV than any instance has free, unusable tables: the fallback's queue
        if (valid && c.rem > 0 && c.need <= kv_max && tb.n_types > 0)
            outcome = capped_first_attempt(tb, c.x, c.y, c.D, c.need, c.d_cap, g, T);
        if (valid && outcome > 0) store(j, g, T, 1u, c.D);
        if (valid && outcome <= 0) GS_COUNT(kCountQueued, 1);
        if (valid && outcome < 0) GS_COUNT(kCountFallback, 1);
        append(queue_full, n_full, valid && outcome == 0, (unsigned)j);
        append(queue_fall, n_fall, valid && outcome < 0, (unsigned)j);
        __syncwarp();
        for (;;) {
            if (n_fall >= 32) drain_fall();
            else if (n_full >= 32) drain_full();
            else break;
        }
    }
    while (n_full > 0) {
        drain_full();
        if (n_fall >= 32) drain_fall();
    }
    while (n_fall > 0) drain_fall();
    if (bad) atomicOr(status, bad);
}

static size_t reroute_smem_bytes(int n_types) {       // the tables of n_types types and the warps' queues
    return route_smem_bytes(n_types, false, false) - (size_t)(route_threads(false, 1) / 32) * kQueueCap * sizeof(unsigned) +
           (size_t)(kRerouteThreads / 32) * 2 * kRerouteQueue * sizeof(unsigned) + (size_t)n_types * kStartBuckets * sizeof(float4);
}

cudaError_t launch_reroute(gs_ctx *ctx, const int32_t *cand_idx, const int64_t *cand_count, int64_t cand_capacity,
                           const int32_t *assigned, const int32_t *generated, const int32_t *pred_len,
                           const float *elapsed, const float *slo, const int32_t *prompt_len, int64_t n_active,
                           int n_instances, int n_types, int32_t *out_inst, float *out_est, float *out_slack, uint8_t *out_tier,
                           cudaStream_t st)
{
    if (cand_capacity == 0) return cudaSuccess;
    const size_t smem = reroute_smem_bytes(n_types);
    int64_t blocks = (cand_capacity + kRerouteThreads - 1) / kRerouteThreads;
    if (blocks > ctx->n_sm) blocks = ctx->n_sm;       // one CTA per SM: its tables fill most of the shared memory
    LaunchTimer timer(ctx, GS_K_REROUTE, st);
    const TableSource src = table_source(ctx, n_instances, n_types);
    reroute_kernel<<<(unsigned)blocks, kRerouteThreads, smem, st>>>(
        cand_idx, cand_count, cand_capacity, assigned, generated, pred_len, elapsed, slo, prompt_len, n_active,
        src, out_inst, out_est, out_slack, out_tier, ctx->s.status);
    return cudaGetLastError();
}

// Raises the dynamic shared-memory limit of the route kernels and looks up how many CTAs fit
// on an SM for each table size (called once per context).
template <int kReq>
static cudaError_t configure_route_kernels()
{
    cudaError_t e = cudaFuncSetAttribute(route_kernel<true, false, false, kReq>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)route_smem_bytes(GS_MAX_TYPES, true, false));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(route_kernel<false, false, false, kReq>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)route_smem_bytes(GS_MAX_TYPES, false, false));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(route_kernel<false, true, false, kReq>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)route_smem_bytes(GS_MAX_TYPES, false, false));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(route_kernel<false, false, true, kReq>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)route_smem_bytes(GS_MAX_TYPES, false, true));
}

cudaError_t configure_route(gs_ctx *ctx)
{
    cudaError_t e = configure_route_kernels<1>();
    if (e != cudaSuccess) return e;
    e = configure_route_kernels<4>();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(reroute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)reroute_smem_bytes(GS_MAX_TYPES));
    if (e != cudaSuccess) return e;
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------
// state advance between rounds of a stream
// ---------------------------------------------------------------------------------------

// One CTA, one thread per instance.  The smoothed queue delay is carried only when an ACCUMULATE
// round has left one since the last advance (the prologue of such a round raises pending[0]).
__global__ void __launch_bounds__(GS_MAX_INSTANCES)
advance_kernel(int32_t *__restrict__ queued, int32_t *__restrict__ batch,
               int32_t *__restrict__ free_kv, float *__restrict__ q_ema, int M,
               unsigned long long *__restrict__ deltas,
               const float *__restrict__ q_by_g, int *__restrict__ pending)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");       // (launched as a programmatic dependent of the routing round)
    const int g = threadIdx.x;
    const bool carry = pending[0] != 0;
    __syncthreads();
    if (g == 0) pending[0] = 0;
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
    if (carry) q_ema[g] = q_by_g[g];
}

cudaError_t launch_advance(gs_ctx *ctx, const gs_instances_mut &inst, cudaStream_t st)
{
    const int M = inst.n_instances;
    LaunchTimer timer(ctx, GS_K_ADVANCE, st);
    return launch_dependent(advance_kernel, dim3(1), dim3(GS_MAX_INSTANCES), 0, st, inst.queued_prefill_tokens,
                            inst.decode_batch, inst.free_kv_tokens, inst.q_ema_ms, M, ctx->s.deltas,
                            (const float *)ctx->s.q_by_g, ctx->s.table_info + 7);
}

// ---------------------------------------------------------------------------------------
// EMA step of the black-box coefficients (Sec. 3.3): c <- alpha * obs + (1 - alpha) * c
// ---------------------------------------------------------------------------------------

// One thread per instance and column; a column without observations (null) is left alone, and
// so is an entry whose observation is negative or NaN (status bit).
__global__ void ema_kernel(float alpha, int M, const float *__restrict__ obs_q, const float *__restrict__ obs_p,
                           const float *__restrict__ obs_d, float *__restrict__ q, float *__restrict__ p,
                           float *__restrict__ d, unsigned *__restrict__ status)
{
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= M) return;
    const float *obs[3] = {obs_q, obs_p, obs_d};
    float *col[3] = {q, p, d};
    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    bool bad = false;
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        if (!obs[c]) continue;
        const float o = obs[c][g];
        if (!(o >= 0.0f)) { bad = true; continue; }
        col[c][g] = __fmaf_rn(alpha, o, __fmul_rn(one_minus_alpha, col[c][g]));
    }
    if (bad) atomicOr(status, (unsigned)GS_DEV_BAD_VALUE);
}

cudaError_t launch_ema(gs_ctx *ctx, float alpha, int M, const float *obs_q, const float *obs_p, const float *obs_d,
                       float *q, float *p, float *d, cudaStream_t st)
{
    LaunchTimer timer(ctx, GS_K_EMA, st);
    ema_kernel<<<(M + 255) / 256, 256, 0, st>>>(alpha, M, obs_q, obs_p, obs_d, q, p, d, ctx->s.status);
    return cudaGetLastError();
}

}  // namespace gs
