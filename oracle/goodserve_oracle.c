/*
 * CPU oracle for the routing hot path of GoodServe.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path
 * computes, written from the paper; it exists so that the CUDA library can be checked
 * against it.  It shares no code with the CUDA path and nothing in the product may call it.
 *
 * What is stated here, and where the paper defines it:
 *   - latency model  T(r,g) = q_g + p_g * (L_in_r - H_{r,g}) + d_g * L_out_r     (Eq. 2); H = 0 in
 *     gso_route_*, sparse per-request hits in gso_route_prefix_*
 *   - queue-delay smoothing  q_g <- alpha * w_g + (1 - alpha) * q_g              (Algorithm 1, EMA step)
 *   - feasible set  C = { g : T(r,g) <= D_r }, restricted to instances whose memory
 *     can hold the request                                                      (Algorithm 1; Sec. 3.1 constraints)
 *   - just-enough choice  g* = argmax_{g in C} d_g                               (Algorithm 1; Sec. 3.4)
 *   - fallback  g* = argmin_g (T(r,g) - D_r)  when C is empty                    (Algorithm 1)
 *   - black-box coefficient smoothing  c <- alpha * obs + (1 - alpha) * c  for q, p, d and
 *     tables given directly                                                    (Sec. 3.3)
 *   - risk test: an ongoing request is flagged when its expected finish time under the
 *     latest estimates exceeds its SLO                                          (Sec. 3.4, second step)
 *
 * Readings taken where the paper is silent (each is listed in the design document):
 *   ties in argmax d_g and in argmin T go to the smallest instance index; d_g is the current
 *   loaded per-token decode latency a_t + b_t * batch_g; w_g (observed wait) is modelled as
 *   queued_prefill_tokens_g * p_g; the EMA steps once per routing round; the memory constraint
 *   is  L_in + L_out <= free_kv_tokens_g ; the fallback prefers instances with KV room
 *   (tier 2) and drops that preference only when no instance has room (tier 3); the risk
 *   test is decode-only:  elapsed + d_assigned * max(pred_len - generated, 0) > slo.
 *
 * Two arithmetic modes, same steps:
 *   *_f64 : every real operation in double from the float inputs (authority for values).
 *   *_f32 : single precision with a fixed operation order, each operation rounded once
 *           (fmaf / one multiply / one subtract) -- the precision in which the kernels take
 *           their decisions, so integer results can be compared bit for bit.
 *
 * Invalid data never aborts: negative counts and negative/NaN q_ema are clamped to 0, an
 * out-of-range type id is read as type 0, an out-of-range assigned instance is clamped into
 * [0, M-1]; a status bit records that it happened.
 *
 * Build:  gcc -O2 -fPIC -shared -ffp-contract=off -fno-fast-math goodserve_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>

enum { GSO_BAD_INSTANCE = 1, GSO_BAD_TYPE = 2, GSO_BAD_VALUE = 4 };

static int32_t clamp_count(int32_t v, unsigned *status) {
    if (v < 0) { *status |= GSO_BAD_VALUE; return 0; }
    return v;
}

/* ------------------------------------------------------------------------------------ */
/* per-instance coefficients of Eq. 2 for one routing round                              */
/* ------------------------------------------------------------------------------------ */

void gso_instance_table_f64(int32_t M, int32_t Tn,
                            const int32_t *type_id, const int32_t *queued_prefill_tokens,
                            const int32_t *decode_batch, const int32_t *free_kv_tokens,
                            const float *q_ema_ms,
                            const float *p_type, const float *a_type, const float *b_type,
                            float ema_alpha,
                            double *q, double *p, double *d, int64_t *kv, unsigned *status)
{
    double alpha = (double)ema_alpha;
    for (int32_t g = 0; g < M; ++g) {
        int32_t t = type_id[g];
        if (t < 0 || t >= Tn) { *status |= GSO_BAD_TYPE; t = 0; }
        double Qtok = (double)clamp_count(queued_prefill_tokens[g], status);
        double B = (double)clamp_count(decode_batch[g], status);
        double qe = (double)q_ema_ms[g];
        if (!(qe >= 0.0)) { *status |= GSO_BAD_VALUE; qe = 0.0; }
        p[g] = (double)p_type[t];
        d[g] = (double)a_type[t] + (double)b_type[t] * B;
        double w = Qtok * p[g];                            /* time to drain the queued prefill work */
        q[g] = alpha * w + (1.0 - alpha) * qe;             /* EMA step */
        kv[g] = (int64_t)clamp_count(free_kv_tokens[g], status);
    }
}

void gso_instance_table_f32(int32_t M, int32_t Tn,
                            const int32_t *type_id, const int32_t *queued_prefill_tokens,
                            const int32_t *decode_batch, const int32_t *free_kv_tokens,
                            const float *q_ema_ms,
                            const float *p_type, const float *a_type, const float *b_type,
                            float ema_alpha,
                            float *q, float *p, float *d, int64_t *kv, unsigned *status)
{
    float one_minus_alpha = 1.0f - ema_alpha;
    for (int32_t g = 0; g < M; ++g) {
        int32_t t = type_id[g];
        if (t < 0 || t >= Tn) { *status |= GSO_BAD_TYPE; t = 0; }
        float Qtok = (float)clamp_count(queued_prefill_tokens[g], status);
        float B = (float)clamp_count(decode_batch[g], status);
        float qe = q_ema_ms[g];
        if (!(qe >= 0.0f)) { *status |= GSO_BAD_VALUE; qe = 0.0f; }
        p[g] = p_type[t];
        d[g] = fmaf(b_type[t], B, a_type[t]);
        float w = Qtok * p[g];
        float keep = one_minus_alpha * qe;
        q[g] = fmaf(ema_alpha, w, keep);
        kv[g] = (int64_t)clamp_count(free_kv_tokens[g], status);
    }
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1 for every request of a round: the literal loop over requests x instances  */
/* ------------------------------------------------------------------------------------ */

void gso_route_f64(int64_t N, const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms,
                   int32_t M, const double *q, const double *p, const double *d, const int64_t *kv,
                   int32_t *instance_idx, double *est_e2e_ms, double *slack_ms, uint8_t *tier,
                   unsigned *status)
{
    for (int64_t r = 0; r < N; ++r) {
        double x = (double)clamp_count(prompt_len[r], status);
        double y = (double)clamp_count(pred_decode_len[r], status);
        double D = (double)slo_ms[r];
        int64_t need = (int64_t)x + (int64_t)y;

        int32_t best_c = -1, best_k = -1, best_a = -1;   /* feasible / KV-ok / all */
        double d_c = 0.0, T_c = 0.0, T_k = 0.0, T_a = 0.0;
        for (int32_t g = 0; g < M; ++g) {
            double T = q[g] + p[g] * x + d[g] * y;        /* Eq. 2, H = 0 */
            int kv_ok = need <= kv[g];
            if (kv_ok && T <= D) {                        /* g joins C */
                if (best_c < 0 || d[g] > d_c) { best_c = g; d_c = d[g]; T_c = T; }
            }
            if (kv_ok && (best_k < 0 || T < T_k)) { best_k = g; T_k = T; }
            if (best_a < 0 || T < T_a) { best_a = g; T_a = T; }
        }
        int32_t g_star; double T_star; uint8_t tr;
        if (best_c >= 0)      { g_star = best_c; T_star = T_c; tr = 1; }
        else if (best_k >= 0) { g_star = best_k; T_star = T_k; tr = 2; }
        else                  { g_star = best_a; T_star = T_a; tr = 3; }
        instance_idx[r] = g_star;
        est_e2e_ms[r] = T_star;
        slack_ms[r] = D - T_star;
        if (tier) tier[r] = tr;
    }
}

void gso_route_f32(int64_t N, const int32_t *prompt_len, const int32_t *pred_decode_len,
                   const float *slo_ms,
                   int32_t M, const float *q, const float *p, const float *d, const int64_t *kv,
                   int32_t *instance_idx, float *est_e2e_ms, float *slack_ms, uint8_t *tier,
                   unsigned *status)
{
    for (int64_t r = 0; r < N; ++r) {
        int32_t xi = clamp_count(prompt_len[r], status);
        int32_t yi = clamp_count(pred_decode_len[r], status);
        float x = (float)xi, y = (float)yi;
        float D = slo_ms[r];
        int64_t need = (int64_t)xi + (int64_t)yi;

        int32_t best_c = -1, best_k = -1, best_a = -1;
        float d_c = 0.0f, T_c = 0.0f, T_k = 0.0f, T_a = 0.0f;
        for (int32_t g = 0; g < M; ++g) {
            float T = fmaf(d[g], y, fmaf(p[g], x, q[g]));
            int kv_ok = need <= kv[g];
            if (kv_ok && T <= D) {
                if (best_c < 0 || d[g] > d_c) { best_c = g; d_c = d[g]; T_c = T; }
            }
            if (kv_ok && (best_k < 0 || T < T_k)) { best_k = g; T_k = T; }
            if (best_a < 0 || T < T_a) { best_a = g; T_a = T; }
        }
        int32_t g_star; float T_star; uint8_t tr;
        if (best_c >= 0)      { g_star = best_c; T_star = T_c; tr = 1; }
        else if (best_k >= 0) { g_star = best_k; T_star = T_k; tr = 2; }
        else                  { g_star = best_a; T_star = T_a; tr = 3; }
        instance_idx[r] = g_star;
        est_e2e_ms[r] = T_star;
        slack_ms[r] = D - T_star;
        if (tier) tier[r] = tr;
    }
}

/* ------------------------------------------------------------------------------------ */
/* SLO-violation risk test over the active requests (Sec. 3.4)                            */
/* ------------------------------------------------------------------------------------ */

static int32_t clamp_instance(int32_t g, int32_t M, unsigned *status) {
    if (g < 0) { *status |= GSO_BAD_INSTANCE; return 0; }
    if (g >= M) { *status |= GSO_BAD_INSTANCE; return M - 1; }
    return g;
}

void gso_risk_f64(int64_t A, const int32_t *assigned_inst, const int32_t *generated_tokens,
                  const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                  int32_t M, const double *d,
                  uint8_t *flag, double *finish_ms, unsigned *status)
{
    for (int64_t i = 0; i < A; ++i) {
        int32_t g = clamp_instance(assigned_inst[i], M, status);
        int64_t gen = clamp_count(generated_tokens[i], status);
        int64_t tot = clamp_count(pred_len[i], status);
        int64_t rem = tot - gen; if (rem < 0) rem = 0;
        double finish = (double)elapsed_ms[i] + d[g] * (double)rem;
        flag[i] = (uint8_t)(finish > (double)slo_ms[i]);
        if (finish_ms) finish_ms[i] = finish;
    }
}

void gso_risk_f32(int64_t A, const int32_t *assigned_inst, const int32_t *generated_tokens,
                  const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                  int32_t M, const float *d,
                  uint8_t *flag, float *finish_ms, unsigned *status)
{
    for (int64_t i = 0; i < A; ++i) {
        int32_t g = clamp_instance(assigned_inst[i], M, status);
        int64_t gen = clamp_count(generated_tokens[i], status);
        int64_t tot = clamp_count(pred_len[i], status);
        int64_t rem = tot - gen; if (rem < 0) rem = 0;
        float finish = fmaf(d[g], (float)rem, elapsed_ms[i]);
        flag[i] = (uint8_t)(finish > slo_ms[i]);
        if (finish_ms) finish_ms[i] = finish;
    }
}

/* Migration candidates: ascending indices of flagged requests, and the packed flag words
 * (bit i%32 of word i/32).  Returns the true count; writes at most `capacity` indices. */
int64_t gso_compact(int64_t A, const uint8_t *flag, uint32_t *flag_bits,
                    int32_t *cand_idx, int64_t capacity)
{
    int64_t count = 0;
    if (flag_bits) for (int64_t w = 0; w < (A + 31) / 32; ++w) flag_bits[w] = 0u;
    for (int64_t i = 0; i < A; ++i) {
        if (!flag[i]) continue;
        if (flag_bits) flag_bits[i >> 5] |= (uint32_t)1u << (i & 31);
        if (cand_idx && count < capacity) cand_idx[count] = (int32_t)i;
        ++count;
    }
    return count;
}

/* ------------------------------------------------------------------------------------ */
/* Between rounds of a stream: every routed request adds its prompt tokens to the chosen   */
/* instance's prefill queue, one slot to its decode batch, and takes L_in + L_out tokens   */
/* of KV room; the smoothed queue delay q_g of this round becomes the carried EMA state.   */
/* ------------------------------------------------------------------------------------ */

void gso_advance(int32_t M, int64_t N, const int32_t *instance_idx,
                 const int32_t *prompt_len, const int32_t *pred_decode_len,
                 int32_t *queued_prefill_tokens, int32_t *decode_batch, int32_t *free_kv_tokens,
                 float *q_ema_ms, const float *q_round)
{
    const int64_t I32_MAX = 2147483647LL;
    int64_t *dq = (int64_t *)calloc((size_t)M, sizeof(int64_t));   /* prompt tokens routed to g */
    int64_t *db = (int64_t *)calloc((size_t)M, sizeof(int64_t));   /* requests routed to g */
    int64_t *dk = (int64_t *)calloc((size_t)M, sizeof(int64_t));   /* KV tokens they will hold */
    for (int64_t r = 0; r < N; ++r) {
        int32_t g = instance_idx[r];
        if (g < 0 || g >= M) continue;
        int64_t x = prompt_len[r] < 0 ? 0 : prompt_len[r];
        int64_t y = pred_decode_len[r] < 0 ? 0 : pred_decode_len[r];
        dq[g] += x; db[g] += 1; dk[g] += x + y;
    }
    for (int32_t g = 0; g < M; ++g) {
        int64_t Q = queued_prefill_tokens[g] < 0 ? 0 : queued_prefill_tokens[g];
        int64_t B = decode_batch[g] < 0 ? 0 : decode_batch[g];
        int64_t K = free_kv_tokens[g] < 0 ? 0 : free_kv_tokens[g];
        Q += dq[g]; if (Q > I32_MAX) Q = I32_MAX;
        B += db[g]; if (B > I32_MAX) B = I32_MAX;
        K -= dk[g]; if (K < 0) K = 0;
        queued_prefill_tokens[g] = (int32_t)Q;
        decode_batch[g] = (int32_t)B;
        free_kv_tokens[g] = (int32_t)K;
        q_ema_ms[g] = q_round[g];
    }
    free(dq); free(db); free(dk);
}

/* ------------------------------------------------------------------------------------ */
/* Re-routing of flagged requests (Sec. 3.4): a request whose expected finish exceeds its */
/* SLO moves to a faster instance, chosen again by the just-enough rule; the migration    */
/* moves token IDs, so the target re-prefills the whole context (prompt + tokens          */
/* generated so far).                                                                      */
/*                                                                                        */
/* Reading: for candidate i on instance c                                                  */
/*   x' = prompt_len + generated,  y' = max(pred_len - generated, 0),  D' = slo - elapsed  */
/*   eligible instances  G_i = { g : d_g < d_c }        (strictly faster per output token) */
/*   Algorithm 1 over G_i with (x', y', D'):  tier 1 just-enough pick, tier 2 / 3 fallback */
/*   to the smallest T among eligible instances with / without KV room;                    */
/*   G_i empty (already on the fastest instance): no move, instance -1, tier 0.            */
/* ------------------------------------------------------------------------------------ */

#define GSO_REROUTE_BODY(REAL, LAT)                                                           \
    for (int64_t j = 0; j < n_cand; ++j) {                                                    \
        int64_t i = cand_idx[j];                                                              \
        int32_t c = clamp_instance(assigned_inst[i], M, status);                              \
        int64_t gen = clamp_count(generated_tokens[i], status);                               \
        int64_t tot = clamp_count(pred_len[i], status);                                       \
        int64_t xin = clamp_count(prompt_len[i], status);                                     \
        int64_t rem = tot - gen; if (rem < 0) rem = 0;                                        \
        int64_t xi = xin + gen;                                                               \
        REAL x = (REAL)xi, y = (REAL)rem;                                                     \
        REAL D = (REAL)slo_ms[i] - (REAL)elapsed_ms[i];                                       \
        int64_t need = xi + rem;                                                              \
        int32_t best_c = -1, best_k = -1, best_a = -1;                                        \
        REAL d_c = 0, T_c = 0, T_k = 0, T_a = 0;                                              \
        for (int32_t g = 0; g < M; ++g) {                                                     \
            if (!(d[g] < d[c])) continue;                  /* only strictly faster instances */ \
            REAL T = LAT;                                                                     \
            int kv_ok = need <= kv[g];                                                        \
            if (kv_ok && T <= D) {                                                            \
                if (best_c < 0 || d[g] > d_c) { best_c = g; d_c = d[g]; T_c = T; }            \
            }                                                                                 \
            if (kv_ok && (best_k < 0 || T < T_k)) { best_k = g; T_k = T; }                    \
            if (best_a < 0 || T < T_a) { best_a = g; T_a = T; }                               \
        }                                                                                     \
        int32_t g_star = -1; REAL T_star = 0; uint8_t tr = 0;                                 \
        if (best_c >= 0)      { g_star = best_c; T_star = T_c; tr = 1; }                      \
        else if (best_k >= 0) { g_star = best_k; T_star = T_k; tr = 2; }                      \
        else if (best_a >= 0) { g_star = best_a; T_star = T_a; tr = 3; }                      \
        new_instance[j] = g_star;                                                             \
        est_ms[j] = T_star;                                                                   \
        slack_ms[j] = tr ? D - T_star : 0;                                                    \
        if (tier) tier[j] = tr;                                                               \
    }

void gso_reroute_f64(int64_t n_cand, const int32_t *cand_idx,
                     const int32_t *assigned_inst, const int32_t *generated_tokens,
                     const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                     const int32_t *prompt_len,
                     int32_t M, const double *q, const double *p, const double *d, const int64_t *kv,
                     int32_t *new_instance, double *est_ms, double *slack_ms, uint8_t *tier,
                     unsigned *status)
{
    GSO_REROUTE_BODY(double, q[g] + p[g] * x + d[g] * y)
}

void gso_reroute_f32(int64_t n_cand, const int32_t *cand_idx,
                     const int32_t *assigned_inst, const int32_t *generated_tokens,
                     const int32_t *pred_len, const float *elapsed_ms, const float *slo_ms,
                     const int32_t *prompt_len,
                     int32_t M, const float *q, const float *p, const float *d, const int64_t *kv,
                     int32_t *new_instance, float *est_ms, float *slack_ms, uint8_t *tier,
                     unsigned *status)
{
    GSO_REROUTE_BODY(float, fmaf(d[g], y, fmaf(p[g], x, q[g])))
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1 with the prefix-cache term of Eq. 2                                        */
/*                                                                                        */
/* H_{r,g} arrives in sparse form: n_slots (instance, hit length) pairs per request,      */
/* slot-major arrays of n_slots * N entries (slot k of request r at k * N + r).           */
/* Reading:                                                                               */
/*   - a slot with a negative instance is empty; an instance >= M names nothing and is    */
/*     ignored (status bit);                                                              */
/*   - a hit length is clamped into [0, L_in] (a negative one, or one longer than the     */
/*     prompt, sets a status bit);                                                        */
/*   - an instance named by several slots keeps its longest hit;                          */
/*   - every other pair has H = 0;                                                        */
/*   - the memory constraint is unchanged: L_in + L_out <= free KV tokens.                */
/* Everything else is the loop of gso_route_* with T taken from the full Eq. 2.           */
/* ------------------------------------------------------------------------------------ */

/* ReusePrefix(r, g): the hit length of request r on instance g */
static int32_t reuse_prefix(int64_t r, int32_t g, int64_t N, int32_t n_slots,
                            const int32_t *prefix_inst, const int32_t *prefix_hit_len, int32_t L_in)
{
    int32_t H = 0;
    for (int32_t k = 0; k < n_slots; ++k) {
        if (prefix_inst[(int64_t)k * N + r] != g) continue;
        int32_t h = prefix_hit_len[(int64_t)k * N + r];
        if (h < 0) h = 0;
        if (h > L_in) h = L_in;
        if (h > H) H = h;
    }
    return H;
}

/* status bits for the slots of request r (kept apart from the search so that it stays plain) */
static void check_slots(int64_t r, int64_t N, int32_t n_slots, int32_t M, const int32_t *prefix_inst,
                        const int32_t *prefix_hit_len, int32_t L_in, unsigned *status)
{
    for (int32_t k = 0; k < n_slots; ++k) {
        int32_t g = prefix_inst[(int64_t)k * N + r];
        if (g < 0) continue;
        if (g >= M) { *status |= GSO_BAD_INSTANCE; continue; }
        int32_t h = prefix_hit_len[(int64_t)k * N + r];
        if (h < 0 || h > L_in) *status |= GSO_BAD_VALUE;
    }
}

#define GSO_ROUTE_PREFIX_BODY(REAL, LAT)                                                      \
    for (int64_t r = 0; r < N; ++r) {                                                         \
        int32_t xi = clamp_count(prompt_len[r], status);                                      \
        int32_t yi = clamp_count(pred_decode_len[r], status);                                 \
        REAL y = (REAL)yi;                                                                    \
        REAL D = (REAL)slo_ms[r];                                                             \
        int64_t need = (int64_t)xi + (int64_t)yi;                                             \
        check_slots(r, N, n_slots, M, prefix_inst, prefix_hit_len, xi, status);               \
        int32_t best_c = -1, best_k = -1, best_a = -1;                                        \
        REAL d_c = 0, T_c = 0, T_k = 0, T_a = 0;                                              \
        for (int32_t g = 0; g < M; ++g) {                                                     \
            int32_t H = reuse_prefix(r, g, N, n_slots, prefix_inst, prefix_hit_len, xi);      \
            REAL xh = (REAL)(xi - H);                      /* tokens left to prefill on g */  \
            REAL T = LAT;                                  /* Eq. 2 */                        \
            int kv_ok = need <= kv[g];                                                        \
            if (kv_ok && T <= D) {                                                            \
                if (best_c < 0 || d[g] > d_c) { best_c = g; d_c = d[g]; T_c = T; }            \
            }                                                                                 \
            if (kv_ok && (best_k < 0 || T < T_k)) { best_k = g; T_k = T; }                    \
            if (best_a < 0 || T < T_a) { best_a = g; T_a = T; }                               \
        }                                                                                     \
        int32_t g_star; REAL T_star; uint8_t tr;                                              \
        if (best_c >= 0)      { g_star = best_c; T_star = T_c; tr = 1; }                      \
        else if (best_k >= 0) { g_star = best_k; T_star = T_k; tr = 2; }                      \
        else                  { g_star = best_a; T_star = T_a; tr = 3; }                      \
        instance_idx[r] = g_star;                                                             \
        est_e2e_ms[r] = T_star;                                                               \
        slack_ms[r] = D - T_star;                                                             \
        if (tier) tier[r] = tr;                                                               \
    }

void gso_route_prefix_f64(int64_t N, const int32_t *prompt_len, const int32_t *pred_decode_len,
                          const float *slo_ms, int32_t n_slots, const int32_t *prefix_inst,
                          const int32_t *prefix_hit_len,
                          int32_t M, const double *q, const double *p, const double *d, const int64_t *kv,
                          int32_t *instance_idx, double *est_e2e_ms, double *slack_ms, uint8_t *tier,
                          unsigned *status)
{
    GSO_ROUTE_PREFIX_BODY(double, q[g] + p[g] * xh + d[g] * y)
}

void gso_route_prefix_f32(int64_t N, const int32_t *prompt_len, const int32_t *pred_decode_len,
                          const float *slo_ms, int32_t n_slots, const int32_t *prefix_inst,
                          const int32_t *prefix_hit_len,
                          int32_t M, const float *q, const float *p, const float *d, const int64_t *kv,
                          int32_t *instance_idx, float *est_e2e_ms, float *slack_ms, uint8_t *tier,
                          unsigned *status)
{
    GSO_ROUTE_PREFIX_BODY(float, fmaf(d[g], y, fmaf(p[g], xh, q[g])))
}

/* ------------------------------------------------------------------------------------ */
/* Black-box coefficients (Sec. 3.3): q_g, p_g, d_g come straight from recent             */
/* observations, each smoothed by an exponential moving average, with no reference to     */
/* GPU type, batch size or queue content.                                                 */
/*                                                                                        */
/* Reading:                                                                               */
/*   - one EMA step per coefficient and instance:  c <- alpha * obs + (1 - alpha) * c ;    */
/*   - an observation that is negative or NaN is no observation: c stays, status bit;     */
/*   - a table handed to the router directly is used as it is (no EMA step inside the      */
/*     round); a negative or NaN coefficient is read as 0 and a negative KV count as 0,    */
/*     with a status bit.                                                                 */
/* ------------------------------------------------------------------------------------ */

void gso_ema_update_f64(int32_t M, float alpha, const float *obs, const double *c_in, double *c_out,
                        unsigned *status)
{
    double a = (double)alpha;
    for (int32_t g = 0; g < M; ++g) {
        double o = (double)obs[g];
        if (!(o >= 0.0)) { *status |= GSO_BAD_VALUE; c_out[g] = c_in[g]; continue; }
        c_out[g] = a * o + (1.0 - a) * c_in[g];
    }
}

void gso_ema_update_f32(int32_t M, float alpha, const float *obs, const float *c_in, float *c_out,
                        unsigned *status)
{
    float one_minus_alpha = 1.0f - alpha;
    for (int32_t g = 0; g < M; ++g) {
        float o = obs[g];
        if (!(o >= 0.0f)) { *status |= GSO_BAD_VALUE; c_out[g] = c_in[g]; continue; }
        float keep = one_minus_alpha * c_in[g];
        c_out[g] = fmaf(alpha, o, keep);
    }
}

/* the table of a round from directly given coefficients (float inputs, as the C ABI takes them) */
void gso_direct_table_f64(int32_t M, const float *q_in, const float *p_in, const float *d_in,
                          const int32_t *free_kv_tokens,
                          double *q, double *p, double *d, int64_t *kv, unsigned *status)
{
    for (int32_t g = 0; g < M; ++g) {
        double qv = (double)q_in[g], pv = (double)p_in[g], dv = (double)d_in[g];
        if (!(qv >= 0.0)) { *status |= GSO_BAD_VALUE; qv = 0.0; }
        if (!(pv >= 0.0)) { *status |= GSO_BAD_VALUE; pv = 0.0; }
        if (!(dv >= 0.0)) { *status |= GSO_BAD_VALUE; dv = 0.0; }
        q[g] = qv; p[g] = pv; d[g] = dv;
        kv[g] = (int64_t)clamp_count(free_kv_tokens[g], status);
    }
}

void gso_direct_table_f32(int32_t M, const float *q_in, const float *p_in, const float *d_in,
                          const int32_t *free_kv_tokens,
                          float *q, float *p, float *d, int64_t *kv, unsigned *status)
{
    for (int32_t g = 0; g < M; ++g) {
        float qv = q_in[g], pv = p_in[g], dv = d_in[g];
        if (!(qv >= 0.0f)) { *status |= GSO_BAD_VALUE; qv = 0.0f; }
        if (!(pv >= 0.0f)) { *status |= GSO_BAD_VALUE; pv = 0.0f; }
        if (!(dv >= 0.0f)) { *status |= GSO_BAD_VALUE; dv = 0.0f; }
        q[g] = qv; p[g] = pv; d[g] = dv;
        kv[g] = (int64_t)clamp_count(free_kv_tokens[g], status);
    }
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1 one request at a time (its literal reading): the requests of a batch are    */
/* taken in arrival order, and each one sees the state left by the ones before it.         */
/*                                                                                        */
/* For request r:                                                                         */
/*   1. every instance takes its EMA step on the current state:                            */
/*        w_g = queued_g * p_g ,  q_g <- alpha * w_g + (1 - alpha) * q_g                   */
/*      and d_g = a_t + b_t * batch_g is read from the current batch;                      */
/*   2. T(r, g), the feasible set, the just-enough pick and the fallback as in gso_route;  */
/*   3. the chosen instance takes the request: queued += L_in, batch += 1,                 */
/*      free KV -= L_in + L_out (saturating like gso_advance), and the smoothed q of step 1 */
/*      becomes the carried state of every instance.                                       */
/* This is the same as rounds of one request each: gso_instance_table, gso_route,          */
/* gso_advance.  Single precision only: the carried state is single precision, and one     */
/* decision that differs changes every later one, so there is no double-precision          */
/* authority to compare values with beyond the first near-tie.                             */
/* The instance state arrays are updated in place.                                         */
/* ------------------------------------------------------------------------------------ */

void gso_route_sequential_f32(int64_t N, const int32_t *prompt_len, const int32_t *pred_decode_len,
                              const float *slo_ms, int32_t M, int32_t Tn, const int32_t *type_id,
                              int32_t *queued_prefill_tokens, int32_t *decode_batch, int32_t *free_kv_tokens,
                              float *q_ema_ms,
                              const float *p_type, const float *a_type, const float *b_type, float ema_alpha,
                              int32_t *instance_idx, float *est_e2e_ms, float *slack_ms, uint8_t *tier,
                              unsigned *status)
{
    const int64_t I32_MAX = 2147483647LL;
    float one_minus_alpha = 1.0f - ema_alpha;
    for (int64_t r = 0; r < N; ++r) {
        int32_t xi = clamp_count(prompt_len[r], status);
        int32_t yi = clamp_count(pred_decode_len[r], status);
        float x = (float)xi, y = (float)yi;
        float D = slo_ms[r];
        int64_t need = (int64_t)xi + (int64_t)yi;

        int32_t best_c = -1, best_k = -1, best_a = -1;
        float d_c = 0.0f, T_c = 0.0f, T_k = 0.0f, T_a = 0.0f;
        for (int32_t g = 0; g < M; ++g) {
            /* step 1: coefficients of g from the current state */
            int32_t t = type_id[g];
            if (t < 0 || t >= Tn) { *status |= GSO_BAD_TYPE; t = 0; }
            float Qtok = (float)clamp_count(queued_prefill_tokens[g], status);
            float B = (float)clamp_count(decode_batch[g], status);
            float qe = q_ema_ms[g];
            if (!(qe >= 0.0f)) { *status |= GSO_BAD_VALUE; qe = 0.0f; }
            float p = p_type[t];
            float d = fmaf(b_type[t], B, a_type[t]);
            float w = Qtok * p;
            float keep = one_minus_alpha * qe;
            float q = fmaf(ema_alpha, w, keep);
            q_ema_ms[g] = q;                               /* carried to the next request */
            int64_t kv = (int64_t)clamp_count(free_kv_tokens[g], status);
            /* step 2 */
            float T = fmaf(d, y, fmaf(p, x, q));
            int kv_ok = need <= kv;
            if (kv_ok && T <= D) {
                if (best_c < 0 || d > d_c) { best_c = g; d_c = d; T_c = T; }
            }
            if (kv_ok && (best_k < 0 || T < T_k)) { best_k = g; T_k = T; }
            if (best_a < 0 || T < T_a) { best_a = g; T_a = T; }
        }
        int32_t g_star; float T_star; uint8_t tr;
        if (best_c >= 0)      { g_star = best_c; T_star = T_c; tr = 1; }
        else if (best_k >= 0) { g_star = best_k; T_star = T_k; tr = 2; }
        else                  { g_star = best_a; T_star = T_a; tr = 3; }
        instance_idx[r] = g_star;
        est_e2e_ms[r] = T_star;
        slack_ms[r] = D - T_star;
        if (tier) tier[r] = tr;
        /* step 3: every instance's counts leave this step clamped as gso_advance leaves them */
        for (int32_t g = 0; g < M; ++g) {
            int64_t Q = queued_prefill_tokens[g] < 0 ? 0 : queued_prefill_tokens[g];
            int64_t Bc = decode_batch[g] < 0 ? 0 : decode_batch[g];
            int64_t K = free_kv_tokens[g] < 0 ? 0 : free_kv_tokens[g];
            if (g == g_star) {
                Q += xi; if (Q > I32_MAX) Q = I32_MAX;
                Bc += 1; if (Bc > I32_MAX) Bc = I32_MAX;
                K -= need; if (K < 0) K = 0;
            }
            queued_prefill_tokens[g] = (int32_t)Q;
            decode_batch[g] = (int32_t)Bc;
            free_kv_tokens[g] = (int32_t)K;
        }
    }
}
