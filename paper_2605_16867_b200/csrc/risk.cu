// gs_risk_scan kernels: the SLO-violation risk test of Sec. 3.4 over all active requests and
// the ordered compaction of the flagged ones (migration candidates).
//
// Pass 1 (risk_flags_kernel) streams the five request columns once, gathers d_g of the
// assigned instance from shared memory, and emits one flag bit per request with a warp
// ballot; every warp-chunk of 1024 requests also leaves its number of flags.
// Pass 2 (scan_counts_kernel) turns the per-chunk counts into exclusive offsets and the total.
// Pass 3 (scatter_candidates_kernel) re-reads only the flag words and writes the ascending
// candidate list; positions inside a word come from popc of the lower lanes' bits.
#include "gs_internal.cuh"

namespace gs {

constexpr int kRiskThreads = 256;
constexpr int kRiskWarps = kRiskThreads / 32;
constexpr int kRiskUnroll = 4;      // independent 32-request groups in flight per warp

__global__ void __launch_bounds__(kRiskThreads)
risk_flags_kernel(const int32_t *__restrict__ assigned, const int32_t *__restrict__ generated,
                  const int32_t *__restrict__ pred_len, const float *__restrict__ elapsed,
                  const float *__restrict__ slo, int64_t n, int M,
                  const float *__restrict__ d_by_g,
                  uint32_t *__restrict__ flag_bits, unsigned *__restrict__ chunk_counts,
                  int64_t n_chunks, unsigned *__restrict__ status)
{
    __shared__ float sh_d[GS_MAX_INSTANCES];
    for (int k = threadIdx.x; k < M; k += blockDim.x) sh_d[k] = d_by_g[k];
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t n_words = (n + 31) >> 5;
    unsigned bad = 0;

    for (int64_t chunk = (int64_t)blockIdx.x * kRiskWarps + warp; chunk < n_chunks;
         chunk += (int64_t)gridDim.x * kRiskWarps) {
        const int64_t first = chunk * kRiskChunk;
        uint32_t my_word = 0;               // lane l ends up holding word l of the chunk
#pragma unroll 1
        for (int w0 = 0; w0 < 32; w0 += kRiskUnroll) {
            int g[kRiskUnroll], gen[kRiskUnroll], tot[kRiskUnroll];
            float el[kRiskUnroll], dl[kRiskUnroll];
            bool valid[kRiskUnroll];
#pragma unroll
            for (int u = 0; u < kRiskUnroll; ++u) {
                const int64_t i = first + (int64_t)(w0 + u) * 32 + lane;
                valid[u] = i < n;
                g[u] = valid[u] ? __ldcs(assigned + i) : 0;
                gen[u] = valid[u] ? __ldcs(generated + i) : 0;
                tot[u] = valid[u] ? __ldcs(pred_len + i) : 0;
                el[u] = valid[u] ? __ldcs(elapsed + i) : 0.f;
                dl[u] = valid[u] ? __ldcs(slo + i) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kRiskUnroll; ++u) {
                int gi = g[u];
                if (gi < 0) { gi = 0; bad |= GS_DEV_BAD_INSTANCE; }
                if (gi >= M) { gi = M - 1; bad |= GS_DEV_BAD_INSTANCE; }
                int ge = gen[u], to = tot[u];
                if (ge < 0) { ge = 0; bad |= GS_DEV_BAD_VALUE; }
                if (to < 0) { to = 0; bad |= GS_DEV_BAD_VALUE; }
                const int rem = max(to - ge, 0);
                const float finish = __fmaf_rn(sh_d[gi], __int2float_rn(rem), el[u]);
                const bool flag = valid[u] && (finish > dl[u]);
                const uint32_t word = __ballot_sync(0xFFFFFFFFu, flag);
                if (lane == w0 + u) my_word = word;
            }
        }
        const int64_t wi = chunk * 32 + lane;
        if (wi < n_words) flag_bits[wi] = my_word;
        const unsigned total = __reduce_add_sync(0xFFFFFFFFu, (unsigned)__popc(my_word));
        if (lane == 0) chunk_counts[chunk] = total;
    }
    if (bad) atomicOr(status, bad);
}

// Exclusive scan of the per-chunk counts, in place, by one CTA; chunk_counts[n_chunks]
// receives the total, which is also written to *cand_count.
__global__ void __launch_bounds__(1024)
scan_counts_kernel(unsigned *__restrict__ chunk_counts, int64_t n_chunks,
                   int64_t *__restrict__ cand_count, int64_t cand_capacity,
                   unsigned *__restrict__ status)
{
    __shared__ unsigned sh_warp[32];
    __shared__ unsigned sh_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) sh_carry = 0;
    __syncthreads();
    const int64_t per_thread = (n_chunks + blockDim.x - 1) / blockDim.x;
    const int64_t lo = min((int64_t)threadIdx.x * per_thread, n_chunks);
    const int64_t hi = min(lo + per_thread, n_chunks);
    unsigned sum = 0;
    for (int64_t k = lo; k < hi; ++k) sum += chunk_counts[k];
    // CTA-wide exclusive scan of the per-thread sums
    unsigned incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) sh_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned w = sh_warp[lane];
        unsigned wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xFFFFFFFFu, wi, off);
            if (lane >= off) wi += v;
        }
        sh_warp[lane] = wi - w;           // exclusive warp offsets
        if (lane == 31) sh_carry = wi;    // grand total
    }
    __syncthreads();
    unsigned run = sh_warp[warp] + (incl - sum);
    for (int64_t k = lo; k < hi; ++k) {
        const unsigned c = chunk_counts[k];
        chunk_counts[k] = run;
        run += c;
    }
    if (threadIdx.x == 0) {
        const unsigned total = sh_carry;
        chunk_counts[n_chunks] = total;
        *cand_count = (int64_t)total;
        if ((int64_t)total > cand_capacity) atomicOr(status, (unsigned)GS_DEV_CAND_TRUNCATED);
    }
}

__global__ void __launch_bounds__(kRiskThreads)
scatter_candidates_kernel(const uint32_t *__restrict__ flag_bits, int64_t n_words,
                          const unsigned *__restrict__ chunk_offsets, int64_t n_chunks,
                          int32_t *__restrict__ cand_idx, int64_t cand_capacity)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int64_t chunk = (int64_t)blockIdx.x * kRiskWarps + warp; chunk < n_chunks;
         chunk += (int64_t)gridDim.x * kRiskWarps) {
        const int64_t wi = chunk * 32 + lane;
        const uint32_t word = wi < n_words ? flag_bits[wi] : 0u;
        const unsigned c = __popc(word);
        unsigned incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += v;
        }
        const unsigned word_off = incl - c;                 // flags in earlier words of the chunk
        const int64_t base = (int64_t)chunk_offsets[chunk];
        if (base >= cand_capacity) continue;                // nothing of this chunk fits
#pragma unroll 4
        for (int k = 0; k < 32; ++k) {
            const uint32_t wk = __shfl_sync(0xFFFFFFFFu, word, k);
            const unsigned ok = __shfl_sync(0xFFFFFFFFu, word_off, k);
            if ((wk >> lane) & 1u) {
                const int64_t pos = base + ok + __popc(wk & lt_mask);
                if (pos < cand_capacity)
                    cand_idx[pos] = (int32_t)(chunk * kRiskChunk + (int64_t)k * 32 + lane);
            }
        }
    }
}

cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n, int M,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st)
{
    const int64_t n_chunks = (n + kRiskChunk - 1) / kRiskChunk;
    const int64_t n_words = (n + 31) >> 5;
    cudaError_t err;
    if (n_chunks > 0) {
        int64_t blocks = (n_chunks + kRiskWarps - 1) / kRiskWarps;
        const int64_t cap = (int64_t)ctx->n_sm * 8;
        if (blocks > cap) blocks = cap;
        LaunchTimer timer(ctx, GS_K_RISK_FLAGS, st);
        risk_flags_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            assigned, generated, pred_len, elapsed, slo, n, M, ctx->s.d_by_g, flag_bits,
            ctx->s.chunk_counts, n_chunks, ctx->s.status);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
    }
    {
        LaunchTimer timer(ctx, GS_K_RISK_OFFSETS, st);
        scan_counts_kernel<<<1, 1024, 0, st>>>(ctx->s.chunk_counts, n_chunks, cand_count, cand_capacity,
                                               ctx->s.status);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
    }
    if (n_chunks > 0 && cand_capacity > 0 && cand_idx != nullptr) {
        int64_t blocks = (n_chunks + kRiskWarps - 1) / kRiskWarps;
        const int64_t cap = (int64_t)ctx->n_sm * 8;
        if (blocks > cap) blocks = cap;
        LaunchTimer timer(ctx, GS_K_RISK_SCATTER, st);
        scatter_candidates_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            flag_bits, n_words, ctx->s.chunk_counts, n_chunks, cand_idx, cand_capacity);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
    }
    return cudaSuccess;
}

}  // namespace gs
