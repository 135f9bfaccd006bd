// gs_risk_scan kernels: the SLO-violation risk test of Sec. 3.4 over all active requests and
// the ordered compaction of the flagged ones (migration candidates).
//
// Pass 1 (risk_flags_kernel) streams the five request columns once, gathers d_g of the
// assigned instance from shared memory, and emits one flag bit per request with a warp
// ballot; every warp-chunk of 1024 requests also leaves its number of flags.
// Pass 2 (scan_counts_kernel) turns the per-chunk counts into exclusive offsets and the total.
// Pass 3 (scatter_candidates_kernel) re-reads only the flag words and writes the ascending
// candidate list; positions inside a word come from popc of the lower lanes' bits.
#include <mutex>

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

// ---------------------------------------------------------------------------------------
// gs_risk_scan_noalloc: the same scan for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------

constexpr int64_t kNoAllocChunks = (GS_NOALLOC_MAX_ACTIVE + kRiskChunk - 1) / kRiskChunk;

// All scratch of the no-allocation entry point.  It lives in the library image: every GPU
// that loads the library holds these ~72 KB until the process exits.
struct NoAllocScratch {
    float d_by_g[GS_MAX_INSTANCES];
    unsigned chunk_counts[kNoAllocChunks + 1];
    unsigned status;
};
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

// Per-instance decode latency d_g = a_t + b_t * batch_g for the scan (the only coefficient
// of Eq. 2 that the risk test of Sec. 3.4 uses), with the same clamping rules as elsewhere.
__global__ void __launch_bounds__(GS_MAX_INSTANCES)
decode_latency_kernel(const int32_t *__restrict__ type_id, const int32_t *__restrict__ batch, int M,
                      const float *__restrict__ a_type, const float *__restrict__ b_type, int n_types,
                      float *__restrict__ d_by_g, unsigned *__restrict__ status)
{
    const int g = threadIdx.x;
    if (g >= M) return;
    unsigned bad = 0;
    int t = type_id[g];
    if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
    int B = batch[g];
    if (B < 0) { bad |= GS_DEV_BAD_VALUE; B = 0; }
    d_by_g[g] = __fmaf_rn(b_type[t], __int2float_rn(B), a_type[t]);
    if (bad) atomicOr(status, bad);
}

}  // namespace gs

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_noalloc_scratch on each GPU, resolved on that GPU's first call.
// In host code the symbol's name is only a handle, never an address a kernel may use.
gs::NoAllocScratch *g_noalloc_ptr[kMaxDevices] = {};
cudaError_t g_noalloc_err[kMaxDevices] = {};
bool g_noalloc_ready[kMaxDevices] = {};
std::mutex g_noalloc_mutex;     // guards the three tables above

}  // namespace

extern "C" GS_API int gs_risk_scan_noalloc(
    const int32_t *assigned_inst, const int32_t *generated_tokens, const int32_t *pred_len,
    const float *elapsed_ms, const float *slo_ms, int64_t n_active,
    const gs_instances *inst, const gs_types *types,
    uint32_t *out_flag_bits, int32_t *out_cand_idx, int64_t cand_capacity,
    int64_t *out_cand_count, unsigned *out_status_bits, void *cuda_stream)
{
    using namespace gs;
    if (!inst || !types || !out_cand_count || n_active < 0 || cand_capacity < 0) return GS_ERR_INVALID_ARG;
    if (n_active > GS_NOALLOC_MAX_ACTIVE) return GS_ERR_TOO_LARGE;
    if (inst->n_instances < 1 || types->n_types < 1) return GS_ERR_INVALID_ARG;
    if (inst->n_instances > GS_MAX_INSTANCES || types->n_types > GS_MAX_TYPES) return GS_ERR_CAPACITY;
    if (!inst->type_id || !inst->decode_batch || !types->tpot_a_ms || !types->tpot_b_ms) return GS_ERR_INVALID_ARG;
    if (cand_capacity > 0 && !out_cand_idx) return GS_ERR_INVALID_ARG;
    if (n_active > 0 && (!assigned_inst || !generated_tokens || !pred_len || !elapsed_ms || !slo_ms || !out_flag_bits))
        return GS_ERR_INVALID_ARG;
    const void *aligned16[] = {assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, out_flag_bits, out_cand_idx};
    for (const void *p : aligned16) if (reinterpret_cast<uintptr_t>(p) & 15u) return GS_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(out_cand_count) & 7u) return GS_ERR_ALIGN;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GS_ERR_NO_DEVICE;
    NoAllocScratch *sc = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ready[dev]) {
            // first call on this GPU (it is the current device): resolve the scratch's address here
            void *p = nullptr;
            g_noalloc_err[dev] = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            g_noalloc_ptr[dev] = static_cast<NoAllocScratch *>(p);
            g_noalloc_ready[dev] = true;
        }
        if (g_noalloc_err[dev] != cudaSuccess || !g_noalloc_ptr[dev]) return GS_ERR_CUDA;
        sc = g_noalloc_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    unsigned *status = out_status_bits ? out_status_bits : &sc->status;
    const int M = inst->n_instances;

    decode_latency_kernel<<<1, GS_MAX_INSTANCES, 0, st>>>(inst->type_id, inst->decode_batch, M, types->tpot_a_ms,
                                                        types->tpot_b_ms, types->n_types, sc->d_by_g, status);
    if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
    const int64_t n_chunks = (n_active + kRiskChunk - 1) / kRiskChunk;
    const int64_t n_words = (n_active + 31) >> 5;
    int n_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1) n_sm = 148;
    int64_t blocks = (n_chunks + kRiskWarps - 1) / kRiskWarps;
    if (blocks > (int64_t)n_sm * 8) blocks = (int64_t)n_sm * 8;
    if (n_chunks > 0) {
        // every count in [0, n_chunks) is rewritten by this pass, so stale contents do not matter
        risk_flags_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, n_active, M, sc->d_by_g,
            out_flag_bits, sc->chunk_counts, n_chunks, status);
        if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
    }
    scan_counts_kernel<<<1, 1024, 0, st>>>(sc->chunk_counts, n_chunks, out_cand_count, cand_capacity, status);
    if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
    if (n_chunks > 0 && cand_capacity > 0) {
        scatter_candidates_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            out_flag_bits, n_words, sc->chunk_counts, n_chunks, out_cand_idx, cand_capacity);
        if (cudaGetLastError() != cudaSuccess) return GS_ERR_CUDA;
    }
    return GS_OK;
}
