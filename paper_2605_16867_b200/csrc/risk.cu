// gs_risk_scan: the SLO-violation risk test of Sec. 3.4 over all active requests and the
// ordered compaction of the flagged ones (migration candidates).
//
// Pass 1 (risk_flags_kernel) streams the five request columns once.  Each CTA first computes
// d_g = a_t + b_t * batch_g for every instance into shared memory; a warp then takes chunks of
// 1024 requests, gathers d_g of the assigned instance, and emits one flag word per 32 requests
// with a warp ballot.  It leaves the chunk's number of flags, and adds it to the total of the
// chunk's group of 64 chunks.
// Pass 2 (scatter_candidates_kernel) re-reads only the flag words.  Every warp owns a
// contiguous run of chunks; it sums the group totals and chunk counts that precede its run
// once, then keeps a running offset, and writes the ascending candidate list: a request's
// position is that offset plus popc of the lower flags.
// There is no device-side wait anywhere in the scan.
//
// The group totals are double-buffered by call parity: pass 2 of one call clears the buffer
// that pass 1 of the next call adds into.
#include <mutex>

#include "gs_internal.cuh"

namespace gs {

constexpr int kRiskThreads = 256;
constexpr int kRiskWarps = kRiskThreads / 32;
constexpr int kRiskUnroll = 4;          // independent 32-request groups in flight per warp
constexpr int kGroupShift = 6;          // 64 chunks per group

__global__ void __launch_bounds__(kRiskThreads)
risk_flags_kernel(const int32_t *__restrict__ assigned, const int32_t *__restrict__ generated,
                  const int32_t *__restrict__ pred_len, const float *__restrict__ elapsed,
                  const float *__restrict__ slo, int64_t n,
                  const int32_t *__restrict__ type_id, const int32_t *__restrict__ batch, int M,
                  const float *__restrict__ a_type, const float *__restrict__ b_type, int n_types,
                  uint32_t *__restrict__ flag_bits, unsigned *__restrict__ chunk_counts,
                  unsigned *__restrict__ group_totals, int64_t n_chunks, unsigned *__restrict__ status)
{
    __shared__ float sh_d[GS_MAX_INSTANCES];
    unsigned bad = 0;
    for (int g = threadIdx.x; g < M; g += blockDim.x) {
        int t = type_id[g];
        if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
        int B = batch[g];
        if (B < 0) { bad |= GS_DEV_BAD_VALUE; B = 0; }
        sh_d[g] = __fmaf_rn(b_type[t], __int2float_rn(B), a_type[t]);   // loaded per-token decode latency
    }
    if (blockIdx.x != 0) bad = 0;           // one CTA reports bad pool data
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t n_words = (n + 31) >> 5;

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
        if (lane == 0) {
            chunk_counts[chunk] = total;
            if (total) atomicAdd(group_totals + (chunk >> kGroupShift), total);
        }
    }
    if (bad) atomicOr(status, bad);
}

__global__ void __launch_bounds__(kRiskThreads)
scatter_candidates_kernel(const uint32_t *__restrict__ flag_bits, int64_t n_words,
                          const unsigned *__restrict__ chunk_counts,
                          const unsigned *__restrict__ group_totals, unsigned *__restrict__ next_group_totals,
                          int64_t n_clear, int64_t n_chunks, int64_t chunks_per_warp,
                          int32_t *__restrict__ cand_idx, int64_t cand_capacity,
                          int64_t *__restrict__ cand_count, unsigned *__restrict__ status)
{
    const int lane = threadIdx.x & 31;
    const int64_t gwarp = (int64_t)blockIdx.x * kRiskWarps + (threadIdx.x >> 5);
     // clear what an earlier call left in the other parity's group totals, for the next call
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n_clear;
         k += (int64_t)gridDim.x * blockDim.x)
        next_group_totals[k] = 0u;

    const int64_t c0 = gwarp * chunks_per_warp;
    if (c0 >= n_chunks) return;
    const int64_t c1 = min(c0 + chunks_per_warp, n_chunks);

    // flags before chunk c0: whole groups, then the chunks of c0's own group
    unsigned part = 0;
    const int64_t g0 = c0 >> kGroupShift;
    for (int64_t k = lane; k < g0; k += 32 * 8) {           // eight independent loads in flight
        unsigned v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = k + 32 * u < g0 ? group_totals[k + 32 * u] : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) part += v[u];
    }
    {
        const int64_t k = (g0 << kGroupShift) + lane;       // at most 64 chunks of c0's own group
        part += (k < c0 ? chunk_counts[k] : 0u) + (k + 32 < c0 ? chunk_counts[k + 32] : 0u);
    }
    int64_t base = (int64_t)__reduce_add_sync(0xFFFFFFFFu, part);

    __shared__ unsigned short sh_stage[kRiskWarps][kRiskChunk];   // a chunk's flagged positions, in order
    unsigned short *stage = sh_stage[threadIdx.x >> 5];
    for (int64_t chunk = c0; chunk < c1; ++chunk) {
        const int64_t wi = chunk * 32 + lane;
        uint32_t word = wi < n_words ? __ldcs(flag_bits + wi) : 0u;
        const unsigned c = __popc(word);
        unsigned incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += v;
        }
        const unsigned total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        // each lane lists the set bits of its own word behind those of the lower words ...
        unsigned at = incl - c;
        const unsigned lane_base = (unsigned)lane << 5;
        while (word) {
            stage[at++] = (unsigned short)(lane_base + (__ffs(word) - 1));
            word &= word - 1;
        }
        __syncwarp();
        // ... and the warp copies the list out with contiguous stores
        const int32_t idx0 = (int32_t)(chunk * kRiskChunk);             // n_active < 2^31
        const int64_t room = cand_capacity - base;
        const unsigned n_out = room <= 0 ? 0u : (room < (int64_t)total ? (unsigned)room : total);
        int32_t *out = cand_idx + base;
        for (unsigned i = lane; i < n_out; i += 32) out[i] = idx0 + (int32_t)stage[i];
        __syncwarp();
        base += total;
    }
    if (c1 == n_chunks && lane == 0) {      // the warp that owns the last chunk knows the total
        *cand_count = base;
        if (base > cand_capacity) atomicOr(status, (unsigned)GS_DEV_CAND_TRUNCATED);
    }
}

// Host side of one scan; `epoch` (host) selects the group-total buffer of this call and
// `dirty[b]` (host) is how many entries of buffer b may be non-zero.
struct ScanLaunch {
    unsigned *chunk_counts;
    unsigned *group_totals;     // two buffers of max_groups entries, both zero before the first call
    size_t max_groups;
    unsigned *epoch;
    int64_t *dirty;
};

static cudaError_t enqueue_scan(const ScanLaunch &sl, int n_sm, gs_ctx *timing_ctx,
                                const int32_t *assigned, const int32_t *generated, const int32_t *pred_len,
                                const float *elapsed, const float *slo, int64_t n,
                                const gs_instances &inst, const gs_types &types,
                                uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                                int64_t *cand_count, unsigned *status, cudaStream_t st)
{
    if (n == 0) return cudaMemsetAsync(cand_count, 0, sizeof(int64_t), st);
    const int64_t n_chunks = (n + kRiskChunk - 1) / kRiskChunk;
    const int64_t n_words = (n + 31) >> 5;
    const unsigned parity = (*sl.epoch)++ & 1u;
    unsigned *totals = sl.group_totals + parity * sl.max_groups;
    unsigned *next_totals = sl.group_totals + (parity ^ 1u) * sl.max_groups;
    int64_t blocks = (n_chunks + kRiskWarps - 1) / kRiskWarps;
    const int64_t cap = (int64_t)n_sm * 8;
    if (blocks > cap) blocks = cap;
    cudaError_t e;
    {
        LaunchTimer timer(timing_ctx, GS_K_RISK_FLAGS, st);
        risk_flags_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            assigned, generated, pred_len, elapsed, slo, n, inst.type_id, inst.decode_batch, inst.n_instances,
            types.tpot_a_ms, types.tpot_b_ms, types.n_types, flag_bits, sl.chunk_counts, totals, n_chunks, status);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    {
        const int64_t warps = blocks * kRiskWarps;
        const int64_t chunks_per_warp = (n_chunks + warps - 1) / warps;
        LaunchTimer timer(timing_ctx, GS_K_RISK_SCATTER, st);
        scatter_candidates_kernel<<<(unsigned)blocks, kRiskThreads, 0, st>>>(
            flag_bits, n_words, sl.chunk_counts, totals, next_totals, sl.dirty[parity ^ 1u], n_chunks,
            chunks_per_warp, cand_idx, cand_capacity, cand_count, status);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    sl.dirty[parity] = (n_chunks + (1 << kGroupShift) - 1) >> kGroupShift;
    sl.dirty[parity ^ 1u] = 0;
    return cudaSuccess;
}

cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n, const gs_instances &inst, const gs_types &types,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st)
{
    ScanLaunch sl{ctx->s.chunk_counts, ctx->s.group_totals, ctx->max_groups, &ctx->scan_epoch, ctx->scan_dirty};
    return enqueue_scan(sl, ctx->n_sm, ctx, assigned, generated, pred_len, elapsed, slo, n, inst, types,
                        flag_bits, cand_idx, cand_capacity, cand_count, ctx->s.status, st);
}

// ---------------------------------------------------------------------------------------
// gs_risk_scan_noalloc: the same scan for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------

constexpr size_t kNoAllocChunks = (GS_NOALLOC_MAX_ACTIVE + kRiskChunk - 1) / kRiskChunk;
constexpr size_t kNoAllocGroups = (kNoAllocChunks + (1u << kGroupShift) - 1) >> kGroupShift;

// All scratch of the no-allocation entry point.  It lives in the library image: every GPU
// that loads the library holds these 66 KB until the process exits.  Zero-initialised.  The
// chunk counts are rewritten by every call before they are read; of the two group-total
// buffers each call adds into one (cleared by the call before it) and clears the other.
struct NoAllocScratch {
    unsigned chunk_counts[kNoAllocChunks];
    unsigned group_totals[2 * kNoAllocGroups];
    unsigned status;
};
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

}  // namespace gs

namespace {

constexpr int kMaxDevices = 64;
// Per GPU: the device address of g_noalloc_scratch, resolved on that GPU's first call (in host
// code the symbol's name is only a handle, never an address a kernel may use), and the host
// side of the scan's bookkeeping.
struct NoAllocDevice {
    gs::NoAllocScratch *ptr = nullptr;
    cudaError_t err = cudaSuccess;
    bool ready = false;
    unsigned epoch = 0;
    int64_t dirty[2] = {0, 0};
};
NoAllocDevice g_noalloc[kMaxDevices];
std::mutex g_noalloc_mutex;     // guards g_noalloc

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
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice &nd = g_noalloc[dev];
    if (!nd.ready) {
        // first call on this GPU (it is the current device): resolve the scratch's address here
        void *p = nullptr;
        nd.err = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        nd.ptr = static_cast<NoAllocScratch *>(p);
        nd.ready = true;
    }
    if (nd.err != cudaSuccess || !nd.ptr) return GS_ERR_CUDA;
    NoAllocScratch *sc = nd.ptr;
    int n_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1) n_sm = 148;
    ScanLaunch sl{sc->chunk_counts, sc->group_totals, kNoAllocGroups, &nd.epoch, nd.dirty};
    const cudaError_t e = enqueue_scan(sl, n_sm, nullptr, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
                                       n_active, *inst, *types, out_flag_bits, out_cand_idx, cand_capacity,
                                       out_cand_count, out_status_bits ? out_status_bits : &sc->status,
                                       (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : GS_ERR_CUDA;
}
