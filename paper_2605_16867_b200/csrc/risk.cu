// gs_risk_scan: the SLO-violation risk test of Sec. 3.4 over all active requests and the
// ordered compaction of the flagged ones (migration candidates), in ONE pass over the data.
//
// A CTA takes tiles of 8192 requests (a ticket from a global counter, so a tile's predecessors
// are always already running).  Each of its 8 warps streams 1024 requests of the five columns,
// gathers d_g of the assigned instance from shared memory (computed per CTA from the raw
// instance state: d_g = a_t + b_t * batch_g), and forms one flag word per 32 requests with a
// warp ballot.  The tile's flag count is published and the tile's offset in the candidate list
// is obtained by a decoupled look-back over the preceding tiles' published counts (each tile
// first publishes its own count, then its inclusive prefix once known).  The candidate indices
// are written straight from the flag words still in registers: a request's position is the
// tile offset plus popc of the lower flags.
//
// The look-back is the only device-side wait.  It is bounded: after kSpinLimit polls the CTA
// sets GS_DEV_TIMEOUT, publishes a prefix anyway so that nobody else waits on it, and goes on
// (that call's candidate list is then invalid; every write stays in bounds).
//
// Tile status words carry the call's epoch, so the status array never needs clearing.
#include <mutex>

#include "gs_internal.cuh"

namespace gs {

constexpr int kRiskThreads = 256;
constexpr int kRiskWarps = kRiskThreads / 32;
constexpr int kRiskUnroll = 4;          // independent 32-request groups in flight per warp
constexpr int kRiskTile = kRiskWarps * kRiskChunk;   // requests per CTA tile
constexpr unsigned kSpinLimit = 4000000u;
constexpr unsigned kFlagAggregate = 1u, kFlagPrefix = 2u;

__device__ __forceinline__ unsigned long long pack_status(unsigned epoch, unsigned flag, unsigned value) {
    return ((unsigned long long)((epoch << 2) | flag) << 32) | value;
}

__device__ __forceinline__ unsigned long long load_status(const unsigned long long *p) {
    return *reinterpret_cast<const volatile unsigned long long *>(p);
}

__device__ __forceinline__ void store_status(unsigned long long *p, unsigned long long v) {
    *reinterpret_cast<volatile unsigned long long *>(p) = v;
}

__global__ void __launch_bounds__(kRiskThreads)
risk_scan_kernel(const int32_t *__restrict__ assigned, const int32_t *__restrict__ generated,
                 const int32_t *__restrict__ pred_len, const float *__restrict__ elapsed,
                 const float *__restrict__ slo, int64_t n,
                 const int32_t *__restrict__ type_id, const int32_t *__restrict__ batch, int M,
                 const float *__restrict__ a_type, const float *__restrict__ b_type, int n_types,
                 uint32_t *__restrict__ flag_bits, int32_t *__restrict__ cand_idx, int64_t cand_capacity,
                 int64_t *__restrict__ cand_count,
                 unsigned long long *__restrict__ tile_status, unsigned *__restrict__ ticket,
                 unsigned ticket_base, unsigned epoch, unsigned n_tiles, unsigned *__restrict__ status)
{
    __shared__ float sh_d[GS_MAX_INSTANCES];
    __shared__ unsigned sh_wcount[kRiskWarps];      // flags per warp, then exclusive offsets
    __shared__ unsigned sh_prefix, sh_tile;

    unsigned bad = 0;
    for (int g = threadIdx.x; g < M; g += blockDim.x) {
        int t = type_id[g];
        if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
        int B = batch[g];
        if (B < 0) { bad |= GS_DEV_BAD_VALUE; B = 0; }
        sh_d[g] = __fmaf_rn(b_type[t], __int2float_rn(B), a_type[t]);   // loaded per-token decode latency
    }
    if (blockIdx.x != 0) bad = 0;           // one CTA reports bad pool data
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t n_words = (n + 31) >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;

    for (;;) {
        __syncthreads();                    // sh_d ready / previous tile done with sh_tile, sh_prefix
        if (threadIdx.x == 0) sh_tile = atomicAdd(ticket, 1u) - ticket_base;
        __syncthreads();
        const unsigned tile = sh_tile;
        if (tile >= n_tiles) break;

        // ---- risk test: lane l ends up holding flag word l of the warp's 1024 requests ----
        const int64_t first = ((int64_t)tile * kRiskWarps + warp) * kRiskChunk;
        uint32_t my_word = 0;
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
        const int64_t wi = (first >> 5) + lane;
        if (wi < n_words) __stcs(flag_bits + wi, my_word);

        // flags in earlier words of this warp's chunk, and the chunk's total
        const unsigned c = __popc(my_word);
        unsigned incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += v;
        }
        const unsigned word_off = incl - c;
        if (lane == 31) sh_wcount[warp] = incl;
        __syncthreads();

        // ---- tile offset: publish the tile's count, look back over the tiles before it -------
        if (warp == 0) {
            const unsigned wc = lane < kRiskWarps ? sh_wcount[lane] : 0u;
            unsigned winc = wc;
#pragma unroll
            for (int off = 1; off < kRiskWarps; off <<= 1) {
                const unsigned v = __shfl_up_sync(0xFFFFFFFFu, winc, off);
                if (lane >= off) winc += v;
            }
            const unsigned agg = __shfl_sync(0xFFFFFFFFu, winc, kRiskWarps - 1);
            if (lane < kRiskWarps) sh_wcount[lane] = winc - wc;
            if (lane == 0 && tile > 0) store_status(tile_status + tile, pack_status(epoch, kFlagAggregate, agg));
            unsigned excl = 0;
            long long look = (long long)tile - 1;      // lane l inspects tile look - l
            unsigned spins = 0;
            bool timed_out = false;
            while (look >= 0) {
                const long long idx = look - lane;
                const unsigned long long w = idx >= 0 ? load_status(tile_status + idx)
                                                      : pack_status(epoch, kFlagPrefix, 0u);
                const unsigned hi = (unsigned)(w >> 32);
                const bool ready = (hi >> 2) == epoch;
                const unsigned ready_mask = __ballot_sync(0xFFFFFFFFu, ready);
                const unsigned prefix_mask = __ballot_sync(0xFFFFFFFFu, ready && (hi & 3u) == kFlagPrefix);
                // lanes up to and including the nearest tile that already knows its prefix
                const int stop = prefix_mask ? __ffs(prefix_mask) - 1 : 31;
                const unsigned need = stop == 31 ? 0xFFFFFFFFu : ((2u << stop) - 1u);
                if ((ready_mask & need) == need) {
                    excl += __reduce_add_sync(0xFFFFFFFFu, lane <= stop ? (unsigned)w : 0u);
                    if (prefix_mask) break;
                    look -= 32;
                    continue;
                }
                if (++spins > kSpinLimit) { timed_out = true; break; }
                __nanosleep(64);
            }
            if (lane == 0) {
                if (timed_out) atomicOr(status, (unsigned)GS_DEV_TIMEOUT);
                store_status(tile_status + tile, pack_status(epoch, kFlagPrefix, excl + agg));
                sh_prefix = excl;
                if (tile == n_tiles - 1) {
                    *cand_count = (int64_t)(excl + agg);
                    if ((int64_t)(excl + agg) > cand_capacity) atomicOr(status, (unsigned)GS_DEV_CAND_TRUNCATED);
                }
            }
        }
        __syncthreads();

        // ---- candidates: ascending indices, straight from the flag words in registers --------
        const int64_t base = (int64_t)sh_prefix + sh_wcount[warp];
        if (base < cand_capacity) {
#pragma unroll 4
            for (int k = 0; k < 32; ++k) {
                const uint32_t wk = __shfl_sync(0xFFFFFFFFu, my_word, k);
                const unsigned ok = __shfl_sync(0xFFFFFFFFu, word_off, k);
                if ((wk >> lane) & 1u) {
                    const int64_t pos = base + ok + __popc(wk & lt_mask);
                    if (pos < cand_capacity) cand_idx[pos] = (int32_t)(first + (int64_t)k * 32 + lane);
                }
            }
        }
    }
    if (bad) atomicOr(status, bad);
}

// Host side of one scan: `state` holds the ticket counter, the epoch and the ticket base.
struct ScanLaunch {
    unsigned long long *tile_status;
    unsigned *ticket;
    unsigned *epoch;        // host
    unsigned *ticket_base;  // host
    size_t max_tiles;
};

static cudaError_t enqueue_scan(const ScanLaunch &sl, int n_sm,
                                const int32_t *assigned, const int32_t *generated, const int32_t *pred_len,
                                const float *elapsed, const float *slo, int64_t n,
                                const gs_instances &inst, const gs_types &types,
                                uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                                int64_t *cand_count, unsigned *status, cudaStream_t st)
{
    if (n == 0) return cudaMemsetAsync(cand_count, 0, sizeof(int64_t), st);
    const unsigned n_tiles = (unsigned)((n + kRiskTile - 1) / kRiskTile);
    if (++*sl.epoch >= (1u << 30)) {
        // epochs are about to repeat: forget every old status word
        cudaError_t e = cudaMemsetAsync(sl.tile_status, 0, sl.max_tiles * sizeof(unsigned long long), st);
        if (e != cudaSuccess) return e;
        *sl.epoch = 1;
    }
    unsigned blocks = n_tiles;
    const unsigned cap = (unsigned)n_sm * 8u;
    if (blocks > cap) blocks = cap;
    risk_scan_kernel<<<blocks, kRiskThreads, 0, st>>>(
        assigned, generated, pred_len, elapsed, slo, n, inst.type_id, inst.decode_batch, inst.n_instances,
        types.tpot_a_ms, types.tpot_b_ms, types.n_types, flag_bits, cand_idx, cand_capacity, cand_count,
        sl.tile_status, sl.ticket, *sl.ticket_base, *sl.epoch, n_tiles, status);
    const cudaError_t e = cudaGetLastError();
    // every tile takes one ticket and every CTA one more (the one that tells it to stop)
    if (e == cudaSuccess) *sl.ticket_base += n_tiles + blocks;
    return e;
}

cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n, const gs_instances &inst, const gs_types &types,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st)
{
    ScanLaunch sl{ctx->s.tile_status, ctx->s.ticket, &ctx->scan_epoch, &ctx->ticket_base, ctx->max_tiles};
    LaunchTimer timer(ctx, GS_K_RISK_SCAN, st);
    return enqueue_scan(sl, ctx->n_sm, assigned, generated, pred_len, elapsed, slo, n, inst, types,
                        flag_bits, cand_idx, cand_capacity, cand_count, ctx->s.status, st);
}

// ---------------------------------------------------------------------------------------
// gs_risk_scan_noalloc: the same scan for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------

constexpr size_t kNoAllocTiles = (GS_NOALLOC_MAX_ACTIVE + kRiskTile - 1) / kRiskTile;

// All scratch of the no-allocation entry point.  It lives in the library image: every GPU
// that loads the library holds these ~16 KB until the process exits.  Zero-initialised; the
// status words and the ticket counter keep their values between calls, which the epoch and
// the ticket base account for.
struct NoAllocScratch {
    unsigned long long tile_status[kNoAllocTiles];
    unsigned ticket;
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
    unsigned epoch = 0, ticket_base = 0;
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
    ScanLaunch sl{sc->tile_status, &sc->ticket, &nd.epoch, &nd.ticket_base, kNoAllocTiles};
    const cudaError_t e = enqueue_scan(sl, n_sm, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
                                       n_active, *inst, *types, out_flag_bits, out_cand_idx, cand_capacity,
                                       out_cand_count, out_status_bits ? out_status_bits : &sc->status,
                                       (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : GS_ERR_CUDA;
}
