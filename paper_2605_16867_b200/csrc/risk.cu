// gs_risk_scan: the SLO-violation risk test of Sec. 3.4 over all active requests and the
// ordered compaction of the flagged ones (migration candidates).
//
// The requests are cut into steps of 128 (four flag words) and the steps dealt out evenly: CTA b
// of G owns the contiguous run of steps [b S / G, (b + 1) S / G).  Both passes use the same G.
//
// Pass 1 (risk_flags_kernel) streams the five request columns once.  Each CTA first computes
// d_g = a_t + b_t * batch_g for every instance into shared memory; its warps then take the
// CTA's steps in turn, four consecutive requests per lane (128-bit column loads), gather d_g of
// the assigned instance and assemble the flag words (a nibble per lane, OR-reduced over each
// eight lanes).  The CTA leaves one number: how many requests it flagged.
// Pass 2 (scatter_candidates_kernel) re-reads only the flag words.  CTA b sums the counts of
// the CTAs before it, then walks its own run 8 x 1024 requests at a time: a warp counts the
// flags of its 1024 requests, the counts of the eight warps are exchanged through shared memory,
// and each warp writes its part of the ascending candidate list word by word: a flagged
// request's position is the running offset plus the number of flagged requests below it in its
// word, so the lanes that hold a flag store to consecutive entries.
//
// Nothing is accumulated with atomics and nothing survives a call: every word of scratch that
// pass 2 reads was stored by pass 1 of the same call.  There is no device-side wait.  Pass 2 is
// launched as a programmatic dependent of pass 1 (its launch overlaps pass 1's tail; it waits
// for pass 1's memory before it reads anything).
#include <mutex>

#include "gs_internal.cuh"

namespace gs {

constexpr int kRiskThreads = 256;
constexpr int kRiskWarps = kRiskThreads / 32;
#ifndef GS_RISK_UNROLL
#define GS_RISK_UNROLL 1
#endif
#ifndef GS_RISK_MIN_CTAS
#define GS_RISK_MIN_CTAS 4
#endif
#ifndef GS_RISK_PDL
#define GS_RISK_PDL 2       // pass 2 as a programmatic dependent of pass 1: 0 no, 1 set up from pass 1's start, 2 from its end
#endif
constexpr int kRiskUnroll = GS_RISK_UNROLL;   // steps of 128 requests a warp works on at a time (as many again are on their way)
constexpr int kRiskMinCtas = GS_RISK_MIN_CTAS;
constexpr int kStepShift = 7;                 // 128 requests per step

// First step of CTA b's run when S steps are dealt to G CTAs.
__host__ __device__ __forceinline__ int64_t first_step_of(int64_t b, int64_t S, int64_t G) { return b * S / G; }

// Risk test of one request (Sec. 3.4): expected finish = elapsed + d_assigned * tokens left;
// flagged when it exceeds the SLO.  Out-of-range data is clamped and reported in `bad`.
__device__ __forceinline__ bool risk_flag(const float *sh_d, int M, int g, int gen, int tot, float el, float dl,
                                          unsigned &bad)
{
    if ((unsigned)g >= (unsigned)M) { g = g < 0 ? 0 : M - 1; bad |= GS_DEV_BAD_INSTANCE; }
    if ((gen | tot) < 0) { gen = max(gen, 0); tot = max(tot, 0); bad |= GS_DEV_BAD_VALUE; }
    const int rem = max(tot - gen, 0);
    return __fmaf_rn(sh_d[g], __int2float_rn(rem), el) > dl;
}

// The five columns of one step (128 requests), four consecutive requests per lane.
struct StepData {
    int4 g, gen, tot;
    float4 el, dl;
};

__device__ __forceinline__ void load_step(StepData &d, const int32_t *__restrict__ assigned,
                                          const int32_t *__restrict__ generated, const int32_t *__restrict__ pred_len,
                                          const float *__restrict__ elapsed, const float *__restrict__ slo,
                                          int64_t step, int lane)
{
    const int64_t i = (step << kStepShift) + lane * 4;
    d.g = __ldcs(reinterpret_cast<const int4 *>(assigned + i));
    d.gen = __ldcs(reinterpret_cast<const int4 *>(generated + i));
    d.tot = __ldcs(reinterpret_cast<const int4 *>(pred_len + i));
    d.el = __ldcs(reinterpret_cast<const float4 *>(elapsed + i));
    d.dl = __ldcs(reinterpret_cast<const float4 *>(slo + i));
}

__global__ void __launch_bounds__(kRiskThreads, kRiskMinCtas)
risk_flags_kernel(const int32_t *__restrict__ assigned, const int32_t *__restrict__ generated,
                  const int32_t *__restrict__ pred_len, const float *__restrict__ elapsed,
                  const float *__restrict__ slo, int64_t n,
                  const int32_t *__restrict__ type_id, const int32_t *__restrict__ batch, int M,
                  const float *__restrict__ a_type, const float *__restrict__ b_type, int n_types,
                  uint32_t *__restrict__ flag_bits, unsigned *__restrict__ cta_counts,
                  int64_t n_steps, unsigned *__restrict__ status)
{
#if GS_RISK_PDL == 1
    // the dependent launch (pass 2) may be set up from now on; it still waits for this grid's end
    asm volatile("griddepcontrol.launch_dependents;");
#endif
    // (launched as a programmatic dependent: the kernel before it may be the one that writes the
    // pool's state, or the previous scan still reading the scratch this one overwrites)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ float sh_d[GS_MAX_INSTANCES];
    __shared__ float sh_a[GS_MAX_TYPES], sh_b[GS_MAX_TYPES];
    __shared__ unsigned sh_count;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t s_begin = first_step_of(blockIdx.x, n_steps, gridDim.x);
    const int64_t s_end = first_step_of((int64_t)blockIdx.x + 1, n_steps, gridDim.x);
    // steps that lie wholly inside the batch and inside this CTA's run take the 128-bit path
    const int64_t s_fast = min(s_end, n >> kStepShift);

    // the warp's first steps are on their way while the CTA works out d_g
    StepData cur[kRiskUnroll];
    int64_t s0 = s_begin + warp;             // warp w takes the steps w, w + 8, .. of the run
#pragma unroll
    for (int u = 0; u < kRiskUnroll; ++u)
        if (s0 + u * kRiskWarps < s_fast) load_step(cur[u], assigned, generated, pred_len, elapsed, slo, s0 + u * kRiskWarps, lane);

    // d_g for every instance: all global loads are issued together (one round trip, not one per
    // dependent step), the type constants go through shared memory
    unsigned bad = 0;
    constexpr int kPerThread = GS_MAX_INSTANCES / kRiskThreads;
    int r_type[kPerThread], r_batch[kPerThread];
#pragma unroll
    for (int k = 0; k < kPerThread; ++k) {
        const int g = threadIdx.x + k * kRiskThreads;
        r_type[k] = g < M ? type_id[g] : 0;
        r_batch[k] = g < M ? batch[g] : 0;
    }
    if (threadIdx.x < n_types) { sh_a[threadIdx.x] = a_type[threadIdx.x]; sh_b[threadIdx.x] = b_type[threadIdx.x]; }
    if (threadIdx.x == 0) sh_count = 0u;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kPerThread; ++k) {
        const int g = threadIdx.x + k * kRiskThreads;
        if (g >= M) break;
        int t = r_type[k], B = r_batch[k];
        if (t < 0 || t >= n_types) { bad |= GS_DEV_BAD_TYPE; t = 0; }
        if (B < 0) { bad |= GS_DEV_BAD_VALUE; B = 0; }
        sh_d[g] = __fmaf_rn(sh_b[t], __int2float_rn(B), sh_a[t]);       // loaded per-token decode latency
    }
    if (blockIdx.x != 0) bad = 0;           // one CTA reports bad pool data
    __syncthreads();

    const unsigned oct_mask = 0xFFu << (lane & 24);     // the eight lanes that share a flag word
    const int nib_shift = (lane & 7) << 2;
    unsigned flagged = 0;                               // flags this lane has seen (its own nibbles)

#pragma unroll 1
    for (; s0 < s_end; s0 += kRiskWarps * kRiskUnroll) {
        const int64_t s_next = s0 + kRiskWarps * kRiskUnroll;
        StepData nxt[kRiskUnroll];
#pragma unroll
        for (int u = 0; u < kRiskUnroll; ++u)            // the next steps are requested before these are worked on
            if (s_next + u * kRiskWarps < s_fast) load_step(nxt[u], assigned, generated, pred_len, elapsed, slo, s_next + u * kRiskWarps, lane);
#pragma unroll
        for (int u = 0; u < kRiskUnroll; ++u) {
            const int64_t s = s0 + u * kRiskWarps;
            if (s >= s_end) break;
            unsigned nib = 0;
            if (s < s_fast) {
                const StepData &d = cur[u];
                nib = risk_flag(sh_d, M, d.g.x, d.gen.x, d.tot.x, d.el.x, d.dl.x, bad) ? 1u : 0u;
                nib |= risk_flag(sh_d, M, d.g.y, d.gen.y, d.tot.y, d.el.y, d.dl.y, bad) ? 2u : 0u;
                nib |= risk_flag(sh_d, M, d.g.z, d.gen.z, d.tot.z, d.el.z, d.dl.z, bad) ? 4u : 0u;
                nib |= risk_flag(sh_d, M, d.g.w, d.gen.w, d.tot.w, d.el.w, d.dl.w, bad) ? 8u : 0u;
            } else {
                // the ragged last step of the batch: request by request
                const int64_t i0 = (s << kStepShift) + lane * 4;
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < n && risk_flag(sh_d, M, assigned[i0 + j], generated[i0 + j], pred_len[i0 + j],
                                                elapsed[i0 + j], slo[i0 + j], bad))
                        nib |= 1u << j;
            }
            flagged += __popc(nib);
            // lanes 8w .. 8w+7 hold the eight nibbles of word w of this step
            const uint32_t word = __reduce_or_sync(oct_mask, nib << nib_shift);
            const int64_t wi = (s << 2) + (lane >> 3);
            if ((lane & 7) == 0 && wi < ((n + 31) >> 5)) flag_bits[wi] = word;
        }
#pragma unroll
        for (int u = 0; u < kRiskUnroll; ++u) cur[u] = nxt[u];
    }
#if GS_RISK_PDL == 2
    // pass 2 may be set up from now on (it still waits for this whole grid before it reads): at
    // 16 M requests that is worth nothing, at 2 M and below it hides pass 2's launch (2 us)
    asm volatile("griddepcontrol.launch_dependents;");
#endif
    flagged = __reduce_add_sync(0xFFFFFFFFu, flagged);
    if (lane == 0 && flagged) atomicAdd(&sh_count, flagged);
    __syncthreads();
    if (threadIdx.x == 0) cta_counts[blockIdx.x] = sh_count;
    if (bad) atomicOr(status, bad);
}

#ifndef GS_SCATTER_THREADS
#define GS_SCATTER_THREADS 512
#endif
constexpr int kScatterThreads = GS_SCATTER_THREADS;      // pass 2 runs more warps per CTA than pass 1: it is bound by latency
constexpr int kScatterWarps = kScatterThreads / 32;
constexpr int kScatterBlocks = 32 / kScatterWarps;        // blocks of 32 flag words (1024 requests) per warp and round: 32 blocks a round

__global__ void __launch_bounds__(kScatterThreads, 2048 / kScatterThreads)
scatter_candidates_kernel(const uint32_t *__restrict__ flag_bits, int64_t n_words,
                          const unsigned *__restrict__ cta_counts, int64_t n_steps,
                          int32_t *__restrict__ cand_idx, int64_t cand_capacity,
                          int64_t *__restrict__ cand_count, unsigned *__restrict__ status,
                          const int64_t *__restrict__ prev_count, int32_t index_base)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    __shared__ unsigned sh_part[kScatterWarps];
    __shared__ unsigned sh_cnt[2][kScatterWarps * kScatterBlocks];
    __shared__ uint2 sh_words[kScatterWarps][32];
    // the CTA's run of flag words; a round covers 32 blocks of 32 words, warp w the blocks
    // w, w + kScatterWarps, .. of the round
    const int64_t w_begin = first_step_of(blockIdx.x, n_steps, gridDim.x) << 2;
    const int64_t w_end = min(first_step_of((int64_t)blockIdx.x + 1, n_steps, gridDim.x) << 2, n_words);
    // everything read below is written by pass 1: wait until that grid is done and visible
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // flags before this CTA's run: the counts of the CTAs before it (fewer than 2^31 in all)
    unsigned part = 0;
    for (int k = threadIdx.x; k < (int)blockIdx.x; k += kScatterThreads) part += __ldcg(cta_counts + k);
    part = __reduce_add_sync(0xFFFFFFFFu, part);
    if (lane == 0) sh_part[warp] = part;
    // (the kernel after this one in the stream may be set up from now on)
    asm volatile("griddepcontrol.launch_dependents;");

    const unsigned lane_bit = 1u << lane, below = lane_bit - 1u;
    // (a scan that continues an earlier one -- the host entry point scans in pieces -- starts
    // its list where that one ended and numbers its requests from index_base)
    int64_t base = prev_count ? *prev_count : 0;
    int buf = 0;
    for (int64_t w0 = w_begin; w0 < w_end; w0 += kScatterWarps * kScatterBlocks * 32, buf ^= 1) {
        uint32_t word[kScatterBlocks];
#pragma unroll
        for (int k = 0; k < kScatterBlocks; ++k) {
            const int64_t wi = w0 + (k * kScatterWarps + warp) * 32 + lane;
            word[k] = wi < w_end ? __ldcs(flag_bits + wi) : 0u;
        }
#pragma unroll
        for (int k = 0; k < kScatterBlocks; ++k) {
            const unsigned total = __reduce_add_sync(0xFFFFFFFFu, (unsigned)__popc(word[k]));
            if (lane == 0) sh_cnt[buf][k * kScatterWarps + warp] = total;
        }
        __syncthreads();                    // (the other buffer is free again after the next barrier)
        if (w0 == w_begin) {
#pragma unroll
            for (int w = 0; w < kScatterWarps; ++w) base += sh_part[w];
        }
        // lane b holds the count of block b of the round: flags before each block, and in all
        const unsigned c = sh_cnt[buf][lane];
        unsigned incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += v;
        }
        const unsigned all = __shfl_sync(0xFFFFFFFFu, incl, 31);
#pragma unroll
        for (int k = 0; k < kScatterBlocks; ++k) {
            const int blk = k * kScatterWarps + warp;
            const unsigned total = __shfl_sync(0xFFFFFFFFu, c, blk);
            const unsigned before = __shfl_sync(0xFFFFFFFFu, incl - c, blk);
            if (total == 0) continue;
            // flags in the block's words before each word (lane = word), then every word and its
            // offset go through shared memory so that the loop below reads them as broadcasts
            unsigned w_incl = __popc(word[k]);
            const unsigned w_cnt = w_incl;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned v = __shfl_up_sync(0xFFFFFFFFu, w_incl, off);
                if (lane >= off) w_incl += v;
            }
            __syncwarp();                   // (the previous block's entries have been read)
            sh_words[warp][lane] = make_uint2(word[k], w_incl - w_cnt);
            __syncwarp();
            const int64_t mine = base + before;             // list position of the block's first flag
            int32_t *out = cand_idx + mine;
            const int32_t idx0 = index_base + (int32_t)((w0 + blk * 32) << 5) + lane;    // n_active < 2^31
            if (mine + total <= cand_capacity) {
#pragma unroll
                for (int w = 0; w < 32; ++w) {
                    const uint2 e = sh_words[warp][w];      // {flag word, flags before it}: same address in all lanes
                    if (e.x & lane_bit) out[e.y + __popc(e.x & below)] = idx0 + (w << 5);
                }
            } else {
                // the list ends inside this block (or has already ended): entries still free
                const int64_t room64 = cand_capacity - mine;
                const unsigned room = room64 <= 0 ? 0u : (unsigned)room64;      // < total <= 1024
#pragma unroll 1
                for (int w = 0; w < 32; ++w) {
                    const uint2 e = sh_words[warp][w];
                    const unsigned at = e.y + __popc(e.x & below);
                    if ((e.x & lane_bit) && at < room) out[at] = idx0 + (w << 5);
                }
            }
        }
        base += all;
    }
    if (w_begin >= w_end) {                 // (a CTA without words still has to know the total if it is the last)
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kScatterWarps; ++w) base += sh_part[w];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {     // the last CTA knows the total
        *cand_count = base;
        if (base > cand_capacity) atomicOr(status, (unsigned)GS_DEV_CAND_TRUNCATED);
    }
}

// CTAs of pass 1 that fit on one SM (looked up once per device).
static int risk_ctas_per_sm(int dev)
{
    static std::mutex mu;
    static int cached[64];
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 0 || dev >= 64) return kRiskMinCtas;
    if (cached[dev] == 0) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, risk_flags_kernel, kRiskThreads, 0) != cudaSuccess || occ < 1)
            occ = kRiskMinCtas;
        cached[dev] = occ;
    }
    return cached[dev];
}

// Number of CTAs (of both passes) for a scan of n requests on a GPU with n_sm SMs: every SM
// full, but no CTA with less than one round of its warps' steps.
static int64_t scan_grid(int64_t n_steps, int dev, int n_sm)
{
    int64_t blocks = (n_steps + kRiskWarps * kRiskUnroll - 1) / (kRiskWarps * kRiskUnroll);
    const int64_t cap = (int64_t)n_sm * risk_ctas_per_sm(dev);
    return blocks > cap ? cap : blocks;
}

// One scan: cta_counts is scratch for one count per CTA (kMaxScanCtas entries).
static cudaError_t enqueue_scan(unsigned *cta_counts, int dev, int n_sm, gs_ctx *timing_ctx,
                                const int32_t *assigned, const int32_t *generated, const int32_t *pred_len,
                                const float *elapsed, const float *slo, int64_t n,
                                const gs_instances &inst, const gs_types &types,
                                uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                                int64_t *cand_count, unsigned *status, cudaStream_t st,
                                const int64_t *prev_count = nullptr, int32_t index_base = 0)
{
    if (n == 0) return cudaMemsetAsync(cand_count, 0, sizeof(int64_t), st);
    const int64_t n_steps = (n + (1 << kStepShift) - 1) >> kStepShift;
    const int64_t n_words = (n + 31) >> 5;
    int64_t blocks = scan_grid(n_steps, dev, n_sm);
    if (blocks > kMaxScanCtas) blocks = kMaxScanCtas;
    cudaError_t e;
    {
        LaunchTimer timer(timing_ctx, GS_K_RISK_FLAGS, st);
        e = launch_dependent(risk_flags_kernel, dim3((unsigned)blocks), dim3(kRiskThreads), 0, st,
                             assigned, generated, pred_len, elapsed, slo, n, inst.type_id, inst.decode_batch, inst.n_instances,
                             types.tpot_a_ms, types.tpot_b_ms, types.n_types, flag_bits, cta_counts, n_steps, status);
        if (e != cudaSuccess) return e;
    }
    {
        LaunchTimer timer(timing_ctx, GS_K_RISK_SCATTER, st);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);           // the same runs of steps as pass 1
        cfg.blockDim = dim3(kScatterThreads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = GS_RISK_PDL ? 1 : 0;
        e = cudaLaunchKernelEx(&cfg, scatter_candidates_kernel, (const uint32_t *)flag_bits, n_words,
                               (const unsigned *)cta_counts, n_steps, cand_idx, cand_capacity, cand_count, status,
                               prev_count, index_base);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_risk(gs_ctx *ctx, const int32_t *assigned, const int32_t *generated,
                        const int32_t *pred_len, const float *elapsed, const float *slo,
                        int64_t n, const gs_instances &inst, const gs_types &types,
                        uint32_t *flag_bits, int32_t *cand_idx, int64_t cand_capacity,
                        int64_t *cand_count, cudaStream_t st, const int64_t *prev_count, int32_t index_base)
{
    return enqueue_scan(ctx->s.scan_counts, ctx->device, ctx->n_sm, ctx, assigned, generated, pred_len, elapsed, slo, n,
                        inst, types, flag_bits, cand_idx, cand_capacity, cand_count, ctx->s.status, st, prev_count,
                        index_base);
}

// ---------------------------------------------------------------------------------------
// gs_risk_scan_noalloc: the same scan for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------

// All scratch of the no-allocation entry point: the per-CTA flag counts that the scan's two
// passes exchange, and a status word.  It lives in the library image: every GPU that loads the
// library holds these 16 KB until the process exits.  Every call stores each count before it
// reads it, so nothing a call computes depends on what an earlier call left here.
struct NoAllocScratch {
    unsigned cta_counts[kMaxScanCtas];
    unsigned status;
};
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

}  // namespace gs

namespace {

constexpr int kMaxDevices = 64;
// Per GPU: the device address of g_noalloc_scratch, resolved on that GPU's first call (in host
// code the symbol's name is only a handle, never an address a kernel may use).
struct NoAllocDevice {
    gs::NoAllocScratch *ptr = nullptr;
    cudaError_t err = cudaSuccess;
    bool ready = false;
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
    const cudaError_t e = enqueue_scan(sc->cta_counts, dev, n_sm, nullptr, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
                                       n_active, *inst, *types, out_flag_bits, out_cand_idx, cand_capacity,
                                       out_cand_count, out_status_bits ? out_status_bits : &sc->status,
                                       (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? GS_OK : GS_ERR_CUDA;
}
