// Host side of the C ABI declared in include/dart.h: argument checks, workspace, launches.
#include "../../include/dart.h"

#include <cuda_runtime.h>

#include <mutex>
#include <new>
#include <vector>

#include "dart_staged.cuh"
#include "dart_sweep.cuh"
#include "dart_onepass.cuh"
#include "dart_resident.cuh"
#include "dart_pair.cuh"

namespace {

constexpr int kSweepChunks = 8;     // column chunks per row tile of the persistent sweep's second pass
constexpr int kSweepChunkMaxP = 16; // ... for up to this many pivots

enum Slot { SLOT_SCORE = 0, SLOT_PIVOT, SLOT_SIM, SLOT_RETAIN, SLOT_GATHER, SLOT_SWEEP, SLOT_ONEPASS, SLOT_RESIDENT, SLOT_PAIR, SLOT_COUNT };
const char *const kSlotNames[SLOT_COUNT] = {"score", "pivot", "sim", "retain", "gather", "sweep", "onepass", "resident", "pair"};

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                      const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct EventPair {
    cudaEvent_t start, stop;
    int slot;
};

} // namespace

struct dart_ctx {
    dart_desc desc;
    int B, S;
    int last_cuda;
    int64_t launches;
    size_t bytes;
    // workspace (device), indexed with the shapes of the current call
    float *l1, *ssq, *sim, *eps;
    int32_t *pivot_idx, *owner;
    void *piv_rows;  // [B_max][P_max rounded to 16][d] bf16: compact copy of the pivot rows (NULL: not available)
    int32_t *len;    // [B_max] packed length of every sample (retention with independent pivots)
    int32_t *cand;   // [B_max][P_max][cand_stride] sorted candidate lists of the two-phase retention (NULL: not available)
    int cand_stride;
    unsigned long long *band; // [B_max][P_max][band_stride] unsorted candidate bands of the band retention (NULL: not available)
    int32_t *band_n;          // [B_max][P_max] their lengths
    int band_stride;
    uint8_t *keep;
    int *status; // device status word, followed by three words of detail
    int32_t status_detail[11];
    // profiling
    bool profiling;
    std::vector<EventPair> pending, spare;
    float slot_ms[SLOT_COUNT];
    int32_t slot_launches[SLOT_COUNT];
    int max_smem_optin;
    // host staging (DART_FLAG_HOST_STAGING): two sets of device buffers for chunks of samples
    int chunk;                      // samples per chunk
    void *st_hidden[2], *st_keys[2], *st_out_hidden[2];
    int32_t *st_out_idx[2];
    int64_t *st_out_pos[2];
    cudaStream_t s_h2d, s_run, s_d2h;
    cudaEvent_t ev_in[2], ev_run[2], ev_out[2];
    // fused path (csrc/dart_sweep.cuh); available when d is a multiple of 64 and the device is sm_100
    bool fused_ok;
    int sm_count, n_atoms;
    int *counters;
    size_t counters_bytes;
    float *sim_share;     // [kSweepChunks][B_max][min(P_max, 16)][S_max]: the column chunks' shares of the similarities (NULL: none)
    TensorMapEncodeFn encode;
    // resident sweep (csrc/dart_resident.cuh)
    bool resident_ok;
    int res_landing;  // landing slots in shared memory
    unsigned long long *res_cand; // [B_max][sm_count][8] candidate keys
    // paired sweeps (csrc/dart_pair.cuh)
    bool pair_ok;
    unsigned long long *pair_cand; // [B_max][sm_count][16] candidate keys
    int32_t *pair_res;             // [B_max][32] resolved pivots and their norms
    // pivots chosen inside the library from other sources than the vision tokens' scores (dart_opts.pivot_source)
    int32_t *pivot_src;            // [B_max][P_max]
    float *text_score;             // [2][B_max][S_max]: L1 scores, then sums of squares, of the text rows (before | after the block)
};

namespace {

int cuda_fail(dart_ctx *ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda = (int)e;
    return e == cudaErrorMemoryAllocation ? DART_ERR_NOMEM : DART_ERR_CUDA;
}

#define DART_CUDA(ctx, call)                                   \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);  \
    } while (0)

template <typename T>
int ws_alloc(dart_ctx *ctx, T **p, size_t count)
{
    size_t bytes = (count * sizeof(T) + 255) / 256 * 256;
    cudaError_t e = cudaMalloc((void **)p, bytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->bytes += bytes;
    return DART_OK;
}

// Scoped device switch: the library never leaves another device current.
struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

struct Prof {
    dart_ctx *ctx;
    cudaStream_t st;
    EventPair ev;
    bool on;
    Prof(dart_ctx *c, cudaStream_t s, int slot) : ctx(c), st(s), on(c->profiling)
    {
        ++ctx->launches;
        if (!on) return;
        if (!ctx->spare.empty()) {
            ev = ctx->spare.back();
            ctx->spare.pop_back();
        } else if (cudaEventCreate(&ev.start) != cudaSuccess || cudaEventCreate(&ev.stop) != cudaSuccess) {
            on = false;
            return;
        }
        ev.slot = slot;
        cudaEventRecord(ev.start, st);
    }
    ~Prof()
    {
        if (!on) return;
        cudaEventRecord(ev.stop, st);
        ctx->pending.push_back(ev);
    }
};

bool overlaps(const void *a, size_t na, const void *b, size_t nb)
{
    if (!a || !b) return false;
    uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + nb && y < x + na;
}

int next_pow2(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

int check_call(const dart_ctx *ctx, const void *hidden, const void *keys, int vis_offset, int n_vis, int n_pivot,
               int n_keep, const void *out_hidden, const void *out_idx, const void *out_pos, bool host = false)
{
    if (!ctx || !hidden || !out_hidden || !out_idx || !out_pos) return DART_ERR_NULL;
    const int S = ctx->S;
    if (ctx->B < 1 || S < 1) return DART_ERR_BAD_SHAPE;
    if (n_pivot < 1 || n_pivot > n_keep || n_keep > n_vis || vis_offset < 0 || n_vis < 1) return DART_ERR_BAD_SHAPE;
    if ((long long)vis_offset + n_vis > S) return DART_ERR_BAD_SHAPE;
    if (n_pivot > ctx->desc.P_max || n_keep > ctx->desc.Kp_max) return DART_ERR_BAD_SHAPE;
    if (!host && (((uintptr_t)hidden | (uintptr_t)keys | (uintptr_t)out_hidden) & 15u)) return DART_ERR_ALIGN;
    if (((uintptr_t)out_idx & 3u) || ((uintptr_t)out_pos & 7u)) return DART_ERR_ALIGN;
    const size_t in_bytes = (size_t)ctx->B * S * ctx->desc.d * 2;
    const size_t S_out = (size_t)S - n_vis + n_keep;
    const size_t out_bytes = (size_t)ctx->B * S_out * ctx->desc.d * 2;
    if (overlaps(out_hidden, out_bytes, hidden, in_bytes) || overlaps(out_hidden, out_bytes, keys, in_bytes))
        return DART_ERR_ALIAS;
    return DART_OK;
}

int copy_debug(dart_ctx *ctx, int B, int n_vis, int P, const dart_debug *dbg, cudaStream_t st)
{
    if (dbg) {
        const size_t nv = (size_t)B * n_vis, np = (size_t)B * P;
        if (dbg->l1) DART_CUDA(ctx, cudaMemcpyAsync(dbg->l1, ctx->l1, nv * 4, cudaMemcpyDeviceToDevice, st));
        if (dbg->ssq) DART_CUDA(ctx, cudaMemcpyAsync(dbg->ssq, ctx->ssq, nv * 4, cudaMemcpyDeviceToDevice, st));
        if (dbg->pivot_idx)
            DART_CUDA(ctx, cudaMemcpyAsync(dbg->pivot_idx, ctx->pivot_idx, np * 4, cudaMemcpyDeviceToDevice, st));
        if (dbg->sim) DART_CUDA(ctx, cudaMemcpyAsync(dbg->sim, ctx->sim, np * n_vis * 4, cudaMemcpyDeviceToDevice, st));
        if (dbg->eps) DART_CUDA(ctx, cudaMemcpyAsync(dbg->eps, ctx->eps, np * 4, cudaMemcpyDeviceToDevice, st));
        if (dbg->keep) DART_CUDA(ctx, cudaMemcpyAsync(dbg->keep, ctx->keep, nv, cudaMemcpyDeviceToDevice, st));
        if (dbg->owner) DART_CUDA(ctx, cudaMemcpyAsync(dbg->owner, ctx->owner, nv * 4, cudaMemcpyDeviceToDevice, st));
    }
    return DART_OK;
}

// Steps 4 and 5a.  Two phases (candidate lists for all pivots at once, then the pivots' turns) when the lists fit
// the workspace and shared memory, else the one-kernel form.
void launch_retention(dart_ctx *ctx, int B, const int64_t *pos_in, int vis_offset, int n_vis, int P, int n_keep,
                      int32_t *out_idx, int64_t *out_pos, const dart_opts &o, cudaStream_t st)
{
    using namespace dart;
    // the tokens shared out beside the pivots: n_keep - P, or up to n_keep when pivots may be text tokens
    const int S = ctx->S, m = o.text_pivots ? n_keep : n_keep - P, mode = o.retention;
    if (o.rule == DART_RULE_GLOBAL) { // one threshold for all pivots: a single selection per sample
        Prof p(ctx, st, SLOT_RETAIN);
        retain_global_kernel<<<B, kSelectThreads, retain_global_smem_bytes(n_vis), st>>>(
            ctx->sim, ctx->pivot_idx, pos_in, S, vis_offset, n_vis, P, n_keep, out_idx, out_pos, ctx->keep, ctx->owner, ctx->eps,
            ctx->status);
        return;
    }
    if (o.rule == DART_RULE_UNION) { // independent pivots: selections, scan of the packed lengths, index lists at their offsets
        {
            Prof p(ctx, st, SLOT_RETAIN);
            retain_union_kernel<<<B, kSelectThreads, retain_union_smem_bytes(n_vis), st>>>(
                ctx->sim, ctx->pivot_idx, S, n_vis, P, n_keep, ctx->keep, ctx->owner, ctx->eps, ctx->len, ctx->status);
        }
        {
            Prof p(ctx, st, SLOT_RETAIN);
            cu_seqlens_kernel<<<1, 256, 0, st>>>(ctx->len, B, o.cu_seqlens, ctx->status);
        }
        Prof p(ctx, st, SLOT_RETAIN);
        pack_varlen_kernel<<<B, kWalkThreads, retain_union_smem_bytes(n_vis), st>>>(ctx->keep, o.cu_seqlens, pos_in, S, vis_offset, n_vis,
                                                                                    out_idx, out_pos, ctx->status);
        return;
    }
    const int m_pad = next_pow2(m > 1 ? m : 1);
    // bands: a list must hold the m tokens of the exact route and fit one staging round of phase 2
    const int band_cap = ctx->band_stride < kPickStageEntries ? ctx->band_stride : kPickStageEntries;
    const bool can_bands = ctx->band && m > 0 && m <= band_cap && n_vis <= kBandMaxTokens && band_smem_bytes(n_vis, band_cap) <= (size_t)ctx->max_smem_optin - 2048 &&
                           pick_smem_bytes(n_vis, P) <= (size_t)ctx->max_smem_optin - 2048;
    // Which form: all do the same selections.  One kernel per sample takes B CTAs through P selections each; sorted
    // lists spread the selections over B * P CTAs, which pays while B CTAs cannot fill the SMs (measured: batch 4-64 up
    // to 4x faster than one kernel); bands need one warp per selection and no sort, which pays once the batch fills the
    // GPU (measured at batch 256: 8 pivots 93 -> 56 us, 32 pivots 0.36 -> 0.16 ms, 128 pivots 1.38 -> 0.49 ms), while for
    // a few samples their turns, one warp per sample, take longer than the sorted lists' walks.
    const bool can_lists = ctx->cand && m <= ctx->cand_stride && m <= kCandMax &&
                               candidates_smem_bytes(n_vis, m_pad) <= (size_t)ctx->max_smem_optin - 2048 &&
                               walk_smem_bytes(n_vis) <= (size_t)ctx->max_smem_optin - 2048;
    // ... and both phases of the bands in one launch for batches that cannot fill the GPU: as many band-building warps as
    // shared memory takes beside the flags
    int band_warps = P < kPickThreads / 32 ? P : kPickThreads / 32;
    while (band_warps > 1 && retain_fused_smem_bytes(n_vis, P, band_cap, band_warps) > (size_t)ctx->max_smem_optin - 2048) --band_warps;
    const bool can_fused = can_bands && retain_fused_smem_bytes(n_vis, P, band_cap, band_warps) <= (size_t)ctx->max_smem_optin - 2048;
    // (measured, us: one sample of 576 tokens 23 -> 20, 64 samples 29 -> 23 against the sorted lists; with more pivots than
    // band-building warps the lists stay ahead: 16 pivots, 8 samples of 2880 tokens 45 vs 55; 32 pivots, 4 samples 66 vs 123)
    if (can_fused && (mode == DART_RETAIN_FUSED || (mode == DART_RETAIN_AUTO && B <= ctx->sm_count && P <= band_warps))) {
        Prof p(ctx, st, SLOT_RETAIN);
        retain_fused_kernel<<<B, kPickThreads, retain_fused_smem_bytes(n_vis, P, band_cap, band_warps), st>>>(
            ctx->sim, ctx->pivot_idx, ctx->band, ctx->band_n, band_cap, pos_in, S, vis_offset, n_vis, P, n_keep, out_idx, out_pos,
            ctx->keep, ctx->owner, ctx->eps, ctx->status, band_warps);
        return;
    }
    const bool bands = can_bands && (mode == DART_RETAIN_BANDS || (mode == DART_RETAIN_AUTO && (B > ctx->sm_count || !can_lists)));
    if (bands) {
        {
            Prof p(ctx, st, SLOT_RETAIN);
            band_kernel<<<dim3((unsigned)P, (unsigned)B), 32, band_smem_bytes(n_vis, band_cap), st>>>(
                ctx->sim, ctx->pivot_idx, n_vis, P, n_keep, band_cap, ctx->band, ctx->band_n, ctx->status);
        }
        Prof p(ctx, st, SLOT_RETAIN);
        retain_pick_kernel<<<B, kPickThreads, pick_smem_bytes(n_vis, P), st>>>(
            ctx->pivot_idx, ctx->band, ctx->band_n, band_cap, pos_in, S, vis_offset, n_vis, P, n_keep, out_idx, out_pos, ctx->keep,
            ctx->owner, ctx->eps, ctx->status);
        return;
    }
    const bool two_phase = can_lists && (mode == DART_RETAIN_LISTS || (mode == DART_RETAIN_AUTO && B <= ctx->sm_count));
    if (!two_phase) {
        Prof p(ctx, st, SLOT_RETAIN);
        retain_kernel<<<B, kSelectThreads, retain_smem_bytes(n_vis, P), st>>>(ctx->sim, ctx->pivot_idx, pos_in, S, vis_offset, n_vis, P,
                                                               n_keep, out_idx, out_pos, ctx->keep, ctx->owner,
                                                               ctx->eps, ctx->status, retain_cache_rows(n_vis, P));
        return;
    }
    if (m > 0) {
        Prof p(ctx, st, SLOT_RETAIN);
        // one CTA per SM at most: big CTAs shorten each selection; more CTAs than SMs: small ones overlap better
        // (measured: 8 x 16 lists 67 -> 54 us with 1024 threads, 64 x 8 lists 36 -> 45 us)
        const int threads = (long long)B * P <= ctx->sm_count ? kCandThreads : 256;
        candidates_kernel<<<dim3((unsigned)P, (unsigned)B), threads, candidates_smem_bytes(n_vis, m_pad), st>>>(
            ctx->sim, ctx->pivot_idx, n_vis, P, n_keep, m_pad, ctx->cand_stride, ctx->cand, ctx->status);
    }
    {
        Prof p(ctx, st, SLOT_RETAIN);
        retain_walk_kernel<<<B, kWalkThreads, walk_smem_bytes(n_vis), st>>>(ctx->sim, ctx->pivot_idx, ctx->cand, ctx->cand_stride, pos_in,
                                                                          S, vis_offset, n_vis, P, n_keep, out_idx, out_pos,
                                                                          ctx->keep, ctx->owner, ctx->eps, ctx->status);
    }
}

// Step 5b.  With independent pivots the rows are packed at the samples' offsets (cu_seqlens) instead of B equal blocks.
void launch_gather(dart_ctx *ctx, int B, const void *hidden, int n_vis, int n_keep, const int32_t *out_idx, void *out_hidden,
                   const dart_opts &o, cudaStream_t st)
{
    using namespace dart;
    const int S = ctx->S, d8 = ctx->desc.d / 8, S_out = S - n_vis + n_keep;
    Prof pr(ctx, st, SLOT_GATHER);
    const long long orows = (long long)B * S_out;
    const unsigned grid = (unsigned)((orows + kGatherWarps - 1) / kGatherWarps);
    if (o.rule == DART_RULE_UNION)
        gather_varlen_kernel<<<grid, kGatherWarps * 32, 0, st>>>((const uint4 *)hidden, out_idx, o.cu_seqlens, B, S, d8, orows,
                                                                ctx->status, (uint4 *)out_hidden);
    else
        gather_kernel<<<grid, kGatherWarps * 32, 0, st>>>((const uint4 *)hidden, out_idx, S, S_out, d8, orows, ctx->status,
                                                         (uint4 *)out_hidden);
}

// Step 2 with the caller's pivots: checked and copied into the workspace.
void launch_pivots_given(dart_ctx *ctx, int B, int vis_offset, int n_vis, int P, const dart_opts &o, cudaStream_t st)
{
    Prof p(ctx, st, SLOT_PIVOT);
    const int lo = o.text_pivots ? -vis_offset : 0, hi = o.text_pivots ? ctx->S - vis_offset : n_vis;
    dart::pivots_given_kernel<<<B, 256, (size_t)((hi - lo + 31) / 32) * 4, st>>>(o.pivots_in, lo, hi, P, ctx->pivot_idx, ctx->status);
}

int launch_staged(dart_ctx *ctx, int B, const void *hidden, const void *keys_in, const int64_t *pos_in, int vis_offset,
                  int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos,
                  const dart_opts &o, const dart_debug *dbg, cudaStream_t st)
{
    using namespace dart;
    const int S = ctx->S, d8 = ctx->desc.d / 8;
    const uint4 *keys = (const uint4 *)(keys_in ? keys_in : hidden);
    const long long rows = (long long)B * n_vis;
    {
        Prof p(ctx, st, SLOT_SCORE);
        unsigned grid = (unsigned)((rows + kScoreWarps - 1) / kScoreWarps);
        score_kernel<<<grid, kScoreWarps * 32, 0, st>>>(keys, S, d8, vis_offset, n_vis, rows, ctx->l1, ctx->ssq);
    }
    if (o.pivots_in) {
        launch_pivots_given(ctx, B, vis_offset, n_vis, P, o, st);
    } else {
        Prof p(ctx, st, SLOT_PIVOT);
        int P_pad = next_pow2(P);
        const bool cached = n_vis <= kPivotCacheMax;
        pivot_kernel<<<B, kSelectThreads, pivot_smem_bytes(n_vis, P_pad, cached), st>>>(o.norm_kind == 2 ? ctx->ssq : ctx->l1, n_vis, P,
                                                                                       P_pad, o.pivot_smallest, cached, ctx->pivot_idx);
    }
    {
        Prof p(ctx, st, SLOT_SIM);
        size_t smem = (size_t)kSimPivotChunk * d8 * 16;
        dim3 grid((n_vis + kSimRowsPerCta - 1) / kSimRowsPerCta, B);
        for (int p0 = 0; p0 < P; p0 += kSimPivotChunk)
            sim_alu_kernel<<<grid, kSimWarps * 32, smem, st>>>(keys, S, d8, vis_offset, n_vis, P, p0, ctx->pivot_idx,
                                                              ctx->ssq, ctx->sim);
        ctx->launches += (P - 1) / kSimPivotChunk;
    }
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

// ---- fused path ------------------------------------------------------------------------------------
int fused_setup(dart_ctx *ctx)
{
    using namespace dart::sweep;
    const dart_desc &D = ctx->desc;
    ctx->fused_ok = false;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, D.device) != cudaSuccess) return DART_ERR_CUDA;
    ctx->sm_count = prop.multiProcessorCount;
    if (prop.major != 10 || D.d % kAtomCols != 0 || D.d * 2 > kMaxRowBytes || !prop.cooperativeLaunch)
        return DART_OK; // staged path only
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess)
        return DART_OK;
    ctx->encode = (TensorMapEncodeFn)fn;
    ctx->n_atoms = D.d / kAtomCols;
    int rc = DART_OK;
    ctx->counters_bytes = (size_t)D.B_max * 2 * sizeof(int);
    if (rc == DART_OK) rc = ws_alloc(ctx, (uint8_t **)&ctx->counters, ctx->counters_bytes);
    if (rc != DART_OK) return rc;
    {   // shares of the similarities for up to 16 pivots; contexts that would need more than 1 GiB go without
        const size_t n = (size_t)kSweepChunks * D.B_max * (D.P_max < kSweepChunkMaxP ? D.P_max : kSweepChunkMaxP) * D.S_max;
        if (n * sizeof(float) <= ((size_t)1 << 30)) rc = ws_alloc(ctx, &ctx->sim_share, n);
        if (rc != DART_OK) return rc;
    }
    if (cudaFuncSetAttribute(sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - kStaticSmemReserve) !=
        cudaSuccess)
        return DART_ERR_CUDA;
    int per_sm = 0;
    int n1 = 0, n2 = 0;
    ring_depths(16, (uint32_t)D.d * 2, ctx->max_smem_optin, n1, n2);
    if (n1 >= 2) { // else the rows are too wide for the persistent sweep's rings: the other tensor-core kernels may still fit
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sweep_kernel, kThreads,
                                                          smem_bytes(16, (uint32_t)D.d * 2, n1, n2)) !=
                cudaSuccess ||
            per_sm < 1)
            return DART_ERR_CUDA;
        ctx->fused_ok = true;
    }
    // the resident sweep: rows of at most 8 KB, two landing slots or more, one CTA per SM
    ctx->resident_ok = false;
    if (D.d * 2 <= dart::resident::kMaxRowBytes && ctx->sm_count <= dart::resident::kMaxGrid) {
        namespace R = dart::resident;
        const int L = R::landing_slots(D.d, ctx->sm_count, ctx->max_smem_optin);
        int res_per_sm = 0;
        if (L >= 2 &&
            cudaFuncSetAttribute(R::resident_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)R::smem_bytes(D.d, ctx->sm_count, L)) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&res_per_sm, R::resident_kernel, R::kThreads,
                                                          R::smem_bytes(D.d, ctx->sm_count, L)) == cudaSuccess &&
            res_per_sm >= 1) {
            rc = ws_alloc(ctx, &ctx->res_cand, (size_t)D.B_max * ctx->sm_count * R::kMaxP);
            if (rc != DART_OK) return rc;
            ctx->res_landing = L;
            ctx->resident_ok = true;
        }
    }
    // paired sweeps: rows of at most 16 KB, two ring-1 stages or more, one CTA per SM
    ctx->pair_ok = false;
    if (ctx->sm_count <= dart::pair::kMaxGrid) {
        namespace Q = dart::pair;
        int n1 = 0, n2 = 0, n3 = 0, per = 0;
        Q::ring_depths(1, (uint32_t)D.d * 2, ctx->sm_count, ctx->max_smem_optin, n1, n2, n3, 0, 2, 2); // the least it takes; checked per call
        if (n1 >= 2 &&
            cudaFuncSetAttribute(Q::pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - Q::kStaticSmemReserve) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, Q::pair_kernel, Q::kThreads,
                                                          Q::smem_bytes(1, (uint32_t)D.d * 2, ctx->sm_count, n1, n2, n3)) == cudaSuccess &&
            per >= 1) {
            rc = ws_alloc(ctx, &ctx->pair_cand, (size_t)D.B_max * ctx->sm_count * Q::kMaxP);
            if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->pair_res, (size_t)D.B_max * 2 * Q::kMaxP);
            if (rc != DART_OK) return rc;
            ctx->pair_ok = true;
        }
    }
    // the one-pass kernel for the caller's pivots uses the same tensor maps
    if (cudaFuncSetAttribute(dart::onepass::onepass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ctx->max_smem_optin - dart::onepass::kStaticSmemReserve) != cudaSuccess)
        return DART_ERR_CUDA;
    return DART_OK;
}

int encode_2d(dart_ctx *ctx, CUtensorMap *tm, const void *base, uint64_t cols, uint64_t rows, uint32_t box_rows)
{
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)dart::sweep::kAtomCols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda = (int)r;
        return DART_ERR_CUDA;
    }
    return DART_OK;
}

bool fused_applies(const dart_ctx *ctx, int P) { return ctx->fused_ok && P <= dart::sweep::kMaxN; }

int launch_fused(dart_ctx *ctx, int B, const void *hidden, const void *keys_in, const int64_t *pos_in, int vis_offset,
                 int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o,
                 const dart_debug *dbg, cudaStream_t st)
{
    using namespace dart;
    using namespace dart::sweep;
    const int S = ctx->S, d8 = ctx->desc.d / 8;
    const void *keys = keys_in ? keys_in : hidden;
    Params p = {};
    p.B = B, p.S = S, p.vis_offset = vis_offset, p.n_vis = n_vis, p.P = P, p.N = (P + 15) / 16 * 16, p.d8 = d8;
    p.n_atoms = ctx->n_atoms, p.n_rt = (n_vis + kTileRows - 1) / kTileRows;
    // Option (dart_opts.tune >= 2): the second pass over a row tile is cut into chunks of columns, one task each (the size of
    // a first-pass task), so that a sample's second pass is spread over all SMs like its first; every chunk writes its share of
    // the similarities and sim_sum_kernel adds them up; the first pass then runs at most `tune` steps ahead of the second.
    // Measured on the 256-sample workload: no gain (1.81-1.89 ms against 1.86 ms): the pivots of a sample take three to
    // four rounds of steps to appear, and holding the first pass back that closely stalls it as much as the L2 then saves.
    p.n_kc = (ctx->sim_share && P <= kSweepChunkMaxP && (o.tune & 0xfff) >= 2) ? (p.n_atoms < kSweepChunks ? p.n_atoms : kSweepChunks) : 1;
    p.apc = (p.n_atoms + p.n_kc - 1) / p.n_kc;
    p.n_kc = (p.n_atoms + p.apc - 1) / p.apc;
    p.T1 = (n_vis + kS1Rows - 1) / kS1Rows, p.T2 = p.n_rt * p.n_kc, p.Tm = p.T1 > p.T2 ? p.T1 : p.T2;
    p.row_bytes = (uint32_t)ctx->desc.d * 2, p.stage1_bytes = stage1_bytes(p.row_bytes);
    ring_depths(p.N, p.row_bytes, ctx->max_smem_optin, p.n1, p.n2);
    if (p.n1 < 2) return DART_ERR_UNSUPPORTED;
    const long long n_all = (long long)B * p.Tm;
    // a row's second sweep follows its first by one sample plus the time the pivots take to appear
    long long lag = (long long)p.Tm + (o.sweep_lag > 0 ? o.sweep_lag : 7 * ctx->sm_count);
    p.lag = (uint32_t)(lag < n_all ? lag : n_all);
    if (n_all + p.lag >= (1ll << 30)) return DART_ERR_UNSUPPORTED;
    p.norm_kind = o.norm_kind, p.smallest = o.pivot_smallest;
    p.withhold_pivots = o.test_withhold_pivots;
    p.keep_l2 = p.n_kc > 1;
    p.ahead = (o.tune & 0xfff) >= 2 ? (uint32_t)(o.tune & 0xfff) : 0u;
    p.wait_ns = o.wait_limit > 0 ? (unsigned long long)o.wait_limit * 1000ull : 2000000000ull;
    p.keys = (const char *)keys;
    p.sim = p.n_kc > 1 ? ctx->sim_share : ctx->sim, p.l1 = ctx->l1, p.ssq = ctx->ssq, p.pivot_idx = ctx->pivot_idx;
    p.s1_done = ctx->counters, p.piv_ready = ctx->counters + B;
    p.status = ctx->status;
    // the same tensor with a 128-row box (full tiles), a 32-row box (short last tiles) and a one-row box (pivot rows)
    CUtensorMap tm_tile, tm_keys, tm_row;
    int rc = encode_2d(ctx, &tm_tile, keys, (uint64_t)ctx->desc.d, (uint64_t)B * S, kTileRows);
    if (rc == DART_OK) rc = encode_2d(ctx, &tm_keys, keys, (uint64_t)ctx->desc.d, (uint64_t)B * S, kSubRows);
    if (rc == DART_OK) rc = encode_2d(ctx, &tm_row, keys, (uint64_t)ctx->desc.d, (uint64_t)B * S, 1);
    if (rc != DART_OK) return rc;
    DART_CUDA(ctx, cudaMemsetAsync(ctx->counters, 0, (size_t)B * 2 * sizeof(int), st));
    {
        Prof pr(ctx, st, SLOT_SWEEP);
        long long grid = n_all < ctx->sm_count ? n_all : ctx->sm_count;
        void *args[4] = {&tm_tile, &tm_keys, &tm_row, &p};
        DART_CUDA(ctx, cudaLaunchCooperativeKernel((const void *)sweep_kernel, dim3((unsigned)grid), dim3(kThreads), args,
                                                   smem_bytes(p.N, p.row_bytes, p.n1, p.n2), st));
    }
    if (p.n_kc > 1) {
        Prof pr(ctx, st, SLOT_SIM);
        const long long n = (long long)B * P * n_vis; // the shares of every chunk lie n floats apart
        const bool vec = n % 4 == 0;
        const long long items = vec ? n / 4 : n, want = (items + kSimSumThreads - 1) / kSimSumThreads;
        const unsigned grid = (unsigned)(want < 8ll * ctx->sm_count ? want : 8ll * ctx->sm_count);
        if (vec)
            sim_sum_kernel<float4><<<grid, kSimSumThreads, 0, st>>>((const float4 *)ctx->sim_share, items, p.n_kc, (float4 *)ctx->sim);
        else
            sim_sum_kernel<float><<<grid, kSimSumThreads, 0, st>>>(ctx->sim_share, items, p.n_kc, ctx->sim);
    }
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

// One pass over `src` (csrc/dart_onepass.cuh) with the pivots already in the workspace: sums of squares of src's rows
// (and their L1 scores unless `scores_elsewhere`: then the scores came from another tensor) and the similarities.
int launch_onepass_kernel(dart_ctx *ctx, int B, const void *src, bool scores_elsewhere, int vis_offset, int n_vis, int P,
                          const dart_opts &o, cudaStream_t st, dart::TileSplit split = dart::TileSplit{1, 0})
{
    using namespace dart;
    using sweep::kSubRows;
    using sweep::kTileRows;
    const int S = ctx->S;
    onepass::Params p = {};
    p.B = B, p.S = S, p.vis_offset = vis_offset, p.n_vis = n_vis, p.P = P, p.N = (P + 15) / 16 * 16;
    p.n_atoms = ctx->n_atoms, p.n_rt = (n_vis + kTileRows - 1) / kTileRows;
    p.split = split, p.n_sel = split.k <= 1 ? p.n_rt : split.n_streamed(p.n_rt);
    if (p.n_sel == 0) return DART_OK; // every tile stayed on the chip
    p.compact = ctx->piv_rows != nullptr && P > onepass::kGatherMaxP;
    // Two row tiles per task share every pivot tile that is fetched (two accumulators per buffer: 4 N <= 512 columns of
    // tensor memory), if that still leaves a ring of three stages and shortens the longest queue of tasks.  With many pivots a
    // pivot tile is as large as a token tile and the SM's share of the L2 bandwidth bounds the kernel; with few, a task of
    // 256 rows halves what is paid per task (measured at batch 256 x 2880 tokens: 8 pivots 1.25 -> 1.01 ms, 16: 1.14 ->
    // 1.00, 32: 1.31 -> 1.04, 64: 1.37 -> 1.22, 128: 1.75 -> 1.61).  (tune bits 0x1000 / 0x2000 force one / two tiles.)
    p.tg = 1;
    const bool two_fit = split.k <= 1 && 4 * p.N <= 512 &&
                         onepass::ring_depth(p.N, onepass::atoms_per_stage(p.N, ctx->max_smem_optin, 2), ctx->max_smem_optin, 2) >= 3;
    // the longest queue of any CTA, in tiles plus 0.4 of a tile per task (the fit above): 8 x 23 tiles on 148 SMs are
    // 2 x 1.4 as single tiles and 1 x 2.4 as pairs (measured 65 and 53 us), 16 x 23 are 3 x 1.4 and 2 x 2.4 (94 and 102 us)
    auto queue_cost = [&](int tg) {
        const long long tasks = (long long)B * ((p.n_rt + tg - 1) / tg);
        return (double)((tasks + ctx->sm_count - 1) / ctx->sm_count) * (tg + 0.4);
    };
    if (two_fit && queue_cost(2) < queue_cost(1) && !(o.tune & 0x1000)) p.tg = 2;
    if (two_fit && (o.tune & 0x2000)) p.tg = 2;
    p.aps = onepass::atoms_per_stage(p.N, ctx->max_smem_optin, p.tg);
    p.n_st = onepass::ring_depth(p.N, p.aps, ctx->max_smem_optin, p.tg);
    if (p.n_st < 2) return DART_ERR_UNSUPPORTED;
    p.wait_ns = o.wait_limit > 0 ? (unsigned long long)o.wait_limit * 1000ull : 2000000000ull;
    p.withhold = o.test_withhold_pivots;
    p.sim = ctx->sim, p.l1 = scores_elsewhere ? nullptr : ctx->l1, p.ssq = ctx->ssq, p.pivot_idx = ctx->pivot_idx;
    p.status = ctx->status;
    CUtensorMap tm_tile, tm_keys, tm_row, tm_piv, tm_pair;
    int rc = encode_2d(ctx, &tm_tile, src, (uint64_t)ctx->desc.d, (uint64_t)B * S, kTileRows);
    if (rc == DART_OK) rc = encode_2d(ctx, &tm_pair, src, (uint64_t)ctx->desc.d, (uint64_t)B * S, 2 * kTileRows);
    if (rc == DART_OK) rc = encode_2d(ctx, &tm_keys, src, (uint64_t)ctx->desc.d, (uint64_t)B * S, kSubRows);
    if (rc == DART_OK) rc = encode_2d(ctx, &tm_row, src, (uint64_t)ctx->desc.d, (uint64_t)B * S, 1);
    if (rc == DART_OK)
        rc = p.compact ? encode_2d(ctx, &tm_piv, ctx->piv_rows, (uint64_t)ctx->desc.d, (uint64_t)B * p.N, (uint32_t)p.N)
                       : encode_2d(ctx, &tm_piv, src, (uint64_t)ctx->desc.d, (uint64_t)B * S, 1); // unused
    if (rc != DART_OK) return rc;
    if (p.compact) { // the sample's pivot rows side by side, so that a pivot tile is one box
        Prof pc(ctx, st, SLOT_PIVOT);
        const long long prow = (long long)B * p.N;
        pivot_rows_kernel<<<(unsigned)((prow + kPivotRowWarps - 1) / kPivotRowWarps), kPivotRowWarps * 32, 0, st>>>(
            (const uint4 *)src, ctx->pivot_idx, S, ctx->desc.d / 8, vis_offset, n_vis, P, p.N, prow, (uint4 *)ctx->piv_rows);
    }
    Prof pr(ctx, st, SLOT_ONEPASS);
    const long long tasks = (long long)B * ((p.n_sel + p.tg - 1) / p.tg);
    const unsigned grid = (unsigned)(tasks < ctx->sm_count ? tasks : ctx->sm_count); // no CTA waits for another
    onepass::onepass_kernel<<<grid, onepass::kThreads, onepass::smem_bytes(p.N, p.aps, p.n_st, p.tg), st>>>(tm_tile, tm_keys, tm_row, tm_piv, tm_pair, p);
    return DART_OK;
}


// The resident sweep applies when a sample's rows fit the chip: at most 8 pivots and, per CTA, no more octets of one
// sample than the exchange warp has lane groups and tensor memory has slots.
bool resident_applies(const dart_ctx *ctx, int n_vis, int P)
{
    namespace R = dart::resident;
    if (!ctx->resident_ok || P > R::kMaxP) return false;
    const int n_oct = (n_vis + R::kOctRows - 1) / R::kOctRows;
    const int per_cta = (n_oct + ctx->sm_count - 1) / ctx->sm_count;
    return per_cta <= R::kMaxOctPerSample && per_cta <= R::tmem_slots(ctx->desc.d);
}

// Steps 1-3 from one read of the keys (csrc/dart_resident.cuh), then steps 4-5.
int launch_resident(dart_ctx *ctx, int B, const void *hidden, const void *keys_in, const int64_t *pos_in, int vis_offset,
                    int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o,
                    const dart_debug *dbg, cudaStream_t st, dart::TileSplit split = dart::TileSplit{1, 0})
{
    namespace R = dart::resident;
    R::Params p = {};
    p.split = split;
    p.B = B, p.S = ctx->S, p.vis_offset = vis_offset, p.n_vis = n_vis, p.P = P, p.d = ctx->desc.d;
    p.n_oct = (n_vis + R::kOctRows - 1) / R::kOctRows;
    p.n_slots = R::tmem_slots(ctx->desc.d), p.n_landing = ctx->res_landing;
    p.norm_kind = o.norm_kind, p.smallest = o.pivot_smallest, p.withhold = o.test_withhold_pivots;
    p.wait_ns = o.wait_limit > 0 ? (unsigned long long)o.wait_limit * 1000ull : 2000000000ull;
    p.keys = (const char *)(keys_in ? keys_in : hidden);
    p.sim = ctx->sim, p.l1 = ctx->l1, p.ssq = ctx->ssq, p.pivot_idx = ctx->pivot_idx;
    p.cand = ctx->res_cand, p.arrived = ctx->counters, p.status = ctx->status;
    DART_CUDA(ctx, cudaMemsetAsync(ctx->counters, 0, (size_t)B * sizeof(int), st));
    {
        Prof pr(ctx, st, SLOT_RESIDENT);
        void *args[1] = {&p};
        // every CTA waits for all others (the candidates of a sample come from all of them): co-residency is required
        DART_CUDA(ctx, cudaLaunchCooperativeKernel((const void *)R::resident_kernel, dim3((unsigned)ctx->sm_count), dim3(R::kThreads),
                                                   args, R::smem_bytes(ctx->desc.d, ctx->sm_count, p.n_landing), st));
    }
    if (split.k > 1) { // the tiles that did not stay on the chip: their norms and similarities from a second read
        int rc = launch_onepass_kernel(ctx, B, p.keys, true, vis_offset, n_vis, P, o, st, split);
        if (rc != DART_OK) return rc;
    }
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

bool pair_applies(const dart_ctx *ctx, int P) { return ctx->pair_ok && P <= dart::pair::kMaxP; }

// Steps 1-3 by the paired sweeps (csrc/dart_pair.cuh), then steps 4-5.
int launch_pair(dart_ctx *ctx, int B, const void *hidden, const void *keys_in, const int64_t *pos_in, int vis_offset, int n_vis,
                int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o, const dart_debug *dbg,
                cudaStream_t st)
{
    namespace Q = dart::pair;
    const void *keys = keys_in ? keys_in : hidden;
    Q::Params p = {};
    p.B = B, p.S = ctx->S, p.vis_offset = vis_offset, p.n_vis = n_vis, p.P = P, p.d = ctx->desc.d;
    p.n_atoms = ctx->n_atoms, p.T1 = (n_vis + Q::kBlockRows - 1) / Q::kBlockRows;
    p.row_bytes = (uint32_t)ctx->desc.d * 2, p.stage1_bytes = Q::stage1_bytes(p.row_bytes);
    p.stage2_bytes = Q::stage2_bytes(P), p.stage3_bytes = Q::stage3_bytes(P);
    Q::ring_depths(P, p.row_bytes, ctx->sm_count, ctx->max_smem_optin, p.n1, p.n2, p.n3, (o.tune >> 8) & 15, (o.tune >> 4) & 15, o.tune & 15);
    if (p.n1 < 2) Q::ring_depths(P, p.row_bytes, ctx->sm_count, ctx->max_smem_optin, p.n1, p.n2, p.n3, 0, 2, 2); // wide rows: the shallowest rings
    if (p.n1 < 2) return DART_ERR_UNSUPPORTED;
    if ((long long)B * p.T1 >= (1ll << 30)) return DART_ERR_UNSUPPORTED;
    p.lead = o.sweep_lag; // tuning: how far the first sweep may run ahead of the second, in samples
    p.norm_kind = o.norm_kind, p.smallest = o.pivot_smallest, p.withhold = o.test_withhold_pivots;
    p.wait_ns = o.wait_limit > 0 ? (unsigned long long)o.wait_limit * 1000ull : 2000000000ull;
    p.keys = (const char *)keys;
    p.sim = ctx->sim, p.l1 = ctx->l1, p.ssq = ctx->ssq, p.pivot_idx = ctx->pivot_idx;
    p.cand = ctx->pair_cand, p.arrived = ctx->counters, p.res_ready = ctx->counters + B, p.res = ctx->pair_res, p.status = ctx->status;
    CUtensorMap tm_blk;
    int rc = encode_2d(ctx, &tm_blk, keys, (uint64_t)ctx->desc.d, (uint64_t)B * ctx->S, Q::kBlockRows);
    if (rc != DART_OK) return rc;
    DART_CUDA(ctx, cudaMemsetAsync(ctx->counters, 0, (size_t)B * 2 * sizeof(int), st));
    {
        Prof pr(ctx, st, SLOT_PAIR);
        const long long blocks = (long long)B * p.T1;
        const unsigned grid = (unsigned)(blocks < ctx->sm_count ? blocks : ctx->sm_count);
        void *args[2] = {&tm_blk, &p};
        // every CTA waits for the lists of all others: co-residency is required
        DART_CUDA(ctx, cudaLaunchCooperativeKernel((const void *)Q::pair_kernel, dim3(grid), dim3(Q::kThreads), args,
                                                   Q::smem_bytes(P, p.row_bytes, (int)grid, p.n1, p.n2, p.n3), st));
    }
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

// The caller's pivots: scores and similarities from one read of the keys, then steps 4-5.
int launch_onepass(dart_ctx *ctx, int B, const void *hidden, const void *keys_in, const int64_t *pos_in, int vis_offset,
                   int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o,
                   const dart_debug *dbg, cudaStream_t st)
{
    launch_pivots_given(ctx, B, vis_offset, n_vis, P, o, st);
    int rc = launch_onepass_kernel(ctx, B, keys_in ? keys_in : hidden, false, vis_offset, n_vis, P, o, st);
    if (rc != DART_OK) return rc;
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

// Two plain passes: the rows of `keys` are read once for the scores that rank the pivots, the rows of `sim_src` once for
// their norms and the similarities (one pass when the tensor-core kernels apply, else the plain kernels: norms, then
// similarities).  sim_src = hidden is dart_opts.cosine_on_hidden; sim_src = keys is the main method without the
// persistent sweep: no launch waits inside for another CTA, which is what small batches want.
int launch_two_pass(dart_ctx *ctx, int B, const void *hidden, const void *keys, const void *sim_src, const int64_t *pos_in,
                    int vis_offset, int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos,
                    const dart_opts &o, const dart_debug *dbg, bool tensor_cores, cudaStream_t st)
{
    using namespace dart;
    const int S = ctx->S, d8 = ctx->desc.d / 8;
    const long long rows = (long long)B * n_vis;
    const unsigned score_grid = (unsigned)((rows + kScoreWarps - 1) / kScoreWarps);
    const bool same = sim_src == keys;
    {
        Prof p(ctx, st, SLOT_SCORE); // the key rows' scores (their sums of squares too when they rank the pivots)
        score_kernel<<<score_grid, kScoreWarps * 32, 0, st>>>((const uint4 *)keys, S, d8, vis_offset, n_vis, rows, ctx->l1,
                                                             (same && (o.norm_kind == 2 || !tensor_cores)) ? ctx->ssq : nullptr);
    }
    if (o.pivots_in) {
        launch_pivots_given(ctx, B, vis_offset, n_vis, P, o, st);
    } else {
        Prof p(ctx, st, SLOT_PIVOT);
        const int P_pad = next_pow2(P);
        const bool cached = n_vis <= kPivotCacheMax;
        pivot_kernel<<<B, kSelectThreads, pivot_smem_bytes(n_vis, P_pad, cached), st>>>(o.norm_kind == 2 ? ctx->ssq : ctx->l1, n_vis, P, P_pad,
                                                                                       o.pivot_smallest, cached, ctx->pivot_idx);
    }
    if (tensor_cores) {
        int rc = launch_onepass_kernel(ctx, B, sim_src, true, vis_offset, n_vis, P, o, st);
        if (rc != DART_OK) return rc;
    } else {
        if (!same) {
            Prof p(ctx, st, SLOT_SCORE); // sums of squares of the hidden rows only
            score_kernel<<<score_grid, kScoreWarps * 32, 0, st>>>((const uint4 *)sim_src, S, d8, vis_offset, n_vis, rows, nullptr,
                                                                 ctx->ssq);
        }
        Prof p(ctx, st, SLOT_SIM);
        const size_t smem = (size_t)kSimPivotChunk * d8 * 16;
        const dim3 grid((n_vis + kSimRowsPerCta - 1) / kSimRowsPerCta, B);
        for (int p0 = 0; p0 < P; p0 += kSimPivotChunk)
            sim_alu_kernel<<<grid, kSimWarps * 32, smem, st>>>((const uint4 *)sim_src, S, d8, vis_offset, n_vis, P, p0,
                                                              ctx->pivot_idx, ctx->ssq, ctx->sim);
        ctx->launches += (P - 1) / kSimPivotChunk;
    }
    launch_retention(ctx, B, pos_in, vis_offset, n_vis, P, n_keep, out_idx, out_pos, o, st);
    launch_gather(ctx, B, hidden, n_vis, n_keep, out_idx, out_hidden, o, st);
    DART_CUDA(ctx, cudaGetLastError());
    return copy_debug(ctx, B, n_vis, P, dbg, st);
}

int launch_reduce(dart_ctx *ctx, int B, const void *hidden, const void *keys, const int64_t *pos_in, int vis_offset,
                  int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o,
                  const dart_debug *dbg, cudaStream_t st);

// Step 2 from another source than the vision tokens' scores (dart_opts.pivot_source): the pivots are written to the
// workspace by a kernel of their own and the call goes on as if the caller had named them.
int launch_with_pivot_source(dart_ctx *ctx, int B, const void *hidden, const void *keys, const int64_t *pos_in, int vis_offset,
                             int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos,
                             const dart_opts &o, const dart_debug *dbg, cudaStream_t st)
{
    using namespace dart;
    const int S = ctx->S, d8 = ctx->desc.d / 8, P_pad = next_pow2(P);
    const uint4 *k = (const uint4 *)(keys ? keys : hidden);
    dart_opts o2 = o;
    o2.pivot_source = 0, o2.pivots_in = ctx->pivot_src;
    if (o.pivot_source == DART_PIVOTS_RANDOM) {
        Prof p(ctx, st, SLOT_PIVOT);
        pivot_random_kernel<<<B, kSelectThreads, (size_t)P_pad * 8, st>>>(o.seed, o.sample_base, n_vis, P, P_pad, ctx->pivot_src);
    } else { // both modalities: the scores of the vision rows and of the text rows before and after them
        const int Pt = o.n_text_pivots, n_after = S - vis_offset - n_vis;
        const size_t half = (size_t)ctx->desc.B_max * ctx->desc.S_max;
        float *tb = ctx->text_score, *ta = ctx->text_score + (size_t)B * vis_offset; // L1 scores; the sums of squares lie `half` further
        {
            Prof p(ctx, st, SLOT_SCORE);
            const long long rows = (long long)B * n_vis;
            score_kernel<<<(unsigned)((rows + kScoreWarps - 1) / kScoreWarps), kScoreWarps * 32, 0, st>>>(k, S, d8, vis_offset, n_vis, rows,
                                                                                                        ctx->l1, ctx->ssq);
            ++ctx->launches;
            if (vis_offset > 0) {
                const long long r = (long long)B * vis_offset;
                score_kernel<<<(unsigned)((r + kScoreWarps - 1) / kScoreWarps), kScoreWarps * 32, 0, st>>>(k, S, d8, 0, vis_offset, r, tb, tb + half);
            }
            if (n_after > 0) {
                const long long r = (long long)B * n_after;
                score_kernel<<<(unsigned)((r + kScoreWarps - 1) / kScoreWarps), kScoreWarps * 32, 0, st>>>(k, S, d8, vis_offset + n_vis, n_after, r,
                                                                                                      ta, ta + half);
            }
        }
        Prof p(ctx, st, SLOT_PIVOT);
        const size_t shift = o.norm_kind == 2 ? half : 0; // which of the two scores ranks the pivots
        pivot_mixed_kernel<<<B, kSelectThreads, (size_t)P_pad * 8, st>>>((o.norm_kind == 2 ? ctx->ssq : ctx->l1), tb + shift, ta + shift, S,
                                                                        vis_offset, n_vis, P - Pt, Pt, P_pad, o.pivot_smallest, ctx->pivot_src);
        o2.text_pivots = 1;
    }
    DART_CUDA(ctx, cudaGetLastError());
    return launch_reduce(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o2, dbg, st);
}

int launch_reduce(dart_ctx *ctx, int B, const void *hidden, const void *keys, const int64_t *pos_in, int vis_offset,
                  int n_vis, int P, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, const dart_opts &o,
                  const dart_debug *dbg, cudaStream_t st)
{
    if (o.pivot_source != DART_PIVOTS_BY_SCORE)
        return launch_with_pivot_source(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg, st);
    const bool fused = o.path == DART_PATH_FUSED || (o.path == DART_PATH_AUTO && fused_applies(ctx, P));
    if (fused && !fused_applies(ctx, P)) return DART_ERR_UNSUPPORTED;
    if (o.path == DART_PATH_RESIDENT || o.path == DART_PATH_SPLIT) {
        if (!resident_applies(ctx, n_vis, P) || o.pivots_in || (o.cosine_on_hidden && keys && keys != hidden))
            return DART_ERR_UNSUPPORTED;
        dart::TileSplit split{1, 0};
        if (o.path == DART_PATH_SPLIT) {
            const int k = o.resident_split == 0 ? 2 : (o.resident_split < 0 ? -o.resident_split : o.resident_split);
            if (k < 2 || k > 64) return DART_ERR_UNSUPPORTED;
            split = dart::TileSplit{k, o.resident_split < 0 ? 1 : 0};
        }
        return launch_resident(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg, st,
                               split);
    }
    if (o.path == DART_PATH_PAIRED) {
        if (!pair_applies(ctx, P) || o.pivots_in || (o.cosine_on_hidden && keys && keys != hidden)) return DART_ERR_UNSUPPORTED;
        return launch_pair(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg, st);
    }
    if (o.cosine_on_hidden && keys && keys != hidden)
        return launch_two_pass(ctx, B, hidden, keys, hidden, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o,
                               dbg, fused, st);
    // AUTO takes the resident sweep for up to four samples: nothing has to be hidden behind other samples there, and
    // rows that stay on the chip save the second read and most of the sweep's waits (measured, 576 tokens: one
    // sample 80 us against 103 us, four samples 96 against 107, eight samples 118 against 113).
    if (o.path == DART_PATH_AUTO && B <= 4 && resident_applies(ctx, n_vis, P) && !o.pivots_in)
        return launch_resident(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg, st);
    // AUTO prefers the three launches below to the persistent sweep in two cases.  (1) Samples with more vision tokens
    // than the sweep's shared-memory score buffer holds: it then selects from global memory and stalls (measured at
    // 4608 tokens, batch 4: 253 us against 111 us).  (2) 32 pivots or more: the sweep fetches pivot tiles four rows per
    // TMA op, the one-pass kernel as one box from a compact copy (batch 256: 32 pivots 2.83 -> 2.71 ms, 128 pivots
    // 6.15 -> 4.65 ms; below that the two are within 1 % of each other at batch 256).  (3) Between half a 128-row tile
    // and two tiles per SM: the persistent sweep has nothing to overlap a sample's pivot dependency with (measured, us per
    // step: 8 samples of 2880 tokens 178 -> 165, 12 samples 218 -> 201, 16 samples of 576 tokens 115 -> 104; with fewer
    // tiles still, the two extra launches cost more: 8 samples of 576 tokens 84 -> 95).
    const long long row_tiles = (long long)B * ((n_vis + dart::sweep::kTileRows - 1) / dart::sweep::kTileRows);
    const bool two_pass = o.path == DART_PATH_TWO_PASS ||
                          (o.path == DART_PATH_AUTO && fused_applies(ctx, P) && !o.pivots_in &&
                           (n_vis > dart::sweep::kSelMax || (P >= 32 && ctx->piv_rows) ||
                            (2 * row_tiles >= ctx->sm_count && row_tiles < 2ll * ctx->sm_count)));
    if (two_pass) {
        if (!fused_applies(ctx, P)) return DART_ERR_UNSUPPORTED;
        const void *k = keys ? keys : hidden;
        return launch_two_pass(ctx, B, hidden, k, k, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg,
                               true, st);
    }
    if (fused && o.pivots_in) // nothing waits for a selection: one pass over the keys
        return launch_onepass(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos, o, dbg, st);
    return fused ? launch_fused(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos,
                                o, dbg, st)
                 : launch_staged(ctx, B, hidden, keys, pos_in, vis_offset, n_vis, P, n_keep, out_hidden, out_idx, out_pos,
                                 o, dbg, st);
}

// Reads the device status word, keeps its detail and clears it.  The caller has synchronised the work that may write it.
int read_status(dart_ctx *ctx)
{
    int word[12] = {0};
    DART_CUDA(ctx, cudaMemcpy(word, ctx->status, sizeof word, cudaMemcpyDeviceToHost));
    if (word[0] != 0) {
        for (int k = 0; k < 11; ++k) ctx->status_detail[k] = word[k + 1];
        DART_CUDA(ctx, cudaMemset(ctx->status, 0, sizeof word));
    }
    return word[0];
}

} // namespace

extern "C" {

int dart_create(dart_ctx **out, const dart_desc *desc)
{
    if (!out || !desc) return DART_ERR_NULL;
    *out = nullptr;
    if (desc->B_max < 1 || desc->S_max < 1 || desc->d < 8 || desc->d % 8 != 0 || desc->P_max < 1 ||
        desc->P_max > desc->Kp_max || desc->Kp_max > desc->S_max || desc->P_max > 1024)
        return DART_ERR_BAD_SHAPE;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || desc->device < 0 || desc->device >= ndev) return DART_ERR_CUDA;
    dart_ctx *ctx = new (std::nothrow) dart_ctx();
    if (!ctx) return DART_ERR_NOMEM;
    ctx->desc = *desc;
    ctx->B = desc->B_max;
    ctx->S = desc->S_max;
    DeviceGuard g(desc->device);
    if (!g.ok) {
        delete ctx;
        return DART_ERR_CUDA;
    }
    const size_t nv = (size_t)desc->B_max * desc->S_max, np = (size_t)desc->B_max * desc->P_max;
    int rc = DART_OK;
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->l1, nv);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->ssq, nv);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->sim, np * desc->S_max);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->eps, np);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->pivot_idx, np);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->owner, nv);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->keep, nv);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->len, (size_t)desc->B_max);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->pivot_src, np);
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->text_score, 2 * nv);
    if (rc == DART_OK) {
        // candidate lists of the two-phase retention: at most kCandMax entries per pivot; contexts whose maxima
        // would need more than 1 GiB go without (they use the one-kernel retention)
        ctx->cand_stride = desc->Kp_max < dart::kCandMax ? desc->Kp_max : dart::kCandMax;
        const size_t entries = np * (size_t)ctx->cand_stride;
        if (entries * sizeof(int32_t) <= ((size_t)1 << 30)) rc = ws_alloc(ctx, &ctx->cand, entries);
    }
    if (rc == DART_OK) {
        // candidate bands of the band retention; contexts whose maxima would need more than 1 GiB go without
        ctx->band_stride = dart::band_stride(desc->Kp_max);
        const size_t entries = np * (size_t)ctx->band_stride;
        if (entries * sizeof(unsigned long long) <= ((size_t)1 << 30)) {
            rc = ws_alloc(ctx, &ctx->band, entries);
            if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->band_n, np);
        }
    }
    if (rc == DART_OK && desc->P_max > dart::onepass::kGatherMaxP) {
        // compact pivot rows for the one-pass kernel; contexts that would need more than 2 GiB go without (gather4 then)
        const size_t bytes = (size_t)desc->B_max * ((desc->P_max + 15) / 16 * 16) * desc->d * 2;
        if (bytes <= ((size_t)2 << 30)) rc = ws_alloc(ctx, (uint8_t **)&ctx->piv_rows, bytes);
    }
    if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->status, 64);
    if (rc == DART_OK && cudaMemset(ctx->status, 0, 256) != cudaSuccess) rc = DART_ERR_CUDA;
    if (rc == DART_OK) {
        cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, desc->device);
        size_t sim_smem = (size_t)dart::kSimPivotChunk * (desc->d / 8) * 16;
        if (sim_smem > (size_t)ctx->max_smem_optin ||
            (size_t)desc->S_max + 16 + dart::kRetainCacheBytes > (size_t)ctx->max_smem_optin)
            rc = DART_ERR_BAD_SHAPE; // rows wider than 8 pivot rows of shared memory are not supported
        else if (cudaFuncSetAttribute(dart::sim_alu_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sim_smem) != cudaSuccess ||
                 cudaFuncSetAttribute(dart::retain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      desc->S_max + 16 + dart::kRetainCacheBytes) != cudaSuccess)
            rc = DART_ERR_CUDA;
    }
    if (rc == DART_OK && (cudaFuncSetAttribute(dart::retain_global_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               ctx->max_smem_optin - 2048) != cudaSuccess ||
                          cudaFuncSetAttribute(dart::retain_union_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               ctx->max_smem_optin - 2048) != cudaSuccess ||
                          cudaFuncSetAttribute(dart::pack_varlen_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               ctx->max_smem_optin - 2048) != cudaSuccess))
        rc = DART_ERR_CUDA;
    if (rc == DART_OK && cudaFuncSetAttribute(dart::pivot_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)dart::pivot_smem_bytes(dart::kPivotCacheMax, 1024, true)) != cudaSuccess)
        rc = DART_ERR_CUDA;
    if (rc == DART_OK && ctx->cand) {
        // the two-phase kernels may use up to the device's shared memory; shapes that need more fall back at launch
        if (cudaFuncSetAttribute(dart::candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - 2048) != cudaSuccess ||
            cudaFuncSetAttribute(dart::retain_walk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - 2048) != cudaSuccess)
            rc = DART_ERR_CUDA;
    }
    if (rc == DART_OK && ctx->band) {
        if (cudaFuncSetAttribute(dart::band_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - 2048) != cudaSuccess ||
            cudaFuncSetAttribute(dart::retain_pick_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - 2048) != cudaSuccess ||
            cudaFuncSetAttribute(dart::retain_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ctx->max_smem_optin - 2048) != cudaSuccess)
            rc = DART_ERR_CUDA;
    }
    if (rc == DART_OK) rc = fused_setup(ctx);
    if (rc == DART_OK && (desc->flags & DART_FLAG_HOST_STAGING)) {
        // chunk = as many samples as fit ~512 MiB of input staging per buffer set (at least one)
        const size_t per_sample = (size_t)desc->S_max * desc->d * 2;
        size_t c = ((size_t)512 << 20) / (2 * per_sample);
        ctx->chunk = (int)(c < 1 ? 1 : (c > (size_t)desc->B_max ? (size_t)desc->B_max : c));
        for (int k = 0; k < 2 && rc == DART_OK; ++k) {
            if (rc == DART_OK) rc = ws_alloc(ctx, (uint8_t **)&ctx->st_hidden[k], ctx->chunk * per_sample);
            if (rc == DART_OK) rc = ws_alloc(ctx, (uint8_t **)&ctx->st_keys[k], ctx->chunk * per_sample);
            if (rc == DART_OK) rc = ws_alloc(ctx, (uint8_t **)&ctx->st_out_hidden[k], ctx->chunk * per_sample);
            if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->st_out_idx[k], (size_t)ctx->chunk * desc->S_max);
            if (rc == DART_OK) rc = ws_alloc(ctx, &ctx->st_out_pos[k], (size_t)ctx->chunk * desc->S_max);
            if (rc == DART_OK && (cudaEventCreateWithFlags(&ctx->ev_in[k], cudaEventDisableTiming) != cudaSuccess ||
                                  cudaEventCreateWithFlags(&ctx->ev_run[k], cudaEventDisableTiming) != cudaSuccess ||
                                  cudaEventCreateWithFlags(&ctx->ev_out[k], cudaEventDisableTiming) != cudaSuccess))
                rc = DART_ERR_CUDA;
        }
        if (rc == DART_OK && (cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking) != cudaSuccess ||
                              cudaStreamCreateWithFlags(&ctx->s_run, cudaStreamNonBlocking) != cudaSuccess ||
                              cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking) != cudaSuccess))
            rc = DART_ERR_CUDA;
    }
    if (rc != DART_OK) {
        dart_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return DART_OK;
}

int dart_destroy(dart_ctx *ctx)
{
    if (!ctx) return DART_OK;
    DeviceGuard g(ctx->desc.device);
    cudaDeviceSynchronize();
    for (auto &e : ctx->pending) ctx->spare.push_back(e);
    for (auto &e : ctx->spare) {
        cudaEventDestroy(e.start);
        cudaEventDestroy(e.stop);
    }
    cudaFree(ctx->l1);
    cudaFree(ctx->ssq);
    cudaFree(ctx->sim);
    cudaFree(ctx->eps);
    cudaFree(ctx->pivot_idx);
    cudaFree(ctx->owner);
    cudaFree(ctx->keep);
    cudaFree(ctx->len);
    cudaFree(ctx->pivot_src);
    cudaFree(ctx->text_score);
    cudaFree(ctx->cand);
    cudaFree(ctx->piv_rows);
    cudaFree(ctx->status);
    cudaFree(ctx->counters);
    cudaFree(ctx->sim_share);
    cudaFree(ctx->res_cand);
    cudaFree(ctx->pair_cand);
    cudaFree(ctx->pair_res);
    for (int k = 0; k < 2; ++k) {
        cudaFree(ctx->st_hidden[k]);
        cudaFree(ctx->st_keys[k]);
        cudaFree(ctx->st_out_hidden[k]);
        cudaFree(ctx->st_out_idx[k]);
        cudaFree(ctx->st_out_pos[k]);
        if (ctx->ev_in[k]) cudaEventDestroy(ctx->ev_in[k]);
        if (ctx->ev_run[k]) cudaEventDestroy(ctx->ev_run[k]);
        if (ctx->ev_out[k]) cudaEventDestroy(ctx->ev_out[k]);
    }
    if (ctx->s_h2d) cudaStreamDestroy(ctx->s_h2d);
    if (ctx->s_run) cudaStreamDestroy(ctx->s_run);
    if (ctx->s_d2h) cudaStreamDestroy(ctx->s_d2h);
    delete ctx;
    return DART_OK;
}

int dart_set_shape(dart_ctx *ctx, int B, int S)
{
    if (!ctx) return DART_ERR_NULL;
    if (B < 1 || S < 1 || B > ctx->desc.B_max || S > ctx->desc.S_max) return DART_ERR_BAD_SHAPE;
    ctx->B = B;
    ctx->S = S;
    return DART_OK;
}

int dart_reduce_ex(dart_ctx *ctx, const void *hidden, const void *keys, const int64_t *pos_in, int vis_offset,
                   int n_vis, int n_pivot, int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos,
                   const dart_opts *opts, const dart_debug *dbg, void *stream)
{
    int rc = check_call(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos);
    if (rc != DART_OK) return rc;
    dart_opts o = {};
    if (opts) o = *opts;
    if (o.norm_kind == 0) o.norm_kind = 1;
    if (o.norm_kind != 1 && o.norm_kind != 2) return DART_ERR_UNSUPPORTED;
    if (o.path != DART_PATH_AUTO && o.path != DART_PATH_STAGED && o.path != DART_PATH_FUSED && o.path != DART_PATH_TWO_PASS &&
        o.path != DART_PATH_RESIDENT && o.path != DART_PATH_SPLIT && o.path != DART_PATH_PAIRED)
        return DART_ERR_UNSUPPORTED;
    if (o.rule != DART_RULE_QUOTAS && o.rule != DART_RULE_GLOBAL && o.rule != DART_RULE_UNION) return DART_ERR_UNSUPPORTED;
    if (o.rule == DART_RULE_UNION) {
        if (!o.cu_seqlens) return DART_ERR_NULL;
        if ((uintptr_t)o.cu_seqlens & 3u) return DART_ERR_ALIGN;
        if (dart::retain_union_smem_bytes(n_vis) > (size_t)ctx->max_smem_optin - 2048) return DART_ERR_UNSUPPORTED;
    }
    if (o.cosine_on_hidden && o.norm_kind != 1) return DART_ERR_UNSUPPORTED; // the hidden rows' sums of squares take the slot
    if ((uintptr_t)o.pivots_in & 3u) return DART_ERR_ALIGN;
    if (o.pivot_source != DART_PIVOTS_BY_SCORE && o.pivot_source != DART_PIVOTS_MIXED && o.pivot_source != DART_PIVOTS_RANDOM)
        return DART_ERR_UNSUPPORTED;
    if (o.pivot_source != DART_PIVOTS_BY_SCORE) {
        // the pivots then reach steps 3-5 like the caller's: only the paths that take those
        if (o.pivots_in) return DART_ERR_UNSUPPORTED;
        if (o.path == DART_PATH_RESIDENT || o.path == DART_PATH_SPLIT || o.path == DART_PATH_PAIRED) return DART_ERR_UNSUPPORTED;
        if (o.pivot_source == DART_PIVOTS_MIXED &&
            (o.n_text_pivots < 0 || o.n_text_pivots > n_pivot || o.n_text_pivots > ctx->S - n_vis || n_pivot - o.n_text_pivots > n_vis))
            return DART_ERR_BAD_SHAPE;
        if (o.sample_base < 0) return DART_ERR_BAD_SHAPE;
    }
    if (o.text_pivots && !o.pivots_in) return DART_ERR_UNSUPPORTED;
    if (o.rule == DART_RULE_GLOBAL &&
        dart::retain_global_smem_bytes(n_vis) > (size_t)ctx->max_smem_optin - 2048)
        return DART_ERR_UNSUPPORTED; // the sample's duplication values must fit shared memory
    if (o.retention != DART_RETAIN_AUTO && o.retention != DART_RETAIN_SERIAL && o.retention != DART_RETAIN_LISTS &&
        o.retention != DART_RETAIN_BANDS && o.retention != DART_RETAIN_FUSED)
        return DART_ERR_UNSUPPORTED;
    if ((uintptr_t)pos_in & 7u) return DART_ERR_ALIGN;
    DeviceGuard g(ctx->desc.device);
    if (!g.ok) return DART_ERR_CUDA;
    return launch_reduce(ctx, ctx->B, hidden, keys, pos_in, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx,
                         out_pos, o, dbg, (cudaStream_t)stream);
}

int dart_reduce(dart_ctx *ctx, const void *hidden, const void *keys, int vis_offset, int n_vis, int n_pivot,
                int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos, void *stream)
{
    return dart_reduce_ex(ctx, hidden, keys, nullptr, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos,
                          nullptr, nullptr, stream);
}

int dart_reduce_host(dart_ctx *ctx, const void *hidden, const void *keys, int vis_offset, int n_vis, int n_pivot,
                     int n_keep, void *out_hidden, int32_t *out_idx, int64_t *out_pos)
{
    int rc = check_call(ctx, hidden, keys, vis_offset, n_vis, n_pivot, n_keep, out_hidden, out_idx, out_pos, true);
    if (rc != DART_OK) return rc;
    if (!(ctx->desc.flags & DART_FLAG_HOST_STAGING)) return DART_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->desc.device);
    if (!g.ok) return DART_ERR_CUDA;
    const int B = ctx->B, S = ctx->S, d = ctx->desc.d, S_out = S - n_vis + n_keep;
    const size_t in_row = (size_t)S * d * 2, out_row = (size_t)S_out * d * 2;
    dart_opts o = {};
    o.norm_kind = 1;
    int n_chunks = (B + ctx->chunk - 1) / ctx->chunk;
    // three streams: copy-in of chunk c+1 and copy-out of chunk c-1 overlap the reduction of chunk c
    for (int c = 0; c < n_chunks; ++c) {
        const int k = c & 1, b0 = c * ctx->chunk, nb = (B - b0 < ctx->chunk) ? B - b0 : ctx->chunk;
        if (c >= 2) { // buffer set k is free once chunk c-2 has been reduced and copied out
            DART_CUDA(ctx, cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_run[k], 0));
            DART_CUDA(ctx, cudaStreamWaitEvent(ctx->s_run, ctx->ev_out[k], 0));
        }
        DART_CUDA(ctx, cudaMemcpyAsync(ctx->st_hidden[k], (const char *)hidden + b0 * in_row, nb * in_row,
                                       cudaMemcpyHostToDevice, ctx->s_h2d));
        if (keys)
            DART_CUDA(ctx, cudaMemcpyAsync(ctx->st_keys[k], (const char *)keys + b0 * in_row, nb * in_row,
                                           cudaMemcpyHostToDevice, ctx->s_h2d));
        DART_CUDA(ctx, cudaEventRecord(ctx->ev_in[k], ctx->s_h2d));
        DART_CUDA(ctx, cudaStreamWaitEvent(ctx->s_run, ctx->ev_in[k], 0));
        rc = launch_reduce(ctx, nb, ctx->st_hidden[k], keys ? ctx->st_keys[k] : nullptr, nullptr, vis_offset, n_vis,
                           n_pivot, n_keep, ctx->st_out_hidden[k], ctx->st_out_idx[k], ctx->st_out_pos[k], o, nullptr,
                           ctx->s_run);
        if (rc != DART_OK) break;
        DART_CUDA(ctx, cudaEventRecord(ctx->ev_run[k], ctx->s_run));
        DART_CUDA(ctx, cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_run[k], 0));
        DART_CUDA(ctx, cudaMemcpyAsync((char *)out_hidden + b0 * out_row, ctx->st_out_hidden[k], nb * out_row,
                                       cudaMemcpyDeviceToHost, ctx->s_d2h));
        DART_CUDA(ctx, cudaMemcpyAsync(out_idx + (size_t)b0 * S_out, ctx->st_out_idx[k], (size_t)nb * S_out * 4,
                                       cudaMemcpyDeviceToHost, ctx->s_d2h));
        DART_CUDA(ctx, cudaMemcpyAsync(out_pos + (size_t)b0 * S_out, ctx->st_out_pos[k], (size_t)nb * S_out * 8,
                                       cudaMemcpyDeviceToHost, ctx->s_d2h));
        DART_CUDA(ctx, cudaEventRecord(ctx->ev_out[k], ctx->s_d2h));
    }
    cudaError_t e1 = cudaStreamSynchronize(ctx->s_h2d), e2 = cudaStreamSynchronize(ctx->s_run),
                e3 = cudaStreamSynchronize(ctx->s_d2h);
    if (rc != DART_OK) return rc;
    DART_CUDA(ctx, e1);
    DART_CUDA(ctx, e2);
    DART_CUDA(ctx, e3);
    // everything has completed: a bounded wait that gave up or a failed self-check made the later kernels skip
    // their writes, so the host buffers must not be handed back with a success code
    return read_status(ctx);
}

int dart_status(dart_ctx *ctx)
{
    if (!ctx) return DART_ERR_NULL;
    DeviceGuard g(ctx->desc.device);
    if (!g.ok) return DART_ERR_CUDA;
    DART_CUDA(ctx, cudaDeviceSynchronize());
    return read_status(ctx);
}

int dart_status_detail(const dart_ctx *ctx, int32_t detail[11])
{
    if (!ctx || !detail) return DART_ERR_NULL;
    for (int k = 0; k < 11; ++k) detail[k] = ctx->status_detail[k];
    return DART_OK;
}

int dart_last_cuda_error(const dart_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }
size_t dart_workspace_bytes(const dart_ctx *ctx) { return ctx ? ctx->bytes : 0; }
int64_t dart_launch_count(const dart_ctx *ctx) { return ctx ? ctx->launches : 0; }

int dart_profile_enable(dart_ctx *ctx, int on)
{
    if (!ctx) return DART_ERR_NULL;
    ctx->profiling = on != 0;
    return DART_OK;
}

int dart_profile_read(dart_ctx *ctx, float *ms, int32_t *launches, const char **names, int *n_slots)
{
    if (!ctx || !ms || !launches || !n_slots) return DART_ERR_NULL;
    DeviceGuard g(ctx->desc.device);
    if (!g.ok) return DART_ERR_CUDA;
    for (auto &e : ctx->pending) {
        float t = 0.f;
        DART_CUDA(ctx, cudaEventSynchronize(e.stop));
        DART_CUDA(ctx, cudaEventElapsedTime(&t, e.start, e.stop));
        ctx->slot_ms[e.slot] += t;
        ctx->slot_launches[e.slot] += 1;
        ctx->spare.push_back(e);
    }
    ctx->pending.clear();
    int n = *n_slots < SLOT_COUNT ? *n_slots : SLOT_COUNT;
    for (int k = 0; k < n; ++k) {
        ms[k] = ctx->slot_ms[k];
        launches[k] = ctx->slot_launches[k];
        if (names) names[k] = kSlotNames[k];
    }
    for (int k = 0; k < SLOT_COUNT; ++k) {
        ctx->slot_ms[k] = 0.f;
        ctx->slot_launches[k] = 0;
    }
    *n_slots = n;
    return DART_OK;
}

// ---- allocation-free pivot selection ---------------------------------------------------------------
// Scratch of dart_pivots_static: L1 scores in the first half, sums of squares in the second.  The
// name below is only a host-side handle; kernels get the address cudaGetSymbolAddress returns.
static __device__ __align__(256) float g_static_scores[2 * DART_STATIC_MAX_ROWS];

namespace {
constexpr int kMaxDevices = 64;
float *g_static_ptr[kMaxDevices]; // device address of g_static_scores, per device; looked up once
std::mutex g_static_mutex;
} // namespace

int dart_pivots_static(const void *keys, int B, int S, int d, int vis_offset, int n_vis, int n_pivot,
                       int32_t *pivot_idx, int device, void *stream)
{
    if (!keys || !pivot_idx) return DART_ERR_NULL;
    if (B < 1 || S < 1 || d < 8 || d % 8 != 0 || vis_offset < 0 || n_vis < 1 || (long long)vis_offset + n_vis > S)
        return DART_ERR_BAD_SHAPE;
    if (n_pivot < 1 || n_pivot > n_vis || n_pivot > 1024) return DART_ERR_BAD_SHAPE;
    if ((long long)B * n_vis > DART_STATIC_MAX_ROWS) return DART_ERR_BAD_SHAPE; // beyond the fixed scratch
    if (((uintptr_t)keys & 15u) || ((uintptr_t)pivot_idx & 3u)) return DART_ERR_ALIGN;
    if (device < 0 || device >= kMaxDevices) return DART_ERR_CUDA;
    DeviceGuard g(device);
    if (!g.ok) return DART_ERR_CUDA;
    float *scratch;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[device]) { // set-up, once per device, with that device current
            // With lazy module loading this is where the library's image (kernels and this array) is placed in
            // device memory: a device whose memory is already handed out answers cudaErrorMemoryAllocation.
            float *ptr = nullptr;
            const cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_static_scores);
            if (e != cudaSuccess || !ptr) {
                cudaGetLastError(); // not sticky: leave no error behind for the caller's next CUDA call
                return e == cudaErrorMemoryAllocation ? DART_ERR_NOMEM : DART_ERR_CUDA;
            }
            g_static_ptr[device] = ptr;
        }
        scratch = g_static_ptr[device];
    }
    using namespace dart;
    cudaStream_t st = (cudaStream_t)stream;
    const long long rows = (long long)B * n_vis;
    float *l1 = scratch, *ssq = scratch + DART_STATIC_MAX_ROWS;
    score_kernel<<<(unsigned)((rows + kScoreWarps - 1) / kScoreWarps), kScoreWarps * 32, 0, st>>>(
        (const uint4 *)keys, S, d / 8, vis_offset, n_vis, rows, l1, ssq);
    const int P_pad = next_pow2(n_pivot);
    pivot_kernel<<<B, kSelectThreads, pivot_smem_bytes(n_vis, P_pad, false), st>>>(l1, n_vis, n_pivot, P_pad, 0, 0, pivot_idx);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DART_OK : e == cudaErrorMemoryAllocation ? DART_ERR_NOMEM : DART_ERR_CUDA;
}

int dart_gather_rows(const void *src, const int32_t *idx, int B, int S, int S_out, int row_bytes, void *out, int device,
                     void *stream)
{
    if (!src || !idx || !out) return DART_ERR_NULL;
    if (B < 1 || S < 1 || S_out < 1 || row_bytes < 16 || row_bytes % 16 != 0) return DART_ERR_BAD_SHAPE;
    if ((((uintptr_t)src | (uintptr_t)out) & 15u) || ((uintptr_t)idx & 3u)) return DART_ERR_ALIGN;
    if (overlaps(out, (size_t)B * S_out * row_bytes, src, (size_t)B * S * row_bytes)) return DART_ERR_ALIAS;
    DeviceGuard g(device);
    if (!g.ok) return DART_ERR_CUDA;
    using namespace dart;
    const long long orows = (long long)B * S_out;
    const unsigned grid = (unsigned)((orows + kGatherWarps - 1) / kGatherWarps);
    gather_kernel<<<grid, kGatherWarps * 32, 0, (cudaStream_t)stream>>>((const uint4 *)src, idx, S, S_out, row_bytes / 16, orows,
                                                                       nullptr, (uint4 *)out);
    return cudaGetLastError() == cudaSuccess ? DART_OK : DART_ERR_CUDA;
}

const char *dart_strerror(int code)
{
    switch (code) {
    case DART_OK: return "ok";
    case DART_ERR_NULL: return "a required pointer is NULL";
    case DART_ERR_BAD_SHAPE: return "sizes violate the shape rules or exceed the context's maxima";
    case DART_ERR_ALIGN: return "a tensor pointer is not sufficiently aligned";
    case DART_ERR_ALIAS: return "an output overlaps an input";
    case DART_ERR_CUDA: return "a CUDA call failed";
    case DART_ERR_NOMEM: return "out of memory";
    case DART_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case DART_ERR_CHECK: return "a device-side self-check failed";
    case DART_ERR_UNSUPPORTED: return "option not available";
    default: return "unknown error code";
    }
}

int dart_version(void) { return DART_VERSION; }

} // extern "C"
