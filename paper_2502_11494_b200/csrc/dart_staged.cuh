// Staged path: one kernel per step of the reduction (Sec. 3.3 of the paper), every intermediate
// in the context's workspace.  It is the plain realisation of the method and the path that
// materialises the per-step outputs.
#pragma once
#include "dart_common.cuh"

namespace dart {

// ------------------------------------------------------------------------------------------------
// Step 1: scores.  One warp per vision token: l1 = sum |k| (the "K-norm" of the Sec. 3.3 footnote),
// ssq = sum k^2 (the squared Euclidean norm in Eq. 7's denominator).  fp32 accumulation, fixed
// order: each lane sums its column groups in order, then a butterfly over the lanes.
// ------------------------------------------------------------------------------------------------
constexpr int kScoreWarps = 8;

__global__ void __launch_bounds__(kScoreWarps * 32)
score_kernel(const uint4 *__restrict__ keys, int S, int d8, int vis_offset, int n_vis, long long rows_total,
             float *__restrict__ l1, float *__restrict__ ssq)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kScoreWarps + (threadIdx.x >> 5);
    if (row >= rows_total) return;
    const int b = (int)(row / n_vis), j = (int)(row % n_vis);
    const uint4 *src = keys + ((size_t)b * S + vis_offset + j) * (size_t)d8;
    float a = 0.f, q = 0.f;
    for (int c0 = 0; c0 < d8; c0 += 32 * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int c = c0 + u * 32 + lane;
            v[u] = (c < d8) ? ld_stream(src + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                float lo = bf16_lo(w[t]), hi = bf16_hi(w[t]);
                a += fabsf(lo);
                a += fabsf(hi);
                q = fmaf(lo, lo, q);
                q = fmaf(hi, hi, q);
            }
        }
    }
    a = warp_sum(a);
    q = warp_sum(q);
    if (lane == 0) { // either output may be NULL (not wanted)
        if (l1) l1[row] = a;
        if (ssq) ssq[row] = q;
    }
}

// ------------------------------------------------------------------------------------------------
// Step 2: pivots (Def. 1; maximum K-norm per the caption of Table 1).  One CTA per sample: radix
// select of the P best scores, then a bitonic sort of the P (key, index) pairs into rank order.
// Dynamic shared memory: P_pad * 8 bytes, P_pad = next power of two >= P.
// ------------------------------------------------------------------------------------------------
constexpr int kSelectThreads = 512;

// n distinct 64-bit entries of `list` in ascending order without a single barrier between compare-exchange stages: every
// thread counts the entries smaller than its own (shared-memory broadcasts) and hands (rank, entry) to `put`.  Cheaper than
// a bitonic sort (log^2 n barriers) while n^2 / threads stays small.
constexpr int kRankSortMax = 1024;
template <typename Put>
__device__ __forceinline__ void rank_sort(const unsigned long long *list, int n, Put put)
{
    for (int t = threadIdx.x; t < n; t += blockDim.x) {
        const unsigned long long x = list[t];
        int r = 0;
        for (int u = 0; u < n; ++u) r += list[u] < x ? 1 : 0;
        put(r, x);
    }
}

inline size_t pivot_smem_bytes(int n_vis, int P_pad, bool cached) { return (size_t)P_pad * 8 + (cached ? (size_t)n_vis * 4 : 0); }
constexpr int kPivotCacheMax = 32768; // scores of a sample that are kept in shared memory as keys (128 KB)

// The k elements of smallest key among n (KeyFn(j, key&) as in block_select_threshold), handed to put(rank, j) in
// ascending (key, index) order.  All threads of the CTA; list: k_pad entries of shared memory.
template <typename KeyFn, typename Put>
__device__ __forceinline__ void cta_smallest_k(KeyFn keyfn, int n, int k, int k_pad, unsigned long long *list, SelectSmem &sel,
                                               uint32_t *n_picked, Put put)
{
    for (int i = threadIdx.x; i < k_pad; i += blockDim.x) list[i] = ~0ull;
    if (threadIdx.x == 0) *n_picked = 0;
    __syncthreads();
    uint32_t T, need_eq, cnt_eq;
    block_select_threshold(CtaGroup(), keyfn, n, (uint32_t)k, sel, T, need_eq, cnt_eq);
    block_select_apply(CtaGroup(), keyfn, n, T, need_eq, cnt_eq, sel, [&](int j, uint32_t key) {
        uint32_t slot = atomicAdd(n_picked, 1u);
        list[slot] = ((unsigned long long)key << 32) | (uint32_t)j;
    });
    rank_sort(list, k, [&](int r, unsigned long long x) { put(r, (int)(x & 0xffffffffu)); });
    __syncthreads();
}

__global__ void __launch_bounds__(kSelectThreads)
pivot_kernel(const float *__restrict__ score, int n_vis, int P, int P_pad, int smallest, int cached,
             int32_t *__restrict__ pivot_idx)
{
    extern __shared__ unsigned long long piv_list[]; // [P_pad], then (cached) the sample's keys [n_vis]
    uint32_t *keys = reinterpret_cast<uint32_t *>(piv_list + P_pad);
    __shared__ SelectSmem sel;
    __shared__ uint32_t n_picked;
    const int b = blockIdx.x;
    const float *s = score + (size_t)b * n_vis;
    // smaller key = better pivot.  The select reads every key five times: from shared memory when the sample fits.
    if (cached)
        for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
            const uint32_t k = order_key(s[j]);
            keys[j] = smallest ? k : ~k;
        }
    auto keyfn = [&](int j, uint32_t &key) {
        if (cached) {
            key = keys[j];
        } else {
            uint32_t k = order_key(s[j]);
            key = smallest ? k : ~k;
        }
        return true;
    };
    // ascending order of (key, index): rank 0 = best score, ties to the lower index
    cta_smallest_k(keyfn, n_vis, P, P_pad, piv_list, sel, &n_picked, [&](int r, int j) { pivot_idx[(size_t)b * P + r] = j; });
}

// Pivots from both modalities (Sec. 5.4; the pivot-selection table fixes "4 visual and 4 text tokens"): the Pv vision
// tokens and the Pt text tokens of best score, the vision pivots in rank order first, then the text pivots in rank order,
// as indices relative to the vision block (a text token before it is negative, one after it >= n_vis).
//   score_vis [B][n_vis]; score_before [B][vis_offset]; score_after [B][S - vis_offset - n_vis]
__global__ void __launch_bounds__(kSelectThreads)
pivot_mixed_kernel(const float *__restrict__ score_vis, const float *__restrict__ score_before, const float *__restrict__ score_after,
                   int S, int vis_offset, int n_vis, int Pv, int Pt, int P_pad, int smallest, int32_t *__restrict__ pivot_idx)
{
    extern __shared__ unsigned long long piv_list[]; // [P_pad]
    __shared__ SelectSmem sel;
    __shared__ uint32_t n_picked;
    const int b = blockIdx.x, P = Pv + Pt, n_after = S - vis_offset - n_vis, n_text = vis_offset + n_after;
    const float *sv = score_vis + (size_t)b * n_vis;
    auto vis_key = [&](int j, uint32_t &key) {
        const uint32_t k = order_key(sv[j]);
        key = smallest ? k : ~k;
        return true;
    };
    if (Pv > 0)
        cta_smallest_k(vis_key, n_vis, Pv, P_pad, piv_list, sel, &n_picked, [&](int r, int j) { pivot_idx[(size_t)b * P + r] = j; });
    // text token t: position t before the block, or vis_offset + n_vis + (t - vis_offset) after it
    auto text_key = [&](int t, uint32_t &key) {
        const float v = t < vis_offset ? score_before[(size_t)b * vis_offset + t] : score_after[(size_t)b * n_after + (t - vis_offset)];
        const uint32_t k = order_key(v);
        key = smallest ? k : ~k;
        return true;
    };
    if (Pt > 0)
        cta_smallest_k(text_key, n_text, Pt, P_pad, piv_list, sel, &n_picked, [&](int r, int t) {
            pivot_idx[(size_t)b * P + Pv + r] = t < vis_offset ? t - vis_offset : n_vis + (t - vis_offset);
        });
}

// Output number k of a SplitMix64 generator seeded with `seed` (Steele, Lea, Flood, OOPSLA 2014): mix(seed + (k + 1) gamma)
__device__ __forceinline__ unsigned long long splitmix64_at(unsigned long long seed, unsigned long long k)
{
    unsigned long long z = seed + (k + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Random pivots (Sec. 5.2 also draws them at random): every vision token of sample b0 + blockIdx.x gets a 32-bit ticket,
// the upper half of output number (sample * 2^32 + token) of the generator; the P smallest tickets win, smallest first,
// equal tickets to the lower index: a uniform draw without replacement.
__global__ void __launch_bounds__(kSelectThreads)
pivot_random_kernel(unsigned long long seed, int b0, int n_vis, int P, int P_pad, int32_t *__restrict__ pivot_idx)
{
    extern __shared__ unsigned long long piv_list[]; // [P_pad]
    __shared__ SelectSmem sel;
    __shared__ uint32_t n_picked;
    const int b = blockIdx.x;
    const unsigned long long hi = (unsigned long long)(uint32_t)(b0 + b) << 32;
    auto keyfn = [&](int j, uint32_t &key) {
        key = (uint32_t)(splitmix64_at(seed, hi | (uint32_t)j) >> 32);
        return true;
    };
    cta_smallest_k(keyfn, n_vis, P, P_pad, piv_list, sel, &n_picked, [&](int r, int j) { pivot_idx[(size_t)b * P + r] = j; });
}

// ------------------------------------------------------------------------------------------------
// Step 3 on the CUDA cores: dup[i][j] = (K_{p_i} . K_j) / (|K_{p_i}| |K_j|)  (Def. 2, Eq. 7).
// A CTA stages up to 8 pivot rows in shared memory and streams a tile of token rows against them,
// 4 rows per warp at a time so that each pivot value read from shared memory feeds 4 FMAs.
// Dynamic shared memory: 8 * d8 * 16 bytes.
// ------------------------------------------------------------------------------------------------
constexpr int kSimWarps = 8;
constexpr int kSimRowsPerWarp = 4;
constexpr int kSimPivotChunk = 8;
constexpr int kSimRowsPerCta = 64;

__global__ void __launch_bounds__(kSimWarps * 32)
sim_alu_kernel(const uint4 *__restrict__ keys, int S, int d8, int vis_offset, int n_vis, int P, int p0,
               const int32_t *__restrict__ pivot_idx, const float *__restrict__ ssq, float *__restrict__ sim)
{
    extern __shared__ uint4 piv_rows[]; // [kSimPivotChunk][d8]
    __shared__ float piv_norm[kSimPivotChunk];
    const int b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint4 *base = keys + ((size_t)b * S + vis_offset) * (size_t)d8;
    const int np = min(kSimPivotChunk, P - p0);
    // a pivot outside [0, n_vis) is a text token of the same sample (checked and clamped to the sample by step 2)
    for (int i = threadIdx.x; i < kSimPivotChunk * d8; i += blockDim.x) {
        int p = i / d8, c = i - p * d8;
        piv_rows[i] = (p < np) ? __ldg(base + (long long)pivot_idx[(size_t)b * P + p0 + p] * d8 + c)
                               : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    // Euclidean norms of the pivots: a vision token's comes from step 1; a text token was not scored, so warp p sums the
    // squares of the staged row p (lanes over 16-byte chunks, fixed order)
    for (int p = warp; p < np; p += kSimWarps) {
        const int pv = pivot_idx[(size_t)b * P + p0 + p];
        float q = 0.f;
        if (pv < 0 || pv >= n_vis) {
            for (int c = lane; c < d8; c += 32) {
                const uint4 w = piv_rows[p * d8 + c];
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float lo = bf16_lo(ww[e]), hi = bf16_hi(ww[e]);
                    q = fmaf(lo, lo, q);
                    q = fmaf(hi, hi, q);
                }
            }
            q = warp_sum(q);
        } else {
            q = ssq[(size_t)b * n_vis + pv];
        }
        if (lane == 0) piv_norm[p] = sqrtf(q);
    }
    __syncthreads();
    const int tile0 = blockIdx.x * kSimRowsPerCta;
    for (int r0 = tile0 + warp * kSimRowsPerWarp; r0 < min(tile0 + kSimRowsPerCta, n_vis);
         r0 += kSimWarps * kSimRowsPerWarp) {
        float acc[kSimRowsPerWarp][kSimPivotChunk];
#pragma unroll
        for (int r = 0; r < kSimRowsPerWarp; ++r)
#pragma unroll
            for (int p = 0; p < kSimPivotChunk; ++p) acc[r][p] = 0.f;
        for (int c = lane; c < d8; c += 32) {
            float x[kSimRowsPerWarp][8];
#pragma unroll
            for (int r = 0; r < kSimRowsPerWarp; ++r) {
                int row = min(r0 + r, n_vis - 1);
                uint4 v = ld_stream(base + (size_t)row * d8 + c);
                x[r][0] = bf16_lo(v.x), x[r][1] = bf16_hi(v.x), x[r][2] = bf16_lo(v.y), x[r][3] = bf16_hi(v.y);
                x[r][4] = bf16_lo(v.z), x[r][5] = bf16_hi(v.z), x[r][6] = bf16_lo(v.w), x[r][7] = bf16_hi(v.w);
            }
#pragma unroll
            for (int p = 0; p < kSimPivotChunk; ++p) {
                uint4 w = piv_rows[p * d8 + c];
                float y[8] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y),
                              bf16_lo(w.z), bf16_hi(w.z), bf16_lo(w.w), bf16_hi(w.w)};
#pragma unroll
                for (int r = 0; r < kSimRowsPerWarp; ++r)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[r][p] = fmaf(x[r][e], y[e], acc[r][p]);
            }
        }
#pragma unroll
        for (int r = 0; r < kSimRowsPerWarp; ++r)
#pragma unroll
            for (int p = 0; p < kSimPivotChunk; ++p) acc[r][p] = warp_sum(acc[r][p]);
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < kSimRowsPerWarp; ++r) {
                int row = r0 + r;
                if (row >= n_vis) break;
                float nj = sqrtf(ssq[(size_t)b * n_vis + row]);
#pragma unroll
                for (int p = 0; p < kSimPivotChunk; ++p) {
                    if (p >= np) break;
                    float den = piv_norm[p] * nj;
                    sim[((size_t)b * P + p0 + p) * n_vis + row] = den > 0.f ? acc[r][p] / den : 0.f;
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Step 2 when the caller names the pivots (Sec. 5.2 compares several ways to choose them): the indices
// are checked - in range, no repeats - and copied into the workspace, clamped so that no later kernel
// can read outside the sample.  A failed check sets DART_ERR_CHECK in the status word (the retention and
// gather kernels then leave the outputs alone).  One CTA per sample; dynamic shared memory: one bit per
// vision token.
// ------------------------------------------------------------------------------------------------
constexpr int kStatusCheck = -8;       // DART_ERR_CHECK
constexpr int kCheckPivotsGiven = 100; // second status word: which check failed

// [lo, hi) is the range a pivot may lie in, relative to the vision block: [0, n_vis), or the whole sequence
// [-vis_offset, S - vis_offset) when text tokens may serve as pivots (Sec. 5.4).
__global__ void __launch_bounds__(256)
pivots_given_kernel(const int32_t *__restrict__ pivots_in, int lo, int hi, int P, int32_t *__restrict__ pivot_idx, int *status)
{
    extern __shared__ uint32_t seen[]; // [(hi - lo + 31) / 32]
    const int b = blockIdx.x;
    for (int w = threadIdx.x; w < (hi - lo + 31) / 32; w += blockDim.x) seen[w] = 0;
    __syncthreads();
    for (int t = threadIdx.x; t < P; t += blockDim.x) {
        const int pv = pivots_in[(size_t)b * P + t];
        bool bad = pv < lo || pv >= hi;
        const int c = min(max(pv, lo), hi - 1);
        if (!bad) bad = (atomicOr(&seen[(c - lo) >> 5], 1u << ((c - lo) & 31)) >> ((c - lo) & 31)) & 1u;
        pivot_idx[(size_t)b * P + t] = c;
        if (bad && atomicCAS(status, 0, kStatusCheck) == 0) {
            status[1] = kCheckPivotsGiven;
            status[2] = b;
            status[3] = t;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Compact copy of every sample's pivot rows, [B][N][d8] with N >= P rows per sample (rows P.. are zero), so that a
// tensor-core kernel can fetch a sample's pivot tile as one box.  One warp per row.
// ------------------------------------------------------------------------------------------------
constexpr int kPivotRowWarps = 8;

__global__ void __launch_bounds__(kPivotRowWarps * 32)
pivot_rows_kernel(const uint4 *__restrict__ keys, const int32_t *__restrict__ pivot_idx, int S, int d8, int vis_offset, int n_vis,
                  int P, int N, long long rows_total, uint4 *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kPivotRowWarps + (threadIdx.x >> 5);
    if (row >= rows_total) return;
    const int b = (int)(row / N), i = (int)(row % N);
    uint4 *dst = out + (size_t)row * d8;
    if (i >= P) {
        for (int c = lane; c < d8; c += 32) dst[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const int pv = min(max(pivot_idx[(size_t)b * P + i], -vis_offset), S - vis_offset - 1); // any row of the sample
    const uint4 *src = keys + ((size_t)b * S + vis_offset + pv) * (size_t)d8;
    for (int c = lane; c < d8; c += 32) dst[c] = __ldg(src + c);
}

// ------------------------------------------------------------------------------------------------
// kept := pivots, for one sample (all threads of the CTA; flags[] zeroed and the CTA synchronised before the call).
// A pivot outside [0, n_vis) is a text token (Sec. 5.4): it takes its turn in step 4 but is no vision token, so it
// is neither flagged nor counted.  Returns Pv, the pivots inside the vision block: the budget left to share out is
// n_keep - Pv.  `word` is a shared scratch word; the CTA is synchronised on return.
// ------------------------------------------------------------------------------------------------
__device__ inline int mark_pivots(const int32_t *__restrict__ piv, int P, int n_vis, uint8_t *flags, int32_t *owner,
                                  uint32_t *word)
{
    if (threadIdx.x == 0) *word = 0;
    __syncthreads();
    uint32_t mine = 0;
    for (int i = threadIdx.x; i < P; i += blockDim.x) {
        const int pv = piv[i];
        if (pv >= 0 && pv < n_vis) {
            flags[pv] = 1;
            if (owner) owner[pv] = P + i;
            ++mine;
        }
    }
    if (mine) atomicAdd(word, mine);
    __syncthreads();
    const int Pv = (int)*word;
    __syncthreads(); // the word may be reused
    return Pv;
}

// ------------------------------------------------------------------------------------------------
// Step 5a for one sample (all threads of the CTA): the packed index list - text rows before, kept vision
// tokens in ascending order (ordered ballot scan over the keep flags), text rows after - and the position
// ids of those rows.  warp_tot: shared scratch, one word per warp.
// ------------------------------------------------------------------------------------------------
__device__ inline void pack_indices(const uint8_t *keep, int S, int vis_offset, int n_vis, int n_keep,
                                    const int64_t *__restrict__ pin, int32_t *__restrict__ oi, int64_t *__restrict__ op,
                                    uint32_t *warp_tot)
{
    for (int t = threadIdx.x; t < vis_offset; t += blockDim.x) {
        oi[t] = t;
        op[t] = pin ? pin[t] : (int64_t)t;
    }
    const int n_after = S - vis_offset - n_vis;
    for (int t = threadIdx.x; t < n_after; t += blockDim.x) {
        const int s = vis_offset + n_vis + t;
        oi[vis_offset + n_keep + t] = s;
        op[vis_offset + n_keep + t] = pin ? pin[s] : (int64_t)s;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    uint32_t base = 0;
    for (int start = 0; start < n_vis; start += blockDim.x) {
        const int j = start + threadIdx.x;
        const bool f = (j < n_vis) && keep[j];
        const uint32_t bal = __ballot_sync(0xffffffffu, f);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        uint32_t before = 0, total = 0;
        for (int w = 0; w < nwarp; ++w) {
            const uint32_t t = warp_tot[w];
            if (w < warp) before += t;
            total += t;
        }
        if (f) {
            const uint32_t t = vis_offset + base + before + __popc(bal & ((1u << lane) - 1u));
            const int s = vis_offset + j;
            oi[t] = s;
            op[t] = pin ? pin[s] : (int64_t)s;
        }
        base += total;
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// Steps 4 and 5a in one kernel: retention (Eq. 9-10) and the packed index list.  One CTA per sample.
// (Used when the two-phase form below does not apply: more than 4096 tokens to keep beside the pivots.)
// kept := pivots; pivot i in rank order selects its q_i not-yet-kept tokens of lowest dup (radix
// select on order-preserving keys, ties to the lower index); eps_i is the selection threshold.
// Then an ordered scan over the keep flags writes the ascending kept indices and position ids.
// Dynamic shared memory: n_vis bytes (keep flags, rounded up to 16) + cache_rows * n_vis * 4 bytes: the
// similarity rows of cache_rows pivots at a time are held as order-preserving keys, so that the select's
// passes read shared memory (cache_rows = 0: every pass reads the row from global memory).
constexpr int kRetainCacheBytes = 96 * 1024; // shared-memory budget of the row cache (two CTAs per SM)
inline int retain_cache_rows(int n_vis, int P)
{
    int r = (int)((size_t)kRetainCacheBytes / ((size_t)n_vis * 4));
    return r > P ? P : r;
}
inline size_t retain_smem_bytes(int n_vis, int P)
{
    return ((size_t)n_vis + 15) / 16 * 16 + (size_t)retain_cache_rows(n_vis, P) * n_vis * 4;
}
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelectThreads)
retain_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, const int64_t *__restrict__ pos_in,
              int S, int vis_offset, int n_vis, int P, int n_keep,
              int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos,
              uint8_t *__restrict__ keep_out, int32_t *__restrict__ owner_out, float *__restrict__ eps_out,
              const int *__restrict__ status, int cache_rows)
{
    extern __shared__ __align__(16) uint8_t keep[]; // [n_vis] flags, then the key cache
    uint32_t *cache = reinterpret_cast<uint32_t *>(keep + ((size_t)n_vis + 15) / 16 * 16); // [cache_rows][n_vis]
    __shared__ SelectSmem sel;
    if (*status != 0) return; // an earlier kernel of this call failed: its outputs are undefined
    const int b = blockIdx.x;
    const int S_out = S - n_vis + n_keep;
    int32_t *owner = owner_out ? owner_out + (size_t)b * n_vis : nullptr;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        keep[j] = 0;
        if (owner) owner[j] = -1;
    }
    __syncthreads();
    const int Pv = mark_pivots(pivot_idx + (size_t)b * P, P, n_vis, keep, owner, &sel.cnt);
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    for (int i = 0; i < P; ++i) {
        const int qi = q + (i < r ? 1 : 0);
        if (qi == 0) {
            if (eps_out && threadIdx.x == 0) eps_out[(size_t)b * P + i] = __int_as_float(0x7fc00000);
            continue;
        }
        const float *row = sim + ((size_t)b * P + i) * n_vis;
        if (cache_rows > 0 && i % cache_rows == 0) { // load the next cache_rows rows (all loads independent)
            const int nr = min(cache_rows, P - i);
            __syncthreads();
            for (int idx = threadIdx.x; idx < nr * n_vis; idx += blockDim.x) cache[idx] = order_key(row[idx]);
            __syncthreads();
        }
        const uint32_t *krow = cache + (size_t)(cache_rows > 0 ? i % cache_rows : 0) * n_vis;
        auto keyfn = [&](int j, uint32_t &key) {
            if (keep[j]) return false;
            key = cache_rows > 0 ? krow[j] : order_key(row[j]);
            return true;
        };
        uint32_t T, need_eq, cnt_eq;
        block_select_threshold(CtaGroup(), keyfn, n_vis, (uint32_t)qi, sel, T, need_eq, cnt_eq);
        // picks only flip flags of elements that stay selected, so keyfn may run while others pick:
        // an element picked by another thread is never examined again by this round's owner thread
        block_select_apply(CtaGroup(), keyfn, n_vis, T, need_eq, cnt_eq, sel, [&](int j, uint32_t) {
            keep[j] = 1;
            if (owner) owner[j] = i;
        });
        if (eps_out && threadIdx.x == 0) eps_out[(size_t)b * P + i] = order_key_inv(T);
    }
    pack_indices(keep, S, vis_offset, n_vis, n_keep, pos_in ? pos_in + (size_t)b * S : nullptr, out_idx + (size_t)b * S_out,
                 out_pos + (size_t)b * S_out, sel.warp_tot);
    if (keep_out)
        for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keep_out[(size_t)b * n_vis + j] = keep[j];
}

// ------------------------------------------------------------------------------------------------
// Steps 4 and 5a in two phases (the default; retain_kernel above is the plain one-kernel form).
//
// Pivot i keeps its q_i not-yet-kept tokens of lowest dup (Eq. 9-10, rank order).  Before its turn at
// most Q_{i-1} = q_0 + ... + q_{i-1} non-pivot tokens have been kept, so its picks are among the
// M_i = Q_{i-1} + q_i = Q_i smallest (dup, index) pairs of its row.  Phase 1 therefore works on all
// (sample, pivot) pairs at once: one CTA selects those M_i candidates (radix select over keys cached in
// shared memory, pivots excluded), sorts them by (dup, index) and stores their indices.  Phase 2, one CTA
// per sample, takes the pivots' turns in rank order: a warp walks pivot i's sorted list 32 entries at a
// time and keeps the first q_i that are still free; eps_i is the dup of the last one kept.  Then the
// ordered scan writes the packed index list as above.  The result equals retain_kernel's exactly.
//
// Dynamic shared memory, phase 1: n_vis * 4 (keys) and n_vis (pivot flags), each rounded to 16, + M_pad * 8 (sort
// buffer, M_pad = next power of two >= n_keep - Pv, Pv = the pivots that are vision tokens).  Phase 2: n_vis rounded to 16 (keep flags) +
// kWalkStageEntries * 4 (staged candidate lists).
// ------------------------------------------------------------------------------------------------
constexpr int kCandThreads = 1024;      // at most; the host launches fewer threads per CTA when there are many CTAs
constexpr int kCandMax = 4096;           // candidates per pivot the sort buffer takes (n_keep - P <= 4096)
constexpr int kWalkThreads = 256;
constexpr int kWalkStageEntries = 12288; // 48 KB of staged candidate indices per round of phase 2

__host__ __device__ inline int quota_prefix(int i, int q, int r) { return (i + 1) * q + (i + 1 < r ? i + 1 : r); } // Q_i

inline size_t candidates_smem_bytes(int n_vis, int m_pad)
{
    return ((size_t)n_vis * 4 + 15) / 16 * 16 + ((size_t)n_vis + 15) / 16 * 16 + (size_t)m_pad * 8;
}
inline size_t walk_smem_bytes(int n_vis) { return ((size_t)n_vis + 15) / 16 * 16 + (size_t)kWalkStageEntries * 4; }

__global__ void __launch_bounds__(kCandThreads)
candidates_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, int n_vis, int P, int n_keep,
                  int m_pad, int cand_stride, int32_t *__restrict__ cand, const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t cand_smem[];
    uint32_t *keys = reinterpret_cast<uint32_t *>(cand_smem);                      // [n_vis] order-preserving keys of the row
    uint8_t *is_pivot = cand_smem + ((size_t)n_vis * 4 + 15) / 16 * 16;            // [n_vis]
    unsigned long long *list = reinterpret_cast<unsigned long long *>(is_pivot + ((size_t)n_vis + 15) / 16 * 16); // [m_pad]
    __shared__ SelectSmem sel;
    __shared__ uint32_t n_picked;
    if (*status != 0) return; // an earlier kernel of this call failed: its outputs are undefined
    const int i = blockIdx.x, b = blockIdx.y;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) is_pivot[j] = 0;
    __syncthreads();
    const int Pv = mark_pivots(pivot_idx + (size_t)b * P, P, n_vis, is_pivot, nullptr, &n_picked);
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    const int qi = q + (i < r ? 1 : 0);
    if (qi == 0) return; // this pivot keeps nothing (and so do all later ones)
    const int M = quota_prefix(i, q, r);
    const float *row = sim + ((size_t)b * P + i) * n_vis;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keys[j] = order_key(row[j]);
    int mp = 1; // this pivot's own sort size
    while (mp < M) mp <<= 1;
    for (int t = threadIdx.x; t < mp; t += blockDim.x) list[t] = ~0ull;
    if (threadIdx.x == 0) n_picked = 0;
    __syncthreads();
    auto keyfn = [&](int j, uint32_t &key) {
        if (is_pivot[j]) return false;
        key = keys[j];
        return true;
    };
    int32_t *out = cand + ((size_t)b * P + i) * cand_stride;
    uint32_t T, need_eq, cnt_eq;
    block_select_threshold(CtaGroup(), keyfn, n_vis, (uint32_t)M, sel, T, need_eq, cnt_eq);
    block_select_apply(CtaGroup(), keyfn, n_vis, T, need_eq, cnt_eq, sel, [&](int j, uint32_t key) {
        const uint32_t slot = atomicAdd(&n_picked, 1u);
        if (slot < (uint32_t)mp) list[slot] = ((unsigned long long)key << 32) | (uint32_t)j;
    });
    if (M <= kRankSortMax) { // lowest dup first, equal dups by index
        rank_sort(list, M, [&](int r, unsigned long long x) { out[r] = (int32_t)(x & 0xffffffffu); });
        return;
    }
    // ascending bitonic sort of (key, index)
    for (int k = 2; k <= mp; k <<= 1) {
        for (int jj = k >> 1; jj > 0; jj >>= 1) {
            for (int t = threadIdx.x; t < mp; t += blockDim.x) {
                const int l = t ^ jj;
                if (l > t) {
                    const unsigned long long x = list[t], y = list[l];
                    const bool up = ((t & k) == 0);
                    if ((x > y) == up) {
                        list[t] = y;
                        list[l] = x;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int t = threadIdx.x; t < M; t += blockDim.x) out[t] = (int32_t)(list[t] & 0xffffffffu);
}

__global__ void __launch_bounds__(kWalkThreads)
retain_walk_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, const int32_t *__restrict__ cand,
                   int cand_stride, const int64_t *__restrict__ pos_in, int S, int vis_offset, int n_vis, int P, int n_keep,
                   int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos, uint8_t *__restrict__ keep_out,
                   int32_t *__restrict__ owner_out, float *__restrict__ eps_out, const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t keep[]; // [n_vis] flags, then the staged candidate lists
    int32_t *stage = reinterpret_cast<int32_t *>(keep + ((size_t)n_vis + 15) / 16 * 16); // [kWalkStageEntries]
    __shared__ uint32_t warp_tot[kWalkThreads / 32];
    if (*status != 0) return;
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S_out = S - n_vis + n_keep;
    int32_t *owner = owner_out ? owner_out + (size_t)b * n_vis : nullptr;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        keep[j] = 0;
        if (owner) owner[j] = -1;
    }
    __syncthreads();
    const int Pv = mark_pivots(pivot_idx + (size_t)b * P, P, n_vis, keep, owner, &warp_tot[0]);
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    if (eps_out)
        for (int i = threadIdx.x; i < P; i += blockDim.x)
            if (q + (i < r ? 1 : 0) == 0) eps_out[(size_t)b * P + i] = __int_as_float(0x7fc00000);
    // rounds: stage the lists of as many pivots as fit, then warp 0 takes their turns in rank order
    const int n_active = q > 0 ? P : r; // pivots with a quota (all later ones keep nothing)
    for (int i0 = 0; i0 < n_active;) {
        int i1 = i0, total = 0;
        while (i1 < n_active && (i1 == i0 || total + quota_prefix(i1, q, r) <= kWalkStageEntries)) {
            total += quota_prefix(i1, q, r);
            ++i1;
        }
        // list of pivot i starts at the sum of the lengths before it (recomputed by every thread: a few adds)
        for (int i = i0, off = 0; i < i1; ++i) {
            const int M = quota_prefix(i, q, r);
            const int32_t *src = cand + ((size_t)b * P + i) * cand_stride;
            for (int t = threadIdx.x; t < M; t += blockDim.x) stage[off + t] = src[t];
            off += M;
        }
        __syncthreads();
        if (warp == 0) {
            for (int i = i0, off = 0; i < i1; ++i) {
                const int M = quota_prefix(i, q, r);
                int remaining = q + (i < r ? 1 : 0), last = -1;
                for (int t = 0; t < M && remaining > 0; t += 32) {
                    const bool valid = t + lane < M;
                    const int j = valid ? stage[off + t + lane] : 0;
                    const bool free = valid && !keep[j];
                    const uint32_t bal = __ballot_sync(0xffffffffu, free);
                    const bool take = free && (int)__popc(bal & ((1u << lane) - 1u)) < remaining;
                    const uint32_t took = __ballot_sync(0xffffffffu, take);
                    if (take) {
                        keep[j] = 1;
                        if (owner) owner[j] = i;
                    }
                    if (took) last = __shfl_sync(0xffffffffu, j, 31 - __clz(took)); // the list is sorted: the highest lane is the largest dup
                    remaining -= __popc(took);
                    __syncwarp(); // the flags are visible to the next chunk and the next pivot
                }
                // eps_i = dup of the last token taken; its index is parked in the output word and turned into the value
                // after the walk by another thread: a load from global memory here would stall every pivot's turn
                if (eps_out && lane == 0) eps_out[(size_t)b * P + i] = __int_as_float(last);
                off += M;
            }
        }
        __syncthreads();
        i0 = i1;
    }
    if (eps_out)
        for (int i = threadIdx.x; i < n_active; i += blockDim.x) {
            const int last = __float_as_int(eps_out[(size_t)b * P + i]);
            eps_out[(size_t)b * P + i] = last >= 0 ? sim[((size_t)b * P + i) * n_vis + last] : __int_as_float(0x7fc00000);
        }
    pack_indices(keep, S, vis_offset, n_vis, n_keep, pos_in ? pos_in + (size_t)b * S : nullptr, out_idx + (size_t)b * S_out,
                 out_pos + (size_t)b * S_out, warp_tot);
    if (keep_out)
        for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keep_out[(size_t)b * n_vis + j] = keep[j];
}

// ------------------------------------------------------------------------------------------------
// Steps 4 and 5a in two phases with candidate BANDS: one warp and one read of the row per (sample, pivot).
//
// Pivot i's picks are among the Q_i smallest (dup, index) pairs of its row (see above), hence among ANY set of its
// row's tokens that contains those Q_i.  Phase 1 (band_kernel) therefore does no exact selection and no sort: it lays
// a histogram of kBandBins equal bins over the row's range [min, max], finds the first bin at which the running count
// reaches Q_i and stores every token up to and including that bin, grouped by bin (a counting sort: the histogram's
// prefix sums are the bins' offsets), each entry tagged with its bin.  The band is a few entries longer than Q_i
// (about one bin's population).  When it would not fit the list (a range stretched by an outlier) the last bin alone is
// cut into kBandBins bins again, up to kBandLevels levels; rows that still do not fit (many equal values) or that hold
// a value that is not finite take the exact route: the Q_i-th smallest key by bitwise search, then every key below it
// and the lowest-index keys equal to it, Q_i entries under one tag.
// Phase 2 (retain_pick_kernel), one CTA per sample, takes the pivots' turns in rank order.  A warp walks pivot i's
// band from its lowest bin, moving the entries that are still free to the front, until it has passed the bin that holds
// the q_i-th free entry; the free entries of the bins before that one are all taken, and the rest of the quota is
// taken from that one bin, smallest (dup, index) first.  eps_i is the last dup taken.  The result equals
// retain_kernel's exactly.
//
// An entry is 64 bits: the order-preserving key of the dup (32), the tag (8), the token's index (24).  Entries with the
// same key share their tag, so comparing entries compares (dup, index).
// Dynamic shared memory, phase 1: n_vis * 4 rounded to 16 + 4 per entry of a list.  Phase 2: n_vis rounded to 16 (keep flags) + P * 4 rounded to
// 16 (band lengths) + 2 * kPickStageEntries * 8 (two buffers of staged bands).
// ------------------------------------------------------------------------------------------------
constexpr int kBandBins = 256;
constexpr int kBandLevels = 3;
constexpr int kBandMaxTokens = 1 << 24; // an entry has 24 bits for the token's index
constexpr int kPickThreads = 256;
constexpr int kPickStageEntries = 6144; // 48 KB of staged entries per buffer of phase 2
constexpr int kPickAhead = 4;           // chunks of 32 entries read ahead in phase 2
inline int band_stride(int m) { return (m + m / 4 + 64 + 1) & ~1; } // entries per list for up to m tokens beside the pivots
__host__ __device__ inline size_t band_smem_bytes(int n_vis, int stride) { return ((size_t)n_vis * 4 + 15) / 16 * 16 + (size_t)stride * 4; }
inline size_t pick_smem_bytes(int n_vis, int P)
{
    return ((size_t)n_vis + 15) / 16 * 16 + ((size_t)P * 4 + 15) / 16 * 16 + (size_t)2 * kPickStageEntries * 8;
}
__device__ __forceinline__ unsigned long long band_entry(uint32_t key, uint32_t tag, uint32_t j)
{
    return ((unsigned long long)key << 32) | (tag << 24) | j;
}
__device__ __forceinline__ uint32_t entry_tag(unsigned long long e) { return ((uint32_t)e >> 24) & 255u; }
__device__ __forceinline__ uint32_t entry_index(unsigned long long e) { return (uint32_t)e & 0xffffffu; }

// Asynchronous copies global -> shared memory that pass no register: many in flight per thread.
template <int kBytes>
__device__ __forceinline__ void copy_async(void *dst_smem, const void *src)
{
    static_assert(kBytes == 8 || kBytes == 16, "cp.async.ca takes 4, 8 or 16 bytes");
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src), "n"(kBytes)
                 : "memory");
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void copy_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

// k-th smallest (k >= 1) of the keys a warp holds, given each lane's count of its keys below a value.
template <typename CountFn>
__device__ __forceinline__ uint32_t warp_kth_key(CountFn count_below, uint32_t k)
{
    uint32_t v = 0; // the largest value with fewer than k keys below it
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t t = v | (1u << bit);
        if (__reduce_add_sync(0xffffffffu, count_below(t)) < k) v = t;
    }
    return v;
}

// Phase 1 for one row, by one warp: the band of pivot i of a sample (row = its dups, piv = the sample's pivots) into
// out[0 .. *out_n).  vs: the warp's shared memory, n_vis rounded up to 4 words for the row + `stride` words for the queue.
struct BandScratch {
    uint32_t hist[kBandBins]; // the bins' counts, then their offsets in the list
    uint32_t n_low;           // entries below the interval of a finer level handed out so far
    uint32_t n_queued;        // the band's tokens found so far
    uint32_t pad[2];
};
__device__ void band_of_row(const float *__restrict__ row, const int32_t *__restrict__ piv, int i, int n_vis, int P, int n_keep,
                            int stride, uint32_t *vs, BandScratch &sc, unsigned long long *__restrict__ out,
                            int32_t *__restrict__ out_n)
{
    const int lane = threadIdx.x & 31;
    const uint32_t lt = (1u << lane) - 1u;
    constexpr uint32_t kNotAToken = 0xffffffffu; // a pivot, or the filler behind the row: a NaN no arithmetic produces
    const int n4 = (n_vis + 3) / 4; // groups of four values
    const bool aligned = (n_vis & 3) == 0; // rows start on 16-byte boundaries
    if (aligned) { // the whole row is on its way before anything else is looked at
        for (int j = lane; j < n4; j += 32) copy_async<16>(vs + 4 * j, row + 4 * j);
        copy_async_commit();
    } else {
#pragma unroll 8
        for (int j = lane; j < n4 * 4; j += 32) vs[j] = __float_as_uint(__ldcs(row + (j < n_vis ? j : 0))); // (filler: a value of the row)
    }
    uint32_t mine = 0;
    for (int t = lane; t < P; t += 32) mine += (piv[t] >= 0 && piv[t] < n_vis) ? 1u : 0u;
    const int Pv = (int)__reduce_add_sync(0xffffffffu, mine);
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    copy_async_wait<0>();
    __syncwarp();
    if (q + (i < r ? 1 : 0) == 0) { // this pivot keeps nothing
        if (lane == 0) *out_n = 0;
        return;
    }
    const uint32_t C = (uint32_t)quota_prefix(i, q, r);
    // the row's smallest and largest value (pivots included: they only stretch the upper end; a NaN is passed over)
    const uint4 *vs4 = reinterpret_cast<const uint4 *>(vs);
    uint32_t *queue = vs + (size_t)n4 * 4; // [stride] the band's tokens, in no order
    float f_lo = __int_as_float(0x7f800000), f_hi = __int_as_float(0xff800000), f_sum = 0.0f;
#pragma unroll 2
    for (int j = lane; j < n4; j += 32) {
        const uint4 v = vs4[j];
        f_lo = fminf(fminf(f_lo, __uint_as_float(v.x)), fminf(fminf(__uint_as_float(v.y), __uint_as_float(v.z)), __uint_as_float(v.w)));
        f_hi = fmaxf(fmaxf(f_hi, __uint_as_float(v.x)), fmaxf(fmaxf(__uint_as_float(v.y), __uint_as_float(v.z)), __uint_as_float(v.w)));
        f_sum += (__uint_as_float(v.x) + __uint_as_float(v.y)) + (__uint_as_float(v.z) + __uint_as_float(v.w));
    }
    f_lo = order_key_inv(__reduce_min_sync(0xffffffffu, order_key(f_lo)));
    f_hi = order_key_inv(__reduce_max_sync(0xffffffffu, order_key(f_hi)));
    f_sum = warp_sum(f_sum);
    for (int t = lane; t < P; t += 32)
        if (piv[t] >= 0 && piv[t] < n_vis) vs[piv[t]] = kNotAToken;
    if (lane < n4 * 4 - n_vis) vs[n_vis + lane] = kNotAToken;
    if (lane == 0) sc.n_queued = 0;
    __syncwarp();
    // The band: every value below lo, and the values of [lo, hi] whose bin is at most last_bin.  A level lays its bins
    // over the smallest and largest value of the interval it looks at; while the band is too long for the list the
    // next level looks at the last bin alone.  (kNotAToken compares false with everything: it is in no interval.)
    // The first level's bins span [min, 2 * mean - min] only (whatever lies above goes into the last bin): a band is the
    // row's low end, and a few large dups - the pivot's own cluster - would otherwise take most of the bins.
    float lo = f_lo, hi = f_hi;
    const float spread = 2.0f * (f_sum / (float)(n4 * 4) - f_lo);
    float scale = (float)kBandBins / (spread > 0.0f && spread < f_hi - f_lo ? spread : f_hi - f_lo);
    // equal values, an infinite one, a NaN, or places that overflow
    bool exact = !(f_hi > f_lo) || !(f_hi - f_lo < 3.0e38f) || !((f_hi - f_lo) * scale < 3.0e38f);
    uint32_t before = 0, last_bin = 0, n_band = 0, my_off = 0;
    int level = 0;
    auto bin_of = [&](float f) { return min((int)((f - lo) * scale), kBandBins - 1); }; // for lo <= f <= hi: not negative, monotone
    uint32_t c[kBandBins / 32];
    while (!exact) {
        for (int t = lane; t < kBandBins; t += 32) sc.hist[t] = 0;
        __syncwarp();
#pragma unroll 2
        for (int j = lane; j < n4; j += 32) {
            const uint4 v = vs4[j];
            const float f[4] = {__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w)};
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (f[t] >= lo && f[t] <= hi) atomicAdd(&sc.hist[bin_of(f[t])], 1u);
        }
        __syncwarp();
        // lane l owns bins [8l, 8l + 8): the first bin at which the running count reaches the rest of C, and the counts there
        const uint32_t want = C - before; // >= 1, and the interval holds at least that many values
        uint32_t sum = 0;
#pragma unroll
        for (int t = 0; t < kBandBins / 32; ++t) {
            c[t] = sc.hist[lane * (kBandBins / 32) + t];
            sum += c[t];
        }
        uint32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        my_off = before + incl - sum; // where this lane's first bin starts in the list
        if (level == 0 && __shfl_sync(0xffffffffu, incl, 31) != (uint32_t)(n_vis - Pv)) { // a NaN among the values
            exact = true;
            break;
        }
        uint32_t my_bin = 0, my_upto = 0, my_cnt = 0;
        const bool here = incl - sum < want && want <= incl; // exactly one lane
        if (here) {
            uint32_t run = incl - sum;
#pragma unroll
            for (int t = 0; t < kBandBins / 32; ++t) {
                if (run < want && want <= run + c[t]) {
                    my_bin = lane * (kBandBins / 32) + t;
                    my_upto = run + c[t];
                    my_cnt = c[t];
                }
                run += c[t];
            }
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, here)) - 1;
        last_bin = __shfl_sync(0xffffffffu, my_bin, src);
        n_band = before + __shfl_sync(0xffffffffu, my_upto, src);
        const uint32_t in_last = __shfl_sync(0xffffffffu, my_cnt, src);
        if (n_band <= (uint32_t)stride) break;
        // look at the last bin alone: its smallest and largest value
        float n_lo = __int_as_float(0x7f800000), n_hi = __int_as_float(0xff800000);
        for (int j = lane; j < n4 * 4; j += 32) {
            const float f = __uint_as_float(vs[j]);
            if (f >= lo && f <= hi && bin_of(f) == (int)last_bin) {
                n_lo = fminf(n_lo, f);
                n_hi = fmaxf(n_hi, f);
            }
        }
        n_lo = order_key_inv(__reduce_min_sync(0xffffffffu, order_key(n_lo)));
        n_hi = order_key_inv(__reduce_max_sync(0xffffffffu, order_key(n_hi)));
        before = n_band - in_last;
        lo = n_lo;
        hi = n_hi;
        scale = (float)kBandBins / (n_hi - n_lo);
        exact = ++level == kBandLevels || !(n_hi > n_lo) || !(scale < 3.0e38f);
    }
    if (!exact) {
        // the bins' offsets
        __syncwarp();
#pragma unroll
        for (int t = 0; t < kBandBins / 32; ++t) {
            sc.hist[lane * (kBandBins / 32) + t] = my_off;
            my_off += c[t];
        }
        if (lane == 0) sc.n_low = 0;
        // the band's tokens: few of the row's, so they are queued first and then handled with all lanes busy
        const float edge = last_bin == kBandBins - 1 ? 3.0e38f : (float)(last_bin + 1); // bin <= last_bin <=> place < edge
#pragma unroll 2
        for (int j = lane; j < n4; j += 32) {
            const uint4 v = vs4[j];
            const float f[4] = {__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w)};
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if ((f[t] - lo) * scale < edge && f[t] <= hi) queue[atomicAdd(&sc.n_queued, 1u)] = (uint32_t)(4 * j + t);
        }
        __syncwarp();
        // every entry asks its bin for the next slot
        for (uint32_t e = lane; e < n_band; e += 32) {
            const uint32_t j = queue[e];
            const float f = __uint_as_float(vs[j]);
            uint32_t slot, tag = 0; // tags grow with the bins; at finer levels tag 0 is what lies below the interval
            if (f < lo) {
                slot = atomicAdd(&sc.n_low, 1u);
            } else {
                const int bin = bin_of(f);
                slot = atomicAdd(&sc.hist[bin], 1u);
                tag = level == 0 ? (uint32_t)bin : (uint32_t)(bin >> 1) + 1u;
            }
            out[slot] = band_entry(order_key(f), tag, j);
        }
        if (lane == 0) *out_n = (int32_t)n_band;
        return;
    }
    // the exact route: C entries (C <= stride by the host's choice of stride), equal keys in index order, one tag
    auto key_of = [&](int j) { return vs[j] == kNotAToken ? 0xffffffffu : min(order_key(__uint_as_float(vs[j])), 0xfffffffeu); };
    const uint32_t T = warp_kth_key(
        [&](uint32_t t) {
            uint32_t n = 0;
            for (int j = lane; j < n_vis; j += 32) n += key_of(j) < t ? 1u : 0u;
            return n;
        },
        C);
    uint32_t below = 0;
    for (int j = lane; j < n_vis; j += 32) below += key_of(j) < T ? 1u : 0u;
    const uint32_t need_eq = C - __reduce_add_sync(0xffffffffu, below);
    uint32_t eq_seen = 0, n_out = 0;
    for (int j0 = 0; j0 < n_vis; j0 += 32) {
        const int j = j0 + lane;
        const uint32_t key = j < n_vis ? key_of(j) : 0xffffffffu;
        const bool eq = j < n_vis && key == T;
        const uint32_t beq = __ballot_sync(0xffffffffu, eq);
        const bool in = j < n_vis && (key < T || (eq && eq_seen + __popc(beq & lt) < need_eq));
        const uint32_t bal = __ballot_sync(0xffffffffu, in);
        if (in) out[n_out + __popc(bal & lt)] = band_entry(key, 0u, (uint32_t)j);
        n_out += __popc(bal);
        eq_seen += __popc(beq);
    }
    if (lane == 0) *out_n = (int32_t)n_out;
}

__global__ void __launch_bounds__(32)
band_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, int n_vis, int P, int n_keep, int stride,
            unsigned long long *__restrict__ band, int32_t *__restrict__ band_n, const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t band_smem[];
    __shared__ BandScratch sc;
    if (*status != 0) return; // an earlier kernel of this call failed: its outputs are undefined
    const int i = blockIdx.x, b = blockIdx.y;
    band_of_row(sim + ((size_t)b * P + i) * n_vis, pivot_idx + (size_t)b * P, i, n_vis, P, n_keep, stride,
                reinterpret_cast<uint32_t *>(band_smem), sc, band + ((size_t)b * P + i) * stride, band_n + (size_t)b * P + i);
}

// Phase 2 for one sample, by a CTA of kPickThreads threads.  keep: [n_vis] flags; len: [P]; stage: two buffers of
// kPickStageEntries entries; warp_tot: one word per warp.
__device__ void pick_sample(const int b, const int32_t *__restrict__ pivot_idx, const unsigned long long *__restrict__ band,
                            const int32_t *__restrict__ band_n, int stride, const int64_t *__restrict__ pos_in, int S, int vis_offset,
                            int n_vis, int P, int n_keep, int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos,
                            uint8_t *__restrict__ keep_out, int32_t *__restrict__ owner_out, float *__restrict__ eps_out,
                            uint8_t *keep, int32_t *len, unsigned long long *stage, uint32_t *warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const int S_out = S - n_vis + n_keep;
    int32_t *owner = owner_out ? owner_out + (size_t)b * n_vis : nullptr;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        keep[j] = 0;
        if (owner) owner[j] = -1;
    }
    for (int i = threadIdx.x; i < P; i += blockDim.x) len[i] = band_n[(size_t)b * P + i];
    __syncthreads();
    const int Pv = mark_pivots(pivot_idx + (size_t)b * P, P, n_vis, keep, owner, &warp_tot[0]);
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    const int n_active = q > 0 ? P : r; // pivots with a quota (all later ones keep nothing)
    if (eps_out)
        for (int i = n_active + threadIdx.x; i < P; i += blockDim.x) eps_out[(size_t)b * P + i] = __int_as_float(0x7fc00000);
    // Rounds: the bands of as many pivots as fit one buffer; while warp 0 takes the turns of one round's pivots in
    // rank order, the next round's bands arrive in the other buffer.
    auto round_end = [&](int i0) { // the pivots [i0, i1) of the round that starts at i0 (every thread computes the same)
        int i1 = i0, total = 0;
        while (i1 < n_active && (i1 == i0 || total + len[i1] <= kPickStageEntries)) total += len[i1++];
        return i1;
    };
    auto fetch = [&](int i0, int i1, unsigned long long *buf) {
        for (int i = i0, off = 0; i < i1; off += len[i], ++i) {
            const unsigned long long *src = band + ((size_t)b * P + i) * stride;
            for (int t = threadIdx.x; t < len[i]; t += blockDim.x) copy_async<8>(buf + off + t, src + t);
        }
        copy_async_commit();
    };
    int i0 = 0, i1 = round_end(0);
    fetch(i0, i1, stage);
    for (int round = 0; i0 < n_active; ++round) {
        unsigned long long *buf = stage + (size_t)(round & 1) * kPickStageEntries;
        const int i2 = round_end(i1);
        fetch(i1, i2, stage + (size_t)((round + 1) & 1) * kPickStageEntries); // (an empty group after the last round)
        copy_async_wait<1>();                                                 // this round's bands have arrived
        __syncthreads();
        if (warp == 0) {
            for (int i = i0, off = 0; i < i1; off += len[i], ++i) {
                unsigned long long *L = buf + off;
                const int n = len[i], qi = q + (i < r ? 1 : 0);
                // the free entries to the front (an entry moves towards the front only), bin after bin, until the bin
                // that holds the qi-th free entry (its tag: tq) has been passed
                int F = 0, tq = -1;
                bool passed = false;
                for (int t0 = 0; t0 < n && !passed; t0 += 32 * kPickAhead) {
                    // kPickAhead chunks of 32 entries and their flags are read, and the votes on them taken, before the
                    // first is looked at (entries move to places before t0 only, and no flag changes here)
                    unsigned long long ent[kPickAhead];
                    bool fr[kPickAhead];
                    uint32_t fb[kPickAhead];
#pragma unroll
                    for (int u = 0; u < kPickAhead; ++u) ent[u] = t0 + 32 * u + lane < n ? L[t0 + 32 * u + lane] : ~0ull;
#pragma unroll
                    for (int u = 0; u < kPickAhead; ++u) fr[u] = ent[u] != ~0ull && !keep[entry_index(ent[u])];
#pragma unroll
                    for (int u = 0; u < kPickAhead; ++u) fb[u] = __ballot_sync(0xffffffffu, fr[u]);
                    int u0 = 0; // the first chunk of the group that is filtered by tag
                    if (tq < 0) {
                        int hit = -1, run = F; // the chunk that holds the qi-th free entry, the free entries before that chunk
#pragma unroll
                        for (int u = 0; u < kPickAhead; ++u) {
                            const int c = __popc(fb[u]);
                            if (hit < 0 && run + c >= qi) hit = u;
                            if (hit < 0) run += c;
                        }
#pragma unroll
                        for (int u = 0; u < kPickAhead; ++u)
                            if (hit < 0 || u < hit) {
                                if (fr[u]) L[F + __popc(fb[u] & lt)] = ent[u];
                                F += __popc(fb[u]);
                            }
                        u0 = kPickAhead;
#pragma unroll
                        for (int u = 0; u < kPickAhead; ++u)
                            if (u == hit) {
                                const uint32_t it = __ballot_sync(0xffffffffu, fr[u] && F + (int)__popc(fb[u] & lt) == qi - 1);
                                tq = __shfl_sync(0xffffffffu, (int)entry_tag(ent[u]), __ffs(it) - 1);
                                u0 = u;
                            }
                    }
                    if (tq >= 0) { // from chunk u0 on: entries up to tag tq only; the first chunk that reaches beyond it is the last
                        uint32_t tb[kPickAhead], gb[kPickAhead];
#pragma unroll
                        for (int u = 0; u < kPickAhead; ++u) {
                            const int tag = (int)entry_tag(ent[u]);
                            tb[u] = __ballot_sync(0xffffffffu, fr[u] && tag <= tq);
                            gb[u] = __ballot_sync(0xffffffffu, ent[u] != ~0ull && tag > tq);
                        }
#pragma unroll
                        for (int u = 0; u < kPickAhead; ++u)
                            if (u >= u0 && !passed) {
                                if (fr[u] && (int)entry_tag(ent[u]) <= tq) L[F + __popc(tb[u] & lt)] = ent[u];
                                F += __popc(tb[u]);
                                passed = gb[u] != 0u;
                            }
                    }
                    __syncwarp();
                }
                unsigned long long best = 0;
                if (F <= 32) {
                    // (the usual case) one entry per lane: those of the bins before tq are all taken, and the rest of the
                    // quota from bin tq, the smallest remaining entry again and again
                    const bool mine = lane < F;
                    const unsigned long long v = mine ? L[lane] : ~0ull;
                    const bool early = mine && (tq < 0 || (int)entry_tag(v) < tq);
                    const int sure = __popc(__ballot_sync(0xffffffffu, early));
                    const int need = (qi < F ? qi : F) - sure;
                    bool take = early;
                    if (need >= F - sure) {
                        take = mine;
                    } else {
                        unsigned long long m = mine && !early ? v : ~0ull;
                        for (int k = 0; k < need; ++k) {
                            const uint32_t hi = __reduce_min_sync(0xffffffffu, (uint32_t)(m >> 32));
                            const uint32_t lo = __reduce_min_sync(0xffffffffu, (uint32_t)(m >> 32) == hi ? (uint32_t)m : 0xffffffffu);
                            if (m == (((unsigned long long)hi << 32) | lo)) {
                                take = true;
                                m = ~0ull;
                            }
                        }
                    }
                    if (take) {
                        keep[entry_index(v)] = 1;
                        if (owner) owner[entry_index(v)] = i;
                    }
                    best = (unsigned long long)__reduce_max_sync(0xffffffffu, take ? (uint32_t)(v >> 32) : 0u) << 32; // eps: the largest taken
                } else {
                    // the free entries of the bins before tq are all taken (they stand first: the band is grouped by bin)
                    int sure = 0;
                    for (int e0 = 0; e0 < F; e0 += 32) {
                        const bool mine = e0 + lane < F && (tq < 0 || (int)entry_tag(L[e0 + lane]) < tq);
                        if (mine) {
                            const uint32_t j = entry_index(L[e0 + lane]);
                            keep[j] = 1;
                            if (owner) owner[j] = i;
                        }
                        const uint32_t bal = __ballot_sync(0xffffffffu, mine);
                        sure += __popc(bal);
                        if (bal != 0xffffffffu) break;
                    }
                    // the rest of the quota from bin tq, L[sure .. F): the smallest remaining entry again and again
                    unsigned long long from = 0;
                    for (int k = sure; k < qi && k < F; ++k) {
                        unsigned long long m = ~0ull;
                        for (int e = sure + lane; e < F; e += 32) {
                            const unsigned long long v = L[e];
                            if (v >= from && v < m) m = v;
                        }
                        const uint32_t hi = __reduce_min_sync(0xffffffffu, (uint32_t)(m >> 32));
                        const uint32_t lo = __reduce_min_sync(0xffffffffu, (uint32_t)(m >> 32) == hi ? (uint32_t)m : 0xffffffffu);
                        best = ((unsigned long long)hi << 32) | lo;
                        from = best + 1;
                        if (lane == 0) {
                            keep[entry_index(best)] = 1;
                            if (owner) owner[entry_index(best)] = i;
                        }
                    }
                    if (F <= qi) { // (fewer free entries than the quota cannot happen; the largest taken, for eps)
                        unsigned long long m = 0;
                        for (int e = lane; e < F; e += 32) m = L[e] > m ? L[e] : m;
                        best = (unsigned long long)__reduce_max_sync(0xffffffffu, (uint32_t)(m >> 32)) << 32;
                    }
                }
                __syncwarp(); // the flags are visible to the next pivot's turn
                if (eps_out && lane == 0)
                    eps_out[(size_t)b * P + i] = F > 0 ? order_key_inv((uint32_t)(best >> 32)) : __int_as_float(0x7fc00000);
            }
        }
        __syncthreads(); // the buffer may be filled again
        i0 = i1;
        i1 = i2;
    }
    copy_async_wait<0>();
    pack_indices(keep, S, vis_offset, n_vis, n_keep, pos_in ? pos_in + (size_t)b * S : nullptr, out_idx + (size_t)b * S_out,
                 out_pos + (size_t)b * S_out, warp_tot);
    if (keep_out)
        for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keep_out[(size_t)b * n_vis + j] = keep[j];
}

__global__ void __launch_bounds__(kPickThreads)
retain_pick_kernel(const int32_t *__restrict__ pivot_idx, const unsigned long long *__restrict__ band,
                   const int32_t *__restrict__ band_n, int stride, const int64_t *__restrict__ pos_in, int S, int vis_offset,
                   int n_vis, int P, int n_keep, int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos,
                   uint8_t *__restrict__ keep_out, int32_t *__restrict__ owner_out, float *__restrict__ eps_out,
                   const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t keep[]; // [n_vis] flags, the bands' lengths, two buffers of staged bands
    int32_t *len = reinterpret_cast<int32_t *>(keep + ((size_t)n_vis + 15) / 16 * 16);                                  // [P]
    unsigned long long *stage = reinterpret_cast<unsigned long long *>(reinterpret_cast<uint8_t *>(len) + ((size_t)P * 4 + 15) / 16 * 16); // [2][kPickStageEntries]
    __shared__ uint32_t warp_tot[kPickThreads / 32];
    if (*status != 0) return;
    pick_sample(blockIdx.x, pivot_idx, band, band_n, stride, pos_in, S, vis_offset, n_vis, P, n_keep, out_idx, out_pos, keep_out,
                owner_out, eps_out, keep, len, stage, warp_tot);
}

// Both phases in one launch, one CTA per sample, for batches that cannot fill the GPU anyway: band_warps warps build the
// sample's bands, a pivot each at a time (through the same workspace in global memory: the CTA reads back what it wrote),
// then the CTA takes the turns.  Dynamic shared memory: the flags and lengths of phase 2, then whichever is larger of
// phase 2's two staging buffers and phase 1's band_warps x (row + queue + scratch).
__host__ __device__ inline size_t fused_warp_bytes(int n_vis, int stride) { return band_smem_bytes(n_vis, stride) + sizeof(BandScratch); }
inline size_t retain_fused_smem_bytes(int n_vis, int P, int stride, int band_warps)
{
    const size_t phase1 = (size_t)band_warps * ((fused_warp_bytes(n_vis, stride) + 15) / 16 * 16);
    const size_t phase2 = (size_t)2 * kPickStageEntries * 8;
    return ((size_t)n_vis + 15) / 16 * 16 + ((size_t)P * 4 + 15) / 16 * 16 + (phase1 > phase2 ? phase1 : phase2);
}
__global__ void __launch_bounds__(kPickThreads)
retain_fused_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, unsigned long long *__restrict__ band,
                    int32_t *__restrict__ band_n, int stride, const int64_t *__restrict__ pos_in, int S, int vis_offset, int n_vis,
                    int P, int n_keep, int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos, uint8_t *__restrict__ keep_out,
                    int32_t *__restrict__ owner_out, float *__restrict__ eps_out, const int *__restrict__ status, int band_warps)
{
    extern __shared__ __align__(16) uint8_t keep[];
    int32_t *len = reinterpret_cast<int32_t *>(keep + ((size_t)n_vis + 15) / 16 * 16);
    uint8_t *work = reinterpret_cast<uint8_t *>(len) + ((size_t)P * 4 + 15) / 16 * 16;
    __shared__ uint32_t warp_tot[kPickThreads / 32];
    if (*status != 0) return;
    const int b = blockIdx.x, warp = threadIdx.x >> 5;
    if (warp < band_warps) {
        const size_t per_warp = (fused_warp_bytes(n_vis, stride) + 15) / 16 * 16;
        uint32_t *vs = reinterpret_cast<uint32_t *>(work + (size_t)warp * per_warp);
        BandScratch &sc = *reinterpret_cast<BandScratch *>(work + (size_t)warp * per_warp + band_smem_bytes(n_vis, stride));
        for (int i = warp; i < P; i += band_warps) {
            band_of_row(sim + ((size_t)b * P + i) * n_vis, pivot_idx + (size_t)b * P, i, n_vis, P, n_keep, stride, vs, sc,
                        band + ((size_t)b * P + i) * stride, band_n + (size_t)b * P + i);
            __syncwarp(); // the row's buffer is free for the next one
        }
    }
    __syncthreads(); // the bands are written; the work area changes hands
    pick_sample(b, pivot_idx, band, band_n, stride, pos_in, S, vis_offset, n_vis, P, n_keep, out_idx, out_pos, keep_out, owner_out,
                eps_out, keep, len, reinterpret_cast<unsigned long long *>(work), warp_tot);
}

// ------------------------------------------------------------------------------------------------
// Steps 4 and 5a with ONE threshold for all pivots (Def. 2 / Eq. 8-9 read with a common eps): a token's
// duplication is its highest dup to any pivot, u_j = max_i dup[i][j]; the n_keep - P non-pivot tokens of
// lowest u_j are kept (radix select on order-preserving keys, ties to the lower index), eps = the largest
// kept u_j.  owner[j] = the pivot token j is most similar to (the first of equals).  One CTA per sample;
// dynamic shared memory: n_vis rounded to 16 (keep flags) + n_vis * 4 (keys of u_j).
// ------------------------------------------------------------------------------------------------
inline size_t retain_global_smem_bytes(int n_vis) { return ((size_t)n_vis + 15) / 16 * 16 + (size_t)n_vis * 4; }

__global__ void __launch_bounds__(kSelectThreads)
retain_global_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, const int64_t *__restrict__ pos_in,
                     int S, int vis_offset, int n_vis, int P, int n_keep,
                     int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos,
                     uint8_t *__restrict__ keep_out, int32_t *__restrict__ owner_out, float *__restrict__ eps_out,
                     const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t keep[]; // [n_vis] flags, then the keys
    uint32_t *ukey = reinterpret_cast<uint32_t *>(keep + ((size_t)n_vis + 15) / 16 * 16); // [n_vis]
    __shared__ SelectSmem sel;
    if (*status != 0) return; // an earlier kernel of this call failed: its outputs are undefined
    const int b = blockIdx.x;
    const int S_out = S - n_vis + n_keep;
    const float *rows = sim + (size_t)b * P * n_vis;
    int32_t *owner = owner_out ? owner_out + (size_t)b * n_vis : nullptr;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        float u = rows[j];
        for (int i = 1; i < P; ++i) u = fmaxf(u, rows[(size_t)i * n_vis + j]); // finite inputs: fmaxf is the plain maximum
        ukey[j] = order_key(u);
        keep[j] = 0;
        if (owner) owner[j] = -1;
    }
    __syncthreads();
    // pivots outside the vision block are text tokens: compared with, but neither marked nor counted
    const int Pv = mark_pivots(pivot_idx + (size_t)b * P, P, n_vis, keep, owner, &sel.cnt);
    const int take = n_keep - Pv;
    float eps = __int_as_float(0x7fc00000);
    if (take > 0) {
        auto keyfn = [&](int j, uint32_t &key) {
            if (keep[j]) return false;
            key = ukey[j];
            return true;
        };
        uint32_t T, need_eq, cnt_eq;
        block_select_threshold(CtaGroup(), keyfn, n_vis, (uint32_t)take, sel, T, need_eq, cnt_eq);
        // picks only flip flags of elements that stay selected, so keyfn may run while others pick
        block_select_apply(CtaGroup(), keyfn, n_vis, T, need_eq, cnt_eq, sel, [&](int j, uint32_t) {
            keep[j] = 1;
            if (owner) {
                int arg = 0;
                float u = rows[j];
                for (int i = 1; i < P; ++i) {
                    const float v = rows[(size_t)i * n_vis + j];
                    if (v > u) {
                        u = v;
                        arg = i;
                    }
                }
                owner[j] = arg;
            }
        });
        eps = order_key_inv(T);
    }
    if (eps_out)
        for (int i = threadIdx.x; i < P; i += blockDim.x) eps_out[(size_t)b * P + i] = eps;
    pack_indices(keep, S, vis_offset, n_vis, n_keep, pos_in ? pos_in + (size_t)b * S : nullptr, out_idx + (size_t)b * S_out,
                 out_pos + (size_t)b * S_out, sel.warp_tot);
    if (keep_out)
        for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keep_out[(size_t)b * n_vis + j] = keep[j];
}

// ------------------------------------------------------------------------------------------------
// Steps 4 and 5a with INDEPENDENT pivots (Eq. 9-10 read literally: R = P u U_i R_i): pivot i takes its q_i
// non-pivot tokens of lowest dup whatever the other pivots took; a token two pivots take is kept once, so a
// sample keeps between P and n_keep vision tokens and the packed length depends on the data.  Three launches:
// the selections (one CTA per sample; writes the keep flags and the sample's packed length), an exclusive
// scan of the lengths (cu_seqlens, the layout variable-length attention kernels take), and the packed index
// lists written at the samples' offsets.
// ------------------------------------------------------------------------------------------------
constexpr int kGatherWarps = 8; // warps per CTA of the gather kernels, one output row each
inline size_t retain_union_smem_bytes(int n_vis) { return ((size_t)n_vis + 15) / 16 * 16; }

__global__ void __launch_bounds__(kSelectThreads)
retain_union_kernel(const float *__restrict__ sim, const int32_t *__restrict__ pivot_idx, int S, int n_vis, int P, int n_keep,
                    uint8_t *__restrict__ keep_out, int32_t *__restrict__ owner_out, float *__restrict__ eps_out,
                    int32_t *__restrict__ len_out, const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t flags[]; // [n_vis] 0 free, 1 kept, 2 pivot
    __shared__ SelectSmem sel;
    if (*status != 0) return; // an earlier kernel of this call failed: its outputs are undefined
    const int b = blockIdx.x;
    int32_t *owner = owner_out ? owner_out + (size_t)b * n_vis : nullptr;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        flags[j] = 0;
        if (owner) owner[j] = -1;
    }
    __syncthreads();
    // pivots outside the vision block are text tokens: they pick like any pivot, but are neither marked nor counted
    __shared__ int n_vis_pivots;
    if (threadIdx.x == 0) n_vis_pivots = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < P; i += blockDim.x) {
        const int pv = pivot_idx[(size_t)b * P + i];
        if (pv >= 0 && pv < n_vis) {
            flags[pv] = 2;
            if (owner) owner[pv] = P + i;
            atomicAdd(&n_vis_pivots, 1);
        }
    }
    __syncthreads();
    const int Pv = n_vis_pivots;
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    for (int i = 0; i < P; ++i) {
        const int qi = q + (i < r ? 1 : 0);
        if (qi == 0) {
            if (eps_out && threadIdx.x == 0) eps_out[(size_t)b * P + i] = __int_as_float(0x7fc00000);
            continue;
        }
        const float *row = sim + ((size_t)b * P + i) * n_vis;
        auto keyfn = [&](int j, uint32_t &key) { // every non-pivot token is a candidate of every pivot
            if (flags[j] == 2) return false;
            key = order_key(row[j]);
            return true;
        };
        uint32_t T, need_eq, cnt_eq;
        block_select_threshold(CtaGroup(), keyfn, n_vis, (uint32_t)qi, sel, T, need_eq, cnt_eq);
        block_select_apply(CtaGroup(), keyfn, n_vis, T, need_eq, cnt_eq, sel, [&](int j, uint32_t) {
            if (flags[j] == 0) { // the first pivot in rank order that takes a token owns it
                flags[j] = 1;
                if (owner) owner[j] = i;
            }
        });
        if (eps_out && threadIdx.x == 0) eps_out[(size_t)b * P + i] = order_key_inv(T);
        __syncthreads();
    }
    int mine = 0;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) {
        const uint8_t f = flags[j] != 0;
        mine += f;
        keep_out[(size_t)b * n_vis + j] = f;
    }
    __shared__ int total;
    if (threadIdx.x == 0) total = 0;
    __syncthreads();
    if (mine) atomicAdd(&total, mine);
    __syncthreads();
    if (threadIdx.x == 0) len_out[b] = S - n_vis + total;
}

// cu[0] = 0, cu[b + 1] = cu[b] + len[b]: one CTA, chunks of blockDim.x lengths with a running carry
__global__ void __launch_bounds__(256) cu_seqlens_kernel(const int32_t *__restrict__ len, int B, int32_t *__restrict__ cu,
                                                         const int *__restrict__ status)
{
    __shared__ int32_t buf[256];
    __shared__ int32_t carry;
    if (*status != 0) return;
    if (threadIdx.x == 0) carry = 0, cu[0] = 0;
    __syncthreads();
    for (int b0 = 0; b0 < B; b0 += blockDim.x) {
        const int b = b0 + threadIdx.x;
        buf[threadIdx.x] = b < B ? len[b] : 0;
        __syncthreads();
        for (int o = 1; o < (int)blockDim.x; o <<= 1) { // inclusive scan
            const int32_t v = threadIdx.x >= (unsigned)o ? buf[threadIdx.x - o] : 0;
            __syncthreads();
            buf[threadIdx.x] += v;
            __syncthreads();
        }
        if (b < B) cu[b + 1] = carry + buf[threadIdx.x];
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry += buf[threadIdx.x];
        __syncthreads();
    }
}

// The packed index list and position ids of every sample at its offset cu[b].
__global__ void __launch_bounds__(kWalkThreads)
pack_varlen_kernel(const uint8_t *__restrict__ keep_in, const int32_t *__restrict__ cu, const int64_t *__restrict__ pos_in, int S,
                   int vis_offset, int n_vis, int32_t *__restrict__ out_idx, int64_t *__restrict__ out_pos,
                   const int *__restrict__ status)
{
    extern __shared__ __align__(16) uint8_t keep[]; // [n_vis]
    __shared__ uint32_t warp_tot[kWalkThreads / 32];
    if (*status != 0) return;
    const int b = blockIdx.x;
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) keep[j] = keep_in[(size_t)b * n_vis + j];
    __syncthreads();
    const int start = cu[b], kept = cu[b + 1] - start - (S - n_vis);
    pack_indices(keep, S, vis_offset, n_vis, kept, pos_in ? pos_in + (size_t)b * S : nullptr, out_idx + start, out_pos + start,
                 warp_tot);
}

// Step 5b for packed rows of variable length: output row t belongs to the sample b with cu[b] <= t < cu[b + 1].
// One warp per output row (as gather_kernel); rows at and beyond cu[B] do not exist.
__global__ void __launch_bounds__(kGatherWarps * 32)
gather_varlen_kernel(const uint4 *__restrict__ hidden, const int32_t *__restrict__ out_idx, const int32_t *__restrict__ cu, int B,
                     int S, int d8, long long rows_cap, const int *__restrict__ status, uint4 *__restrict__ out_hidden)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kGatherWarps + (threadIdx.x >> 5);
    if (row >= rows_cap || *status != 0 || row >= cu[B]) return;
    int lo = 0, hi = B; // the largest b with cu[b] <= row
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)cu[mid] <= row) lo = mid;
        else hi = mid;
    }
    const int s = out_idx[row];
    const uint4 *src = hidden + ((size_t)lo * S + s) * (size_t)d8;
    uint4 *dst = out_hidden + (size_t)row * (size_t)d8;
    for (int c = lane; c < d8; c += 32) st_stream(dst + c, ld_stream(src + c));
}

// ------------------------------------------------------------------------------------------------
// Step 5b: gather the kept hidden rows into the packed sequence.  One warp per output row,
// 128-bit loads and streaming stores, 8 loads in flight per lane.
// ------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kGatherWarps * 32)
gather_kernel(const uint4 *__restrict__ hidden, const int32_t *__restrict__ out_idx, int S, int S_out, int d8,
              long long rows_total, const int *__restrict__ status, uint4 *__restrict__ out_hidden)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kGatherWarps + (threadIdx.x >> 5);
    if (row >= rows_total || (status && *status != 0)) return; // after a failed kernel out_idx is undefined
    const int b = (int)(row / S_out);
    const int s = out_idx[row];
    const uint4 *src = hidden + ((size_t)b * S + s) * (size_t)d8;
    uint4 *dst = out_hidden + (size_t)row * (size_t)d8;
    for (int c0 = 0; c0 < d8; c0 += 32 * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int c = c0 + u * 32 + lane;
            if (c < d8) v[u] = ld_stream(src + c);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int c = c0 + u * 32 + lane;
            if (c < d8) st_stream(dst + c, v[u]);
        }
    }
}

// Adds up the column chunks' shares of the similarities (the persistent sweep cuts every row tile into chunks of columns
// so that all SMs re-read a sample at the same time): sim[i] = share[0][i] + share[1][i] + ... in this fixed order.
constexpr int kSimSumThreads = 256;
template <typename V>
__global__ void __launch_bounds__(kSimSumThreads) sim_sum_kernel(const V *__restrict__ share, long long n, int n_kc, V *__restrict__ sim)
{
    for (long long i = (long long)blockIdx.x * kSimSumThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kSimSumThreads) {
        V a = __ldcs(share + i);
        for (int k = 1; k < n_kc; ++k) {
            const V b = __ldcs(share + (size_t)k * n + i);
            if constexpr (sizeof(V) == 16) {
                a.x += b.x, a.y += b.y, a.z += b.z, a.w += b.w;
            } else {
                a += b;
            }
        }
        sim[i] = a;
    }
}

} // namespace dart
