// One-pass path for pivots that are known before the step starts (the caller's pivots): scores and
// similarities from ONE read of the key rows.
//
// With the pivots given, nothing in a row's dot products (Eq. 7's numerator) waits for another row, so a
// row tile is streamed once and used twice while it sits in shared memory: the tensor cores multiply it
// with the sample's pivot rows (tokens = M 128, pivots = N, bf16 -> fp32 in TMEM, accumulating over all
// of d), and four warps add up |x| (the K-norm of the Sec. 3.3 footnote) and x^2 (Eq. 7's denominator)
// of the same 128 rows, and of the pivot rows that came with the tile.  The epilogue divides by the two
// norms and writes dup(p_i, x_j) (Eq. 7).  No CTA depends on another one: tasks (sample, row tile) are
// dealt out round-robin to a persistent grid of one CTA per SM.
//
// Per CTA (384 threads):
//   warp 0     producer: per 64-column atom one or two 128-row TMA tiles (128-byte swizzle) and the pivot rows - as
//              ONE box from a compact copy of the sample's pivot rows, or, where the context has no room for that
//              copy, by tile::gather4 straight from the key tensor (4 rows per op, ~13 ops per us: slower) -
//              up to four atoms per stage of a ring
//   warp 1     one thread issues tcgen05.mma; tcgen05.commit releases the stage on the tensor cores' behalf
//   warps 4-7  norms: thread t owns tile row t and sums its 128 bytes of every atom, in column order whatever
//              the swizzle did to the chunks, so a row's norm does not depend on where in a tile it was read
//   warps 2-3  the same for the pivot rows of the stage's pivot tile (thread u: rows u, u + 64, ...)
//   warps 8-11 epilogue: TMEM -> normalised similarities [B][P][n_vis]
// Every wait is bounded in time; on expiry the kernel records DART_ERR_TIMEOUT in the status word, lets the
// copies and MMAs in flight finish, frees TMEM and exits normally.  Results are bitwise reproducible.
#pragma once
#include "dart_sweep.cuh"

namespace dart {
namespace onepass {

using namespace sweep; // PTX wrappers, Ctl, Ring, tile constants

constexpr int kThreads = 384;
constexpr int kNormWarp0 = 4, kNormWarps = 4;
constexpr int kPivWarp0 = 2, kPivWarps = 2, kPivThreads = kPivWarps * 32;
constexpr int kEpi0 = 8;          // kEpi0 % 4 == 0: warp w reads TMEM lanes 32 (w % 4) ...
constexpr int kStages = 10;       // at most
constexpr int kMaxAtomsPerStage = 4; // a stage holds up to four 64-column atoms: the producer's issue latency (wait, expect,
                                     // issue: ~0.3 us) is paid per stage; measured at 8 pivots: 1 atom 1.40 ms, 2 1.14, 4 1.02
constexpr int kGatherMaxP = 0;    // up to this many pivots the pivot rows come by gather4 even when the compact copy exists: none
                                  // (gather4 ops issue at ~13 per us and SM: at 8 pivots 128 of them per row tile cost more than
                                  // the copy; measured per launch, 256 x 2880 tokens, 8 pivots: 1.01 -> 0.95 ms)
constexpr int kStaticSmemReserve = 8192;
enum { kWaitStageFree = 64, kWaitStageMma, kWaitStageNorm, kWaitAccumFree1, kWaitAccumFull1, kWaitNormFree, kWaitNormFull };

struct Params {
    int B, S, vis_offset, n_vis, P, N; // N = P rounded up to a multiple of 16 (MMA N)
    int n_atoms, n_rt;                 // 64-column atoms per row; row tiles per sample
    int n_st, aps;                     // ring depth; atoms per stage (<= kMaxAtomsPerStage)
    int tg;                            // row tiles per task (1 or 2): two tiles share every pivot tile that is fetched
    int compact;                       // pivot tiles come from the compact copy [B][N][d] (tm_piv), not by gather4
    int n_sel;                         // row tiles per sample this launch takes: n_rt, or the streamed tiles of `split`
    TileSplit split;                   // k <= 1: all tiles
    int withhold;                      // test hook: the first pivot-norm warp never hands its norms over, so that the bounded waits expire
    unsigned long long wait_ns;
    float *sim;                        // [B][P][n_vis] dup(p_i, x_j)
    float *l1, *ssq;                   // [B][n_vis]; l1 may be NULL (the scores come from another tensor)
    const int32_t *pivot_idx;          // [B][P], checked and clamped; outside [0, n_vis): a text row of the sample
    int *status;
};

struct Shared {
    unsigned long long full[kStages], empty[kStages];
    unsigned long long tmem_full[2], tmem_empty[2], norm_full[2], norm_empty[2];
    unsigned long long mma_drain;
    uint32_t tmem_base;
    int abort_flag;
    float row_ssq[2][2][kTileRows]; // per accumulator buffer and tile of the task: sum of squares of the tile's rows
    float piv_ssq[2][kMaxN];     // ... and of the sample's pivot rows
};
static_assert(sizeof(Shared) + 64 <= kStaticSmemReserve, "static shared memory exceeds its reserve");

__host__ __device__ inline uint32_t stage_bytes(int N, int aps, int tg = 1) { return (uint32_t)aps * ((uint32_t)tg * kAtomBytes + b_stage_bytes(N)); }
__host__ inline int ring_depth(int N, int aps, size_t smem_limit, int tg = 1)
{
    const size_t n = (smem_limit - 1024 - kStaticSmemReserve) / stage_bytes(N, aps, tg);
    return (int)(n > (size_t)kStages ? (size_t)kStages : n);
}
// As many atoms per stage as still leave three stages (with many pivots the pivot tiles crowd them out)
__host__ inline int atoms_per_stage(int N, size_t smem_limit, int tg = 1)
{
    int aps = kMaxAtomsPerStage;
    while (aps > 1 && ring_depth(N, aps, smem_limit, tg) < 3) aps >>= 1;
    return aps;
}
__host__ inline size_t smem_bytes(int N, int aps, int n_st, int tg = 1) { return 1024 + (size_t)n_st * stage_bytes(N, aps, tg); }

// |x| and x^2 of one 128-byte row of a 128B-swizzled tile, added to the four running sums in column order:
// logical 16-byte chunk c of row r sits at chunk position c ^ (r & 7)
__device__ __forceinline__ void add_row(uint32_t tile, int r, float &a0, float &a1, float &q0, float &q1)
{
    const uint32_t row = tile + (uint32_t)r * 128u;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint4 v = lds128(row + (uint32_t)((c ^ (r & 7)) * 16));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float lo = bf16_lo(w[e]), hi = bf16_hi(w[e]);
            a0 += fabsf(lo);
            a1 += fabsf(hi);
            q0 = fmaf(lo, lo, q0);
            q1 = fmaf(hi, hi, q1);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
onepass_kernel(const __grid_constant__ CUtensorMap tm_tile, const __grid_constant__ CUtensorMap tm_keys,
               const __grid_constant__ CUtensorMap tm_row, const __grid_constant__ CUtensorMap tm_piv,
               const __grid_constant__ CUtensorMap tm_pair, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bstage = b_stage_bytes(p.N);
    // stage s: p.aps x p.tg token tiles (atom-major), then p.aps pivot tiles
    auto a_addr = [&](int s, int h, int w = 0) {
        return smem0 + (uint32_t)s * stage_bytes(p.N, p.aps, p.tg) + (uint32_t)(h * p.tg + w) * kAtomBytes;
    };
    auto b_addr = [&](int s, int h) {
        return smem0 + (uint32_t)s * stage_bytes(p.N, p.aps, p.tg) + (uint32_t)(p.aps * p.tg) * kAtomBytes + (uint32_t)h * bstage;
    };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    // the epilogue waits for everything else, so its waits are nearest to whatever is missing: shortest limit; then the producer
    const Ctl ctl{&sh.abort_flag, p.status, warp >= kEpi0 ? limit : warp == 0 ? limit + limit / 8 : limit + limit / 4};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), 1 + kNormWarps + kPivWarps); // the MMAs' commit and every norm warp
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh.tmem_full[a]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[a]), kEpiWarps);
            mbar_init(smem_u32(&sh.norm_full[a]), kNormWarps + kPivWarps);
            mbar_init(smem_u32(&sh.norm_empty[a]), kEpiWarps);
        }
        mbar_init(smem_u32(&sh.mma_drain), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * (uint32_t)p.tg * p.N) tmem_cols <<= 1;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;
    const uint32_t per_sample = (uint32_t)(p.n_sel + p.tg - 1) / (uint32_t)p.tg;
    const uint32_t total = (uint32_t)p.B * per_sample; // tasks: (sample, first row tile), sample-major
    // task g -> (sample, row tile); with a split only the tiles that did not stay on the chip are taken (one tile per task then)
    auto task = [&](uint32_t g, int &b, int &rt) {
        b = (int)(g / per_sample);
        const int i = (int)(g - (uint32_t)b * per_sample) * p.tg;
        rt = p.split.k <= 1 ? i : p.split.streamed(i);
    };
    auto tile_rows = [&](int rt, int w) { return max(0, min(kTileRows, p.n_vis - (rt + w) * kTileRows)); }; // 0: no such tile
    const int na = p.n_atoms;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        unsigned long long pol_keep, pol_drop;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));  // pivot rows: every tile of the sample
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_drop)); // token rows: read once
        Ring ring(p.n_st);
        long long issued = 0;
        bool ok = true;
        int cur_b = -1;
        int my_piv[kMaxN / 128][4]; // lane l loads pivot ranks 4l..4l+3, 4(l+32).., as rows of the key tensor
        for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
            int b, rt;
            task(g, b, rt);
            if (b != cur_b) {
#pragma unroll
                for (int k = 0; k < kMaxN / 128; ++k)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = min(4 * (lane + 32 * k) + e, p.P - 1); // ranks beyond P repeat the last pivot
                        my_piv[k][e] = b * p.S + min(max(p.vis_offset + __ldg(p.pivot_idx + (size_t)b * p.P + i), 0), p.S - 1); // any row of the sample
                    }
                cur_b = b;
            }
            const int y0 = b * p.S + p.vis_offset + rt * kTileRows;
            const bool pair_box = p.tg == 2 && tile_rows(rt, 0) == kTileRows && tile_rows(rt, 1) == kTileRows;
            uint32_t tile_tx = 0; // bytes of one atom of the task's tiles
            for (int w = 0; w < p.tg; ++w) {
                const int rows = tile_rows(rt, w);
                tile_tx += rows == kTileRows ? (uint32_t)kAtomBytes : (uint32_t)((rows + kSubRows - 1) / kSubRows) * kSubBytes;
            }
            for (int a = 0; a < na; a += p.aps) {
                const int nh = min(p.aps, na - a); // atoms in this stage
                const uint32_t full = smem_u32(&sh.full[ring.stage]);
                if (lane == 0) {
                    ok = ctl.wait_bar(smem_u32(&sh.empty[ring.stage]), ring.phase ^ 1u, kWaitStageFree, g);
                    if (ok)
                        mbar_arrive_expect_tx(full, (uint32_t)nh * (tile_tx + (p.compact ? (uint32_t)p.N * 128u : (uint32_t)((p.P + 3) / 4) * 512u)));
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                for (int h = 0; h < nh; ++h) {
                    const int x = (a + h) * kAtomCols;
                    if (pair_box) { // two whole tiles, one below the other in the tensor and in the stage: one box of 256 rows
                        if (lane == h) tma_load_2d(a_addr(ring.stage, h, 0), &tm_pair, x, y0, full, pol_drop);
                    } else
                    for (int w = 0; w < p.tg; ++w) {
                        const int rows = tile_rows(rt, w), n_sub = (rows + kSubRows - 1) / kSubRows;
                        const uint32_t dst = a_addr(ring.stage, h, w);
                        if (rows == kTileRows) {
                            if (lane == h + kMaxAtomsPerStage * 2 * w) tma_load_2d(dst, &tm_tile, x, y0 + w * kTileRows, full, pol_drop); // one lane per tile: issued side by side
                        } else if (lane < n_sub) {
                            tma_load_2d(dst + (uint32_t)lane * kSubBytes, &tm_keys, x, y0 + w * kTileRows + lane * kSubRows, full, pol_drop);
                        }
                    }
                    if (p.compact) { // rows b N .. b N + N - 1 of the compact copy: the sample's pivots in rank order, zero padded
                        if (lane == kMaxAtomsPerStage + h) tma_load_2d(b_addr(ring.stage, h), &tm_piv, x, b * p.N, full, pol_keep);
                    } else {
#pragma unroll
                        for (int k = 0; k < kMaxN / 128; ++k) {
                            const int q = lane + 32 * k; // pivot ranks 4q..4q+3 -> rows 4q..4q+3 of the pivot tile
                            if (4 * q < p.P)
                                tma_gather4(b_addr(ring.stage, h) + (uint32_t)q * 512u, &tm_row, x, my_piv[k][0], my_piv[k][1],
                                            my_piv[k][2], my_piv[k][3], full, pol_keep);
                        }
                    }
                }
                ring.advance();
                ++issued;
            }
        }
        if ((!ok || ctl.aborted()) && lane == 0) // let the copies already issued land before the CTA may exit
            for (long long i = issued > p.n_st ? issued - p.n_st : 0; i < issued; ++i)
                ctl.wait_landed(smem_u32(&sh.full[i % p.n_st]), (uint32_t)((i / p.n_st) & 1));
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(p.N);
            Ring ring(p.n_st);
            uint32_t n = 0;
            bool ok = true;
            for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
                const uint32_t acc = n & 1u;
                ok = ctl.wait_bar(smem_u32(&sh.tmem_empty[acc]), ((n >> 1) & 1u) ^ 1u, kWaitAccumFree1, g);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)(p.tg * p.N);
                int rt_b, rt_t;
                task(g, rt_b, rt_t);
                const int nt = p.tg > 1 && tile_rows(rt_t, 1) > 0 ? 2 : 1; // tiles of this task
                for (int a = 0; a < na; a += p.aps) {
                    ok = ctl.wait_bar(smem_u32(&sh.full[ring.stage]), ring.phase, kWaitStageMma, g);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    for (int h = 0; h < min(p.aps, na - a); ++h) {
                        const unsigned long long db = umma_desc(b_addr(ring.stage, h));
                        for (int w = 0; w < nt; ++w) { // the task's tiles share the pivot tile
                            const unsigned long long da = umma_desc(a_addr(ring.stage, h, w));
#pragma unroll
                            for (int k = 0; k < kAtomCols / 16; ++k) // 16 columns = 32 bytes per MMA: advance the start address
                                umma_bf16(d_tmem + (uint32_t)(w * p.N), da + (unsigned long long)(2 * k), db + (unsigned long long)(2 * k),
                                          idesc, (a | h | k) != 0);
                        }
                    }
                    umma_commit(smem_u32(&sh.empty[ring.stage])); // the tensor cores' share of releasing the stage
                    ring.advance();
                }
                if (!ok) break;
                umma_commit(smem_u32(&sh.tmem_full[acc]));
                ++n;
            }
            if (!ok || ctl.aborted()) { // TMEM is freed at the end: first let the MMAs issued so far finish
                umma_commit(smem_u32(&sh.mma_drain));
                ctl.wait_landed(smem_u32(&sh.mma_drain), 0);
            }
        }
    } else if (warp >= kNormWarp0 && warp < kNormWarp0 + kNormWarps) {
        // ------------------------------------------------------------------ norms of the tile's rows and of the pivot rows
        const int t = (int)threadIdx.x - kNormWarp0 * 32; // tile row owned by this thread
        Ring ring(p.n_st);
        uint32_t n = 0;
        bool dead = false; // warp-uniform
        for (uint32_t g = blockIdx.x; !dead && g < total; g += gridDim.x) {
            int b, rt;
            task(g, b, rt);
            const int rows = tile_rows(rt, 0), rows2 = p.tg > 1 ? tile_rows(rt, 1) : 0;
            float a0 = 0.f, a1 = 0.f, q0 = 0.f, q1 = 0.f; // own row of the task's first tile
            float c0 = 0.f, c1 = 0.f, r0 = 0.f, r1 = 0.f; // ... and of its second tile
            for (int a = 0; a < na; a += p.aps) {
                dead = !ctl.wait_bar(smem_u32(&sh.full[ring.stage]), ring.phase, kWaitStageNorm, g);
                dead = __any_sync(0xffffffffu, dead);
                if (dead) break;
                for (int h = 0; h < min(p.aps, na - a); ++h) { // atoms in column order: the sums do not depend on the staging
                    if (t < rows) add_row(a_addr(ring.stage, h), t, a0, a1, q0, q1);
                    if (t < rows2) add_row(a_addr(ring.stage, h, 1), t, c0, c1, r0, r1);
                }
                __syncwarp(); // the warp's reads of the stage are done
                if (lane == 0) mbar_arrive(smem_u32(&sh.empty[ring.stage]));
                ring.advance();
            }
            if (dead) break;
            const uint32_t acc = n & 1u;
            // the slot is free once the epilogue has used the norms of the task two before
            dead = !ctl.wait_bar(smem_u32(&sh.norm_empty[acc]), ((n >> 1) & 1u) ^ 1u, kWaitNormFree, g);
            dead = __any_sync(0xffffffffu, dead);
            if (dead) break;
            const float q = q0 + q1, r = r0 + r1;
            sh.row_ssq[acc][0][t] = t < rows ? q : 0.f;
            sh.row_ssq[acc][1][t] = t < rows2 ? r : 0.f;
            if (t < rows) {
                const size_t o = (size_t)b * p.n_vis + rt * kTileRows + t;
                if (p.l1) p.l1[o] = a0 + a1;
                p.ssq[o] = q;
            }
            if (t < rows2) {
                const size_t o = (size_t)b * p.n_vis + (rt + 1) * kTileRows + t;
                if (p.l1) p.l1[o] = c0 + c1;
                p.ssq[o] = r;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.norm_full[acc])); // release: the warp's norms are ordered before it
            ++n;
        }
    } else if (warp >= kPivWarp0 && warp < kPivWarp0 + kPivWarps) {
        // ------------------------------------------------------------------ norms of the pivot rows that come with every tile
        const int u = (int)threadIdx.x - kPivWarp0 * 32; // pivot rows u, u + 64, u + 128, u + 192
        Ring ring(p.n_st);
        uint32_t n = 0;
        bool dead = false; // warp-uniform
        for (uint32_t g = blockIdx.x; !dead && g < total; g += gridDim.x) {
            float pq[kMaxN / kPivThreads][2]; // sums of squares only
#pragma unroll
            for (int k = 0; k < kMaxN / kPivThreads; ++k) pq[k][0] = pq[k][1] = 0.f;
            for (int a = 0; a < na; a += p.aps) {
                dead = !ctl.wait_bar(smem_u32(&sh.full[ring.stage]), ring.phase, kWaitStageNorm, g);
                dead = __any_sync(0xffffffffu, dead);
                if (dead) break;
                for (int h = 0; h < min(p.aps, na - a); ++h)
#pragma unroll
                    for (int k = 0; k < kMaxN / kPivThreads; ++k)
                        if (u + kPivThreads * k < p.P) {
                            float x0 = 0.f, x1 = 0.f;
                            add_row(b_addr(ring.stage, h), u + kPivThreads * k, x0, x1, pq[k][0], pq[k][1]);
                        }
                __syncwarp(); // the warp's reads of the stage are done
                if (lane == 0) mbar_arrive(smem_u32(&sh.empty[ring.stage]));
                ring.advance();
            }
            if (dead) break;
            const uint32_t acc = n & 1u;
            dead = !ctl.wait_bar(smem_u32(&sh.norm_empty[acc]), ((n >> 1) & 1u) ^ 1u, kWaitNormFree, g);
            dead = __any_sync(0xffffffffu, dead);
            if (dead) break;
#pragma unroll
            for (int k = 0; k < kMaxN / kPivThreads; ++k)
                if (u + kPivThreads * k < p.P) sh.piv_ssq[acc][u + kPivThreads * k] = pq[k][0] + pq[k][1];
            __syncwarp();
            if (lane == 0 && !(p.withhold && warp == kPivWarp0)) mbar_arrive(smem_u32(&sh.norm_full[acc]));
            ++n;
        }
    } else if (warp >= kEpi0 && warp < kEpi0 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue (warps independent)
        const int quarter = warp & 3;        // TMEM lane quarter this warp may read
        const int row = quarter * 32 + lane; // tile row owned by this thread
        uint32_t n = 0;
        for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
            int b, rt;
            task(g, b, rt);
            const uint32_t acc = n & 1u;
            bool ok = ctl.wait_bar(smem_u32(&sh.norm_full[acc]), (n >> 1) & 1u, kWaitNormFull, g);
            if (ok) ok = ctl.wait_bar(smem_u32(&sh.tmem_full[acc]), (n >> 1) & 1u, kWaitAccumFull1, g);
            if (!__all_sync(0xffffffffu, ok)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int w = 0; w < p.tg; ++w) { // the task's tiles, one accumulator each
                const int rows = tile_rows(rt, w);
                if (rows == 0) break;
                const int j = (rt + w) * kTileRows + row;
                const float nj = sqrtf(sh.row_ssq[acc][w][row]);
                const uint32_t taddr = tmem_base + acc * (uint32_t)(p.tg * p.N) + (uint32_t)(w * p.N) + ((uint32_t)(quarter * 32) << 16);
                float *dst = p.sim + (size_t)b * p.P * p.n_vis + j;
                for (int c0 = 0; c0 < p.P; c0 += 8) {
                    float v[8];
                    tmem_ld8(taddr + (uint32_t)c0, v); // warp-collective: rows outside the tile still take part
                    if (row < rows) {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + e < p.P) { // dup = dot / (|pivot| |row|); a zero norm gives 0; a warp writes 128 contiguous bytes
                                const float den = sqrtf(sh.piv_ssq[acc][c0 + e]) * nj;
                                dst[(size_t)(c0 + e) * p.n_vis] = den > 0.f ? v[e] / den : 0.f;
                            }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.tmem_empty[acc]));
                mbar_arrive(smem_u32(&sh.norm_empty[acc]));
            }
            ++n;
        }
    }
    // ---------------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
}

} // namespace onepass
} // namespace dart
