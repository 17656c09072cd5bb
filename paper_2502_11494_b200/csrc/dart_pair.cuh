// Paired sweeps: scores, pivots and similarities (Sec. 3.3 steps 1-3; Def. 1-2, Eq. 7) in one persistent kernel in which
// the SAME CTA reads a block of 16 key rows twice, a short time apart, so that the second read is served by the L2.
//
// A sample's pivots exist only when all of its rows are scored, and Eq. 7 needs the rows again.  What decides whether
// that second read hits the L2 is how many newer bytes pass between a row's two reads.  Here that distance is one
// sample plus what streams while the pivots are found:
//   * every sample is cut into blocks of 16 rows, block t of the batch belongs to CTA t mod G for BOTH sweeps, so all
//     SMs work on the same one or two samples at any time and a sample's second sweep takes as long as its first;
//   * every CTA keeps the best P rows of its own blocks of a sample and publishes them (P keys) with one counter
//     increment; one CTA per sample merges the G short lists as soon as the counter is full and publishes the pivots,
//     so between a sample's last row and its first re-read lie two publications, two polls, one load of 9 KB and a
//     merge of sorted lists;
//   * the second sweep takes the CTA's blocks of a sample together (one or two at the large shapes), stage by stage
//     of 8 atoms (512 columns): the pivot rows' columns of the stage come through a ring of their own, one plain bulk
//     copy of 1 KB per pivot, up to a whole sample ahead (rows 16 bytes further apart than their length, which makes
//     8-row matrix loads conflict-free; four rows per TMA gather op were too slow at this granularity, and copies
//     that travel with the token tiles expose the L2 latency per stage), every block's 16 x 512 token tile as
//     128-byte-swizzled TMA boxes through another; four warps multiply with
//     mma.sync.m16n8k16 (tokens = M 16: exactly one block; pivots = N 8; bf16 -> fp32), two atoms of every stage
//     each, and add their partial products in a fixed order; the first of them normalises (Eq. 7) and writes
//     dup(p_i, x_j).  (tcgen05.mma takes ~120 cycles per 16-column step whatever the tile height: fine for
//     128-row tiles, eight times too slow when a block has 16 rows.)
//
// Per CTA (512 threads):
//   warp 0      sweep-1 producer: bulk copies of four rows per stage into ring 1 (L2 evict_last)
//   warps 4-7   sweep-1 workers: one row per warp and stage: L1 norm (K-norm footnote) and sum of squares
//   warp 12     publisher: keeps the CTA's best P rows of the current sample; writes the list when its last block is in
//   warps 13-14 announcers: make the list visible GPU-wide and count the CTA in (the fence is slow: samples in turn)
//   warp 15     merger (for the samples whose block 0 this CTA owns): waits for the sample's counter, merges the G lists,
//               publishes the pivots and their norms
//   warp 3      resolver: takes every sample's pivots from its merger and hands pivot rows and norms to sweep 2
//   warp 2      sweep-2 producer (token tiles), warp 1: pivot columns, warps 8-11: multiply and epilogue
// Limits: P <= 16, d % 64 == 0, d <= 8192.  Every wait is bounded in time; on expiry the kernel records
// DART_ERR_TIMEOUT in the status words, lets copies and MMAs in flight finish, frees TMEM and exits normally.
// Results are bitwise reproducible: every sum runs in a fixed order.
#pragma once
#include "dart_sweep.cuh"

namespace dart {
namespace pair {
using namespace sweep; // PTX wrappers, bounded waits, rings

constexpr int kBlockRows = 16;            // rows per block: the unit of both sweeps
constexpr int kStageRows = 4;             // sweep 1: rows per ring-1 stage, one per worker warp
constexpr int kStageAtoms = 8;            // sweep 2: 64-column atoms per ring-2 stage
constexpr int kTokAtomBytes = kBlockRows * 128; // 2 KB: 16 rows x 128 bytes, 128B-swizzled
constexpr int kMaxP = 16;                 // pivots: one or two n8 tiles of the MMA
constexpr int kThreads = 512;
constexpr int kProd2Warp = 2, kResolveWarp = 3, kWorker0 = 4, kWorkerWarps = 4, kMul0 = 8, kMulWarps = 4, kPubWarp = 12, kMergeWarp = 15, kPivWarp = 1, kAnn0 = 13, kAnnWarps = 2;
constexpr int kAnn = 4;                   // hand-over slots between the publisher and the announcers
constexpr int kPivPitch = kStageAtoms * 128 + 16; // bytes between pivot rows of a stage in shared memory
constexpr int kMaxStages1 = 6, kMaxStages2 = 6, kMaxStages3 = 8;
constexpr int kMaxBlk = 4;                // blocks of a sample that one CTA multiplies in one pass over the pivot columns
constexpr int kPivSlots = 4;              // samples whose pivots may be resolved ahead of the second sweep
constexpr int kMaxGrid = 192;             // lists per lane of the merge: kMaxGrid / 32
constexpr int kStaticSmemReserve = 12288;
// second status word of a wait that expired
enum { kWaitS1Stage = 40, kWaitS1Rows, kWaitMailFree, kWaitMailFull, kWaitPublished, kWaitPivSlot, kWaitResolved, kWaitS2Stage,
       kWaitS2Tile, kWaitS2Piv, kWaitPivots2, kWaitNorms, kWaitThrottle, kWaitLoaderStage, kWaitAnnFree, kWaitAnnFull };

struct Params {
    int B, S, vis_offset, n_vis, P, d;
    int n_atoms;                       // 64-column atoms per row
    int T1;                            // blocks per sample
    int n1, n2, n3;                    // ring depths: first sweep, token tiles, pivot columns
    int lead;                          // sweep 1 runs at most this many of the CTA's samples ahead of sweep 2 (0: no limit)
    uint32_t row_bytes, stage1_bytes, stage2_bytes, stage3_bytes;
    int norm_kind, smallest;
    int withhold;                      // test hook: 1 = never publish, 2 = never hand the norms to the epilogue
    unsigned long long wait_ns;
    const char *keys;                  // [B][S][d] bf16
    float *sim;                        // [B][P][n_vis]
    float *l1, *ssq;                   // [B][n_vis]
    int32_t *pivot_idx;                // [B][P]
    unsigned long long *cand;          // [B][G][kMaxP]: rank key << 32 | ~index, best first; 0 = none
    int *arrived;                      // [B] CTAs that have published, zero at launch
    int *res_ready;                    // [B] 1 once the sample's pivots are in res, zero at launch
    int32_t *res;                      // [B][2 kMaxP]: pivot indices, then the bits of the pivots' Euclidean norms
    int *status;
};

__host__ __device__ inline uint32_t stage2_bytes(int) { return (uint32_t)kStageAtoms * kTokAtomBytes; }
__host__ __device__ inline uint32_t stage3_bytes(int P) { return ((uint32_t)(P <= 8 ? 8 : 16) * kPivPitch + 127u) / 128u * 128u; }
__host__ __device__ inline uint32_t stage1_bytes(uint32_t row_bytes) { return (kStageRows * row_bytes + 1023u) / 1024u * 1024u; }
__host__ __device__ inline uint32_t cand_smem_bytes(int G, int P) { return (uint32_t)G * (uint32_t)((P + 1) / 2 * 2) * 8u; }
// ring depths for a shared-memory budget: `want3` stages of pivot columns (0: eight = one sample ahead at d = 4096),
// `want2` token stages (0: three), the rest (up to six, or `want1`) for the first sweep
__host__ inline void ring_depths(int P, uint32_t row_bytes, int G, size_t smem_limit, int &n1, int &n2, int &n3, int want1 = 0,
                                 int want2 = 0, int want3 = 0)
{
    n2 = want2 >= 2 && want2 <= kMaxStages2 ? want2 : 3;
    n3 = want3 >= 2 && want3 <= kMaxStages3 ? want3 : (P <= 8 ? 7 : 3);
    const long long left = (long long)smem_limit - kStaticSmemReserve - 1024 - cand_smem_bytes(G, P) - 1024 -
                           (long long)n2 * stage2_bytes(P) - (long long)n3 * stage3_bytes(P);
    long long a = left / (long long)stage1_bytes(row_bytes);
    a = a > kMaxStages1 ? kMaxStages1 : a;
    if (want1 >= 2 && want1 < a) a = want1;
    n1 = (int)(a < 0 ? 0 : a);
}
__host__ inline size_t smem_bytes(int P, uint32_t row_bytes, int G, int n1, int n2, int n3)
{
    return 1024 + (size_t)n2 * stage2_bytes(P) + (size_t)n3 * stage3_bytes(P) + (size_t)n1 * stage1_bytes(row_bytes) + 1024 +
           cand_smem_bytes(G, P);
}

struct Shared {
    unsigned long long full1[kMaxStages1], empty1[kMaxStages1], full2[kMaxStages2], empty2[kMaxStages2];
    unsigned long long full3[kMaxStages3], empty3[kMaxStages3];
    unsigned long long mail_full[kMail], mail_empty[kMail];
    int4 mail[kMail];                      // (sample, block within the sample, 1 if it is this CTA's last block of the sample, -)
    uint32_t mail_keys[kMail][kBlockRows]; // rank keys of the block's rows, larger = better pivot; 0 = no row
    unsigned long long ann_full[kAnn], ann_empty[kAnn];
    int ann[kAnn];                         // samples whose lists are written: to be counted (sample < 0 ends the stream)
    int abort_flag;
    float part[2][kMulWarps][32][8];       // per block parity: every multiplier warp's partial products (fragment order)
    volatile uint32_t resolved;            // own samples whose pivot rows are in piv_row
    volatile uint32_t normed;              // ... whose pivot norms are in piv_norm
    volatile uint32_t s2_done;             // own samples whose second sweep is complete
    long long piv_row[kPivSlots][kMaxP];   // row of the key tensor that holds pivot i
    float piv_norm[kPivSlots][kMaxP];
};
static_assert(sizeof(Shared) + 64 <= kStaticSmemReserve, "static shared memory exceeds its reserve");

// The blocks of one CTA in schedule order: t = c, c + G, ...; sample n = t / T1, block u = t % T1; ord counts the
// samples in which the CTA owns a block.
struct Own {
    uint32_t t, total, G;
    int T1, n, u, ord;
    __device__ Own(const Params &p) : t(blockIdx.x), total((uint32_t)p.B * (uint32_t)p.T1), G(gridDim.x), T1(p.T1), n(-1), u(0), ord(-1) { set(); }
    __device__ __forceinline__ bool valid() const { return t < total; }
    __device__ __forceinline__ void set()
    {
        if (!valid()) return;
        const int nn = (int)(t / (uint32_t)T1);
        u = (int)(t - (uint32_t)nn * (uint32_t)T1);
        if (nn != n) {
            n = nn;
            ++ord;
        }
    }
    __device__ __forceinline__ void next()
    {
        t += G;
        set();
    }
    __device__ __forceinline__ bool last_of_sample() const
    {
        const uint32_t t2 = t + G;
        return t2 >= total || (int)(t2 / (uint32_t)T1) != n;
    }
    // skips to the first block of the next sample in which this CTA owns one
    __device__ __forceinline__ void next_sample()
    {
        const int cur = n;
        while (valid() && n == cur) next();
    }
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Polls a shared-memory counter until it reaches `target`, sleeping between polls (bounded like every other wait).
__device__ inline bool wait_count(const Ctl &ctl, const volatile uint32_t *word, uint32_t target, int where, long long task)
{
    for (int it = 0; it < 8; ++it)
        if (*word >= target) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (*word >= target) return true;
        __nanosleep(40);
        if ((it & 31u) == 31u) {
            if (ctl.aborted()) return false;
            if ((unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                ctl.give_up(where, task);
                return false;
            }
        }
    }
}

// Sixteen warps share four instruction schedulers, and most of them wait most of the time: a warp that polls a barrier in a
// tight loop takes issue slots from the warps that work (the scoring warps ran several times slower next to tight polls).
// So one lane polls and sleeps between polls; the other lanes wait at the shuffle.
constexpr unsigned kPollNs = 32;
__device__ inline bool polite_bar(const Ctl &ctl, uint32_t bar, uint32_t parity, int where, long long task)
{
    for (int it = 0; it < 2; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        __nanosleep(kPollNs);
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 31u) == 31u) {
            if (ctl.aborted()) return false;
            if ((unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                ctl.give_up(where, task);
                return false;
            }
        }
    }
}
// Warp-collective form for warps that read what the barrier guards: lane 0 polls, then every lane observes the completed phase.
__device__ inline bool warp_bar(const Ctl &ctl, uint32_t bar, uint32_t parity, int where, long long task)
{
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = polite_bar(ctl, bar, parity, where, task);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    if (ok) mbar_try_wait(bar, parity);
    return ok;
}

// The largest 64-bit key of the warp in two warp-wide reductions (lanes without a key pass 0); the same in all lanes.
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long key)
{
    const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
    const uint32_t top_hi = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t top_lo = __reduce_max_sync(0xffffffffu, hi == top_hi ? lo : 0u);
    return ((unsigned long long)top_hi << 32) | top_lo;
}

__global__ void __launch_bounds__(kThreads, 1) pair_kernel(const __grid_constant__ CUtensorMap tm_blk, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x, c = (int)blockIdx.x;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // token ring, pivot ring, first-sweep ring, candidate lists
    const uint32_t ring3_0 = smem0 + (uint32_t)p.n2 * p.stage2_bytes;
    const uint32_t ring1_0 = ring3_0 + (uint32_t)p.n3 * p.stage3_bytes;
    const uint32_t cand_off = (ring1_0 - smem_u32(smem_raw)) + (uint32_t)p.n1 * p.stage1_bytes + 1024u;
    unsigned long long *cand_sm = reinterpret_cast<unsigned long long *>(smem_raw + cand_off);
    auto a1_addr = [&](int s) { return ring1_0 + (uint32_t)s * p.stage1_bytes; };
    auto tok_addr = [&](int s) { return smem0 + (uint32_t)s * p.stage2_bytes; };
    auto piv_addr = [&](int s) { return ring3_0 + (uint32_t)s * p.stage3_bytes; };
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    // the waits nearest a possible cause report first: those for another CTA (merger, resolver), then those for this CTA's
    // resolver and memory traffic (first multiplier warp, scoring warps), then the roles that merely depend on them
    const bool waits_for_others = warp == kResolveWarp || warp == kMergeWarp;
    const bool waits_for_those = warp == kMul0 || (warp >= kWorker0 && warp < kWorker0 + kWorkerWarps);
    const Ctl ctl{&sh.abort_flag, p.status, waits_for_others ? limit : waits_for_those ? limit + limit / 8 : limit + limit / 4};
    const int stages_per_block = (p.n_atoms + kStageAtoms - 1) / kStageAtoms;
    const int Ppad = (p.P + 1) / 2 * 2; // list length in shared and global memory (16-byte units)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages1; ++s) {
            mbar_init(smem_u32(&sh.full1[s]), 1);
            mbar_init(smem_u32(&sh.empty1[s]), kWorkerWarps);
        }
        for (int s = 0; s < kMaxStages2; ++s) {
            mbar_init(smem_u32(&sh.full2[s]), 1);
            mbar_init(smem_u32(&sh.empty2[s]), kMulWarps); // every multiplier warp releases a stage by itself
        }
        for (int s = 0; s < kMaxStages3; ++s) {
            mbar_init(smem_u32(&sh.full3[s]), 1);
            mbar_init(smem_u32(&sh.empty3[s]), kMulWarps);
        }
        for (int m = 0; m < kMail; ++m) {
            mbar_init(smem_u32(&sh.mail_full[m]), 1);
            mbar_init(smem_u32(&sh.mail_empty[m]), 1);
        }
        for (int m = 0; m < kAnn; ++m) {
            mbar_init(smem_u32(&sh.ann_full[m]), 1);
            mbar_init(smem_u32(&sh.ann_empty[m]), 1);
        }
        sh.abort_flag = 0;
        sh.resolved = 0, sh.normed = 0, sh.s2_done = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ sweep-1 producer
        if (lane == 0) {
            unsigned long long pol_keep; // the same CTA reads the row again a few microseconds later
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            Ring ring(p.n1);
            long long issued = 0;
            bool ok = true;
            for (Own o(p); ok && o.valid(); o.next()) {
                if (p.lead > 0 && o.ord >= p.lead) // not too far ahead of the second sweep: its re-reads should still hit the L2
                    ok = wait_count(ctl, &sh.s2_done, (uint32_t)(o.ord - p.lead + 1), kWaitThrottle, o.t);
                if (!ok) break;
                const int row0 = o.u * kBlockRows, rows = min(kBlockRows, p.n_vis - row0);
                const char *src = p.keys + ((size_t)o.n * p.S + p.vis_offset + row0) * (size_t)p.row_bytes;
                for (int r = 0; r < rows; r += kStageRows) {
                    const uint32_t bytes = (uint32_t)min(kStageRows, rows - r) * p.row_bytes;
                    ok = polite_bar(ctl, smem_u32(&sh.empty1[ring.stage]), ring.phase ^ 1u, kWaitS1Stage, o.t);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&sh.full1[ring.stage]);
                    mbar_arrive_expect_tx(full, bytes);
                    bulk_load(a1_addr(ring.stage), src + (size_t)r * p.row_bytes, bytes, full, pol_keep);
                    ring.advance();
                    ++issued;
                }
            }
            if (!ok || ctl.aborted()) // drain: let the copies already issued land before the CTA may exit
                for (long long i = issued > p.n1 ? issued - p.n1 : 0; i < issued; ++i)
                    ctl.wait_landed(smem_u32(&sh.full1[i % p.n1]), (uint32_t)((i / p.n1) & 1));
        }
    } else if (warp >= kWorker0 && warp < kWorker0 + kWorkerWarps) {
        // ------------------------------------------------------------------ sweep-1 workers: one row per warp and stage
        const int wq = warp - kWorker0, wt = (int)threadIdx.x - kWorker0 * 32;
        const int d8 = p.d / 8;
        Ring ring(p.n1);
        int ms = 0;
        uint32_t mph = 0;
        bool dead = false; // warp-uniform inside a block, group-uniform after every workers_any()
        for (Own o(p); o.valid(); o.next()) {
            const int row0 = o.u * kBlockRows, rows = min(kBlockRows, p.n_vis - row0);
            uint32_t key[kBlockRows / kStageRows];
#pragma unroll
            for (int k = 0; k < kBlockRows / kStageRows; ++k) key[k] = 0;
#pragma unroll
            for (int k = 0; k < kBlockRows / kStageRows; ++k) {
                const int r = k * kStageRows;
                if (r >= rows) break;
                // warp-uniform: either the whole warp reads the stage and releases it, or none of it does
                if (!dead) dead = !warp_bar(ctl, smem_u32(&sh.full1[ring.stage]), ring.phase, kWaitS1Rows, o.t);
                if (!dead && r + wq < rows) {
                    const uint32_t base = a1_addr(ring.stage) + (uint32_t)wq * p.row_bytes + (uint32_t)lane * 16u;
                    float a0 = 0.f, a1 = 0.f, q0 = 0.f, q1 = 0.f;
                    // lanes read consecutive 16-byte chunks (no bank conflicts).  Kept as a small loop on purpose: sixteen warps
                    // run nine different roles, and with the sums unrolled eight loads deep the same work took 1.7x as long
#pragma unroll 1
                    for (int ch = lane; ch < d8; ch += 64) {
                        const uint4 v0 = lds128(base + (uint32_t)(ch - lane) * 16u);
                        const uint4 v1 = ch + 32 < d8 ? lds128(base + (uint32_t)(ch - lane + 32) * 16u) : make_uint4(0, 0, 0, 0);
                        const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float lo = bf16_lo(w[e]), hi = bf16_hi(w[e]);
                            a0 += fabsf(lo);
                            a1 += fabsf(hi);
                            q0 = fmaf(lo, lo, q0);
                            q1 = fmaf(hi, hi, q1);
                        }
                    }
                    const float a = warp_sum(a0 + a1), q = warp_sum(q0 + q1); // fixed order; every lane gets the sum
                    if (lane == 0) {
                        const size_t at = (size_t)o.n * p.n_vis + row0 + r + wq;
                        p.l1[at] = a;
                        p.ssq[at] = q;
                    }
                    const uint32_t okey = order_key(p.norm_kind == 2 ? q : a);
                    key[k] = p.smallest ? ~okey : okey;
                    if (key[k] == 0) key[k] = 1; // 0 marks "no row"
                }
                __syncwarp(); // the warp's reads of the stage are done
                if (!dead && lane == 0) mbar_arrive(smem_u32(&sh.empty1[ring.stage]));
                ring.advance();
            }
            // hand the block's keys to the publisher: a free mail slot, the keys, then the mail itself
            if (wt == 0 && !dead) dead = !polite_bar(ctl, smem_u32(&sh.mail_empty[ms]), mph ^ 1u, kWaitMailFree, o.t);
            dead = workers_any(dead);
            if (!dead && lane == 0)
#pragma unroll
                for (int k = 0; k < kBlockRows / kStageRows; ++k) sh.mail_keys[ms][k * kStageRows + wq] = key[k];
            dead = workers_any(dead);
            if (wt == 0 && !dead) {
                sh.mail[ms] = make_int4(o.n, o.u, o.last_of_sample() ? 1 : 0, 0);
                mbar_arrive(smem_u32(&sh.mail_full[ms])); // release: the group's scores and keys are ordered before it
            }
            if (++ms == kMail) {
                ms = 0;
                mph ^= 1u;
            }
            if (dead) break;
        }
        dead = workers_any(dead);
        if (wt == 0) { // end mark (also after a failure, so that the publisher exits): needs a free slot, bounded
            if (polite_bar(ctl, smem_u32(&sh.mail_empty[ms]), mph ^ 1u, kWaitMailFree, -1)) {
                sh.mail[ms] = make_int4(-1, 0, 0, 0);
                mbar_arrive(smem_u32(&sh.mail_full[ms]));
            }
        }
    } else if (warp == kPubWarp) {
        // ------------------------------------------------------------------ publisher: the CTA's best P rows of the current sample
        // Lanes 0-15 take the 16 rows of the block that came in, lanes 16-31 hold the list so far; P rounds of a warp-wide
        // maximum give the new list (keys are distinct: they carry the row index).
        unsigned long long held = 0ull; // lane 16 + i: the i-th best row so far
        uint32_t handed = 0;
        for (uint32_t m = 0;; ++m) {
            const int slot = (int)(m % kMail);
            bool ok = true;
            if (lane == 0) ok = polite_bar(ctl, smem_u32(&sh.mail_full[slot]), (m / kMail) & 1u, kWaitMailFull, m);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            mbar_try_wait(smem_u32(&sh.mail_full[slot]), (m / kMail) & 1u); // every lane observes the completed phase
            const int4 mail = sh.mail[slot];
            if (mail.x < 0) break;
            unsigned long long pool = held;
            if (lane < kBlockRows) {
                const uint32_t rk = sh.mail_keys[slot][lane];
                const uint32_t idx = (uint32_t)(mail.y * kBlockRows + lane);
                pool = rk ? ((unsigned long long)rk << 32) | (0xffffffffu - idx) : 0ull; // equal scores: lower index first
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.mail_empty[slot]));
            unsigned long long sel = 0ull; // lane i: the i-th best of list and block together
#pragma unroll 1
            for (int i = 0; i < p.P; ++i) {
                const unsigned long long best = warp_max_key(pool);
                if (lane == i) sel = best;
                if (pool == best) pool = 0ull;
            }
            held = __shfl_sync(0xffffffffu, sel, lane & 15);
            if (lane < 16 || lane - 16 >= p.P) held = 0ull;
            if (mail.z) { // the CTA's last block of this sample: the list, then (by an announcer warp) the count
                const unsigned long long k0 = __shfl_sync(0xffffffffu, sel, (2 * lane) & 31), k1 = __shfl_sync(0xffffffffu, sel, (2 * lane + 1) & 31);
                if (2 * lane < Ppad)
                    __stcg(reinterpret_cast<ulonglong2 *>(p.cand + ((size_t)mail.x * G + c) * kMaxP + 2 * lane),
                           make_ulonglong2(k0, 2 * lane + 1 < p.P ? k1 : 0ull));
                held = 0ull;
                const int as = (int)(handed % kAnn);
                if (lane == 0) ok = polite_bar(ctl, smem_u32(&sh.ann_empty[as]), ((handed / kAnn) & 1u) ^ 1u, kWaitAnnFree, mail.x);
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0; // also orders the lanes' list stores before the hand-over
                if (!ok) break;
                if (lane == 0) {
                    sh.ann[as] = mail.x;
                    mbar_arrive(smem_u32(&sh.ann_full[as])); // release: the warp's list stores are ordered before it
                }
                ++handed;
            }
        }
        // end marks for both announcers (also after a failure: their own waits are bounded anyway)
        for (int e = 0; e < kAnnWarps; ++e) {
            const int as = (int)(handed % kAnn);
            bool ok = true;
            if (lane == 0) ok = polite_bar(ctl, smem_u32(&sh.ann_empty[as]), ((handed / kAnn) & 1u) ^ 1u, kWaitAnnFree, -1);
            if (lane == 0 && ok) {
                sh.ann[as] = -1;
                mbar_arrive(smem_u32(&sh.ann_full[as]));
            }
            ++handed;
        }
    } else if (warp == kAnn0 || warp == kAnn0 + 1) {
        // ------------------------------------------------------------------ announcers: fence and count, one thread each, samples in turn
        // The fence that makes the list and the scores visible GPU-wide takes microseconds under load; two warps take
        // the samples in turn so that it is not paid once per sample in a row.
        if (lane == 0) {
            for (uint32_t j = (uint32_t)(warp - kAnn0);; j += kAnnWarps) {
                const int as = (int)(j % kAnn);
                if (!polite_bar(ctl, smem_u32(&sh.ann_full[as]), (j / kAnn) & 1u, kWaitAnnFull, j)) break;
                const int n = sh.ann[as];
                mbar_arrive(smem_u32(&sh.ann_empty[as]));
                if (n < 0) break;
                __threadfence(); // the list and the workers' scores (ordered before the hand-over) become visible GPU-wide
                if (p.withhold != 1) atomicAdd(p.arrived + n, 1);
            }
        }
    } else if (warp == kMergeWarp) {
        // ------------------------------------------------------------------ merger: the pivots of the samples whose block 0 this CTA owns
        // ONE CTA per sample merges the G lists and publishes the pivots with their norms; every CTA (this one too) takes
        // them from there.  A load of all lists and a merge in every CTA took longer than a sample takes to stream.  The
        // merger waits for nothing but the lists, so the merges of consecutive samples, in different CTAs, overlap.
        const int n_lists = (G + 31) / 32;
        const int contributors = p.T1 < G ? p.T1 : G;
        bool ok = true;
        for (int n = 0; ok && n < p.B; ++n) {
            const uint32_t first = (uint32_t)(((long long)n * p.T1) % G); // owner of the sample's block 0
            if (c != (int)first) continue;
            if (lane == 0) ok = ctl.wait_flag(p.arrived + n, kWaitPublished, n, contributors);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            // the G lists into shared memory, 16 bytes per copy, all copies of the warp in flight at once
            auto owns = [&](int cc) { return cc < G && (uint32_t)((cc - (int)first + G) % G) < (uint32_t)p.T1; }; // CTA cc owns blocks of this sample
            const int per_list = Ppad / 2, n_copies = G * per_list;
            for (int id = lane; id < n_copies; id += 32) {
                const int cc = id / per_list, i = id - cc * per_list;
                if (owns(cc)) cp_async16(smem_u32(cand_sm + (size_t)cc * Ppad + 2 * i), p.cand + ((size_t)n * G + cc) * kMaxP + 2 * i);
            }
            cp_async_commit();
            cp_async_wait<0>();
            __syncwarp(); // every lane's copies have landed
            // lane l merges the lists of CTAs l, l + 32, ...
            int head[kMaxGrid / 32];
#pragma unroll
            for (int u = 0; u < kMaxGrid / 32; ++u) head[u] = (u < n_lists && owns(lane + 32 * u)) ? 0 : kMaxP;
            unsigned long long cur[kMaxGrid / 32]; // the head of every list; only the list that wins reads its next key
            unsigned long long mine = 0ull;
#pragma unroll
            for (int u = 0; u < kMaxGrid / 32; ++u) {
                cur[u] = head[u] < p.P ? cand_sm[(size_t)(lane + 32 * u) * Ppad] : 0ull;
                mine = cur[u] > mine ? cur[u] : mine;
            }
            int my_piv = 0;
#pragma unroll 1
            for (int i = 0; i < p.P; ++i) { // P rounds: the warp's best key wins, its lane moves that list on
                const unsigned long long best = warp_max_key(mine);
                if (lane == i) my_piv = (int)(0xffffffffu - (uint32_t)best);
                if (best != 0ull && mine == best) {
                    mine = 0ull;
#pragma unroll
                    for (int u = 0; u < kMaxGrid / 32; ++u) {
                        if (cur[u] == best) {
                            ++head[u];
                            cur[u] = head[u] < p.P ? cand_sm[(size_t)(lane + 32 * u) * Ppad + head[u]] : 0ull;
                        }
                        mine = cur[u] > mine ? cur[u] : mine;
                    }
                }
            }
            my_piv = min(max(my_piv, 0), p.n_vis - 1);
            if (lane < p.P) {
                // the pivots' sums of squares were written by the CTAs that scored them, before they published
                const float my_norm = sqrtf(__ldcg(p.ssq + (size_t)n * p.n_vis + my_piv));
                p.pivot_idx[(size_t)n * p.P + lane] = my_piv;
                __stcg(p.res + (size_t)n * (2 * kMaxP) + lane, my_piv);
                __stcg(p.res + (size_t)n * (2 * kMaxP) + kMaxP + lane, (int)__float_as_uint(my_norm));
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence();
                st_release(p.res_ready + n, 1);
            }
        }
    } else if (warp == kResolveWarp) {
        // ------------------------------------------------------------------ resolver: the pivots of this CTA's samples, in order
        bool ok = true;
        for (Own o(p); ok && o.valid(); o.next_sample()) {
            const int n = o.n, ord = o.ord;
            // the slot is free once the second sweep of the sample kPivSlots before this one is complete
            if (ord >= kPivSlots) ok = wait_count(ctl, &sh.s2_done, (uint32_t)(ord - kPivSlots + 1), kWaitPivSlot, n);
            if (ok && lane == 0) ok = ctl.wait_flag(p.res_ready + n, kWaitPivots2, n, 1);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            const int slot = ord % kPivSlots;
            if (lane < p.P) {
                const int piv = min(max(__ldcg(p.res + (size_t)n * (2 * kMaxP) + lane), 0), p.n_vis - 1);
                sh.piv_row[slot][lane] = (long long)n * p.S + p.vis_offset + piv;
                sh.piv_norm[slot][lane] = __uint_as_float((uint32_t)__ldcg(p.res + (size_t)n * (2 * kMaxP) + kMaxP + lane));
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                sh.resolved = (uint32_t)(ord + 1); // the second sweep of this sample may start
                if (p.withhold != 2) sh.normed = (uint32_t)(ord + 1);
            }
        }
    } else if (warp == kProd2Warp) {
        // ------------------------------------------------------------------ sweep-2 producer: token tiles, stage by stage over the pass's blocks
        unsigned long long pol_drop;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_drop)); // the row's last use
        Ring ring(p.n2);
        long long issued = 0;
        bool ok = true;
        for (Own o(p); ok && o.valid();) {
            const int n = o.n, ord = o.ord;
            int us[kMaxBlk], cnt = 0;
            while (o.valid() && o.n == n && cnt < kMaxBlk) us[cnt++] = o.u, o.next(); // one pass: up to kMaxBlk own blocks of the sample
            if (lane == 0) ok = wait_count(ctl, &sh.resolved, (uint32_t)(ord + 1), kWaitResolved, n);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            for (int st = 0; ok && st < stages_per_block; ++st) {
                const int a0 = st * kStageAtoms, na = min(kStageAtoms, p.n_atoms - a0);
#pragma unroll
                for (int b = 0; b < kMaxBlk; ++b) {
                    if (b >= cnt || !ok) break;
                    const uint32_t full = smem_u32(&sh.full2[ring.stage]);
                    if (lane == 0) {
                        ok = polite_bar(ctl, smem_u32(&sh.empty2[ring.stage]), ring.phase ^ 1u, kWaitS2Stage, n);
                        if (ok) mbar_arrive_expect_tx(full, (uint32_t)na * kTokAtomBytes); // rows past the tensor's end are filled, and counted
                    }
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (!ok) break;
                    if (lane < na) // one lane per atom: issued side by side
                        tma_load_2d(tok_addr(ring.stage) + (uint32_t)lane * kTokAtomBytes, &tm_blk, (a0 + lane) * kAtomCols,
                                    n * p.S + p.vis_offset + us[b] * kBlockRows, full, pol_drop);
                    ring.advance();
                    ++issued;
                }
            }
        }
        if ((!ok || ctl.aborted()) && lane == 0) // drain: let the copies already issued land before the CTA may exit
            for (long long i = issued > p.n2 ? issued - p.n2 : 0; i < issued; ++i)
                ctl.wait_landed(smem_u32(&sh.full2[i % p.n2]), (uint32_t)((i / p.n2) & 1));
    } else if (warp == kPivWarp) {
        // ------------------------------------------------------------------ pivot columns: one bulk copy per pivot and stage
        unsigned long long pol_keep;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep)); // every CTA reads the pivot rows
        Ring ring(p.n3);
        long long issued = 0;
        bool ok = true;
        for (Own o(p); ok && o.valid();) {
            const int n = o.n, ord = o.ord;
            int cnt = 0;
            while (o.valid() && o.n == n && cnt < kMaxBlk) ++cnt, o.next(); // one pass over the pivot columns per kMaxBlk own blocks
            if (lane == 0) ok = wait_count(ctl, &sh.resolved, (uint32_t)(ord + 1), kWaitResolved, n);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            const char *src = lane < p.P ? p.keys + (size_t)sh.piv_row[ord % kPivSlots][lane] * p.row_bytes : nullptr;
            for (int st = 0; st < stages_per_block; ++st) {
                const int a0 = st * kStageAtoms, na = min(kStageAtoms, p.n_atoms - a0);
                const uint32_t full = smem_u32(&sh.full3[ring.stage]);
                if (lane == 0) {
                    ok = polite_bar(ctl, smem_u32(&sh.empty3[ring.stage]), ring.phase ^ 1u, kWaitLoaderStage, n);
                    if (ok) mbar_arrive_expect_tx(full, (uint32_t)p.P * (uint32_t)na * 128u);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                if (lane < p.P)
                    bulk_load(piv_addr(ring.stage) + (uint32_t)lane * kPivPitch, src + (size_t)a0 * 128u, (uint32_t)na * 128u, full, pol_keep);
                ring.advance();
                ++issued;
            }
        }
        if ((!ok || ctl.aborted()) && lane == 0) // drain: let the copies already issued land before the CTA may exit
            for (long long i = issued > p.n3 ? issued - p.n3 : 0; i < issued; ++i)
                ctl.wait_landed(smem_u32(&sh.full3[i % p.n3]), (uint32_t)((i / p.n3) & 1));
    } else if (warp >= kMul0 && warp < kMul0 + kMulWarps) {
        // ------------------------------------------------------------------ sweep 2: multiply, add up, normalise, write
        const int mw = warp - kMul0;       // this warp takes atoms 2 mw and 2 mw + 1 of every stage
        const int g = lane >> 2, t = lane & 3;
        const int n_tiles = p.P > 8 ? 2 : 1; // n8 tiles of pivots
        // ldmatrix row addresses.  Tokens, inside a 128B-swizzled atom (rows of 128 bytes; 16-byte chunk ch of row r at
        // position ch ^ (r & 7)): matrix lane / 8 = (rows 0-7 | rows 8-15) x (chunk 2k | chunk 2k + 1).  Pivots, plain rows
        // kPivPitch bytes apart: rows 0-7, chunk 2k | 2k + 1 of the atom.
        const int ar = (lane & 7) + ((lane >> 3) & 1) * 8, ac = lane >> 4;
        const int br = lane & 7, bc = (lane >> 3) & 1;
        Ring ring2(p.n2), ring3(p.n3);
        uint32_t nb = 0;
        bool dead = false; // warp-uniform inside a pass, group-uniform after every group_any()
        for (Own o(p); o.valid();) {
            const int n = o.n, ord = o.ord;
            int us[kMaxBlk], cnt = 0;
            while (o.valid() && o.n == n && cnt < kMaxBlk) us[cnt++] = o.u, o.next();
            const bool last_pass = !(o.valid() && o.n == n);
            float acc[kMaxBlk][2][4];
#pragma unroll
            for (int b = 0; b < kMaxBlk; ++b)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[b][nt][e] = 0.f;
            for (int st = 0; st < stages_per_block; ++st) {
                const int na = min(kStageAtoms, p.n_atoms - st * kStageAtoms);
                if (!dead) dead = !warp_bar(ctl, smem_u32(&sh.full3[ring3.stage]), ring3.phase, kWaitS2Piv, n);
#pragma unroll
                for (int b = 0; b < kMaxBlk; ++b) {
                    if (b >= cnt) break;
                    if (!dead) dead = !warp_bar(ctl, smem_u32(&sh.full2[ring2.stage]), ring2.phase, kWaitS2Tile, n);
                    if (!dead) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int a = 2 * mw + h;
                            if (a < na) {
                                const uint32_t ta = tok_addr(ring2.stage) + (uint32_t)a * kTokAtomBytes + (uint32_t)ar * 128u;
                                const uint32_t pa = piv_addr(ring3.stage) + (uint32_t)br * kPivPitch + (uint32_t)a * 128u;
#pragma unroll
                                for (int k = 0; k < kAtomCols / 16; ++k) {
                                    uint32_t a0, a1, a2, a3, b0, b1;
                                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                                                 : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                                                 : "r"(ta + (uint32_t)(((2 * k + ac) ^ (ar & 7)) * 16)));
                                    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];"
                                                 : "=r"(b0), "=r"(b1)
                                                 : "r"(pa + (uint32_t)((2 * k + bc) * 16)));
                                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                                 : "+f"(acc[b][0][0]), "+f"(acc[b][0][1]), "+f"(acc[b][0][2]), "+f"(acc[b][0][3])
                                                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
                                    if (n_tiles > 1) { // pivots 8-15
                                        asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];"
                                                     : "=r"(b0), "=r"(b1)
                                                     : "r"(pa + 8u * kPivPitch + (uint32_t)((2 * k + bc) * 16)));
                                        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                                     : "+f"(acc[b][1][0]), "+f"(acc[b][1][1]), "+f"(acc[b][1][2]), "+f"(acc[b][1][3])
                                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
                                    }
                                }
                            }
                        }
                    }
                    __syncwarp(); // the warp's reads of the token stage are done
                    if (!dead && lane == 0) mbar_arrive(smem_u32(&sh.empty2[ring2.stage]));
                    ring2.advance();
                }
                __syncwarp(); // ... and of the pivot stage
                if (!dead && lane == 0) mbar_arrive(smem_u32(&sh.empty3[ring3.stage]));
                ring3.advance();
            }
            // per block: the four warps' partial products, added in a fixed order by the first of them
            if (mw == 0 && !dead && lane == 0) dead = !wait_count(ctl, &sh.normed, (uint32_t)(ord + 1), kWaitNorms, n);
#pragma unroll
            for (int b = 0; b < kMaxBlk; ++b) {
                if (b >= cnt) break;
                const int rows = min(kBlockRows, p.n_vis - us[b] * kBlockRows);
                float nj[2] = {0.f, 0.f};
                if (mw == 0 && !dead) { // the rows' sums of squares were written by this CTA's workers during the first sweep
                    const float *q = p.ssq + (size_t)n * p.n_vis + us[b] * kBlockRows;
                    if (g < rows) nj[0] = __ldcg(q + g);
                    if (g + 8 < rows) nj[1] = __ldcg(q + g + 8);
                }
                float *mine = sh.part[nb & 1][mw][lane];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) mine[nt * 4 + e] = acc[b][nt][e];
                dead = group_any<3, kMulWarps * 32>(dead); // everyone's partial products are written
                if (dead) break;
                if (mw == 0) {
                    const float *pn = sh.piv_norm[ord % kPivSlots];
                    float v[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = sh.part[nb & 1][0][lane][e];
                    for (int w = 1; w < kMulWarps; ++w)
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] += sh.part[nb & 1][w][lane][e];
                    // fragment order: v[4 nt + 2 hi + e] = row g + 8 hi, pivot 8 nt + 2 t + e
                    float *dst = p.sim + (size_t)n * p.P * p.n_vis + us[b] * kBlockRows;
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int hi = 0; hi < 2; ++hi)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int i = 8 * nt + 2 * t + e, r = g + 8 * hi;
                                if (i < p.P && r < rows) { // dup = dot / (|pivot| |row|); a zero norm gives 0
                                    const float den = pn[i] * sqrtf(nj[hi]);
                                    dst[(size_t)i * p.n_vis + r] = den > 0.f ? v[4 * nt + 2 * hi + e] / den : 0.f;
                                }
                            }
                }
                ++nb;
            }
            if (dead) break;
            if (mw == 0 && last_pass) {
                __syncwarp();
                if (lane == 0) {
                    __threadfence_block();
                    sh.s2_done = (uint32_t)(ord + 1);
                }
            }
        }
    }
}

} // namespace pair
} // namespace dart
