// Fused path, sweeps: ONE persistent kernel computes the scores (sweep 1), the pivots and the
// pivot x token dot products (sweep 2) of a whole batch, so that the second read of a key row can be
// served by the L2 cache instead of HBM.
//
// Sweep-1 task: 16 whole key rows (one contiguous block of 16 * d * 2 bytes), streamed through shared
// memory four rows at a time; each of four worker warps sums one row (L1 norm: the K-norm of the
// Sec. 3.3 footnote; sum of squares: Eq. 7's denominator) and writes the final values - no partial sums.
// Sweep-2 task: 128 rows x all d columns, streamed as 128-byte-swizzled TMA tiles of 64 columns and
// multiplied on the tensor cores with the sample's pivot rows, accumulating over all of d in TMEM
// (Eq. 7's numerator); the epilogue divides by the two norms and writes dup(p_i, x_j) (Eq. 7).
// Both kinds of task sit in one global, static order: step q = (sweep-1 slot q, sweep-2 slot q - lag),
// CTA c runs steps c, c + grid, ...  A sweep-2 task therefore follows the sweep-1 pass over its sample
// by `lag` steps: enough for the sample's pivots to have been selected and published meanwhile.
//
// Per CTA (512 threads; warp 3 idles):
//   warp 0     sweep-1 producer: bulk copies into ring 1
//   warp 2     sweep-2 producer: waits for the sample's pivots, then TMA tiles (L2 evict_first) and the
//              pivot rows (tile::gather4 straight from the key tensor) into ring 2
//   warp 1     sweep 2: one thread issues tcgen05.mma (tokens = M 128, pivots = N, bf16 -> fp32 in TMEM)
//   warps 4-7  sweep-1 workers (one row per warp and stage)
//   warps 8-11 sweep-2 epilogue: TMEM -> normalised similarities [B][P][n_vis] in global memory
//   warp 12    counter: counts finished sweep-1 tasks (the fence and the atomic are kept off the
//              workers by a mailbox); when it counts a sample's LAST task it hands the sample over to
//   warps 13-15 selection: wait until all of the sample's tasks are counted, select the pivots (Def. 1)
//              by a radix select in shared memory and publish them.  Counting never waits for a selection.
// Each ring has one producer and one consumer role, so no role ever skips a barrier phase.
// Every result is bitwise reproducible: all sums run in a fixed order.
//
// Every wait (mbarrier, flag or lock) is bounded in time; on expiry the kernel records
// DART_ERR_TIMEOUT in the status word, drains and exits normally.
#pragma once
#include <cuda.h>

#include "dart_common.cuh"

namespace dart {
namespace sweep {

constexpr int kTileRows = 128;   // sweep-2 tile rows (MMA M)
constexpr int kAtomCols = 64;    // 64 bf16 = 128 bytes = one swizzle row
constexpr int kSubRows = 32;     // rows per TMA box of a short last tile
constexpr int kS1Rows = 16;      // rows per sweep-1 task
constexpr int kS1StageRows = 4;  // rows per sweep-1 stage: one per worker warp
constexpr int kMaxRowBytes = 16384; // widest row the fused path takes (d <= 8192)
constexpr int kMaxStages = 8;    // per ring
constexpr int kAtomBytes = kTileRows * 128; // 16 KB: 128 rows x 128 bytes, 128B-swizzled, K-major
constexpr int kSubBytes = kSubRows * 128;
constexpr int kThreads = 512;
constexpr int kProducer2Warp = 2;
constexpr int kWorkerWarp0 = 4, kWorkerWarps = 4, kWorkers = kWorkerWarps * 32;
constexpr int kEpiWarp0 = 8, kEpiWarps = 4; // kEpiWarp0 % 4 == 0: warp w reads TMEM lanes 32 (w % 4) ...
constexpr int kCountWarp = 12, kSelWarp0 = 13, kSelWarps = 3, kSel = kSelWarps * 32;
constexpr int kDuty = 4;         // samples waiting for their selection
constexpr int kMaxN = 256;       // pivots per MMA (N dimension)
constexpr int kMail = 8;         // mailbox slots between the workers and the counter warp
constexpr int kSelMax = 4096;    // scores of a sample that fit the shared-memory select buffer
constexpr int kArgminMaxP = 32;  // up to this many pivots: P rounds of group-wide argmin; above: radix select
constexpr int kStaticSmemReserve = 28672;
constexpr int kStatusTimeout = -7;
// which wait expired (second status word)
enum { kWaitPivots = 1, kWaitEmptyStage, kWaitDrain, kWaitAccumFree, kWaitStageMma, kWaitStageRows, kWaitAccumFull,
       kWaitMailSlot, kWaitMail, kWaitTasks, kWaitDutySlot, kWaitDuty, kWaitAhead };

using Workers = WarpGroup<kWorkerWarp0, kWorkerWarps, 1>;
using Selectors = WarpGroup<kSelWarp0, kSelWarps, 2>;

struct Params {
    int B, S, vis_offset, n_vis, P, N; // N = P rounded up to a multiple of 16 (MMA N)
    int d8;                            // row width in 16-byte units
    int n_atoms, n_rt;                 // sweep 2: 64-column atoms per row; row tiles per sample
    int n_kc, apc;                     // sweep 2: column chunks per row tile (tasks per tile) and atoms per chunk
    int T1, T2, Tm;                    // tasks per sample: sweep 1, sweep 2; slots per sample = max of both
    int n1, n2;                        // depth of ring 1 and ring 2 (<= kMaxStages each)
    uint32_t row_bytes, stage1_bytes;  // d * 2; shared-memory bytes of a ring-1 stage (4 rows, 1 KB granules)
    uint32_t lag;                      // steps between the two sweeps (Tm <= lag <= B * Tm)
    int norm_kind, smallest;
    int withhold_pivots;               // test hook: never publish pivots, so that the bounded waits expire
    int keep_l2;                       // first-pass reads ask the L2 to keep the row (the second pass follows within microseconds)
    uint32_t ahead;                    // 0: no limit; else the first pass runs at most this many steps ahead of the CTA's second pass
    unsigned long long wait_ns;        // time limit of every wait
    const char *keys;                  // [B][S][d] bf16
    float *sim;                        // [B][P][n_vis] dup(p_i, x_j); with n_kc > 1: [n_kc][B][P][n_vis], every chunk's share of it
    float *l1, *ssq;                   // [B][n_vis]
    int32_t *pivot_idx;                // [B][P]
    int *s1_done;                      // [B] sweep-1 tasks counted per sample
    int *piv_ready;                    // [B] 1 once the pivots of the sample are published
    int *status;
};

struct Task {
    int b;
    int u;      // sweep 1: task index within the sample (rows 16 u ...)
    int rt, kc; // sweep 2: row tile and column chunk
};

// Schedule.  Every sample owns Tm consecutive slots in each sweep (a slot beyond the sweep's own task count is
// empty).  Step q = (sweep-1 slot q, sweep-2 slot q - lag).  The host guarantees B * Tm + lag < 2^30.
__device__ __forceinline__ uint32_t total_steps(const Params &p) { return (uint32_t)p.B * (uint32_t)p.Tm + p.lag; }

// kind 0: sweep-1 task of step q; kind 1: its sweep-2 task.  Returns false if the step has no such task.
__device__ __forceinline__ bool decode(const Params &p, uint32_t q, int kind, Task &t)
{
    const uint32_t n_all = (uint32_t)p.B * (uint32_t)p.Tm;
    if (kind == 0 ? q >= n_all : q < p.lag) return false;
    const uint32_t n = kind ? q - p.lag : q, Tm = (uint32_t)p.Tm;
    t.b = (int)(n / Tm);
    const uint32_t u = n - (uint32_t)t.b * Tm;
    t.u = (int)u;
    if (kind == 0) return u < (uint32_t)p.T1;
    // a sample's T2 sweep-2 tasks are spread evenly over its Tm slots (every stride-th slot carries one)
    const uint32_t stride = Tm / (uint32_t)p.T2, idx = u / stride;
    t.rt = (int)(idx / (uint32_t)p.n_kc), t.kc = (int)(idx - (uint32_t)t.rt * (uint32_t)p.n_kc); // a tile's chunks side by side
    return u % stride == 0 && idx < (uint32_t)p.T2;
}


// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *ptr) { return (uint32_t)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return ok != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar,
                                            unsigned long long policy)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
                 "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(policy)
                 : "memory");
}
// Plain bulk copy of `bytes` contiguous bytes (16-byte aligned, a multiple of 16) into shared memory.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, unsigned long long policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}
// Four rows (given by index) x one box width of columns -> four consecutive 128-byte rows at dst.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *tm, int x, int r0, int r1, int r2, int r3,
                                            uint32_t bar, unsigned long long policy)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;" ::"r"(dst),
                 "l"(tm), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ int ld_acquire(const int *ptr)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int *ptr, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// OR of a predicate over a 128-thread warp group; doubles as the group's barrier
template <int kBarrierId, int kCount>
__device__ __forceinline__ bool group_any(bool pred)
{
    uint32_t r;
    asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbar.red.or.pred p, %2, %3, q;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(r)
                 : "r"((uint32_t)pred), "n"(kBarrierId), "n"(kCount)
                 : "memory");
    return r != 0;
}
__device__ __forceinline__ bool workers_any(bool pred) { return group_any<1, kWorkers>(pred); }
__device__ __forceinline__ bool selectors_any(bool pred) { return group_any<2, kSel>(pred); }

// Shared-memory matrix descriptor of a K-major, 128B-swizzled bf16 tile (rows at a 128-byte pitch,
// groups of 8 rows 1024 bytes apart).
__device__ __forceinline__ unsigned long long umma_desc(uint32_t saddr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((saddr & 0x3ffffu) >> 4);  // start address
    d |= (unsigned long long)1 << 16;                    // leading byte offset (unused for this layout)
    d |= (unsigned long long)(1024 >> 4) << 32;          // stride byte offset: 8 rows x 128 bytes
    d |= (unsigned long long)1 << 46;                    // descriptor version of sm_100
    d |= (unsigned long long)2 << 61;                    // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileRows >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, unsigned long long da, unsigned long long db, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
                 "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float *v)
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// ---- bounded waits --------------------------------------------------------------------------------
struct Ctl {
    volatile int *abort_flag; // shared memory
    int *status;              // global status word
    unsigned long long limit_cycles; // SM clock cycles (the clock runs at <= 2.1 GHz)
    __device__ __forceinline__ bool aborted() const { return *abort_flag != 0; }
    // records the first wait that expired: status[1] = where (kWait*), status[2] = task index, status[3] = CTA
    __device__ void give_up(int where, long long task) const
    {
        *abort_flag = 1;
        if (atomicCAS(status, 0, kStatusTimeout) == 0) {
            status[1] = where;
            status[2] = (int)task;
            status[3] = (int)blockIdx.x;
        }
    }
    // Waits poll without any bookkeeping first; only a wait that lasts starts reading the SM's cycle
    // counter (cheap, unlike the global nanosecond timer) and compares it with the limit.
    __device__ bool wait_bar(uint32_t bar, uint32_t parity, int where, long long task) const
    {
        for (int it = 0; it < 64; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        const long long t0 = clock64();
        for (uint32_t it = 0;; ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((it & 31u) == 31u) {
                if (aborted()) return false;
                if ((unsigned long long)(clock64() - t0) > limit_cycles) {
                    give_up(where, task);
                    return false;
                }
            }
        }
    }
    // After a failure: waits for work that is already in flight (a copy into shared memory, an MMA), whatever the
    // abort flag says: a CTA must not exit, nor free TMEM, while such work is pending.  Bounded by the time limit only.
    __device__ void wait_landed(uint32_t bar, uint32_t parity) const
    {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity))
            if ((unsigned long long)(clock64() - t0) > limit_cycles) return;
    }
    // waits until *flag >= target
    __device__ bool wait_flag(const int *flag, int where, long long task, int target = 1) const
    {
        for (int it = 0; it < 16; ++it) {
            if (ld_acquire(flag) >= target) return true;
            __nanosleep(32);
        }
        const long long t0 = clock64();
        for (uint32_t it = 0;; ++it) {
            if (ld_acquire(flag) >= target) return true;
            __nanosleep(64);
            if ((it & 15u) == 15u) {
                if (aborted()) return false;
                if ((unsigned long long)(clock64() - t0) > limit_cycles) {
                    give_up(where, task);
                    return false;
                }
            }
        }
    }
};

struct Ring {
    int depth;
    int stage = 0;
    uint32_t phase = 0;
    __device__ explicit Ring(int d) : depth(d) {}
    __device__ __forceinline__ void advance()
    {
        if (++stage == depth) {
            stage = 0;
            phase ^= 1u;
        }
    }
};

struct Shared {
    unsigned long long full1[kMaxStages], empty1[kMaxStages], full2[kMaxStages], empty2[kMaxStages];
    unsigned long long tmem_full[2], tmem_empty[2], mail_full[kMail], mail_empty[kMail];
    unsigned long long mma_drain; // abort path: completes when the MMAs issued so far have finished
    unsigned long long duty_full[kDuty], duty_empty[kDuty];
    int duty[kDuty]; // samples whose last task has been counted; < 0 ends the stream
    int4 mail[kMail]; // (sample, task index, 1 if it is the sample's last task, -); sample < 0 ends the stream
    // pivot selection (the selection warps, one sample at a time)
    uint32_t sel_keys[kSelMax];
    unsigned long long sel_list[kMaxN];
    SelectSmem sel;
    uint32_t tmem_base, n_picked;
    float pivot_norm[kEpiWarps][kMaxN]; // per epilogue warp: Euclidean norms of the current sample's pivots
    int abort_flag;
    volatile uint32_t s2_step;          // the step whose second-pass task the MMA issuer looks at next
};
static_assert(sizeof(Shared) + 64 <= kStaticSmemReserve, "static shared memory exceeds its reserve");

__host__ __device__ inline uint32_t b_stage_bytes(int N) { return (uint32_t)((N * 128 + 1023) / 1024 * 1024); }
__host__ __device__ inline uint32_t stage1_bytes(uint32_t row_bytes)
{
    return (kS1StageRows * row_bytes + 1023u) / 1024u * 1024u;
}
// Ring depths for a shared-memory budget: a little over half to ring 2 (its stages are freed only when the MMAs
// that read them have completed, so it needs more in flight than ring 1), the rest to ring 1.  Measured at
// N = 16, d = 4096: 2 + 6 stages 1.80 ms, 3 + 5 1.83 ms, 4 + 3 1.94 ms per launch of the 256-sample sweep.
__host__ inline void ring_depths(int N, uint32_t row_bytes, size_t smem_limit, int &n1, int &n2)
{
    const size_t budget = smem_limit - 1024 - kStaticSmemReserve; // alignment slack and static shared memory
    const size_t s1 = stage1_bytes(row_bytes), s2 = kAtomBytes + b_stage_bytes(N);
    size_t b = budget * 11 / 20 / s2;
    b = b < 2 ? 2 : (b > (size_t)kMaxStages ? (size_t)kMaxStages : b);
    size_t a = budget > b * s2 ? (budget - b * s2) / s1 : 0;
    a = a > (size_t)kMaxStages ? (size_t)kMaxStages : a;
    n1 = (int)a;
    n2 = (int)b;
}
__host__ inline size_t smem_bytes(int N, uint32_t row_bytes, int n1, int n2)
{
    return 1024 + (size_t)n1 * stage1_bytes(row_bytes) + (size_t)n2 * (kAtomBytes + b_stage_bytes(N));
}

// The selection warps: the pivots of sample b (Def. 1) = its P best scores in rank order, equal scores to the
// lower index.  Radix select over order-preserving keys held in shared memory, then a bitonic sort of the
// P winners.
__device__ void select_pivots(const Params &p, Shared &sh, int b)
{
    const Selectors g;
    const int lane = g.tid(); // 0 .. kSel-1
    const float *score = (p.norm_kind == 2 ? p.ssq : p.l1) + (size_t)b * p.n_vis;
    const int smallest = p.smallest;
    const bool cached = p.n_vis <= kSelMax;
    if (cached) { // the scores were written by other SMs: read them from L2, eight loads in flight per lane
        for (int j0 = lane; j0 < p.n_vis; j0 += kSel * 16) {
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = (j0 + kSel * u < p.n_vis) ? __ldcg(score + j0 + kSel * u) : 0.f;
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (j0 + kSel * u < p.n_vis) {
                    const uint32_t k = order_key(v[u]);
                    sh.sel_keys[j0 + kSel * u] = smallest ? k : ~k; // smaller key = better pivot
                }
        }
    }
    if (cached && p.P <= kArgminMaxP) {
        // few pivots: every thread keeps the best (key, index) among its own scores; each round the group's
        // minimum is the next pivot, and only its owner looks for a new best.  (key, index) pairs are unique,
        // so this is the same order as a full sort: best score first, equal scores by index.
        g.sync();
        auto scan = [&]() {
            unsigned long long best = ~0ull;
            for (int j = lane; j < p.n_vis; j += kSel) {
                const unsigned long long k = ((unsigned long long)sh.sel_keys[j] << 32) | (uint32_t)j;
                best = k < best ? k : best;
            }
            return best;
        };
        unsigned long long mine = scan();
        for (int r = 0; r < p.P; ++r) {
            unsigned long long w = mine;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long x = __shfl_xor_sync(0xffffffffu, w, o);
                w = x < w ? x : w;
            }
            if ((lane & 31) == 0) sh.sel_list[(r & 1) * kSelWarps + (lane >> 5)] = w; // double-buffered by round
            g.sync();
            unsigned long long win = sh.sel_list[(r & 1) * kSelWarps];
#pragma unroll
            for (int k = 1; k < kSelWarps; ++k) {
                const unsigned long long x = sh.sel_list[(r & 1) * kSelWarps + k];
                win = x < win ? x : win;
            }
            const uint32_t idx = (uint32_t)(win & 0xffffffffu);
            if (lane == 0) p.pivot_idx[(size_t)b * p.P + r] = (int32_t)min(idx, (uint32_t)(p.n_vis - 1));
            if (mine == win) { // the owner: retire the winner and find this thread's next best
                sh.sel_keys[idx] = 0xffffffffu;
                mine = scan();
            }
        }
        __threadfence();
        g.sync();
        if (lane == 0 && !p.withhold_pivots) st_release(p.piv_ready + b, 1);
        return;
    }
    int P_pad = 1;
    while (P_pad < p.P) P_pad <<= 1;
    for (int i = lane; i < P_pad; i += kSel) sh.sel_list[i] = ~0ull;
    if (lane == 0) sh.n_picked = 0;
    g.sync();
    auto keyfn = [&](int j, uint32_t &key) {
        if (cached) {
            key = sh.sel_keys[j];
        } else {
            const uint32_t k = order_key(__ldcg(score + j));
            key = smallest ? k : ~k;
        }
        return true;
    };
    uint32_t T, need_eq, cnt_eq;
    block_select_threshold(g, keyfn, p.n_vis, (uint32_t)p.P, sh.sel, T, need_eq, cnt_eq);
    block_select_apply(g, keyfn, p.n_vis, T, need_eq, cnt_eq, sh.sel, [&](int j, uint32_t key) {
        const uint32_t slot = atomicAdd(&sh.n_picked, 1u);
        if (slot < (uint32_t)kMaxN) sh.sel_list[slot] = ((unsigned long long)key << 32) | (uint32_t)j;
    });
    for (int k = 2; k <= P_pad; k <<= 1) { // ascending bitonic sort of (key, index): rank 0 = best
        for (int jj = k >> 1; jj > 0; jj >>= 1) {
            for (int i = lane; i < P_pad; i += kSel) {
                const int l = i ^ jj;
                if (l > i) {
                    const unsigned long long x = sh.sel_list[i], y = sh.sel_list[l];
                    const bool up = ((i & k) == 0);
                    if ((x > y) == up) {
                        sh.sel_list[i] = y;
                        sh.sel_list[l] = x;
                    }
                }
            }
            g.sync();
        }
    }
    for (int i = lane; i < p.P; i += kSel)
        p.pivot_idx[(size_t)b * p.P + i] = (int32_t)min((uint32_t)(sh.sel_list[i] & 0xffffffffu), (uint32_t)(p.n_vis - 1));
    __threadfence();
    g.sync();
    if (lane == 0 && !p.withhold_pivots) st_release(p.piv_ready + b, 1);
}

__global__ void __launch_bounds__(kThreads, 1)
sweep_kernel(const __grid_constant__ CUtensorMap tm_tile, const __grid_constant__ CUtensorMap tm_keys,
             const __grid_constant__ CUtensorMap tm_row, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bstage = b_stage_bytes(p.N);
    // ring 1: n1 stages of four plain rows; ring 2: n2 swizzled key tiles followed by n2 pivot tiles
    const uint32_t ring2_0 = smem0 + (uint32_t)p.n1 * p.stage1_bytes;
    auto a1_addr = [&](int s) { return smem0 + (uint32_t)s * p.stage1_bytes; };
    auto a2_addr = [&](int s) { return ring2_0 + (uint32_t)s * kAtomBytes; };
    auto b2_addr = [&](int s) { return ring2_0 + (uint32_t)p.n2 * kAtomBytes + (uint32_t)s * bstage; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    // consumers get a longer limit than the producers, so that the wait nearest the cause reports first
    const Ctl ctl{&sh.abort_flag, p.status, (warp == 0 || warp == kProducer2Warp) ? limit : limit + limit / 4};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&sh.full1[s]), 1);
            mbar_init(smem_u32(&sh.empty1[s]), kWorkerWarps); // every worker warp releases a stage by itself
            mbar_init(smem_u32(&sh.full2[s]), 1);
            mbar_init(smem_u32(&sh.empty2[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh.tmem_full[a]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[a]), kEpiWarps);
        }
        mbar_init(smem_u32(&sh.mma_drain), 1);
        for (int m = 0; m < kMail; ++m) {
            mbar_init(smem_u32(&sh.mail_full[m]), 1);
            mbar_init(smem_u32(&sh.mail_empty[m]), 1);
        }
        for (int m = 0; m < kDuty; ++m) {
            mbar_init(smem_u32(&sh.duty_full[m]), 1);
            mbar_init(smem_u32(&sh.duty_empty[m]), 1);
        }
        sh.abort_flag = 0;
        sh.s2_step = blockIdx.x;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * p.N) tmem_cols <<= 1;
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
    const uint32_t total = total_steps(p);

    if (warp == 0) {
        // ------------------------------------------------------------------ sweep-1 producer
        if (lane == 0) {
            // With the second pass cut into column chunks a row is read again a few microseconds later: the L2 is asked to keep
            // it.  With whole-tile tasks the second read comes ~100 MB of newer rows later, and nothing is kept.
            unsigned long long pol_keep;
            if (p.keep_l2)
                asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            else
                asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_keep));
            Ring ring(p.n1);
            long long issued = 0;
            bool ok = true;
            for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
                Task t;
                if (!decode(p, g, 0, t)) continue;
                if (p.ahead) { // not too far ahead of the second pass: what it reads again should still be in the L2
                    const long long t0 = clock64();
                    for (uint32_t it = 0; g > p.ahead && sh.s2_step < g - p.ahead; ++it) {
                        __nanosleep(64);
                        if ((it & 31u) == 31u && (ctl.aborted() || (unsigned long long)(clock64() - t0) > ctl.limit_cycles)) {
                            if (!ctl.aborted()) ctl.give_up(kWaitAhead, g);
                            ok = false;
                            break;
                        }
                    }
                    if (!ok) break;
                }
                const int row0 = t.u * kS1Rows, rows = min(kS1Rows, p.n_vis - row0);
                const char *src = p.keys + ((size_t)t.b * p.S + p.vis_offset + row0) * (size_t)p.row_bytes;
                for (int r = 0; r < rows; r += kS1StageRows) {
                    const uint32_t bytes = (uint32_t)min(kS1StageRows, rows - r) * p.row_bytes;
                    ok = ctl.wait_bar(smem_u32(&sh.empty1[ring.stage]), ring.phase ^ 1u, kWaitEmptyStage, g);
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
    } else if (warp == kProducer2Warp) {
        // ------------------------------------------------------------------ sweep-2 producer
        unsigned long long pol_keep, pol_drop;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_drop));
        Ring ring(p.n2);
        long long issued = 0;
        bool ok = true;
        int cur_b = -1;
        int my_piv[kMaxN / 128][4]; // lane l loads pivot ranks 4l..4l+3, 4(l+32).., as rows of the key tensor
        for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
            Task t;
            if (!decode(p, g, 1, t)) continue;
            if (t.b != cur_b) {
                if (lane == 0) {
                    ok = ctl.wait_flag(p.piv_ready + t.b, kWaitPivots, g);
                    if (!ok && p.status[1] == kWaitPivots && p.status[3] == (int)blockIdx.x) {
                        p.status[4] = t.b;
                        p.status[5] = ld_acquire(p.s1_done + t.b);
                    }
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
#pragma unroll
                for (int k = 0; k < kMaxN / 128; ++k)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = min(4 * (lane + 32 * k) + e, p.P - 1); // ranks beyond P repeat the last pivot
                        const int piv = min(max(__ldcg(p.pivot_idx + (size_t)t.b * p.P + i), 0), p.n_vis - 1);
                        my_piv[k][e] = t.b * p.S + p.vis_offset + piv;
                    }
                cur_b = t.b;
            }
            const int a_lo = t.kc * p.apc, na = min(p.n_atoms, a_lo + p.apc);
            const int rows = min(kTileRows, p.n_vis - t.rt * kTileRows);
            const int n_sub = (rows + kSubRows - 1) / kSubRows;
            const int y0 = t.b * p.S + p.vis_offset + t.rt * kTileRows;
            for (int a = a_lo; a < na; ++a) {
                const uint32_t full = smem_u32(&sh.full2[ring.stage]);
                if (lane == 0) {
                    ok = ctl.wait_bar(smem_u32(&sh.empty2[ring.stage]), ring.phase ^ 1u, kWaitEmptyStage, g);
                    if (ok)
                        mbar_arrive_expect_tx(full, (rows == kTileRows ? (uint32_t)kAtomBytes : (uint32_t)n_sub * kSubBytes) +
                                                        (uint32_t)((p.P + 3) / 4) * 512u);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const int x = a * kAtomCols;
                const uint32_t dst = a2_addr(ring.stage);
                if (rows == kTileRows) {
                    if (lane == 0) tma_load_2d(dst, &tm_tile, x, y0, full, pol_drop);
                } else if (lane < n_sub) {
                    tma_load_2d(dst + (uint32_t)lane * kSubBytes, &tm_keys, x, y0 + lane * kSubRows, full, pol_drop);
                }
#pragma unroll
                for (int k = 0; k < kMaxN / 128; ++k) {
                    const int q = lane + 32 * k; // pivot ranks 4q..4q+3 -> rows 4q..4q+3 of the B tile
                    if (4 * q < p.P)
                        tma_gather4(b2_addr(ring.stage) + (uint32_t)q * 512u, &tm_row, x, my_piv[k][0], my_piv[k][1],
                                    my_piv[k][2], my_piv[k][3], full, pol_keep);
                }
                ring.advance();
                ++issued;
            }
        }
        if ((!ok || ctl.aborted()) && lane == 0) // drain, as above
            for (long long i = issued > p.n2 ? issued - p.n2 : 0; i < issued; ++i)
                ctl.wait_landed(smem_u32(&sh.full2[i % p.n2]), (uint32_t)((i / p.n2) & 1));
    } else if (warp == 1) {
        // ------------------------------------------------------------------ sweep-2 MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(p.N);
            Ring ring(p.n2);
            uint32_t s2n = 0;
            bool ok = true;
            for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
                Task t;
                sh.s2_step = g;
                if (!decode(p, g, 1, t)) continue;
                const int a_lo = t.kc * p.apc, na = min(p.n_atoms, a_lo + p.apc);
                const uint32_t acc = s2n & 1u;
                ok = ctl.wait_bar(smem_u32(&sh.tmem_empty[acc]), ((s2n >> 1) & 1u) ^ 1u, kWaitAccumFree, g);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.N;
                for (int a = a_lo; a < na; ++a) {
                    ok = ctl.wait_bar(smem_u32(&sh.full2[ring.stage]), ring.phase, kWaitStageMma, g);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned long long da = umma_desc(a2_addr(ring.stage)), db = umma_desc(b2_addr(ring.stage));
#pragma unroll
                    for (int k = 0; k < kAtomCols / 16; ++k) // 16 columns = 32 bytes per MMA: advance the start address
                        umma_bf16(d_tmem, da + (unsigned long long)(2 * k), db + (unsigned long long)(2 * k), idesc,
                                  ((a - a_lo) | k) != 0);
                    umma_commit(smem_u32(&sh.empty2[ring.stage])); // frees the stage once the MMAs have read it
                    ring.advance();
                }
                if (!ok) break;
                umma_commit(smem_u32(&sh.tmem_full[acc]));
                ++s2n;
            }
            sh.s2_step = 0xfffffff0u; // nothing holds the first pass back any more
            if (!ok || ctl.aborted()) { // TMEM is freed at the end: first let the MMAs issued so far finish
                umma_commit(smem_u32(&sh.mma_drain));
                ctl.wait_landed(smem_u32(&sh.mma_drain), 0);
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // ------------------------------------------------------------------ sweep-2 epilogue (warps independent)
        const int quarter = warp & 3;        // TMEM lane quarter this warp may read
        const int row = quarter * 32 + lane; // tile row owned by this thread
        float *pn = sh.pivot_norm[quarter];
        int cur_b = -1;
        uint32_t s2n = 0;
        for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
            Task t;
            if (!decode(p, g, 1, t)) continue;
            const int rows = min(kTileRows, p.n_vis - t.rt * kTileRows);
            const int j = t.rt * kTileRows + row;
            const uint32_t acc = s2n & 1u;
            bool ok = ctl.wait_bar(smem_u32(&sh.tmem_full[acc]), (s2n >> 1) & 1u, kWaitAccumFull, g);
            if (!__all_sync(0xffffffffu, ok)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // the accumulator exists, so the sample's pivots and all of its norms were published long ago
            if (t.b != cur_b) {
                __syncwarp();
                for (int i = lane; i < p.P; i += 32) {
                    const int piv = min(max(__ldcg(p.pivot_idx + (size_t)t.b * p.P + i), 0), p.n_vis - 1);
                    pn[i] = sqrtf(__ldcg(p.ssq + (size_t)t.b * p.n_vis + piv));
                }
                __syncwarp();
                cur_b = t.b;
            }
            const float nj = row < rows ? sqrtf(__ldcg(p.ssq + (size_t)t.b * p.n_vis + j)) : 0.f;
            const uint32_t taddr = tmem_base + acc * (uint32_t)p.N + ((uint32_t)(quarter * 32) << 16);
            // a chunk's share of dup: its part of the dot product over the same two norms; the shares are added up afterwards
            float *dst = p.sim + ((size_t)t.kc * p.B + t.b) * p.P * p.n_vis + j;
            for (int c0 = 0; c0 < p.P; c0 += 8) {
                float v[8];
                tmem_ld8(taddr + (uint32_t)c0, v); // warp-collective: rows outside the tile still take part
                if (row < rows) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (c0 + e < p.P) { // dup = dot / (|pivot| |row|); a zero norm gives 0; a warp writes 128 contiguous bytes
                            const float den = pn[c0 + e] * nj;
                            dst[(size_t)(c0 + e) * p.n_vis] = den > 0.f ? v[e] / den : 0.f;
                        }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.tmem_empty[acc]));
            }
            ++s2n;
        }
    } else if (warp >= kWorkerWarp0 && warp < kWorkerWarp0 + kWorkerWarps) {
        // ------------------------------------------------------------------ sweep-1 workers: one row per warp and stage
        const int wq = warp - kWorkerWarp0, wt = threadIdx.x - kWorkerWarp0 * 32;
        Ring ring(p.n1);
        int ms = 0;
        uint32_t mph = 0;
        bool dead = false; // warp-uniform inside a task, group-uniform after every workers_any()
        auto post = [&](int4 m) { // thread wt == 0: hand a finished task (or an end mark) to a control warp
            bool ok = ctl.wait_bar(smem_u32(&sh.mail_empty[ms]), mph ^ 1u, kWaitMailSlot, 0);
            if (ok) {
                sh.mail[ms] = m;
                mbar_arrive(smem_u32(&sh.mail_full[ms])); // release: the group's scores are ordered before it
            }
            if (++ms == kMail) {
                ms = 0;
                mph ^= 1u;
            }
            return ok;
        };
        for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
            Task t;
            if (!decode(p, g, 0, t)) continue;
            const int row0 = t.u * kS1Rows, rows = min(kS1Rows, p.n_vis - row0);
            for (int r = 0; r < rows; r += kS1StageRows) {
                // warp-uniform: either the whole warp reads the stage and releases it, or none of it does
                if (!dead) dead = !ctl.wait_bar(smem_u32(&sh.full1[ring.stage]), ring.phase, kWaitStageRows, g);
                dead = __any_sync(0xffffffffu, dead);
                if (!dead && r + wq < rows) {
                    const uint32_t base = a1_addr(ring.stage) + (uint32_t)wq * p.row_bytes + (uint32_t)lane * 16u;
                    float a0 = 0.f, a1 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll 4
                    for (int c = lane; c < p.d8; c += 32) { // lanes read consecutive 16-byte chunks: no bank conflicts
                        const uint4 v = lds128(base + (uint32_t)(c - lane) * 16u);
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
                    const float a = warp_sum(a0 + a1), q = warp_sum(q0 + q1); // fixed order; every lane gets the sum
                    if (lane == 0) {
                        const size_t o = (size_t)t.b * p.n_vis + row0 + r + wq;
                        p.l1[o] = a;
                        p.ssq[o] = q;
                    }
                }
                __syncwarp(); // the warp's reads of the stage are done
                if (!dead && lane == 0) mbar_arrive(smem_u32(&sh.empty1[ring.stage]));
                ring.advance();
            }
            dead = workers_any(dead); // every warp's scores of this task are issued
            if (wt == 0 && !dead && !post(make_int4(t.b, t.u, t.u == p.T1 - 1, 0))) dead = true;
        }
        workers_any(dead);
        if (wt == 0) post(make_int4(-1, 0, 0, 0)); // end mark (also after a failure, so that the control warps exit)
    } else if (warp == kCountWarp) {
        // ------------------------------------------------------------------ counter (one thread)
        if (lane == 0) {
            int ds = 0;
            uint32_t dph = 0;
            auto hand_over = [&](int b) { // sample b is complete once s1_done[b] reaches T1: the selectors' job
                bool ok = ctl.wait_bar(smem_u32(&sh.duty_empty[ds]), dph ^ 1u, kWaitDutySlot, b);
                if (ok) {
                    sh.duty[ds] = b;
                    mbar_arrive(smem_u32(&sh.duty_full[ds]));
                }
                if (++ds == kDuty) {
                    ds = 0;
                    dph ^= 1u;
                }
                return ok;
            };
            for (uint32_t m = 0;; ++m) {
                const int slot = (int)(m % kMail);
                if (!ctl.wait_bar(smem_u32(&sh.mail_full[slot]), (m / kMail) & 1u, kWaitMail, 0)) break;
                const int4 mail = sh.mail[slot];
                mbar_arrive(smem_u32(&sh.mail_empty[slot]));
                if (mail.x < 0) break;
                __threadfence(); // the workers' scores (ordered before the mail) become visible GPU-wide
                atomicAdd(p.s1_done + mail.x, 1);
                if (mail.z && !hand_over(mail.x)) break;
            }
            hand_over(-1); // end mark for the selectors (also after a failure)
        }
    } else if (warp >= kSelWarp0 && warp < kSelWarp0 + kSelWarps) {
        // ------------------------------------------------------------------ selection
        const Selectors sg;
        const int st = sg.tid();
        for (uint32_t m = 0;; ++m) {
            const int slot = (int)(m % kDuty);
            bool fail = !ctl.wait_bar(smem_u32(&sh.duty_full[slot]), (m / kDuty) & 1u, kWaitDuty, 0);
            if (selectors_any(fail)) break;
            const int b = sh.duty[slot];
            sg.sync(); // everyone has read the slot
            if (st == 0) mbar_arrive(smem_u32(&sh.duty_empty[slot]));
            if (b < 0) break;
            // the sample's last task has been counted; the other tasks precede it in the schedule, so their
            // counts do not depend on anything this CTA still has to do
            fail = st == 0 && !ctl.wait_flag(p.s1_done + b, kWaitTasks, b, p.T1);
            if (selectors_any(fail)) break;
            select_pivots(p, sh, b);
        }
    }
    // ---------------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
}

} // namespace sweep
} // namespace dart
