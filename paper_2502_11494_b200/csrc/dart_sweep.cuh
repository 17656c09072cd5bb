// Fused path, sweeps: ONE persistent kernel computes the scores (sweep 1), the pivots and the
// pivot x token dot products (sweep 2) of a whole batch, so that the second read of every key row
// is served by the L2 cache instead of HBM.
//
// Work is cut into tasks of 128 token rows x 512 columns (128 KB of keys).  Every task appears
// twice in one global, static order: as a sweep-1 task (row L1 norms and sums of squares: the
// K-norm of the Sec. 3.3 footnote and Eq. 7's denominator) and, `lag` tasks later, as a sweep-2
// task (dot products with the sample's pivot rows: Eq. 7's numerator).  CTA c executes tasks
// c, c + grid, c + 2 grid, ...  Because a task is only 128 KB, all SMs together hold < 20 MB in
// flight, and the distance between the two reads of a row is the sample size plus the lag.
//
// Per CTA (512 threads; warp 3 idles):
//   warps 0, 2 sweep-1 producer and sweep-2 producer: TMA loads of key tiles into two
//              shared-memory rings, one per sweep, each with its own producer and exactly one consumer
//              role, so that neither sweep blocks the other and no role ever skips a barrier phase; the
//              sweep-2 producer also gathers the sample's pivot rows (tile::gather4 boxes straight from
//              the key tensor).  L2 evict_last on the first read of a tile, evict_first on the second.
//   warp 1     sweep 2: one thread issues tcgen05.mma (tokens = M 128, pivots = N, bf16 -> fp32 in TMEM)
//   warps 4-7  sweep-1 workers: each thread owns one tile row and sums it from shared memory.
//   warps 8-11 sweep-2 epilogue: read the accumulators out of TMEM and store the partial dot products
//              (separate from the workers so that neither sweep ever waits for the other; the sweep-1
//              producer only stays within one round of the CTA's sweep-2 progress, which bounds the
//              distance between the two reads of a tile).
//   warps 12-15 control: everything that needs a global-memory round trip, fed by a mailbox so that the
//              workers never wait for it: counts finished column slabs; the CTA that delivers a row
//              tile's last slab adds the slab partials up (fixed order) and leaves the tile's P best
//              (score, index) candidates; the CTA that delivers a sample's last row tile merges the
//              candidates into the pivots (Def. 1) and publishes them.
// Every result is bitwise reproducible: partial sums are added in slab order by one thread per row.
//
// Every wait (mbarrier or global flag) is bounded in time; on expiry the kernel records
// DART_ERR_TIMEOUT in the status word, drains and exits normally.
#pragma once
#include <cuda.h>

#include "dart_common.cuh"

namespace dart {
namespace sweep {

constexpr int kTileRows = 128;
constexpr int kAtomCols = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int kSubRows = 32;   // rows per TMA box of the key tensor
constexpr int kSlabAtoms = 8;  // a task spans 8 atoms = 512 columns
constexpr int kMaxStages = 8;  // per ring; fewer when many pivots make the sweep-2 stages large
constexpr int kAtomBytes = kTileRows * 128; // 16 KB: 128 rows x 128 bytes, 128B-swizzled, K-major
constexpr int kSubBytes = kSubRows * 128;
constexpr int kThreads = 512;
constexpr int kWorkerWarp0 = 4, kWorkerWarps = 4, kWorkers = kWorkerWarps * 32;
constexpr int kEpiWarp0 = 8, kEpiWarps = 4; // kEpiWarp0 % 4 == 0: warp w reads TMEM lanes 32 (w % 4) ...
constexpr int kCtrlWarp0 = 12, kCtrlWarps = 4, kCtrl = kCtrlWarps * 32;
constexpr int kProducer2Warp = 2;
constexpr int kMaxN = 256;      // pivots per MMA (N dimension)
constexpr int kMail = 8;        // mailbox slots between workers and control warps
constexpr int kMergeMax = 1024; // candidates merged in shared memory; beyond that a radix select over all scores
constexpr int kStaticSmemReserve = 12288;
constexpr int kStatusTimeout = -7;
// which wait expired (second status word)
enum { kWaitPivots = 1, kWaitEmptyStage, kWaitDrain, kWaitAccumFree, kWaitStageMma, kWaitStageRows, kWaitAccumFull,
       kWaitMailSlot, kWaitMail, kWaitSlabs, kWaitRowTiles, kWaitSweep2 };

using Workers = WarpGroup<kWorkerWarp0, kWorkerWarps, 1>;
using Control = WarpGroup<kCtrlWarp0, kCtrlWarps, 2>;

struct Params {
    int B, S, vis_offset, n_vis, P, N; // N = P rounded up to a multiple of 16 (MMA N)
    int Pc;                            // candidates a row tile leaves: min(P, 128)
    int d8;                            // row width in 16-byte units
    int n_atoms, KS, n_rt, T;          // atoms per row; column slabs; row tiles per sample; tasks per sample and sweep
    int n1, n2;                        // depth of the sweep-1 and of the sweep-2 ring (<= kMaxStages each)
    uint32_t lag;                      // tasks between a task's first and second sweep (T <= lag <= B * T)
    int norm_kind, smallest;
    unsigned long long wait_ns;        // time limit of every wait
    float *pl1, *pssq;                 // [B][KS][n_vis] per-slab partial sums
    float *psim;                       // [B][KS][n_vis][P] per-slab partial dot products
    float *l1, *ssq;                   // [B][n_vis]
    unsigned long long *cand;          // [B][n_rt][Pc] best (key, index) pairs of every row tile, best first
    int32_t *pivot_idx;                // [B][P]
    int *rt_done;                      // [B][n_rt] column slabs finished per row tile
    int *s1_done;                      // [B] row tiles finished per sample
    int *piv_ready;                    // [B] 1 once the pivots of the sample are published
    int *status;
};

struct Task {
    int kind; // 0 = sweep 1, 1 = sweep 2
    int b, rt, ks;
};

// Schedule.  Step q of the global order is the pair (sweep-1 task q, sweep-2 task q - lag); CTA c runs steps
// c, c + grid, ... and, within a step, the sweep-1 task first.  So every CTA alternates between the two kinds
// of task, and a sweep-2 task comes `lag` steps after the sweep-1 task of the same tile (lag >= T, hence after
// the whole sample has been scored).  The host guarantees B * T + lag < 2^31.
__device__ __forceinline__ uint32_t total_steps(const Params &p) { return (uint32_t)p.B * (uint32_t)p.T + p.lag; }

// kind 0: sweep-1 task of step q; kind 1: its sweep-2 task.  Returns false if the step has no such task.
__device__ __forceinline__ bool decode(const Params &p, uint32_t q, int kind, Task &t)
{
    const uint32_t n_all = (uint32_t)p.B * (uint32_t)p.T;
    if (kind == 0 ? q >= n_all : q < p.lag) return false;
    const uint32_t n = kind ? q - p.lag : q, T = (uint32_t)p.T, KS = (uint32_t)p.KS;
    t.kind = kind;
    t.b = (int)(n / T);
    const uint32_t u = n - (uint32_t)t.b * T;
    t.rt = (int)(u / KS);
    t.ks = (int)(u - (uint32_t)t.rt * KS);
    return true;
}

__device__ __forceinline__ int slab_atoms(const Params &p, int ks) { return min(kSlabAtoms, p.n_atoms - ks * kSlabAtoms); }

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
template <int kBarrierId>
__device__ __forceinline__ bool group_any(bool pred)
{
    uint32_t r;
    asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbar.red.or.pred p, %2, 128, q;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(r)
                 : "r"((uint32_t)pred), "n"(kBarrierId)
                 : "memory");
    return r != 0;
}
__device__ __forceinline__ bool workers_any(bool pred) { return group_any<1>(pred); }
__device__ __forceinline__ bool control_any(bool pred) { return group_any<2>(pred); }

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
    // waits until a shared-memory counter reaches target
    __device__ bool wait_count(const volatile int *cnt, int target, int where, long long task) const
    {
        if (*cnt >= target) return true;
        const long long t0 = clock64();
        for (uint32_t it = 0;; ++it) {
            if (*cnt >= target) return true;
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
    int4 mail[kMail]; // (sample, row tile, column slab, valid rows); sample < 0 ends the stream
    union {
        unsigned long long cand[kMergeMax]; // candidate merge
        struct {
            SelectSmem sel; // radix-select path for very many pivots
            unsigned long long list[kMaxN];
        } rs;
    } u;
    unsigned long long ckey[kTileRows]; // (key, index) of the rows of the tile being finalised
    uint32_t tmem_base, n_picked;
    int abort_flag;
    volatile int s2_step; // last schedule step whose sweep-2 task this CTA has finished (-1: none yet)
};
static_assert(sizeof(Shared) + 64 <= kStaticSmemReserve, "static shared memory exceeds its reserve");

__host__ __device__ inline uint32_t b_stage_bytes(int N) { return (uint32_t)((N * 128 + 1023) / 1024 * 1024); }
// Ring depths for a shared-memory budget: half of it to the sweep-2 ring (at least 2 stages), the rest to sweep 1.
__host__ inline void ring_depths(int N, size_t smem_limit, int &n1, int &n2)
{
    const size_t budget = smem_limit - 1024 - kStaticSmemReserve; // alignment slack and static shared memory
    const size_t s2 = kAtomBytes + b_stage_bytes(N);
    size_t b = budget / 2 / s2;
    b = b < 2 ? 2 : (b > (size_t)kMaxStages ? (size_t)kMaxStages : b);
    size_t a = budget > b * s2 ? (budget - b * s2) / kAtomBytes : 0;
    a = a > (size_t)kMaxStages ? (size_t)kMaxStages : a;
    n1 = (int)a;
    n2 = (int)b;
}
__host__ inline size_t smem_bytes(int N, int n1, int n2)
{
    return 1024 + (size_t)n1 * kAtomBytes + (size_t)n2 * (kAtomBytes + b_stage_bytes(N));
}

// (key, index) composite of a score: smaller composite = better pivot, equal scores -> lower index first
__device__ __forceinline__ unsigned long long pivot_key(const Params &p, float score, int j)
{
    const uint32_t k = order_key(score);
    return ((unsigned long long)(p.smallest ? k : ~k) << 32) | (uint32_t)j;
}

// Control warps, row tile (b, rt) complete: add up the slab partials of every row in slab order, store the
// final sums, and leave the tile's Pc best candidates, best first.
__device__ void finalize_row_tile(const Params &p, Shared &sh, int b, int rt, int rows)
{
    const Control g;
    const int r = g.tid(), j = rt * kTileRows + r;
    unsigned long long mine = ~0ull;
    if (r < rows) {
        float s1 = 0.f, s2 = 0.f;
        for (int k0 = 0; k0 < p.KS; k0 += 8) {
            float a[8], q[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const size_t o = ((size_t)b * p.KS + min(k0 + k, p.KS - 1)) * p.n_vis + j;
                a[k] = __ldcg(p.pl1 + o);
                q[k] = __ldcg(p.pssq + o);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k0 + k < p.KS) {
                    s1 += a[k];
                    s2 += q[k];
                }
        }
        p.l1[(size_t)b * p.n_vis + j] = s1;
        p.ssq[(size_t)b * p.n_vis + j] = s2;
        mine = pivot_key(p, p.norm_kind == 2 ? s2 : s1, j);
    }
    sh.ckey[r] = mine;
    g.sync();
    int rank = 0;
#pragma unroll 8
    for (int i = 0; i < kTileRows; ++i) rank += (sh.ckey[i] < mine) ? 1 : 0;
    unsigned long long *dst = p.cand + ((size_t)b * p.n_rt + rt) * p.Pc;
    if (r < rows) {
        if (rank < p.Pc) dst[rank] = mine;
    } else if (r < p.Pc) {
        dst[r] = ~0ull; // a short tile has fewer rows than candidate slots: slots rows..Pc-1 stay empty
    }
}

// Control warps, sample b complete: pivots (Def. 1) = the P best of the row tiles' candidates, in rank order.
__device__ void merge_pivots(const Params &p, Shared &sh, int b)
{
    const Control g;
    const int tid = g.tid();
    const int C = p.n_rt * p.Pc;
    if (C <= kMergeMax) {
        const unsigned long long *src = p.cand + (size_t)b * C;
        for (int i = tid; i < C; i += kCtrl) sh.u.cand[i] = __ldcg(src + i);
        g.sync();
        for (int i = tid; i < C; i += kCtrl) {
            const unsigned long long mine = sh.u.cand[i];
            if (mine == ~0ull) continue;
            int rank = 0;
#pragma unroll 8
            for (int k = 0; k < C; ++k) rank += (sh.u.cand[k] < mine) ? 1 : 0;
            if (rank < p.P) p.pivot_idx[(size_t)b * p.P + rank] = (int32_t)(mine & 0xffffffffu);
        }
    } else {
        // very many pivots: radix select over all scores of the sample, then sort the winners
        const float *score = (p.norm_kind == 2 ? p.ssq : p.l1) + (size_t)b * p.n_vis;
        const int smallest = p.smallest;
        auto keyfn = [&](int j, uint32_t &key) {
            uint32_t k = order_key(__ldcg(score + j));
            key = smallest ? k : ~k;
            return true;
        };
        int P_pad = 1;
        while (P_pad < p.P) P_pad <<= 1;
        for (int i = tid; i < P_pad; i += kCtrl) sh.u.rs.list[i] = ~0ull;
        if (tid == 0) sh.n_picked = 0;
        uint32_t T, need_eq, cnt_eq;
        block_select_threshold(g, keyfn, p.n_vis, (uint32_t)p.P, sh.u.rs.sel, T, need_eq, cnt_eq);
        block_select_apply(g, keyfn, p.n_vis, T, need_eq, cnt_eq, sh.u.rs.sel, [&](int j, uint32_t key) {
            uint32_t slot = atomicAdd(&sh.n_picked, 1u);
            if (slot < (uint32_t)kMaxN) sh.u.rs.list[slot] = ((unsigned long long)key << 32) | (uint32_t)j;
        });
        for (int k = 2; k <= P_pad; k <<= 1) {
            for (int jj = k >> 1; jj > 0; jj >>= 1) {
                for (int i = tid; i < P_pad; i += kCtrl) {
                    int l = i ^ jj;
                    if (l > i) {
                        unsigned long long x = sh.u.rs.list[i], y = sh.u.rs.list[l];
                        bool up = ((i & k) == 0);
                        if ((x > y) == up) {
                            sh.u.rs.list[i] = y;
                            sh.u.rs.list[l] = x;
                        }
                    }
                }
                g.sync();
            }
        }
        for (int i = tid; i < p.P; i += kCtrl)
            p.pivot_idx[(size_t)b * p.P + i] = (int32_t)min((uint32_t)(sh.u.rs.list[i] & 0xffffffffu), (uint32_t)(p.n_vis - 1));
    }
    __threadfence();
    g.sync();
    if (tid == 0) st_release(p.piv_ready + b, 1);
}

__global__ void __launch_bounds__(kThreads, 1)
sweep_kernel(const __grid_constant__ CUtensorMap tm_tile, const __grid_constant__ CUtensorMap tm_keys,
             const __grid_constant__ CUtensorMap tm_row, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bstage = b_stage_bytes(p.N);
    // ring 1: n1 key tiles; ring 2: n2 key tiles followed by n2 pivot tiles
    auto a1_addr = [&](int s) { return smem0 + (uint32_t)s * kAtomBytes; };
    auto a2_addr = [&](int s) { return smem0 + (uint32_t)(p.n1 + s) * kAtomBytes; };
    auto b2_addr = [&](int s) { return smem0 + (uint32_t)(p.n1 + p.n2) * kAtomBytes + (uint32_t)s * bstage; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    // consumers get a longer limit than the producer, so that the wait nearest the cause reports first
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
        for (int m = 0; m < kMail; ++m) {
            mbar_init(smem_u32(&sh.mail_full[m]), 1);
            mbar_init(smem_u32(&sh.mail_empty[m]), 1);
        }
        sh.abort_flag = 0;
        sh.s2_step = -1;
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
        // ------------------------------------------------------------------ sweep-1 producer (lane 0 waits, lanes issue)
        unsigned long long pol_keep;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
        Ring ring(p.n1);
        long long issued = 0;
        bool ok = true;
        for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
            Task t;
            if (!decode(p, g, 0, t)) continue;
            // stay within one round of this CTA's sweep-2 progress: the step one round back has a sweep-2
            // task if it is >= lag, and that task must be finished before more tiles are pulled in
            if (g >= gridDim.x && g - gridDim.x >= p.lag) {
                if (lane == 0) ok = ctl.wait_count(&sh.s2_step, (int)(g - gridDim.x), kWaitSweep2, g);
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
            }
            const int na = slab_atoms(p, t.ks);
            const int rows = min(kTileRows, p.n_vis - t.rt * kTileRows);
            const int n_sub = (rows + kSubRows - 1) / kSubRows;
            const int y0 = t.b * p.S + p.vis_offset + t.rt * kTileRows;
            for (int a = 0; a < na; ++a) {
                const uint32_t full = smem_u32(&sh.full1[ring.stage]);
                if (lane == 0) {
                    ok = ctl.wait_bar(smem_u32(&sh.empty1[ring.stage]), ring.phase ^ 1u, kWaitEmptyStage, g);
                    if (ok) mbar_arrive_expect_tx(full, rows == kTileRows ? (uint32_t)kAtomBytes : (uint32_t)n_sub * kSubBytes);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const int x = (t.ks * kSlabAtoms + a) * kAtomCols;
                const uint32_t dst = a1_addr(ring.stage);
                if (rows == kTileRows) { // a full tile is one 128-row box; a short last tile is 32-row boxes
                    if (lane == 0) tma_load_2d(dst, &tm_tile, x, y0, full, pol_keep);
                } else if (lane < n_sub) {
                    tma_load_2d(dst + (uint32_t)lane * kSubBytes, &tm_keys, x, y0 + lane * kSubRows, full, pol_keep);
                }
                ring.advance();
                ++issued;
            }
        }
        if (!ok && lane == 0) // drain: let the copies already issued land before the CTA may exit
            for (long long i = issued > p.n1 ? issued - p.n1 : 0; i < issued; ++i)
                ctl.wait_bar(smem_u32(&sh.full1[i % p.n1]), (uint32_t)((i / p.n1) & 1), kWaitDrain, i);
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
                        for (int r = 0; r < 6 && r < p.n_rt; ++r)
                            p.status[6 + r] = ld_acquire(p.rt_done + (size_t)t.b * p.n_rt + r);
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
            const int na = slab_atoms(p, t.ks);
            const int rows = min(kTileRows, p.n_vis - t.rt * kTileRows);
            const int n_sub = (rows + kSubRows - 1) / kSubRows;
            const int y0 = t.b * p.S + p.vis_offset + t.rt * kTileRows;
            for (int a = 0; a < na; ++a) {
                const uint32_t full = smem_u32(&sh.full2[ring.stage]);
                if (lane == 0) {
                    ok = ctl.wait_bar(smem_u32(&sh.empty2[ring.stage]), ring.phase ^ 1u, kWaitEmptyStage, g);
                    if (ok)
                        mbar_arrive_expect_tx(full, (rows == kTileRows ? (uint32_t)kAtomBytes : (uint32_t)n_sub * kSubBytes) +
                                                        (uint32_t)((p.P + 3) / 4) * 512u);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const int x = (t.ks * kSlabAtoms + a) * kAtomCols;
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
        if (!ok && lane == 0)
            for (long long i = issued > p.n2 ? issued - p.n2 : 0; i < issued; ++i)
                ctl.wait_bar(smem_u32(&sh.full2[i % p.n2]), (uint32_t)((i / p.n2) & 1), kWaitDrain, i);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ sweep-2 MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(p.N);
            Ring ring(p.n2);
            uint32_t s2n = 0;
            bool ok = true;
            for (uint32_t g = blockIdx.x; ok && g < total; g += gridDim.x) {
                Task t;
                if (!decode(p, g, 1, t)) continue;
                const int na = slab_atoms(p, t.ks);
                const uint32_t acc = s2n & 1u;
                ok = ctl.wait_bar(smem_u32(&sh.tmem_empty[acc]), ((s2n >> 1) & 1u) ^ 1u, kWaitAccumFree, g);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.N;
                for (int a = 0; a < na; ++a) {
                    ok = ctl.wait_bar(smem_u32(&sh.full2[ring.stage]), ring.phase, kWaitStageMma, g);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned long long da = umma_desc(a2_addr(ring.stage)), db = umma_desc(b2_addr(ring.stage));
#pragma unroll
                    for (int k = 0; k < kAtomCols / 16; ++k) // 16 columns = 32 bytes per MMA: advance the start address
                        umma_bf16(d_tmem, da + (unsigned long long)(2 * k), db + (unsigned long long)(2 * k), idesc,
                                  (a | k) != 0);
                    umma_commit(smem_u32(&sh.empty2[ring.stage])); // frees the stage once the MMAs have read it
                    ring.advance();
                }
                if (!ok) break;
                umma_commit(smem_u32(&sh.tmem_full[acc]));
                ++s2n;
            }
        }
    } else if (warp >= kWorkerWarp0 && warp < kWorkerWarp0 + kWorkerWarps) {
        // ------------------------------------------------------------------ sweep-1 workers
        const int wt = threadIdx.x - kWorkerWarp0 * 32; // 0..127 = tile row owned by this thread
        const int row = wt;
        Ring ring(p.n1);
        int ms = 0;
        uint32_t mph = 0;
        bool dead = false; // warp-uniform inside a task, group-uniform after every workers_any()
        auto post = [&](int4 m) { // thread wt == 0: hand a finished slab (or the end mark) to the control warps
            bool ok = ctl.wait_bar(smem_u32(&sh.mail_empty[ms]), mph ^ 1u, kWaitMailSlot, 0);
            if (ok) {
                sh.mail[ms] = m;
                mbar_arrive(smem_u32(&sh.mail_full[ms])); // release: the group's partial sums are ordered before it
            }
            return ok;
        };
        for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
            Task t;
            if (!decode(p, g, 0, t)) continue;
            const int rows = min(kTileRows, p.n_vis - t.rt * kTileRows);
            const int j = t.rt * kTileRows + row;
            const int na = slab_atoms(p, t.ks);
            float a0 = 0.f, a1 = 0.f, q0 = 0.f, q1 = 0.f;
            for (int a = 0; a < na; ++a) {
                // warp-uniform: either the whole warp reads the stage and releases it, or none of it does
                if (!dead) dead = !ctl.wait_bar(smem_u32(&sh.full1[ring.stage]), ring.phase, kWaitStageRows, g);
                dead = __any_sync(0xffffffffu, dead);
                if (!dead && row < rows) {
                    const uint32_t base = a1_addr(ring.stage) + (uint32_t)row * 128u;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        // logical 16-byte chunk c of this row sits at chunk c ^ (row & 7)
                        const uint4 v = lds128(base + (uint32_t)((c ^ (row & 7)) << 4));
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
                __syncwarp(); // the warp's reads of the stage are done
                if (!dead && lane == 0) mbar_arrive(smem_u32(&sh.empty1[ring.stage]));
                ring.advance();
            }
            if (!dead && row < rows) {
                const size_t o = ((size_t)t.b * p.KS + t.ks) * p.n_vis + j;
                p.pl1[o] = a0 + a1;
                p.pssq[o] = q0 + q1;
            }
            dead = workers_any(dead); // every worker's partial sums are issued
            if (!dead && wt == 0 && !post(make_int4(t.b, t.rt, t.ks, rows))) dead = true;
            if (++ms == kMail) {
                ms = 0;
                mph ^= 1u;
            }
        }
        workers_any(dead);
        if (wt == 0) post(make_int4(-1, 0, 0, 0)); // end of the stream (also after a failure, so that control exits)
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // ------------------------------------------------------------------ sweep-2 epilogue (warps independent)
        const int quarter = warp & 3;        // TMEM lane quarter this warp may read
        const int row = quarter * 32 + lane; // tile row owned by this thread
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
            const uint32_t taddr = tmem_base + acc * (uint32_t)p.N + ((uint32_t)(quarter * 32) << 16);
            float *dst = p.psim + (((size_t)t.b * p.KS + t.ks) * p.n_vis + j) * p.P;
            for (int c0 = 0; c0 < p.P; c0 += 8) {
                float v[8];
                tmem_ld8(taddr + (uint32_t)c0, v); // warp-collective: rows outside the tile still take part
                if (row < rows) {
                    if (c0 + 8 <= p.P && (p.P & 3) == 0) {
                        *reinterpret_cast<float4 *>(dst + c0) = make_float4(v[0], v[1], v[2], v[3]);
                        *reinterpret_cast<float4 *>(dst + c0 + 4) = make_float4(v[4], v[5], v[6], v[7]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + e < p.P) dst[c0 + e] = v[e];
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.tmem_empty[acc]));
                if (quarter == 0) sh.s2_step = (int)g; // progress mark for the sweep-1 producer's throttle
            }
            ++s2n;
        }
    } else if (warp >= kCtrlWarp0 && warp < kCtrlWarp0 + kCtrlWarps) {
        // ------------------------------------------------------------------ control
        const Control cg;
        const int ct = cg.tid();
        int mi = 0;
        uint32_t mph = 0;
        for (;;) {
            bool fail = !ctl.wait_bar(smem_u32(&sh.mail_full[mi]), mph, kWaitMail, 0);
            if (control_any(fail)) break;
            const int4 m = sh.mail[mi];
            cg.sync(); // everyone has read the slot
            if (ct == 0) mbar_arrive(smem_u32(&sh.mail_empty[mi]));
            if (++mi == kMail) {
                mi = 0;
                mph ^= 1u;
            }
            if (m.x < 0) break;
            // Who finalises is fixed by the schedule, not by arrival order: the CTA that holds slab
            // (b + rt) % KS of a row tile finalises it, and the one that finalises a sample's LAST row tile
            // merges the sample, so that it only ever waits for work that precedes its own in the schedule
            // (its own later mails can then never be what it waits for).  Letting the last arriver do it
            // instead makes a busy control group ever later, hence ever last.
            int *slabs = p.rt_done + (size_t)m.x * p.n_rt + m.y;
            const bool fin_tile = m.z == (m.x + m.y) % p.KS, fin_sample = fin_tile && m.y == p.n_rt - 1;
            bool late = false;
            if (ct == 0) {
                __threadfence(); // the workers' partial sums (ordered before the mail) become visible GPU-wide
                atomicAdd(slabs, 1);
                if (fin_tile) late = !ctl.wait_flag(slabs, kWaitSlabs, m.x, p.KS);
            }
            if (control_any(late)) break;
            if (fin_tile) {
                finalize_row_tile(p, sh, m.x, m.y, m.w);
                __threadfence();
                cg.sync();
                if (ct == 0) {
                    atomicAdd(p.s1_done + m.x, 1);
                    if (fin_sample) late = !ctl.wait_flag(p.s1_done + m.x, kWaitRowTiles, m.x, p.n_rt);
                }
                if (control_any(late)) break;
                if (fin_sample) merge_pivots(p, sh, m.x);
            }
        }
    }
    // ---------------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
}

// Adds up the per-slab partial dot products in slab order and normalises them (Eq. 7):
// sim[b][i][j] = (sum_ks psim[b][ks][j][i]) / (|K_{p_i}| |K_j|); a zero norm gives 0.
constexpr int kFinalizeThreads = 128;

__global__ void __launch_bounds__(kFinalizeThreads)
finalize_sim_kernel(const float *__restrict__ psim, const float *__restrict__ ssq, const int32_t *__restrict__ pivot_idx,
                    int n_vis, int P, int KS, const int *__restrict__ status, float *__restrict__ sim)
{
    const int b = blockIdx.y, j = blockIdx.x * kFinalizeThreads + threadIdx.x;
    if (j >= n_vis || *status != 0) return; // after a failed sweep the pivots are undefined
    const float nj = sqrtf(ssq[(size_t)b * n_vis + j]);
    const int32_t *piv = pivot_idx + (size_t)b * P;
    for (int p0 = 0; p0 < P; p0 += 4) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int ks = 0; ks < KS; ++ks) {
            const float *src = psim + (((size_t)b * KS + ks) * n_vis + j) * P + p0;
            if ((P & 3) == 0) {
                const float4 v = __ldcs(reinterpret_cast<const float4 *>(src));
                acc[0] += v.x, acc[1] += v.y, acc[2] += v.z, acc[3] += v.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (p0 + e < P) acc[e] += __ldcs(src + e);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (p0 + e >= P) break;
            const float den = sqrtf(ssq[(size_t)b * n_vis + piv[p0 + e]]) * nj;
            sim[((size_t)b * P + p0 + e) * n_vis + j] = den > 0.f ? acc[e] / den : 0.f;
        }
    }
}

} // namespace sweep
} // namespace dart
