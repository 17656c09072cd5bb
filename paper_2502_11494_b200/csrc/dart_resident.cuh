// Resident sweep: scores, pivots and similarities from ONE read of the keys (Sec. 3.3, steps 1-3; Def. 1-2, Eq. 7).
//
// The pivots of a sample are known only after all of its rows have been scored, so a kernel that streams the rows
// has to read them again for Eq. 7 - unless the sample is still on the chip.  One sample of the large workloads
// (2880 rows x 8 KB = 23.6 MB) does not fit one SM, but it fits the GPU: shared memory and tensor memory of all
// SMs together hold about three samples.  This kernel therefore spreads every sample over ALL CTAs (one per SM,
// launched cooperatively) and keeps the rows on the chip until the sample's pivots are known:
//
//   * A sample's rows are cut into octets (8 consecutive rows).  Octet t = n * n_oct + o of the whole batch belongs
//     to CTA t mod G, so every CTA holds 2-3 octets of every sample and the assignment rotates from sample to
//     sample (equal load without a remainder).
//   * producer warp: one bulk copy per row into a landing slot of shared memory (rows 16 bytes further apart than
//     their length, which makes 8-row matrix loads conflict-free).
//   * scorer warps (four, two rows of every octet each): L1 norm and sum of squares of the landed rows.
//   * worker warp q (four, one per 32-lane quarter of tensor memory): reads a landed octet with ldmatrix in the
//     register layout of an mma.sync B operand (token = column of the product) and parks the fragments in tensor
//     memory with tcgen05.st: tensor memory serves as 256 KB of spill space per SM, each thread reads back exactly
//     what it wrote.  When scorers and worker are done the landing slot is free again.
//   * exchange warp: the CTA's best P rows of the sample go to global memory (score key and index), a counter per
//     sample counts the CTAs that have published; when all have, every CTA merges the sorted lists itself (each
//     lane its share of the lists, then a butterfly of 8-entry merges across the lanes) and fetches the P pivot
//     rows into shared memory.
//   * worker warp again: fragments back from tensor memory (tcgen05.ld), pivot rows as the A operand (ldmatrix),
//     mma.sync m16n8k16 with fp32 accumulation: D[pivot][token]; normalised and written as dup(p_i, x_j).
//
// Every octet is read from HBM once; the pivot rows are read again by every CTA (P rows per sample, from L2).
// The time between a row's arrival and its sample's pivots (scoring, two global round trips, the merge, the pivot
// fetch) has to be covered by the octets that wait on the chip: tensor-memory slots plus landing slots, 2.4 samples
// of 2880 x 4096.  Measured on a B200 that time is ~27 us per sample where one read at full bandwidth allows 3.4 us
// per sample, so the kernel runs at about half the speed of the two-read sweep there; it is an option, not a default.
//
// Limits (else the caller takes another path): P <= 8, d % 64 == 0, d <= 4096, at most min(4, slots) octets per
// CTA and sample.  All waits are bounded; a wait that expires sets the status words and every role winds down.
#pragma once
#include "dart_sweep.cuh"

namespace dart {
namespace resident {
using namespace sweep; // PTX wrappers, bounded waits

constexpr int kThreads = 320; // 204 registers per thread
constexpr int kProducerWarp = 0, kExchangeWarp = 1, kWorker0 = 4, kWorkers = 4; // kWorker0 % 4 == 0: worker q owns TMEM lanes 32 q ..
constexpr int kScorers = 4; // warps 2, 3, 8, 9: scorer w takes rows 2w and 2w + 1 of every octet
constexpr int kMeta = 64;                 // ring of per-octet scores: more than tensor-memory plus landing slots
constexpr int kOctRows = 8;
constexpr int kOctPerTile = kTileRows / kOctRows; // octets per 128-row tile (the unit of Params::split)
constexpr int kMaxP = 8;
constexpr int kMaxRowBytes = 8192;     // d <= 4096: one octet fills a quarter of tensor memory
constexpr int kRowPad = 16;            // bytes between rows in shared memory beyond their length
constexpr int kTmemCols = 512;
constexpr int kMaxSlotsPerQuarter = 8; // tensor-memory slots: 4 x min(8, 512 / (d / 8))
constexpr int kMaxSlots = 4 * kMaxSlotsPerQuarter;
constexpr int kMaxLanding = 8;
constexpr int kMaxOctPerSample = 4;    // per CTA: 32 rows, one per lane of the exchange warp
constexpr int kMaxGrid = 192;          // lists per lane of the merge: kMaxGrid / 32
constexpr int kStaticSmemReserve = 8192;
// second status word of a wait that expired
constexpr int kWaitLandingFree = 80, kWaitWorker = 81, kWaitScored = 82, kWaitPublished = 83, kWaitPivotBufFree = 84,
              kWaitLanded = 85, kWaitPivotNorms = 86;

struct Params {
    int B, S, vis_offset, n_vis, P, d;
    int n_oct;      // octets per sample
    int n_slots;    // tensor-memory slots (a multiple of 4)
    int n_landing;  // landing slots in shared memory
    int norm_kind, smallest;
    TileSplit split;   // which 128-row tiles stay on the chip; the octets of the others are scored here and nothing else
    int withhold;      // test hook: no CTA ever counts itself in after publishing its candidates, so that the bounded waits expire
    unsigned long long wait_ns;
    const char *keys;  // [B][S][d] bf16
    float *sim;        // [B][P][n_vis]
    float *l1, *ssq;   // [B][n_vis]
    int32_t *pivot_idx; // [B][P]
    unsigned long long *cand; // [B][G][kMaxP]: score key << 32 | ~index, best first; 0 = none
    int *arrived;      // [B] CTAs that have published their candidates, zero at launch
    int *status;
};

__host__ __device__ inline uint32_t row_pitch(int d) { return (uint32_t)d * 2u + kRowPad; }
__host__ __device__ inline uint32_t oct_bytes(int d) { return kOctRows * row_pitch(d); }
__host__ __device__ inline int tmem_slots(int d)
{
    int per = kTmemCols / (d / 8); // an octet takes d / 8 columns of its quarter
    if (per > kMaxSlotsPerQuarter) per = kMaxSlotsPerQuarter;
    return 4 * per;
}
__host__ __device__ inline uint32_t cand_smem_bytes(int G) { return (uint32_t)G * kMaxP * 8u; }
inline int landing_slots(int d, int G, int smem_limit)
{
    const long long left = (long long)smem_limit - kStaticSmemReserve - 128 - oct_bytes(d) - cand_smem_bytes(G);
    long long n = left / (long long)oct_bytes(d);
    return (int)(n > kMaxLanding ? kMaxLanding : n);
}
inline size_t smem_bytes(int d, int G, int n_landing) { return 128 + (size_t)(1 + n_landing) * oct_bytes(d) + cand_smem_bytes(G); }

struct Shared {
    unsigned long long full[kMaxLanding], empty[kMaxLanding]; // landing slots
    unsigned long long piv_full;                              // pivot rows of the current sample have landed
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile uint32_t armed;      // pivot fetches started so far (the barrier's phase of sample number ord is ord)
    volatile uint32_t pssq_ready; // samples whose pivot norms are in piv_ssq
    volatile uint32_t issued;     // octets whose copies have been started (octet s is phase s / L of full[s % L])
    volatile uint32_t mma_seq[kMaxSlots]; // octet number + 1 whose similarities have been written
    uint32_t scored[kMeta];       // scorer warps that are done with the octets of this ring entry, all uses added up
    float meta_ssq[kMeta][kOctRows];
    uint32_t meta_key[kMeta][kOctRows]; // ranking key of the row, larger = better pivot; 0 = no row
    float piv_ssq[kMaxP];
};

// The octets of one CTA in the order in which every role of the CTA meets them.
struct Seq {
    int G, c, n_oct, B, step;
    int n, off, o, ord; // sample, (n * n_oct) mod G, octet within the sample, samples with octets of this CTA so far - 1
    long long s;        // running number of the octet within the CTA
    __device__ Seq(int G_, int c_, int n_oct_, int B_) : G(G_), c(c_), n_oct(n_oct_), B(B_), step(n_oct_ % G_), n(-1), off(0), o(n_oct_), ord(-1), s(-1)
    {
        next();
    }
    __device__ __forceinline__ bool valid() const { return n < B; }
    __device__ __forceinline__ int first_octet() const { return (c - off + G) % G; }
    __device__ __forceinline__ bool last_of_sample() const { return o + G >= n_oct; }
    __device__ void next()
    {
        o += G;
        while (o >= n_oct) {
            if (++n >= B) return;
            off = n == 0 ? 0 : (off + step) % G;
            o = first_octet();
            if (o < n_oct) ++ord;
        }
        ++s;
    }
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D (16 pivots x 8 tokens, fp32) += A (16 x 16 bf16, rows 8-15 zero) * B (16 x 8 bf16)
__device__ __forceinline__ void mma_16816(float (&acc)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    const uint32_t z = 0;
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
                 : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}
#define DART_R8(r, o) "r"(r[o]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])
#define DART_W8(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
                 DART_R8(r, 0), DART_R8(r, 8), DART_R8(r, 16), DART_R8(r, 24)
                 : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t *r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), DART_R8(r, 0) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : DART_W8(r, 0), DART_W8(r, 8), DART_W8(r, 16), DART_W8(r, 24)
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// The same load without the wait, and the wait with the registers tied to it: the loaded values exist only after
// the wait, so nothing may read or move the registers between the two statements.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : DART_W8(r, 0), DART_W8(r, 8), DART_W8(r, 16), DART_W8(r, 24)
                 : "r"(taddr));
}
#define DART_T8(r, o) "+r"(r[o]), "+r"(r[o + 1]), "+r"(r[o + 2]), "+r"(r[o + 3]), "+r"(r[o + 4]), "+r"(r[o + 5]), "+r"(r[o + 6]), "+r"(r[o + 7])
__device__ __forceinline__ void tmem_ld32_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : DART_T8(r, 0), DART_T8(r, 8), DART_T8(r, 16), DART_T8(r, 24)::"memory");
}
#undef DART_T8
__device__ __forceinline__ void tmem_ld8u(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : DART_W8(r, 0) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
#undef DART_R8
#undef DART_W8

// |x| and x^2 of the two bf16 values in one word
__device__ __forceinline__ void add_pair(uint32_t w, float &l1, float &ssq)
{
    const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xffff0000u);
    l1 += fabsf(lo) + fabsf(hi);
    ssq = fmaf(lo, lo, ssq);
    ssq = fmaf(hi, hi, ssq);
}

// Waits in this kernel last long (a sample's pivots take tens of microseconds) and several warps wait at any time.
// Polls go through the same shared-memory pipe as the shuffles and loads of the warps that work, so a waiting warp
// sleeps between polls: tight polling slowed the working warps down several times over.
constexpr unsigned kPollNs = 100;

// Polls a shared-memory word until it reaches `target` (bounded like every other wait).
__device__ inline bool wait_seq(const Ctl &ctl, const volatile uint32_t *word, uint32_t target, int where, long long task)
{
    for (int it = 0; it < 4; ++it)
        if (*word >= target) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (*word >= target) return true;
        __nanosleep(kPollNs);
        if ((it & 31u) == 31u) {
            if (ctl.aborted()) return false;
            if ((unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                ctl.give_up(where, task);
                return false;
            }
        }
    }
}

// Bounded wait for a barrier phase, sleeping between polls.
__device__ inline bool wait_bar_polite(const Ctl &ctl, uint32_t bar, uint32_t parity, int where, long long task)
{
    for (int it = 0; it < 4; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(kPollNs);
        if ((it & 31u) == 31u) {
            if (ctl.aborted()) return false;
            if ((unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                ctl.give_up(where, task);
                return false;
            }
        }
    }
}

// The largest 64-bit key of the warp in two warp-wide reductions (lanes without a key pass 0); the same in all lanes.
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long key)
{
    const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
    const uint32_t top_hi = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t top_lo = __reduce_max_sync(0xffffffffu, hi == top_hi ? lo : 0u);
    return ((unsigned long long)top_hi << 32) | top_lo;
}

__global__ void __launch_bounds__(kThreads, 1) resident_kernel(const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x, c = (int)blockIdx.x;
    const uint32_t pitch = row_pitch(p.d), octb = oct_bytes(p.d), row_bytes = (uint32_t)p.d * 2u;
    const uint32_t smem0 = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t piv_buf = smem0;                         // P pivot rows at the landing pitch
    const uint32_t land0 = smem0 + octb;                    // n_landing octets
    const uint32_t cand_off = (1u + (uint32_t)p.n_landing) * octb; // [G][kMaxP] candidate keys of the current sample
    unsigned long long *cand_sm = reinterpret_cast<unsigned long long *>(smem_raw + ((smem0 - smem_u32(smem_raw)) + cand_off));
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    // the exchange warp is the one that waits for other CTAs: shortest limit, so that its wait reports first; then the producer
    const Ctl ctl{&sh.abort_flag, p.status, warp == kExchangeWarp ? limit : warp == kProducerWarp ? limit + limit / 8 : limit + limit / 4};
    const int L = p.n_landing, n_slots = p.n_slots;
    const uint32_t cols_per_oct = (uint32_t)p.d / 8u;

    if (threadIdx.x == 0) {
        for (int j = 0; j < kMaxLanding; ++j) {
            mbar_init(smem_u32(&sh.full[j]), 1);
            mbar_init(smem_u32(&sh.empty[j]), 1 + kScorers); // the worker that parks the octet and every scorer
        }
        mbar_init(smem_u32(&sh.piv_full), 1);
        sh.abort_flag = 0;
        sh.armed = 0;
        sh.pssq_ready = 0;
        sh.issued = 0;
        for (int j = 0; j < kMaxSlots; ++j) sh.mma_seq[j] = 0;
        for (int j = 0; j < kMeta; ++j) sh.scored[j] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kExchangeWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer: one bulk copy per row
        unsigned long long pol_drop;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_drop)); // read once
        long long issued = 0;
        for (Seq q(G, c, p.n_oct, p.B); q.valid(); q.next()) {
            const int j = (int)(q.s % L);
            const uint32_t par = (uint32_t)((q.s / L) & 1);
            bool ok = true;
            if (lane == 0) ok = wait_bar_polite(ctl, smem_u32(&sh.empty[j]), par ^ 1u, kWaitLandingFree, q.s);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            const int rows = min(kOctRows, p.n_vis - q.o * kOctRows);
            const uint32_t full = smem_u32(&sh.full[j]);
            if (lane == 0) {
                mbar_arrive_expect_tx(full, (uint32_t)rows * row_bytes);
                sh.issued = (uint32_t)(q.s + 1); // from here on the barrier is in this octet's phase until the octet is parked
            }
            __syncwarp();
            if (lane < rows) {
                const char *src = p.keys + ((size_t)q.n * p.S + p.vis_offset + (size_t)q.o * kOctRows + lane) * row_bytes;
                bulk_load(land0 + (uint32_t)j * octb + (uint32_t)lane * pitch, src, row_bytes, full, pol_drop);
            }
            issued = q.s + 1;
        }
        if (ctl.aborted() && lane == 0) // copies in flight must land before the CTA exits
            for (long long s = issued > L ? issued - L : 0; s < issued; ++s)
                ctl.wait_landed(smem_u32(&sh.full[s % L]), (uint32_t)((s / L) & 1));
    } else if (warp == kExchangeWarp) {
        // ------------------------------------------------------------------ exchange: candidates out, pivots in
        unsigned long long pol_keep;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep)); // pivot rows: every CTA reads them
        const int n_lists = (G + 31) / 32;
        long long prev_s[kMaxOctPerSample];
        int prev_k = 0;
        uint32_t armed = 0; // pivot fetches armed so far
        bool ok = true;
        for (Seq q(G, c, p.n_oct, p.B); ok && q.valid();) {
            const int n = q.n, off = q.off;
            long long s_of[kMaxOctPerSample];
            int o_of[kMaxOctPerSample];
            int k = 0;
            while (q.valid() && q.n == n) { // this CTA's octets of sample n
                if (k < kMaxOctPerSample) s_of[k] = q.s, o_of[k] = q.o, ++k;
                q.next();
            }
            // 1. the octets' scores: lane 8u + r takes row r of the sample's u-th octet here
            unsigned long long key = 0ull;
#pragma unroll
            for (int u = 0; u < kMaxOctPerSample; ++u)
                if (u < k) {
                    const int m = (int)(s_of[u] % kMeta);
                    ok = ok && wait_seq(ctl, &sh.scored[m], (uint32_t)(kScorers * (s_of[u] / kMeta + 1)), kWaitScored, s_of[u]);
                    if (ok && (lane >> 3) == u) {
                        const uint32_t rk = sh.meta_key[m][lane & 7];
                        const uint32_t idx = (uint32_t)(o_of[u] * kOctRows + (lane & 7));
                        key = rk ? ((unsigned long long)rk << 32) | (0xffffffffu - idx) : 0ull;
                    }
                }
            if (!__all_sync(0xffffffffu, ok)) break;
            // 2. the CTA's best P rows, best first (equal scores: lower index first): lane i keeps the winner of round i
            unsigned long long rec = 0ull;
#pragma unroll 1
            for (int i = 0; i < p.P; ++i) {
                const unsigned long long best = warp_max_key(key);
                if (lane == i) rec = best;
                if (key == best) key = 0ull; // keys are distinct (they carry the index): one lane, or nobody when best is 0
            }
            if (lane < kMaxP) __stcg(p.cand + ((size_t)n * G + c) * kMaxP + lane, rec);
            __threadfence();
            __syncwarp();
            const int contributors = p.n_oct < G ? p.n_oct : G;
            if (lane == 0) {
                if (!p.withhold) atomicAdd(p.arrived + n, 1);
                ok = ctl.wait_flag(p.arrived + n, kWaitPublished, n, contributors);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            // 3. merge: lane l reads the sorted lists of CTAs l, l + 32, ... (64 bytes each; all loads in flight at
            // once) and merges them into its own best 8; a butterfly over the lanes leaves the sample's best 8 in all
            int head[kMaxGrid / 32];
#pragma unroll
            for (int h = 0; h < kMaxGrid / 32; h += 3) { // three lists (twelve loads) at a time
                uint4 v[3][4];
#pragma unroll
                for (int u = h; u < h + 3; ++u) {
                    const int cc = lane + 32 * u;
                    const bool has = u < n_lists && cc < G && (cc - off + G) % G < p.n_oct; // that CTA holds rows of this sample
                    head[u] = has ? 0 : 8;
                    const uint4 *src = reinterpret_cast<const uint4 *>(p.cand + ((size_t)n * G + cc) * kMaxP);
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[u - h][i] = has ? __ldcg(src + i) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = h; u < h + 3; ++u) {
                    uint4 *dst = reinterpret_cast<uint4 *>(cand_sm + (size_t)(lane + 32 * u) * kMaxP);
                    if (u < n_lists && lane + 32 * u < G)
#pragma unroll
                        for (int i = 0; i < 4; ++i) dst[i] = v[u - h][i];
                }
            }
            unsigned long long cur[kMaxGrid / 32]; // the head of every list; only the list that wins reads its next key
            unsigned long long mine = 0ull;        // the best of them
#pragma unroll
            for (int u = 0; u < kMaxGrid / 32; ++u) {
                cur[u] = head[u] < 8 ? cand_sm[(lane + 32 * u) * kMaxP] : 0ull;
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
                            cur[u] = head[u] < 8 ? cand_sm[(lane + 32 * u) * kMaxP + head[u]] : 0ull;
                        }
                        mine = cur[u] > mine ? cur[u] : mine;
                    }
                }
            }
            my_piv = min(max(my_piv, 0), p.n_vis - 1);
            if (lane < p.P && c == off) p.pivot_idx[(size_t)n * p.P + lane] = my_piv; // the CTA that holds the sample's octet 0
            // the pivots' sums of squares were written by the CTAs that scored them, before they published
            float my_pssq = 0.f;
            if (lane < p.P) my_pssq = __ldcg(p.ssq + (size_t)n * p.n_vis + my_piv);
            // 4. the pivot buffer is free once the previous sample's similarities are written
            for (int u = 0; u < prev_k; ++u)
                ok = ok && wait_seq(ctl, &sh.mma_seq[prev_s[u] % n_slots], (uint32_t)(prev_s[u] + 1), kWaitPivotBufFree, prev_s[u]);
            if (!__all_sync(0xffffffffu, ok)) break;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); // the workers' reads of the buffer precede the copies
            __syncwarp();
            const uint32_t bar = smem_u32(&sh.piv_full);
            if (lane == 0) {
                mbar_arrive_expect_tx(bar, (uint32_t)p.P * row_bytes);
                sh.armed = armed + 1; // from here on the barrier is in this sample's phase until the workers are done with it
            }
            __syncwarp();
            if (lane < p.P)
                bulk_load(piv_buf + (uint32_t)lane * pitch, p.keys + ((size_t)n * p.S + p.vis_offset + my_piv) * row_bytes, row_bytes,
                          bar, pol_keep);
            if (lane < p.P) sh.piv_ssq[lane] = my_pssq; // needed at the end of the multiplication only
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                sh.pssq_ready = armed + 1;
            }
            ++armed;
            prev_k = k;
            for (int u = 0; u < k; ++u) prev_s[u] = s_of[u];
        }
        if (ctl.aborted() && armed && lane == 0) ctl.wait_landed(smem_u32(&sh.piv_full), (armed - 1) & 1u);
    } else if (warp == 2 || warp == 3 || warp == 8 || warp == 9) {
        // ------------------------------------------------------------------ scorers: L1 norm and sum of squares of two rows
        const int w = warp < 4 ? warp - 2 : warp - 6;
        const uint32_t n_chunks = row_bytes / 16u;
        bool ok = true;
        for (Seq q(G, c, p.n_oct, p.B); ok && q.valid(); q.next()) {
            const int j = (int)(q.s % L), m = (int)(q.s % kMeta);
            // a parity test is only meaningful once the barrier has reached this octet's phase
            ok = wait_seq(ctl, &sh.issued, (uint32_t)(q.s + 1), kWaitLanded, q.s);
            if (ok && lane == 0) ok = wait_bar_polite(ctl, smem_u32(&sh.full[j]), (uint32_t)((q.s / L) & 1), kWaitLanded, q.s);
            if (!__all_sync(0xffffffffu, ok)) break;
            mbar_try_wait(smem_u32(&sh.full[j]), (uint32_t)((q.s / L) & 1)); // every lane observes the completed phase itself
            const int rows = min(kOctRows, p.n_vis - q.o * kOctRows);
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = 2 * w + rr;
                uint32_t rk = 0;
                float l1 = 0.f, ssq = 0.f;
                if (r < rows) {
                    const uint32_t base = land0 + (uint32_t)j * octb + (uint32_t)r * pitch;
                    float l1a[4] = {0.f, 0.f, 0.f, 0.f}, ssqa[4] = {0.f, 0.f, 0.f, 0.f}; // four chains: the sums are latency bound
                    for (uint32_t ch = lane; ch < n_chunks; ch += 128) { // four loads in flight (row lengths are multiples of 128 bytes)
                        uint4 v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) v[e] = ch + 32u * e < n_chunks ? lds128(base + (ch + 32u * e) * 16u) : make_uint4(0, 0, 0, 0);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            add_pair(v[e].x, l1a[0], ssqa[0]);
                            add_pair(v[e].y, l1a[1], ssqa[1]);
                            add_pair(v[e].z, l1a[2], ssqa[2]);
                            add_pair(v[e].w, l1a[3], ssqa[3]);
                        }
                    }
                    l1 = warp_sum((l1a[0] + l1a[1]) + (l1a[2] + l1a[3]));
                    ssq = warp_sum((ssqa[0] + ssqa[1]) + (ssqa[2] + ssqa[3]));
                    const uint32_t ok_ = order_key(p.norm_kind == 2 ? ssq : l1);
                    rk = p.smallest ? ~ok_ : ok_;
                    if (rk == 0) rk = 1; // 0 marks "no row"
                }
                if (lane == 0) {
                    if (r < rows) {
                        const size_t at = (size_t)q.n * p.n_vis + (size_t)q.o * kOctRows + r;
                        p.l1[at] = l1;
                        p.ssq[at] = ssq;
                    }
                    sh.meta_key[m][r] = rk;
                    sh.meta_ssq[m][r] = ssq;
                }
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence(); // the global sums of squares are read by other CTAs once this CTA has published
                mbar_arrive(smem_u32(&sh.empty[j]));
                atomicAdd(&sh.scored[m], 1u);
            }
        }
    } else if (warp >= kWorker0 && warp < kWorker0 + kWorkers) {
        // ------------------------------------------------------------------ workers: park, then multiply
        const int quarter = warp - kWorker0;
        const uint32_t tq = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int g = lane >> 2, t = lane & 3;
        // this lane's row address within an 8-row, 32-column block: row lane % 8, 16-byte chunk lane / 8
        const uint32_t lm_off = (uint32_t)(lane & 7) * pitch + (uint32_t)(lane >> 3) * 16u;
        Seq cs(G, c, p.n_oct, p.B), ms(G, c, p.n_oct, p.B); // next octet to park, next octet to multiply
        while (cs.valid() && (cs.s & 3) != quarter) cs.next();
        while (ms.valid() && (ms.s & 3) != quarter) ms.next();
        long long t0 = 0;
        uint32_t idle = 0;
        bool failed = false;
        while (ms.valid() && !failed) {
            bool did = false;
            if (cs.valid() && cs.s - ms.s < n_slots) { // the slot's previous octet has been multiplied
                const int j = (int)(cs.s % L);
                if (!p.split.on_chip(cs.o / kOctPerTile)) {
                    // an octet of a streamed tile: nothing to park.  The landing slot still counts this warp among those
                    // that release it, and its barrier is in this octet's phase once the copies have been started.
                    if (sh.issued > (uint32_t)cs.s) {
                        if (lane == 0) mbar_arrive(smem_u32(&sh.empty[j]));
                        do cs.next();
                        while (cs.valid() && (cs.s & 3) != quarter);
                        did = true;
                    }
                } else
                // a parity test is only meaningful once the barrier has reached this octet's phase
                if (sh.issued > (uint32_t)cs.s && mbar_try_wait(smem_u32(&sh.full[j]), (uint32_t)((cs.s / L) & 1))) {
                    // ---- park octet cs.s: shared memory -> registers -> tensor memory
                    const int slot = (int)(cs.s % n_slots);
                    const uint32_t tcol = tq + (uint32_t)(slot >> 2) * cols_per_oct;
                    const uint32_t src = land0 + (uint32_t)j * octb + lm_off;
                    const int n32 = p.d / 256, n8 = (p.d % 256) / 64; // batches of 32 and of 8 registers
                    for (int bt = 0; bt < n32; ++bt) {
                        uint32_t r[32];
#pragma unroll
                        for (int it = 0; it < 8; ++it)
                            ldmatrix_x4(src + (uint32_t)(bt * 8 + it) * 64u, r[4 * it], r[4 * it + 1], r[4 * it + 2], r[4 * it + 3]);
                        tmem_st32(tcol + (uint32_t)bt * 32u, r);
                    }
                    for (int bt = 0; bt < n8; ++bt) {
                        uint32_t r[8];
#pragma unroll
                        for (int it = 0; it < 2; ++it)
                            ldmatrix_x4(src + (uint32_t)(n32 * 8 + bt * 2 + it) * 64u, r[4 * it], r[4 * it + 1], r[4 * it + 2], r[4 * it + 3]);
                        tmem_st8(tcol + (uint32_t)n32 * 32u + (uint32_t)bt * 8u, r);
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh.empty[j])); // this warp is done with the landing slot
                    do cs.next();
                    while (cs.valid() && (cs.s & 3) != quarter);
                    did = true;
                }
            }
            if (!did && ms.s < cs.s + (cs.valid() ? 0 : (1ll << 40))) { // parked and waiting for its sample's pivots
                if (!p.split.on_chip(ms.o / kOctPerTile)) { // never parked: nothing of it waits for the pivot buffer
                    if (lane == 0) sh.mma_seq[ms.s % n_slots] = (uint32_t)(ms.s + 1);
                    do ms.next();
                    while (ms.valid() && (ms.s & 3) != quarter);
                    did = true;
                } else
                // a parity test is only meaningful once the barrier has reached this sample's phase
                if (sh.armed > (uint32_t)ms.ord && mbar_try_wait(smem_u32(&sh.piv_full), (uint32_t)(ms.ord & 1))) {
                    // ---- multiply octet ms.s: D[pivot][token] over all columns, four accumulators in turn
                    const int slot = (int)(ms.s % n_slots), m = (int)(ms.s % kMeta);
                    const uint32_t tcol = tq + (uint32_t)(slot >> 2) * cols_per_oct;
                    const uint32_t asrc = piv_buf + lm_off;
                    float acc[4][4];
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[a][e] = 0.f;
                    const int n32 = p.d / 256, n8 = (p.d % 256) / 64;
                    auto multiply = [&](int bt, const uint32_t(&r)[32]) {
#pragma unroll
                        for (int it = 0; it < 8; ++it) { // 32 columns: two k16 blocks
                            uint32_t a0, a2, a0n, a2n;
                            ldmatrix_x4(asrc + (uint32_t)(bt * 8 + it) * 64u, a0, a2, a0n, a2n);
                            mma_16816(acc[(2 * it) & 3], a0, a2, r[4 * it], r[4 * it + 1]);
                            mma_16816(acc[(2 * it + 1) & 3], a0n, a2n, r[4 * it + 2], r[4 * it + 3]);
                        }
                    };
                    {   // two register sets in turn: the next batch is on its way while this one is multiplied
                        uint32_t ra[32], rb[32];
                        if (n32 > 0) tmem_ld32_issue(tcol, ra);
                        for (int bt = 0; bt < n32; bt += 2) {
                            tmem_ld32_wait(ra);
                            if (bt + 1 < n32) tmem_ld32_issue(tcol + (uint32_t)(bt + 1) * 32u, rb);
                            multiply(bt, ra);
                            if (bt + 1 < n32) {
                                tmem_ld32_wait(rb);
                                if (bt + 2 < n32) tmem_ld32_issue(tcol + (uint32_t)(bt + 2) * 32u, ra);
                                multiply(bt + 1, rb);
                            }
                        }
                    }
                    for (int bt = 0; bt < n8; ++bt) {
                        uint32_t r[8];
                        tmem_ld8u(tcol + (uint32_t)n32 * 32u + (uint32_t)bt * 8u, r);
#pragma unroll
                        for (int it = 0; it < 2; ++it) {
                            uint32_t a0, a2, a0n, a2n;
                            ldmatrix_x4(asrc + (uint32_t)(n32 * 8 + bt * 2 + it) * 64u, a0, a2, a0n, a2n);
                            mma_16816(acc[(2 * it) & 3], a0, a2, r[4 * it], r[4 * it + 1]);
                            mma_16816(acc[(2 * it + 1) & 3], a0n, a2n, r[4 * it + 2], r[4 * it + 3]);
                        }
                    }
                    // the pivots' norms come by another route than their rows
                    if (!wait_seq(ctl, &sh.pssq_ready, (uint32_t)(ms.ord + 1), kWaitPivotNorms, ms.s)) failed = true;
                    failed = __any_sync(0xffffffffu, failed);
                    // thread (g, t): pivot g x tokens 2t, 2t + 1 of the octet
                    const int rows = min(kOctRows, p.n_vis - ms.o * kOctRows);
                    if (!failed && g < p.P) {
                        const float np_ = sqrtf(sh.piv_ssq[g]);
                        float *dst = p.sim + ((size_t)ms.n * p.P + g) * p.n_vis + (size_t)ms.o * kOctRows;
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int tok = 2 * t + e;
                            if (tok < rows) { // dup = dot / (|pivot| |row|); a zero norm gives 0
                                const float v = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
                                const float den = np_ * sqrtf(sh.meta_ssq[m][tok]);
                                dst[tok] = den > 0.f ? v / den : 0.f;
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        __threadfence_block();
                        sh.mma_seq[slot] = (uint32_t)(ms.s + 1);
                    }
                    do ms.next();
                    while (ms.valid() && (ms.s & 3) != quarter);
                    did = true;
                }
            }
            if (did) {
                idle = 0;
            } else if (idle < 64) {
                ++idle;
                __nanosleep(kPollNs);
            } else if (++idle > 64) { // a wait that lasts: start the clock, then check it now and then
                __nanosleep(2 * kPollNs);
                if (idle == 65) t0 = clock64();
                if ((idle & 31u) == 0u) {
                    bool stop = ctl.aborted();
                    if (!stop && (unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                        if (lane == 0) ctl.give_up(kWaitWorker, ms.s);
                        stop = true;
                    }
                    if (__any_sync(0xffffffffu, stop)) break;
                }
            }
        }
    }
    // ---------------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == kExchangeWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    // the CTA whose wait expired first adds where its pipeline stood: status words 4-10
    if (threadIdx.x == 0 && sh.abort_flag && p.status[0] == kStatusTimeout && p.status[3] == c && p.status[1] >= kWaitLandingFree) {
        for (int j = 0; j < 4; ++j) p.status[4 + j] = (int)sh.mma_seq[j];
        p.status[8] = (int)sh.issued, p.status[9] = (int)sh.pssq_ready, p.status[10] = (int)sh.armed;
    }
}

} // namespace resident
} // namespace dart
