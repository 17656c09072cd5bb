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
//   * worker warp q (four, one per 32-lane quarter of tensor memory): reads a landed octet with ldmatrix in the
//     register layout of an mma.sync B operand (token = column of the product), accumulates the rows' L1 norms and
//     sums of squares on the way and parks the fragments in tensor memory with tcgen05.st: tensor memory serves as
//     256 KB of spill space per SM, each thread reads back exactly what it wrote.  The landing slot is free again.
//   * exchange warp: the CTA's best P rows of the sample go to global memory (score key, index, sum of squares), a
//     counter per sample counts the CTAs that have published; when all have, every CTA merges the sorted lists
//     itself (P rounds over the lists' heads) and fetches the P pivot rows into shared memory.
//   * worker warp again: fragments back from tensor memory (tcgen05.ld), pivot rows as the A operand (ldmatrix),
//     mma.sync m16n8k16 with fp32 accumulation: D[pivot][token]; normalised and written as dup(p_i, x_j).
//
// Every octet is read from HBM once; the pivot rows are read again by every CTA (P rows per sample, from L2).
// The time between a row's arrival and its sample's pivots (two global round trips, the merge, the pivot fetch)
// is covered by the octets that wait on the chip: tensor-memory slots plus landing slots.
//
// Limits (else the caller takes another path): P <= 8, d % 64 == 0, d <= 4096, at most min(4, slots) octets per
// CTA and sample.  All waits are bounded; a wait that expires sets the status words and every role winds down.
#pragma once
#include "dart_sweep.cuh"

namespace dart {
namespace resident {
using namespace sweep; // PTX wrappers, bounded waits

constexpr int kThreads = 256;
constexpr int kProducerWarp = 0, kExchangeWarp = 1, kWorker0 = 4, kWorkers = 4; // kWorker0 % 4 == 0: worker q owns TMEM lanes 32 q ..
constexpr int kOctRows = 8;
constexpr int kMaxP = 8;
constexpr int kMaxRowBytes = 8192;     // d <= 4096: one octet fills a quarter of tensor memory
constexpr int kRowPad = 16;            // bytes between rows in shared memory beyond their length
constexpr int kTmemCols = 512;
constexpr int kMaxSlotsPerQuarter = 8; // tensor-memory slots: 4 x min(8, 512 / (d / 8))
constexpr int kMaxSlots = 4 * kMaxSlotsPerQuarter;
constexpr int kMaxLanding = 8;
constexpr int kMaxOctPerSample = 4;    // per CTA: 32 rows, one per lane of the exchange warp
constexpr int kMaxGrid = 192;          // lists per lane of the merge: kMaxGrid / 32
constexpr int kStaticSmemReserve = 4096;
// second status word of a wait that expired
constexpr int kWaitLandingFree = 80, kWaitWorker = 81, kWaitConverted = 82, kWaitPublished = 83, kWaitPivotBufFree = 84;

struct Params {
    int B, S, vis_offset, n_vis, P, d;
    int n_oct;      // octets per sample
    int n_slots;    // tensor-memory slots (a multiple of 4)
    int n_landing;  // landing slots in shared memory
    int norm_kind, smallest;
    unsigned long long wait_ns;
    const char *keys;  // [B][S][d] bf16
    float *sim;        // [B][P][n_vis]
    float *l1, *ssq;   // [B][n_vis]
    int32_t *pivot_idx; // [B][P]
    uint4 *cand;       // [B][G][kMaxP]: {score key, ~index, sum of squares, 0}, best first
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
__host__ __device__ inline uint32_t cand_smem_bytes(int G) { return (uint32_t)G * kMaxP * 16u; }
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
    volatile uint32_t armed;               // pivot fetches started so far (the barrier's phase of sample number ord is ord)
    volatile uint32_t issued;              // octets whose copies have been started (octet s is phase s / L of full[s % L])
    volatile uint32_t conv_seq[kMaxSlots]; // octet number + 1 whose fragments and norms the slot holds
    volatile uint32_t mma_seq[kMaxSlots];  // octet number + 1 whose similarities have been written
    float slot_ssq[kMaxSlots][kOctRows];
    uint32_t slot_key[kMaxSlots][kOctRows]; // ranking key of the row, larger = better pivot; 0 = no row
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

// Polls a shared-memory word until it reaches `target` (bounded like every other wait).
__device__ inline bool wait_seq(const Ctl &ctl, const volatile uint32_t *word, uint32_t target, int where, long long task)
{
    for (int it = 0; it < 64; ++it)
        if (*word >= target) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (*word >= target) return true;
        __nanosleep(20);
        if ((it & 31u) == 31u) {
            if (ctl.aborted()) return false;
            if ((unsigned long long)(clock64() - t0) > ctl.limit_cycles) {
                ctl.give_up(where, task);
                return false;
            }
        }
    }
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
    const uint32_t cand_off = (1u + (uint32_t)p.n_landing) * octb; // [G][kMaxP] candidate records of the current sample
    uint4 *cand_sm = reinterpret_cast<uint4 *>(smem_raw + ((smem0 - smem_u32(smem_raw)) + cand_off));
    const unsigned long long limit = 2ull * p.wait_ns; // ns -> cycles at the highest SM clock: never shorter than asked
    const Ctl ctl{&sh.abort_flag, p.status, warp == kProducerWarp ? limit : limit + limit / 4};
    const int L = p.n_landing, n_slots = p.n_slots;
    const uint32_t cols_per_oct = (uint32_t)p.d / 8u;

    if (threadIdx.x == 0) {
        for (int j = 0; j < kMaxLanding; ++j) {
            mbar_init(smem_u32(&sh.full[j]), 1);
            mbar_init(smem_u32(&sh.empty[j]), 1);
        }
        mbar_init(smem_u32(&sh.piv_full), 1);
        sh.abort_flag = 0;
        sh.armed = 0;
        sh.issued = 0;
        for (int j = 0; j < kMaxSlots; ++j) sh.conv_seq[j] = 0, sh.mma_seq[j] = 0;
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
            if (lane == 0) ok = ctl.wait_bar(smem_u32(&sh.empty[j]), par ^ 1u, kWaitLandingFree, q.s);
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
            // 1. the octets' norms
            unsigned long long key = 0;
            float my_ssq = 0.f;
#pragma unroll
            for (int u = 0; u < kMaxOctPerSample; ++u)
                if (u < k) {
                    const int slot = (int)(s_of[u] % n_slots);
                    ok = ok && wait_seq(ctl, &sh.conv_seq[slot], (uint32_t)(s_of[u] + 1), kWaitConverted, s_of[u]);
                    if (ok && (lane >> 3) == u) {
                        const uint32_t rk = sh.slot_key[slot][lane & 7];
                        const uint32_t idx = (uint32_t)(o_of[u] * kOctRows + (lane & 7));
                        key = rk ? ((unsigned long long)rk << 32) | (0xffffffffu - idx) : 0ull;
                        my_ssq = sh.slot_ssq[slot][lane & 7];
                    }
                }
            if (!__all_sync(0xffffffffu, ok)) break;
            // 2. the CTA's best P rows, best first (equal scores: lower index first)
            uint4 rec = make_uint4(0, 0, 0, 0);
            for (int i = 0; i < p.P; ++i) {
                unsigned long long best = key;
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) {
                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, m);
                    best = other > best ? other : best;
                }
                const uint32_t who = __ballot_sync(0xffffffffu, best != 0ull && key == best);
                const int wl = who ? __ffs(who) - 1 : 0;
                const float wssq = __shfl_sync(0xffffffffu, my_ssq, wl);
                if (lane == i) rec = make_uint4((uint32_t)(best >> 32), (uint32_t)best, __float_as_uint(wssq), 0u);
                if (who && lane == wl) key = 0ull;
            }
            uint4 *mine = p.cand + ((size_t)n * G + c) * kMaxP;
            if (lane < p.P) __stcg(mine + lane, rec);
            __threadfence();
            __syncwarp();
            const int contributors = p.n_oct < G ? p.n_oct : G;
            if (lane == 0) {
                atomicAdd(p.arrived + n, 1);
                ok = ctl.wait_flag(p.arrived + n, kWaitPublished, n, contributors);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            // 3. merge: lane l walks the sorted lists of CTAs l, l + 32, ...
            int head[kMaxGrid / 32];
#pragma unroll
            for (int u = 0; u < kMaxGrid / 32; ++u) {
                const int cc = lane + 32 * u;
                const bool has = u < n_lists && cc < G && (cc - off + G) % G < p.n_oct; // that CTA holds rows of this sample
                head[u] = has ? 0 : p.P;
                if (has) {
                    const uint4 *src = p.cand + ((size_t)n * G + cc) * kMaxP;
                    for (int i = 0; i < p.P; ++i) cand_sm[cc * kMaxP + i] = __ldcg(src + i);
                }
            }
            __syncwarp();
            int my_piv = 0;
            float my_pssq = 0.f;
            for (int i = 0; i < p.P; ++i) {
                unsigned long long best = 0ull;
                int bu = 0;
                float bssq = 0.f;
#pragma unroll
                for (int u = 0; u < kMaxGrid / 32; ++u)
                    if (head[u] < p.P) {
                        const uint4 r = cand_sm[(lane + 32 * u) * kMaxP + head[u]];
                        const unsigned long long kk = ((unsigned long long)r.x << 32) | r.y;
                        if (kk > best) best = kk, bu = u, bssq = __uint_as_float(r.z);
                    }
                unsigned long long top = best;
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) {
                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, top, m);
                    top = other > top ? other : top;
                }
                const uint32_t who = __ballot_sync(0xffffffffu, top != 0ull && best == top);
                const int wl = who ? __ffs(who) - 1 : 0; // keys are distinct (they carry the index): one lane
                const float wssq = __shfl_sync(0xffffffffu, bssq, wl);
                if (lane == i) my_piv = (int)(0xffffffffu - (uint32_t)top), my_pssq = wssq;
                if (who && lane == wl) {
#pragma unroll
                    for (int u = 0; u < kMaxGrid / 32; ++u)
                        if (u == bu) ++head[u];
                }
            }
            if (lane < p.P) {
                my_piv = min(max(my_piv, 0), p.n_vis - 1);
                if (c == off) p.pivot_idx[(size_t)n * p.P + lane] = my_piv; // the CTA that holds the sample's octet 0
            }
            // 4. the pivot buffer is free once the previous sample's similarities are written
            for (int u = 0; u < prev_k; ++u)
                ok = ok && wait_seq(ctl, &sh.mma_seq[prev_s[u] % n_slots], (uint32_t)(prev_s[u] + 1), kWaitPivotBufFree, prev_s[u]);
            if (!__all_sync(0xffffffffu, ok)) break;
            if (lane < p.P) sh.piv_ssq[lane] = my_pssq;
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
            ++armed;
            prev_k = k;
            for (int u = 0; u < k; ++u) prev_s[u] = s_of[u];
        }
        if (ctl.aborted() && armed && lane == 0) ctl.wait_landed(smem_u32(&sh.piv_full), (armed - 1) & 1u);
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
        while (ms.valid()) {
            bool did = false;
            if (cs.valid() && cs.s - ms.s < n_slots) { // the slot's previous octet has been multiplied
                const int j = (int)(cs.s % L);
                // a parity test is only meaningful once the barrier has reached this octet's phase
                if (sh.issued > (uint32_t)cs.s && mbar_try_wait(smem_u32(&sh.full[j]), (uint32_t)((cs.s / L) & 1))) {
                    // ---- park octet cs.s: shared memory -> registers (+ norms) -> tensor memory
                    const int slot = (int)(cs.s % n_slots);
                    const uint32_t tcol = tq + (uint32_t)(slot >> 2) * cols_per_oct;
                    const uint32_t src = land0 + (uint32_t)j * octb + lm_off;
                    float l1 = 0.f, ssq = 0.f;
                    const int n32 = p.d / 256, n8 = (p.d % 256) / 64; // batches of 32 and of 8 registers
                    for (int bt = 0; bt < n32; ++bt) {
                        uint32_t r[32];
#pragma unroll
                        for (int it = 0; it < 8; ++it)
                            ldmatrix_x4(src + (uint32_t)(bt * 8 + it) * 64u, r[4 * it], r[4 * it + 1], r[4 * it + 2], r[4 * it + 3]);
#pragma unroll
                        for (int e = 0; e < 32; ++e) add_pair(r[e], l1, ssq);
                        tmem_st32(tcol + (uint32_t)bt * 32u, r);
                    }
                    for (int bt = 0; bt < n8; ++bt) {
                        uint32_t r[8];
#pragma unroll
                        for (int it = 0; it < 2; ++it)
                            ldmatrix_x4(src + (uint32_t)(n32 * 8 + bt * 2 + it) * 64u, r[4 * it], r[4 * it + 1], r[4 * it + 2], r[4 * it + 3]);
#pragma unroll
                        for (int e = 0; e < 8; ++e) add_pair(r[e], l1, ssq);
                        tmem_st8(tcol + (uint32_t)n32 * 32u + (uint32_t)bt * 8u, r);
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    // the four lanes of a group hold the four column classes of row g
                    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
                    ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
                    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
                    ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
                    const int rows = min(kOctRows, p.n_vis - cs.o * kOctRows);
                    if (t == 0) {
                        uint32_t rk = 0;
                        if (g < rows) {
                            const size_t at = (size_t)cs.n * p.n_vis + (size_t)cs.o * kOctRows + g;
                            p.l1[at] = l1;
                            p.ssq[at] = ssq;
                            const uint32_t ok_ = order_key(p.norm_kind == 2 ? ssq : l1);
                            rk = p.smallest ? ~ok_ : ok_;
                            if (rk == 0) rk = 1; // 0 marks "no row"
                        }
                        sh.slot_key[slot][g] = rk;
                        sh.slot_ssq[slot][g] = ssq;
                    }
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&sh.empty[j])); // the landing slot may be overwritten
                        __threadfence_block();
                        sh.conv_seq[slot] = (uint32_t)(cs.s + 1);
                    }
                    do cs.next();
                    while (cs.valid() && (cs.s & 3) != quarter);
                    did = true;
                }
            }
            if (!did && ms.s < cs.s + (cs.valid() ? 0 : (1ll << 40))) { // parked and waiting for its sample's pivots
                // a parity test is only meaningful once the barrier has reached this sample's phase
                if (sh.armed > (uint32_t)ms.ord && mbar_try_wait(smem_u32(&sh.piv_full), (uint32_t)(ms.ord & 1))) {
                    // ---- multiply octet ms.s: D[pivot][token] over all columns, four accumulators in turn
                    const int slot = (int)(ms.s % n_slots);
                    const uint32_t tcol = tq + (uint32_t)(slot >> 2) * cols_per_oct;
                    const uint32_t asrc = piv_buf + lm_off;
                    float acc[4][4];
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[a][e] = 0.f;
                    const int n32 = p.d / 256, n8 = (p.d % 256) / 64;
                    for (int bt = 0; bt < n32; ++bt) {
                        uint32_t r[32];
                        tmem_ld32(tcol + (uint32_t)bt * 32u, r);
#pragma unroll
                        for (int it = 0; it < 8; ++it) { // 32 columns: two k16 blocks
                            uint32_t a0, a2, a0n, a2n;
                            ldmatrix_x4(asrc + (uint32_t)(bt * 8 + it) * 64u, a0, a2, a0n, a2n);
                            mma_16816(acc[(2 * it) & 3], a0, a2, r[4 * it], r[4 * it + 1]);
                            mma_16816(acc[(2 * it + 1) & 3], a0n, a2n, r[4 * it + 2], r[4 * it + 3]);
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
                    // thread (g, t): pivot g x tokens 2t, 2t + 1 of the octet
                    const int rows = min(kOctRows, p.n_vis - ms.o * kOctRows);
                    if (g < p.P) {
                        const float np_ = sqrtf(sh.piv_ssq[g]);
                        float *dst = p.sim + ((size_t)ms.n * p.P + g) * p.n_vis + (size_t)ms.o * kOctRows;
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int tok = 2 * t + e;
                            if (tok < rows) { // dup = dot / (|pivot| |row|); a zero norm gives 0
                                const float v = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
                                const float den = np_ * sqrtf(sh.slot_ssq[slot][tok]);
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
            } else if (++idle > 64) { // a wait that lasts: start the clock, then check it now and then
                __nanosleep(32);
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
        for (int j = 0; j < 3; ++j) p.status[4 + j] = (int)sh.conv_seq[j], p.status[7 + j] = (int)sh.mma_seq[j];
        p.status[10] = (int)sh.armed;
    }
}

} // namespace resident
} // namespace dart
