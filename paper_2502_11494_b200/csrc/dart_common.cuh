// Shared device helpers of the DART reduction kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dart {

constexpr int kWarp = 32;

// ---- memory access -------------------------------------------------------------------------
// 128-bit read-only load that does not allocate in L1: every key/hidden byte is used once per sweep.
__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 128-bit streaming store (evict-first): packed rows are not read again by this library.
__device__ __forceinline__ void st_stream(uint4 *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// ---- bf16 pairs ----------------------------------------------------------------------------
// A 32-bit word holds two bf16 values; each widens to fp32 by placing its 16 bits on top.
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- order-preserving float keys --------------------------------------------------------------
// Unsigned key whose order equals the float order (-0 and +0 are merged first so that they tie).
__device__ __forceinline__ uint32_t order_key(float f)
{
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float order_key_inv(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- which row tiles stay on the chip ------------------------------------------------------------
// The split path shares a sample's 128-row tiles between two kernels: the resident sweep keeps some of them in
// tensor memory until the sample's pivots are known, the rest is streamed a second time by the one-pass kernel.
// k <= 1: every tile stays on the chip.  inv == 0: tiles with rt % k == 0 stay (a fraction 1/k); inv == 1: tiles
// with rt % k != 0 stay (a fraction 1 - 1/k).
struct TileSplit {
    int k, inv;
    __host__ __device__ __forceinline__ bool on_chip(int rt) const { return k <= 1 || ((rt % k == 0) != (inv != 0)); }
    // tiles among n_rt that are streamed, and the i-th of them
    __host__ __device__ __forceinline__ int n_streamed(int n_rt) const
    {
        if (k <= 1) return 0;
        const int zero = (n_rt + k - 1) / k; // tiles with rt % k == 0
        return inv ? zero : n_rt - zero;
    }
    __host__ __device__ __forceinline__ int streamed(int i) const { return inv ? i * k : i + i / (k - 1) + 1; }
};

// ---- thread groups ---------------------------------------------------------------------------------
// The selection helpers below run either on a whole CTA or on a group of warps inside one
// (a named barrier), so that a few warps of a persistent kernel can select while others stream.
struct CtaGroup {
    __device__ __forceinline__ int tid() const { return threadIdx.x; }
    __device__ __forceinline__ int size() const { return blockDim.x; }
    __device__ __forceinline__ void sync() const { __syncthreads(); }
};
template <int kFirstWarp, int kWarps, int kBarrierId>
struct WarpGroup {
    __device__ __forceinline__ int tid() const { return (int)threadIdx.x - kFirstWarp * 32; }
    __device__ __forceinline__ int size() const { return kWarps * 32; }
    __device__ __forceinline__ void sync() const
    {
        asm volatile("bar.sync %0, %1;" ::"n"(kBarrierId), "n"(kWarps * 32) : "memory");
    }
};

// ---- group-wide selection of the k smallest (key, index) pairs -----------------------------------
// Radix select over 32-bit keys, 8 bits per pass, most significant first.  KeyFn(j, key&) returns
// whether element j takes part and, if so, its key.  After the call every thread holds the same
// threshold key T (the k-th smallest), the number `need_eq` of elements with key == T that belong to
// the selection (those of lowest index) and the number `cnt_eq` of elements with key == T.
struct SelectSmem {
    uint32_t hist[256];
    uint32_t warp_tot[32];
    uint32_t bin, before, cnt;
};

template <typename Group, typename KeyFn>
__device__ void block_select_threshold(Group g, KeyFn keyfn, int n, uint32_t k, SelectSmem &sm, uint32_t &T,
                                       uint32_t &need_eq, uint32_t &cnt_eq)
{
    uint32_t prefix = 0, mask = 0, remaining = k, cnt = 0;
    const int tid = g.tid(), gsz = g.size();
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += gsz) sm.hist[i] = 0;
        g.sync();
        // histogram with one cheap aggregation: the lanes of a warp that share the first valid lane's bin add
        // once (scores of real tokens share their leading key bytes, which would otherwise serialise one
        // atomic per lane); lanes in other bins add individually
        for (int j0 = 0; j0 < n; j0 += gsz) {
            const int j = j0 + tid;
            uint32_t key = 0;
            const bool v = j < n && keyfn(j, key) && (key & mask) == prefix;
            const uint32_t bin = (key >> shift) & 255u;
            const uint32_t valid = __ballot_sync(0xffffffffu, v);
            if (valid == 0) continue;
            const uint32_t bin0 = __shfl_sync(0xffffffffu, bin, __ffs(valid) - 1);
            const uint32_t same = __ballot_sync(0xffffffffu, v && bin == bin0);
            if (v) {
                if (bin != bin0)
                    atomicAdd(&sm.hist[bin], 1u);
                else if ((tid & 31) == __ffs(same) - 1)
                    atomicAdd(&sm.hist[bin], (uint32_t)__popc(same));
            }
        }
        g.sync();
        if (tid < kWarp) {
            // lane l owns bins [8l, 8l+8); find the bin where the running count reaches `remaining`
            uint32_t c[8], s = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                c[t] = sm.hist[tid * 8 + t];
                s += c[t];
            }
            uint32_t incl = s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                if (tid >= o) incl += v;
            }
            uint32_t excl = incl - s;
            if (excl < remaining && remaining <= incl) {
                uint32_t run = excl;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (run < remaining && remaining <= run + c[t]) {
                        sm.bin = tid * 8 + t;
                        sm.before = run;
                        sm.cnt = c[t];
                    }
                    run += c[t];
                }
            }
        }
        g.sync();
        prefix |= sm.bin << shift;
        mask |= 255u << shift;
        remaining -= sm.before;
        cnt = sm.cnt;
        g.sync();
    }
    T = prefix;
    need_eq = remaining;
    cnt_eq = cnt;
}

// Invoke pick(j, key) for every selected element: all with key < T, and the need_eq lowest-index
// elements with key == T.  Group-uniform control flow; ends with a group sync.
template <typename Group, typename KeyFn, typename PickFn>
__device__ void block_select_apply(Group g, KeyFn keyfn, int n, uint32_t T, uint32_t need_eq, uint32_t cnt_eq,
                                   SelectSmem &sm, PickFn pick)
{
    const bool all_eq = (need_eq == cnt_eq);
    const int tid = g.tid(), gsz = g.size();
    for (int j = tid; j < n; j += gsz) {
        uint32_t key;
        if (keyfn(j, key) && (key < T || (all_eq && key == T))) pick(j, key);
    }
    if (!all_eq) {
        // ties at the threshold: walk the indices in order and take the first need_eq
        const int lane = tid & 31, warp = tid >> 5, nwarp = gsz >> 5;
        uint32_t base = 0;
        for (int start = 0; start < n && base < need_eq; start += gsz) {
            int j = start + tid;
            uint32_t key = 0;
            bool f = (j < n) && keyfn(j, key) && key == T;
            uint32_t bal = __ballot_sync(0xffffffffu, f);
            if (lane == 0) sm.warp_tot[warp] = __popc(bal);
            g.sync();
            uint32_t before = 0, total = 0;
            for (int w = 0; w < nwarp; ++w) {
                uint32_t t = sm.warp_tot[w];
                if (w < warp) before += t;
                total += t;
            }
            uint32_t rank = base + before + __popc(bal & ((1u << lane) - 1u));
            if (f && rank < need_eq) pick(j, key);
            base += total;
            g.sync();
        }
    }
    g.sync();
}

} // namespace dart
