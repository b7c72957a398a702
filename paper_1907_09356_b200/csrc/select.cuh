// Pieces shared by the selection kernels (top_a / random_a of the paper's Appendix C) and by
// the update kernel, which collects the next step's candidates while it still holds
// x - x^ in registers.
#pragma once

#include "common.cuh"
#include "internal.h"

namespace choco {

constexpr int kSelThreads = 1024;
constexpr int kSelThreadsSmall = 256; // blocks for short rows: several of them share an SM
enum { SEL_TOPK = 0, SEL_RANDK = 1 };

// Ordering key: larger key = kept first.  top_a: |v| without its sign bit, shifted up so that
// all 32 bits carry order information (+0 and -0 tie).  random_a: complement of the Philox
// word, so that the k smallest words win.
template <int KIND>
__device__ __forceinline__ uint32_t order_key(uint32_t bits)
{
    return KIND == SEL_TOPK ? (bits << 1) : ~bits;
}

// Exclusive prefix sum over the block (NT threads, NT a multiple of 32, at most 1024).
// `sm` needs 33 words.  Returns the exclusive prefix; *total gets the block sum.
template <int NT>
__device__ __forceinline__ uint32_t block_scan_excl(uint32_t v, uint32_t* sm, uint32_t* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads(); // protect sm from the previous use
    if (lane == 31) sm[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < NT / 32 ? sm[lane] : 0u;
        uint32_t winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        sm[lane] = winc - w;
        if (lane == 31) sm[32] = winc;
    }
    __syncthreads();
    *total = sm[32];
    return sm[warp] + inc - v;
}

// Given hist[0..nbins) (shared memory) find the largest digit D with
// sum_{b >= D} hist[b] >= need; *above = sum_{b > D} hist[b].  nbins <= R * NT: a thread looks
// at R consecutive bins.  All threads return the same values.  `sm` needs 36 words.
template <int NT, int R = 2>
__device__ __forceinline__ void block_find_digit(const uint32_t* hist, int nbins, uint32_t need,
                                                 uint32_t* sm, uint32_t* digit, uint32_t* above)
{
    uint32_t hv[R], sum = 0u;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        const int r = R * (int)threadIdx.x + i; // bins are walked from the top
        hv[i] = r < nbins ? hist[nbins - 1 - r] : 0u;
        sum += hv[i];
    }
    uint32_t total;
    uint32_t run = block_scan_excl<NT>(sum, sm, &total);
    if (threadIdx.x == 0) { sm[34] = 0u; sm[35] = 0u; }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < R; ++i) {
        if (run < need && need <= run + hv[i]) {
            sm[34] = (uint32_t)(nbins - 1 - (R * (int)threadIdx.x + i));
            sm[35] = run;
        }
        run += hv[i];
    }
    __syncthreads();
    *digit = sm[34];
    *above = sm[35];
}

// A block of NT threads holds, per thread and per iteration `it` < NIT, cnt[it] <= 4 chosen
// coordinates of its tile; thread t's quad in iteration it covers coordinates
// (it * NT + t) * 4 ... + 3.  Computes the slot of each thread's first chosen coordinate in
// ascending coordinate order (start[it]) and the number chosen in the whole tile.
// NIT is 2 or 4 (16-bit fields: a tile holds fewer than 65536 coordinates).
// `sm` needs 2 x (NT / 32 + 1) words; contains two block barriers, or one with FRESH, when
// the caller knows that no thread of the block still reads `sm` from an earlier use.
template <int NT, int NIT, bool FRESH = false>
__device__ __forceinline__ void ordered_starts(const uint32_t cnt[NIT], uint32_t (*sm)[NT / 32 + 1],
                                               uint32_t start[NIT], uint32_t* total)
{
    static_assert(NIT == 2 || NIT == 4, "two 16-bit fields per word");
    static_assert(NT * NIT * 4 < 65536, "per-iteration totals must fit 16 bits");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t wa = cnt[0] | (cnt[1] << 16);
    uint32_t wb = 0u;
    if constexpr (NIT == 4) wb = cnt[2] | (cnt[3] << 16);
    uint32_t ia = wa, ib = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o);
        if (lane >= o) ia += ta;
        if constexpr (NIT == 4) {
            const uint32_t tb = __shfl_up_sync(0xffffffffu, ib, o);
            if (lane >= o) ib += tb;
        }
    }
    if (!FRESH) __syncthreads(); // protect sm from the previous use
    if (lane == 31) {
        sm[0][warp] = ia;
        if constexpr (NIT == 4) sm[1][warp] = ib;
    }
    __syncthreads();
    uint32_t pa = 0, pb = 0, ta = 0, tb = 0; // exclusive over warps, totals
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        const uint32_t xa = sm[0][w];
        if (w < warp) pa += xa;
        ta += xa;
        if constexpr (NIT == 4) {
            const uint32_t xb = sm[1][w];
            if (w < warp) pb += xb;
            tb += xb;
        }
    }
    const uint32_t ea = pa + ia - wa, eb = pb + ib - wb; // exclusive, per thread
    const uint32_t t0 = ta & 0xFFFFu, t1 = ta >> 16, t2 = tb & 0xFFFFu, t3 = tb >> 16;
    start[0] = ea & 0xFFFFu;
    start[1] = t0 + (ea >> 16);
    if constexpr (NIT == 4) {
        start[2] = t0 + t1 + (eb & 0xFFFFu);
        start[3] = t0 + t1 + t2 + (eb >> 16);
    }
    *total = t0 + t1 + t2 + t3;
}

} // namespace choco
