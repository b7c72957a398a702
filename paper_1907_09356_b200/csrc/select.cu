// Per-row selection of the k largest ordering keys: top_a and random_a of the paper's
// Appendix C ("Compression Schemes").
//
// Ordering key of a coordinate: top_a -> bit pattern of |x - x^| (monotone for finite
// floats; +0 and -0 tie); random_a -> complement of the coordinate's Philox word (so the k smallest words
// win).  Ties go to the lower coordinate.  The message lists the chosen coordinates in
// ascending order with their values x - x^, plus a table tile_ptr[t] = number of chosen
// coordinates below 4096 t that lets a reader find any 4096-coordinate tile directly.
//
// Pipeline (all device-side, no host decisions):
//   prepare : histogram of the top 11 key bits -> lower key bound per row that keeps at
//             least k coordinates -> collect those coordinates ("candidates") tile by tile,
//             in ascending order inside a tile.
//   emit    : one block per row: exact k-th key by radix refinement over the candidates,
//             tie ranks, ordered compaction into the message.
//   exact   : rows whose candidates are unusable (too many equal keys, overflow) run a
//             one-block exact selection straight from the dense row.
#include "common.cuh"
#include "internal.h"

namespace choco {

constexpr int kSelThreads = 1024;
enum { SEL_TOPK = 0, SEL_RANDK = 1 };

template <int KIND>
__device__ __forceinline__ uint32_t order_key(uint32_t bits)
{
    // |v| without its sign bit, shifted up so that all 32 bits carry order information
    return KIND == SEL_TOPK ? (bits << 1) : ~bits;
}

// value bits of the four coordinates of a quad (top-k: x - x^; random-k: Philox words)
template <int KIND, bool VEC>
__device__ __forceinline__ void quad_bits(const Dev& dv, const StepArgs& a, int row, int64_t c,
                                          uint32_t out[4])
{
    if (KIND == SEL_TOPK) {
        const float4 x = load_quad<VEC>(a.X + (int64_t)row * dv.ld, c, dv.d);
        const float4 h = load_quad<VEC>(a.Xhat + (int64_t)row * dv.ld, c, dv.d);
        out[0] = __float_as_uint(__fsub_rn(x.x, h.x));
        out[1] = __float_as_uint(__fsub_rn(x.y, h.y));
        out[2] = __float_as_uint(__fsub_rn(x.z, h.z));
        out[3] = __float_as_uint(__fsub_rn(x.w, h.w));
    } else {
        const uint4 w = coord_words(dv.seed, a.step, (uint32_t)row, kStreamRandK, c);
        out[0] = w.x; out[1] = w.y; out[2] = w.z; out[3] = w.w;
    }
}

// ---------------------------------------------------------------------------------------
// block-wide helpers
// ---------------------------------------------------------------------------------------

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
// sum_{b >= D} hist[b] >= need; *above = sum_{b > D} hist[b].  nbins <= 2 * NT.
// All threads return the same values.  `sm` needs 36 words.
template <int NT>
__device__ __forceinline__ void block_find_digit(const uint32_t* hist, int nbins, uint32_t need,
                                                 uint32_t* sm, uint32_t* digit, uint32_t* above)
{
    const int r0 = 2 * threadIdx.x, r1 = r0 + 1;
    const uint32_t h0 = r0 < nbins ? hist[nbins - 1 - r0] : 0u;
    const uint32_t h1 = r1 < nbins ? hist[nbins - 1 - r1] : 0u;
    uint32_t total;
    const uint32_t ex = block_scan_excl<NT>(h0 + h1, sm, &total);
    if (threadIdx.x == 0) { sm[34] = 0u; sm[35] = 0u; }
    __syncthreads();
    if (ex < need && need <= ex + h0) {
        sm[34] = (uint32_t)(nbins - 1 - r0);
        sm[35] = ex;
    } else if (ex + h0 < need && need <= ex + h0 + h1) {
        sm[34] = (uint32_t)(nbins - 1 - r1);
        sm[35] = ex + h0;
    }
    __syncthreads();
    *digit = sm[34];
    *above = sm[35];
}

// ---------------------------------------------------------------------------------------
// prepare 1: histogram of the top 11 bits of |x - x^| (top-k only)
// ---------------------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(kThreads) hist_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t h[kHistBins];
    const int row = blockIdx.y;
    for (int b = threadIdx.x; b < kHistBins; b += kThreads) h[b] = 0u;
    __syncthreads();
    const int64_t c0 = (int64_t)blockIdx.x * kTile;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        if (c < dv.d) {
            uint32_t bits[4];
            quad_bits<SEL_TOPK, VEC>(dv, a, row, c, bits);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (c + e < dv.d) atomicAdd(&h[order_key<SEL_TOPK>(bits[e]) >> 21], 1u);
        }
    }
    __syncthreads();
    uint32_t* g = dv.hist + (int64_t)row * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kThreads)
        if (h[b]) atomicAdd(&g[b], h[b]);
}

// prepare 2: per row, the lowest first digit that must be kept
__global__ void __launch_bounds__(kSelThreads) bound_kernel(Dev dv)
{
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[36];
    const int row = blockIdx.x;
    uint32_t* g = dv.hist + (int64_t)row * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) {
        h[b] = g[b];
        g[b] = 0u; // ready for the next use
    }
    __syncthreads();
    uint32_t digit, above;
    block_find_digit<kSelThreads>(h, kHistBins, (uint32_t)dv.k, sm, &digit, &above);
    if (threadIdx.x == 0) {
        dv.row_lo[row] = digit << 21;
        dv.row_count[row] = 0u;
        // every coordinate with this digit or a higher one becomes a candidate
        dv.row_flags[row] = ((int64_t)above + (int64_t)h[digit] > dv.cap) ? kRowExact : 0u;
    }
}

// random-k: the bound is a fixed fraction of the word range, so that about
// k + 6 sqrt(k) + 16 coordinates qualify
__global__ void randk_bound_kernel(Dev dv, uint32_t lo)
{
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row < dv.n) {
        dv.row_lo[row] = lo;
        dv.row_count[row] = 0u;
        dv.row_flags[row] = 0u;
    }
}

// ---------------------------------------------------------------------------------------
// prepare 3: collect candidates, ascending inside each 4096-coordinate tile
// ---------------------------------------------------------------------------------------
template <int KIND, bool VEC>
__global__ void __launch_bounds__(kThreads) collect_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t sm[2][9];
    __shared__ uint32_t s_base;
    const int row = blockIdx.y;
    if (dv.row_flags[row] & kRowExact) return;
    const uint32_t lo = dv.row_lo[row];
    const int64_t c0 = (int64_t)blockIdx.x * kTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    uint32_t bits[kIters][4];
    uint32_t take = 0; // bit (4 it + e)
    uint32_t cnt[kIters];
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        cnt[it] = 0;
        if (c < dv.d) {
            quad_bits<KIND, VEC>(dv, a, row, c, bits[it]);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (c + e < dv.d && order_key<KIND>(bits[it][e]) >= lo) {
                    take |= 1u << (4 * it + e);
                    ++cnt[it];
                }
        }
    }
    // ordered slots: order is (iteration, thread, element).  Counts are scanned over the
    // threads for the four iterations at once, two 16-bit fields per word.
    uint32_t wa = cnt[0] | (cnt[1] << 16), wb = cnt[2] | (cnt[3] << 16);
    uint32_t ia = wa, ib = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o);
        const uint32_t tb = __shfl_up_sync(0xffffffffu, ib, o);
        if (lane >= o) { ia += ta; ib += tb; }
    }
    if (lane == 31) { sm[0][warp] = ia; sm[1][warp] = ib; }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ra = 0, rb = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            const uint32_t ta = sm[0][w], tb = sm[1][w];
            sm[0][w] = ra; sm[1][w] = rb;
            ra += ta; rb += tb;
        }
        sm[0][8] = ra; sm[1][8] = rb;
        const uint32_t total = (ra & 0xFFFFu) + (ra >> 16) + (rb & 0xFFFFu) + (rb >> 16);
        const uint32_t base = total ? atomicAdd(&dv.row_count[row], total) : 0u;
        dv.seg_off[(int64_t)row * dv.ntiles + blockIdx.x] = base;
        dv.seg_cnt[(int64_t)row * dv.ntiles + blockIdx.x] = total;
        s_base = base;
        if ((int64_t)base + total > dv.cap) s_base = 0xFFFFFFFFu; // overflow: emit sees count > cap
    }
    __syncthreads();
    if (s_base == 0xFFFFFFFFu) return;
    const uint32_t ea = sm[0][warp] + ia - wa, eb = sm[1][warp] + ib - wb; // exclusive, per thread
    const uint32_t ta = sm[0][8], tb = sm[1][8];
    uint32_t start[kIters];
    start[0] = ea & 0xFFFFu;
    start[1] = (ta & 0xFFFFu) + (ea >> 16);
    start[2] = (ta & 0xFFFFu) + (ta >> 16) + (eb & 0xFFFFu);
    start[3] = (ta & 0xFFFFu) + (ta >> 16) + (tb & 0xFFFFu) + (eb >> 16);
    uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cap + s_base;
    uint32_t* cv = dv.cand_val + (int64_t)row * dv.cap + s_base;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        uint32_t p = start[it];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (take & (1u << (4 * it + e))) {
                ci[p] = (uint32_t)(c + e);
                cv[p] = bits[it][e];
                ++p;
            }
    }
}

// ---------------------------------------------------------------------------------------
// emit: exact selection among the candidates of a row, ordered output
// ---------------------------------------------------------------------------------------
template <int KIND>
__global__ void __launch_bounds__(kSelThreads) emit_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[36];
    __shared__ uint32_t s_carry[2];
    const int row = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ncand = dv.row_count[row];
    const uint32_t flags = dv.row_flags[row];
    const uint32_t k = (uint32_t)dv.k;
    __syncthreads();
    if ((flags & kRowExact) || ncand > (uint32_t)dv.cap || ncand < k) {
        if (threadIdx.x == 0) {
            dv.row_flags[row] = kRowExact;
            dv.row_count[row] = 0u;
        }
        return;
    }
    const uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cap;
    const uint32_t* cv = dv.cand_val + (int64_t)row * dv.cap;

    // k-th largest key T by three radix digits (11, 11, 10 bits)
    uint32_t prefix = 0, pmask = 0, need = k;
    const int shifts[3] = {21, 10, 0};
    const int nbins[3] = {2048, 2048, 1024};
    for (int pass = 0; pass < 3; ++pass) {
        for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0u;
        __syncthreads();
        for (uint32_t p = threadIdx.x; p < ncand; p += kSelThreads) {
            const uint32_t key = order_key<KIND>(cv[p]);
            if ((key & pmask) == prefix) atomicAdd(&h[(key >> shifts[pass]) & (nbins[pass] - 1)], 1u);
        }
        __syncthreads();
        uint32_t digit, above;
        block_find_digit<kSelThreads>(h, nbins[pass], need, sm, &digit, &above);
        need -= above;
        prefix |= digit << shifts[pass];
        pmask |= (uint32_t)(nbins[pass] - 1) << shifts[pass];
        __syncthreads();
    }
    const uint32_t T = prefix;  // k-th largest key
    const uint32_t r = need;    // how many coordinates with key == T are kept (lowest first)

    // per tile: candidates above T, candidates equal to T
    const uint32_t* so = dv.seg_off + (int64_t)row * dv.ntiles;
    const uint32_t* sc = dv.seg_cnt + (int64_t)row * dv.ntiles;
    uint32_t* tgt = dv.tile_a + (int64_t)row * dv.ntiles;
    uint32_t* teq = dv.tile_b + (int64_t)row * dv.ntiles;
    for (int64_t t = warp; t < dv.ntiles; t += kSelThreads / 32) {
        const uint32_t off = so[t], cnt = sc[t];
        uint32_t gt = 0, eq = 0;
        for (uint32_t p = lane; p < cnt; p += 32) {
            const uint32_t key = order_key<KIND>(cv[off + p]);
            gt += key > T;
            eq += key == T;
        }
        gt = __reduce_add_sync(0xffffffffu, gt);
        eq = __reduce_add_sync(0xffffffffu, eq);
        if (lane == 0) { tgt[t] = gt; teq[t] = eq; }
    }
    if (threadIdx.x == 0) { s_carry[0] = 0u; s_carry[1] = 0u; }
    __syncthreads();
    // prefix over tiles: tile_ptr = (#above before) + min(#equal before, r); teq <- #equal before
    uint32_t* tp = dv.tile_ptr + (int64_t)row * (dv.ntiles + 1);
    for (int64_t t0 = 0; t0 < dv.ntiles; t0 += kSelThreads) {
        const int64_t t = t0 + threadIdx.x;
        const uint32_t gt = t < dv.ntiles ? tgt[t] : 0u;
        const uint32_t eq = t < dv.ntiles ? teq[t] : 0u;
        uint32_t tot_gt, tot_eq;
        const uint32_t ex_gt = block_scan_excl<kSelThreads>(gt, sm, &tot_gt);
        const uint32_t ex_eq = block_scan_excl<kSelThreads>(eq, sm, &tot_eq);
        const uint32_t cg = s_carry[0], ce = s_carry[1];
        if (t < dv.ntiles) {
            const uint32_t eqb = ce + ex_eq;
            tp[t] = cg + ex_gt + (eqb < r ? eqb : r);
            teq[t] = eqb;
        }
        __syncthreads();
        if (threadIdx.x == 0) { s_carry[0] = cg + tot_gt; s_carry[1] = ce + tot_eq; }
        __syncthreads();
    }
    if (threadIdx.x == 0) tp[dv.ntiles] = k;
    __syncthreads();
    // ordered compaction, one warp per tile
    uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch;
    float* mv = dv.msg_val + (int64_t)row * dv.kpitch;
    const float* xr = a.X + (int64_t)row * dv.ld;
    const float* hr = a.Xhat + (int64_t)row * dv.ld;
    const uint32_t lt = (1u << lane) - 1u;
    for (int64_t t = warp; t < dv.ntiles; t += kSelThreads / 32) {
        const uint32_t off = so[t], cnt = sc[t];
        uint32_t out = tp[t], eqrank = teq[t];
        for (uint32_t p0 = 0; p0 < cnt; p0 += 32) {
            const uint32_t p = p0 + lane;
            const bool act = p < cnt;
            const uint32_t idx = act ? ci[off + p] : 0u;
            const uint32_t bits = act ? cv[off + p] : 0u;
            const uint32_t key = order_key<KIND>(bits);
            const bool iseq = act && key == T;
            const uint32_t eqb = __ballot_sync(0xffffffffu, iseq);
            const bool sel = act && (key > T || (iseq && eqrank + __popc(eqb & lt) < r));
            const uint32_t sb = __ballot_sync(0xffffffffu, sel);
            if (sel) {
                const uint32_t pos = out + __popc(sb & lt);
                mi[pos] = idx;
                mv[pos] = KIND == SEL_TOPK ? __uint_as_float(bits) : __fsub_rn(xr[idx], hr[idx]);
            }
            out += __popc(sb);
            eqrank += __popc(eqb);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        dv.row_count[row] = 0u;
        atomicAdd(&dv.stats->recompressed_rows, 1ull);
    }
}

// ---------------------------------------------------------------------------------------
// exact: one block selects straight from the dense row (three radix passes and an ordered
// compaction pass).  Slow; only for rows whose candidates could not be used.
// ---------------------------------------------------------------------------------------
template <int KIND, bool VEC>
__global__ void __launch_bounds__(kSelThreads) exact_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[36];
    const int row = blockIdx.x;
    if (!(dv.row_flags[row] & kRowExact)) return;
    const uint32_t k = (uint32_t)dv.k;
    const int64_t span = (int64_t)kSelThreads * kQuad; // 4096 = one tile per iteration
    uint32_t prefix = 0, pmask = 0, need = k;
    const int shifts[3] = {21, 10, 0};
    const int nbins[3] = {2048, 2048, 1024};
    for (int pass = 0; pass < 3; ++pass) {
        for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0u;
        __syncthreads();
        for (int64_t c = (int64_t)threadIdx.x * kQuad; c < dv.d; c += span) {
            uint32_t bits[4];
            quad_bits<KIND, VEC>(dv, a, row, c, bits);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t key = order_key<KIND>(bits[e]);
                if (c + e < dv.d && (key & pmask) == prefix)
                    atomicAdd(&h[(key >> shifts[pass]) & (nbins[pass] - 1)], 1u);
            }
        }
        __syncthreads();
        uint32_t digit, above;
        block_find_digit<kSelThreads>(h, nbins[pass], need, sm, &digit, &above);
        need -= above;
        prefix |= digit << shifts[pass];
        pmask |= (uint32_t)(nbins[pass] - 1) << shifts[pass];
        __syncthreads();
    }
    const uint32_t T = prefix, r = need;
    uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch;
    float* mv = dv.msg_val + (int64_t)row * dv.kpitch;
    uint32_t* tp = dv.tile_ptr + (int64_t)row * (dv.ntiles + 1);
    const float* xr = a.X + (int64_t)row * dv.ld;
    const float* hr = a.Xhat + (int64_t)row * dv.ld;
    uint32_t run_gt = 0, run_eq = 0; // coordinates above / equal to T before this tile
    for (int64_t t = 0; t < dv.ntiles; ++t) {
        const int64_t c = t * span + (int64_t)threadIdx.x * kQuad;
        uint32_t bits[4] = {0u, 0u, 0u, 0u};
        uint32_t gtm = 0, eqm = 0;
        if (c < dv.d) {
            quad_bits<KIND, VEC>(dv, a, row, c, bits);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t key = order_key<KIND>(bits[e]);
                if (c + e < dv.d) {
                    gtm |= (uint32_t)(key > T) << e;
                    eqm |= (uint32_t)(key == T) << e;
                }
            }
        }
        uint32_t tot;
        const uint32_t ex = block_scan_excl<kSelThreads>(__popc(gtm) | (__popc(eqm) << 16), sm, &tot);
        if (threadIdx.x == 0) tp[t] = run_gt + (run_eq < r ? run_eq : r);
        uint32_t g = run_gt + (ex & 0xFFFFu), q = run_eq + (ex >> 16);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool isgt = (gtm >> e) & 1u, iseq = (eqm >> e) & 1u;
            if (isgt || (iseq && q < r)) {
                const uint32_t pos = g + (q < r ? q : r);
                mi[pos] = (uint32_t)(c + e);
                mv[pos] = KIND == SEL_TOPK ? __uint_as_float(bits[e])
                                           : __fsub_rn(xr[c + e], hr[c + e]);
            }
            g += isgt;
            q += iseq;
        }
        run_gt += tot & 0xFFFFu;
        run_eq += tot >> 16;
    }
    if (threadIdx.x == 0) {
        tp[dv.ntiles] = k;
        dv.row_flags[row] = 0u;
        atomicAdd(&dv.stats->exact_rows, 1ull);
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------

template <int KIND>
static cudaError_t prepare_impl(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    const dim3 grid((unsigned)dv.ntiles, (unsigned)dv.n);
    if (KIND == SEL_TOPK) {
        if (a.vec) hist_kernel<true><<<grid, kThreads, 0, st>>>(dv, a);
        else hist_kernel<false><<<grid, kThreads, 0, st>>>(dv, a);
        bound_kernel<<<dv.n, kSelThreads, 0, st>>>(dv);
        *a.launches += 2;
    } else {
        // keep words <= hi: about k + 6 sqrt(k) + 16 of d coordinates
        const double kk = (double)dv.k;
        double frac = (kk + 6.0 * sqrt(kk) + 16.0) / (double)dv.d;
        uint32_t hi = frac >= 1.0 ? 0xFFFFFFFFu : (uint32_t)(frac * 4294967296.0);
        randk_bound_kernel<<<(dv.n + 127) / 128, 128, 0, st>>>(dv, ~hi);
        *a.launches += 1;
    }
    if (a.vec) collect_kernel<KIND, true><<<grid, kThreads, 0, st>>>(dv, a);
    else collect_kernel<KIND, false><<<grid, kThreads, 0, st>>>(dv, a);
    *a.launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_prepare(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? prepare_impl<SEL_TOPK>(dv, a, st)
                                   : prepare_impl<SEL_RANDK>(dv, a, st);
}

template <int KIND>
static cudaError_t emit_impl(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    emit_kernel<KIND><<<dv.n, kSelThreads, 0, st>>>(dv, a);
    if (a.vec) exact_kernel<KIND, true><<<dv.n, kSelThreads, 0, st>>>(dv, a);
    else exact_kernel<KIND, false><<<dv.n, kSelThreads, 0, st>>>(dv, a);
    *a.launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_select_emit(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? emit_impl<SEL_TOPK>(dv, a, st) : emit_impl<SEL_RANDK>(dv, a, st);
}

} // namespace choco
