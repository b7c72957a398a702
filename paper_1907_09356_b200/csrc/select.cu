// Per-row selection of the k largest ordering keys: top_a and random_a of the paper's
// Appendix C ("Compression Schemes").
//
// Ties go to the lower coordinate.  The message lists the chosen coordinates in ascending
// order with their values x - x^, plus a table tile_ptr[t] = number of chosen coordinates
// below kTile * t that lets a reader find any tile of coordinates directly.
//
// Pipeline (all device-side, no host decisions):
//   prepare : histogram of the top 11 key bits -> lower key bound per row that keeps at
//             least k coordinates -> collect those coordinates ("candidates") tile by tile,
//             in ascending order inside a tile.  (For top-k the update kernel of the previous
//             step normally did this already, with a bound guessed from that step.)
//   emit    : one block per row: exact k-th key by radix refinement over the candidates,
//             tie ranks, ordered compaction into the message; the candidate bound for the
//             next step.
//   exact   : rows whose candidates are unusable (too many, too few, overflow) run a
//             one-block exact selection straight from the dense row.
#include "select.cuh"

namespace choco {

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
// prepare 1: histogram of the top 11 bits of the key of x - x^ (top-k only)
// ---------------------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(kThreads) hist_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t h[kHistBins];
    const int row = blockIdx.y;
    for (int b = threadIdx.x; b < kHistBins; b += kThreads) h[b] = 0u;
    __syncthreads();
    const int64_t c0 = (int64_t)blockIdx.x * kSpan;
#pragma unroll
    for (int it = 0; it < kDenseIters; ++it) {
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
    // keep down to rank 3.5 k (not just k) so that emit can place the next step's bound
    const uint64_t want = 3 * (uint64_t)dv.k + (uint64_t)dv.k / 2;
    const uint32_t need = (uint32_t)(want < (uint64_t)dv.d ? want : (uint64_t)dv.d);
    uint32_t digit, above;
    block_find_digit<kSelThreads>(h, kHistBins, need, sm, &digit, &above);
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
// prepare 3: collect candidates, ascending inside each tile
// ---------------------------------------------------------------------------------------
template <int KIND, bool VEC>
__global__ void __launch_bounds__(kTileThreads) collect_kernel(Dev dv, StepArgs a)
{
    __shared__ uint32_t sm[2][kTileThreads / 32 + 1];
    __shared__ uint32_t s_base;
    const int row = blockIdx.y;
    if (dv.row_flags[row] & kRowExact) return;
    const uint32_t lo = dv.row_lo[row];
    const int64_t c0 = (int64_t)blockIdx.x * kTile;

    uint32_t bits[kTileIters][4];
    uint32_t take = 0; // bit (4 it + e)
    uint32_t cnt[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kTileThreads + threadIdx.x) * kQuad;
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
    uint32_t start[kTileIters], total;
    ordered_starts<kTileThreads, kTileIters>(cnt, sm, start, &total);
    if (threadIdx.x == 0) {
        const uint32_t base = total ? atomicAdd(&dv.row_count[row], total) : 0u;
        dv.seg_off[(int64_t)row * dv.ntiles + blockIdx.x] = base;
        dv.seg_cnt[(int64_t)row * dv.ntiles + blockIdx.x] = total;
        // past the capacity nothing is written; emit sees row_count > cap and gives up
        s_base = ((int64_t)base + total > dv.cap) ? 0xFFFFFFFFu : base;
    }
    __syncthreads();
    if (s_base == 0xFFFFFFFFu) return;
    uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cap + s_base;
    uint32_t* cv = dv.cand_val + (int64_t)row * dv.cap + s_base;
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kTileThreads + threadIdx.x) * kQuad;
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

// Radix refinement over the candidate values cv[0..ncand): the key of rank `rank`
// (1 = largest) and how many candidates are strictly above it.
template <int KIND>
__device__ __forceinline__ void rank_key(const uint32_t* cv, uint32_t ncand, uint32_t rank,
                                         uint32_t* h, uint32_t* sm, uint32_t* key_out,
                                         uint32_t* above_out)
{
    uint32_t prefix = 0, pmask = 0, need = rank, above_total = 0;
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
        above_total += above;
        prefix |= digit << shifts[pass];
        pmask |= (uint32_t)(nbins[pass] - 1) << shifts[pass];
        __syncthreads();
    }
    *key_out = prefix;
    *above_out = above_total;
}

// Tell every reader of worker `row` where row's message enters each tile (tp[t] .. tp[t+1]),
// in the reader's own CSR position, with the reader's own weight.  Called by all threads of
// the block after tp[] is complete and visible.
__device__ __forceinline__ void publish_ranges(const Dev& dv, int row, const uint32_t* tp)
{
    for (int e = dv.row_ptr[row]; e < dv.row_ptr[row + 1]; ++e) {
        const int64_t reader = dv.col[e];
        const int pos = dv.rd_pos[e];
        const uint32_t wbits = __float_as_uint(dv.rd_w[e]);
        uint4* rec = dv.rec + (reader * dv.ntiles) * dv.maxdeg + pos;
        for (int64_t t = threadIdx.x; t < dv.ntiles; t += blockDim.x) {
            const uint32_t lo = tp[t];
            rec[t * dv.maxdeg] = make_uint4((uint32_t)row, lo, tp[t + 1] - lo, wbits);
        }
    }
}

// Lower a key bound by `eighths` eighths of an octave (about 8 % of the value each).
__device__ __forceinline__ uint32_t lower_bound_key(uint32_t key, uint32_t eighths)
{
    const uint32_t dec = eighths << 21;
    return key > dec ? key - dec : 0u;
}

// Rank aimed at by the candidate bound: 3.5 k (the k chosen leave, about 2.5 k stay)
__host__ __device__ __forceinline__ uint64_t target_rank(uint64_t k) { return 3 * k + k / 2; }

// lo: bound the ncand candidates were collected with (their rank-ncand key, roughly);
// T: key of rank k.  Linear in the key between the two ranks, at most half an octave down.
__device__ __forceinline__ uint32_t next_bound(uint32_t lo, uint32_t T, uint32_t ncand, uint32_t k)
{
    if (ncand <= k || T < lo) return lower_bound_key(lo, 4u);
    const uint64_t span = T - lo, want = target_rank(k), den = ncand - k;
    if (ncand >= want) return lo + (uint32_t)((ncand - want) * span / den);
    uint64_t dec = (want - ncand) * span / den;
    if (dec > (4ull << 21)) dec = 4ull << 21;
    return lo > dec ? (uint32_t)(lo - dec) : 0u;
}

template <int KIND>
__global__ void __launch_bounds__(kSelThreads) emit_kernel(Dev dv, StepArgs a, int fused)
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

    uint32_t T, above;
    rank_key<KIND>(cv, ncand, k, h, sm, &T, &above);
    const uint32_t r = k - above; // how many coordinates with key == T are kept (lowest first)

    if (KIND == SEL_TOPK) {
        // Candidate bound for the next step: only a guess (the next step verifies that it kept
        // at least k coordinates and otherwise selects exactly from the dense row).  The k
        // chosen coordinates drop to ~0, so aim the bound at today's rank 3.5 k, reading the
        // key of that rank off a straight line through (rank k, T) and (rank ncand, bound).
        if (threadIdx.x == 0) dv.row_lo[row] = next_bound(dv.row_lo[row], T, ncand, k);
    }

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
    publish_ranges(dv, row, tp);
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
        atomicAdd(fused ? &dv.stats->prepared_rows : &dv.stats->recompressed_rows, 1ull);
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
    const int64_t span = (int64_t)kSelThreads * kQuad; // coordinates per block iteration
    const int64_t nspan = (dv.d + span - 1) / span;
    constexpr int kTilesPerSpan = (kSelThreads * kQuad) / kTile;
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
    uint32_t run_gt = 0, run_eq = 0; // coordinates above / equal to T before this span
    for (int64_t sp = 0; sp < nspan; ++sp) {
        const int64_t c = sp * span + (int64_t)threadIdx.x * kQuad;
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
        uint32_t g = run_gt + (ex & 0xFFFFu), q = run_eq + (ex >> 16);
        // the first thread of every tile records how many coordinates were chosen before it
        if ((threadIdx.x % (kTile / kQuad)) == 0) {
            const int64_t t = sp * kTilesPerSpan + threadIdx.x / (kTile / kQuad);
            if (t < dv.ntiles) tp[t] = g + (q < r ? q : r);
        }
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
    if (threadIdx.x == 0) tp[dv.ntiles] = k;
    __syncthreads();
    publish_ranges(dv, row, tp);
    if (threadIdx.x == 0) {
        dv.row_flags[row] = 0u;
        dv.row_count[row] = 0u;
        if (KIND == SEL_TOPK) dv.row_lo[row] = lower_bound_key(T, 3u);
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
        const dim3 hgrid((unsigned)dv.nspans, (unsigned)dv.n);
        if (a.vec) hist_kernel<true><<<hgrid, kThreads, 0, st>>>(dv, a);
        else hist_kernel<false><<<hgrid, kThreads, 0, st>>>(dv, a);
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
    if (a.vec) collect_kernel<KIND, true><<<grid, kTileThreads, 0, st>>>(dv, a);
    else collect_kernel<KIND, false><<<grid, kTileThreads, 0, st>>>(dv, a);
    *a.launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_prepare(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? prepare_impl<SEL_TOPK>(dv, a, st)
                                   : prepare_impl<SEL_RANDK>(dv, a, st);
}

template <int KIND>
static cudaError_t emit_impl(const Dev& dv, const StepArgs& a, bool fused, cudaStream_t st)
{
    emit_kernel<KIND><<<dv.n, kSelThreads, 0, st>>>(dv, a, fused ? 1 : 0);
    if (a.vec) exact_kernel<KIND, true><<<dv.n, kSelThreads, 0, st>>>(dv, a);
    else exact_kernel<KIND, false><<<dv.n, kSelThreads, 0, st>>>(dv, a);
    *a.launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_select_emit(const Dev& dv, const StepArgs& a, bool fused, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? emit_impl<SEL_TOPK>(dv, a, fused, st)
                                   : emit_impl<SEL_RANDK>(dv, a, fused, st);
}

} // namespace choco
