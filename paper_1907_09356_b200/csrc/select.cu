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
//   exact   : rows whose candidates are unusable (too many, too few, overflow) are selected
//             exactly, by the same block, straight from the dense row.
#include <cooperative_groups.h>

#include <algorithm>

#include "bulk.cuh"
#include "select.cuh"

namespace choco {

// Rank the candidate bound aims at, in units of k / 256, kept per row: it starts at 3 k,
// creeps down to 1.75 k while the guesses keep holding (fewer candidates = less work in the
// emit kernel) and jumps back to 3 k when a row had to be selected exactly.  (A start at
// 2.5 k missed on 24 row-steps during steps 5-7 of a 32 x 25.6 M top-0.1 % run, where one
// exact selection from the 102 MB row takes about 30 ms; from 3 k none missed.)
constexpr uint32_t kAimStart = 768u, kAimMin = 448u, kAimAfterMiss = 768u, kAimStep = 8u;

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
        const uint4 w = coord_words(dv.seed, step_of(a), (uint32_t)row, kStreamRandK, c);
        out[0] = w.x; out[1] = w.y; out[2] = w.z; out[3] = w.w;
    }
}

// ---------------------------------------------------------------------------------------
// prepare 1: histogram of the top 11 bits of the key of x - x^ (top-k only)
// ---------------------------------------------------------------------------------------
// True (for every thread of the block) if any row carries one of the flags in `mask`.  The
// rescue kernels ask this first: the rows' flags are read side by side rather than one after
// the other, so a launch with nothing to do is over in about a microsecond.
__device__ __forceinline__ bool any_row_flagged(const Dev& dv, uint32_t mask)
{
    int mine = 0;
    for (int r = threadIdx.x; r < dv.n; r += blockDim.x) mine |= (dv.row_flags[r] & mask) != 0u;
    return __syncthreads_or(mine) != 0;
}

// level 0 counts the first digit (top 11 bits) of every key; level 1 serves rows flagged
// kRowRefine only and counts the next 11 bits of the keys whose first digit is the one row_lo
// holds.  With `rescue` only rows flagged kRowRescue are served.  Whenever rows are picked by
// flag the grid is one-dimensional and its blocks stride over the spans of those rows
// (normally there are none, and every block returns at once).
template <bool VEC>
__global__ void __launch_bounds__(kThreads) hist_kernel(Dev dv, StepArgs a, int rescue, int level)
{
    __shared__ uint32_t h[kHistBins];
    // rows served: those flagged for the rescue (if this is one) and, at level 1, for refinement;
    // with either condition the grid is one-dimensional and strides over the rows that qualify
    const uint32_t need = (rescue ? kRowRescue : 0u) | (level ? kRowRefine : 0u);
    const bool strided = need != 0u;
    if (strided && !any_row_flagged(dv, kRowRefine | kRowRescue)) return;
    const int row_begin = strided ? 0 : (int)blockIdx.y, row_end = strided ? dv.n : (int)blockIdx.y + 1;
    for (int row = row_begin; row < row_end; ++row) {
        if (need && (dv.row_flags[row] & need) != need) continue;
        const uint32_t first = level ? dv.row_lo[row] >> 21 : 0u;
        for (int64_t sp = blockIdx.x; sp < dv.nspans; sp += strided ? (int64_t)gridDim.x : dv.nspans) {
            for (int b = threadIdx.x; b < kHistBins; b += kThreads) h[b] = 0u;
            __syncthreads();
            const int64_t c0 = sp * kSpan;
#pragma unroll
            for (int it = 0; it < kDenseIters; ++it) {
                const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
                if (c < dv.d) {
                    uint32_t bits[4];
                    quad_bits<SEL_TOPK, VEC>(dv, a, row, c, bits);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t key = order_key<SEL_TOPK>(bits[e]);
                        if (c + e >= dv.d) continue;
                        if (!level) atomicAdd(&h[key >> 21], 1u);
                        else if ((key >> 21) == first) atomicAdd(&h[(key >> 10) & (kHistBins - 1)], 1u);
                    }
                }
            }
            __syncthreads();
            uint32_t* g = dv.hist + (int64_t)row * kHistBins;
            for (int b = threadIdx.x; b < kHistBins; b += kThreads)
                if (h[b]) atomicAdd(&g[b], h[b]);
            __syncthreads();
        }
    }
}

// prepare 2: per row, the lowest first digit that must be kept
__global__ void __launch_bounds__(kSelThreads) bound_kernel(Dev dv, int rescue, int level)
{
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[36];
    const int row = blockIdx.x;
    const uint32_t flags = dv.row_flags[row];
    if (rescue && !(flags & kRowRescue)) return;
    if (level && !(flags & kRowRefine)) return;
    uint32_t* g = dv.hist + (int64_t)row * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) {
        h[b] = g[b];
        g[b] = 0u; // ready for the next use
    }
    __syncthreads();
    // keep down to rank 2.5 k (not just k) so that emit can place the next step's bound
    const uint64_t want = 2 * (uint64_t)dv.k + (uint64_t)dv.k / 2;
    const uint32_t rank = (uint32_t)(want < (uint64_t)dv.d ? want : (uint64_t)dv.d);
    // level 1: the keys above the first digit's bin are already counted
    const uint32_t before = level ? dv.row_above[row] : 0u;
    uint32_t digit, above;
    block_find_digit<kSelThreads>(h, kHistBins, rank - before, sm, &digit, &above);
    if (threadIdx.x == 0) {
        // Every coordinate with this digit or a higher one becomes a candidate.  If the digit's
        // own bin makes that more than the capacity, the bins above it alone will do as long as
        // they hold k coordinates.  Otherwise the bin is both needed and too full: after a
        // first digit the next 11 bits are resolved (the keys of a row whose largest entries
        // were just sent crowd under the last threshold); after those the row is left to the
        // exact selection.
        const int64_t upto = (int64_t)before + above; // keys above the bin
        bool full = false;
        if (upto + (int64_t)h[digit] > dv.cap) {
            if (upto >= dv.k && digit + 1u < (uint32_t)kHistBins) digit += 1u;
            else full = true;
        }
        const uint32_t keep = rescue ? kRowRescue : 0u;
        if (!level) {
            dv.row_lo[row] = digit << 21;
            dv.row_above[row] = above;
            dv.row_aim[row] = kAimStart;
            dv.row_count[row] = 0u;
            dv.row_ovf[row] = 0u;
            dv.row_flags[row] = keep | (full ? kRowRefine : 0u);
        } else {
            dv.row_lo[row] = (dv.row_lo[row] & 0xFFE00000u) | (digit << 10);
            dv.row_flags[row] = keep | (full ? kRowExact : 0u);
        }
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
        dv.row_ovf[row] = 0u;
        dv.row_flags[row] = 0u;
    }
}

// ---------------------------------------------------------------------------------------
// prepare 3: collect candidates, ascending inside each tile
// ---------------------------------------------------------------------------------------
// With `rescue`: one-dimensional grid striding over the tiles of the rows flagged kRowRescue.
template <int KIND, bool VEC>
__global__ void __launch_bounds__(kTileThreads) collect_kernel(Dev dv, StepArgs a, int rescue)
{
    __shared__ uint32_t sm[2][kTileThreads / 32 + 1];
    __shared__ uint32_t s_base;
    if (rescue && !any_row_flagged(dv, kRowRescue)) return;
    const int row_begin = rescue ? 0 : (int)blockIdx.y, row_end = rescue ? dv.n : (int)blockIdx.y + 1;
    for (int row = row_begin; row < row_end; ++row) {
        const uint32_t flags = dv.row_flags[row];
        if (rescue && !(flags & kRowRescue)) continue;
        if (flags & kRowExact) continue;
        const uint32_t lo = dv.row_lo[row];
        for (int64_t tile = blockIdx.x; tile < dv.ntiles; tile += rescue ? (int64_t)gridDim.x : dv.ntiles) {
            const int64_t c0 = tile * kTile;
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
                dv.seg_off[(int64_t)row * dv.ntiles + tile] = base;
                dv.seg_cnt[(int64_t)row * dv.ntiles + tile] = total;
                // past the capacity nothing is written; emit sees row_count > cap and gives up
                s_base = ((int64_t)base + total > dv.cap) ? 0xFFFFFFFFu : base;
            }
            __syncthreads();
            const uint32_t base = s_base;
            __syncthreads(); // s_base and sm are written again by the next tile
            if (base == 0xFFFFFFFFu) continue;
            uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cand_pitch + base;
            uint32_t* cv = dv.cand_val + (int64_t)row * dv.cand_pitch + base;
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
    }
}

// ---------------------------------------------------------------------------------------
// emit: exact selection among the candidates of a row, ordered output
// ---------------------------------------------------------------------------------------

// The key of rank `rank` (1 = largest) among key(0..ncand) and how many keys are strictly
// above it.  `key` is any callable p -> uint32_t.  Histogram refinement over the range the
// keys actually span: candidates share their leading bits, so a fixed radix digit would pile
// them into a handful of bins (and serialise the shared-memory atomics); bins spread over
// [min, max] instead, then over the chosen bin, until a bin is one key wide.
// Block-wide minimum and maximum of per-thread values (NT threads); `sm` needs 64 words.
template <int NT>
__device__ __forceinline__ void block_min_max(uint32_t& lo, uint32_t& hi, uint32_t* sm)
{
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    __syncthreads(); // protect sm from the previous use
    if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = lo; sm[32 + (threadIdx.x >> 5)] = hi; }
    __syncthreads();
    for (int w = 0; w < NT / 32; ++w) {
        lo = sm[w] < lo ? sm[w] : lo;
        hi = sm[32 + w] > hi ? sm[32 + w] : hi;
    }
    __syncthreads();
}

constexpr int kListCap = 1024; // a histogram bin this small is resolved by direct comparison

// NT threads; a list of at most min(NT, kListCap) keys is ranked with one key per thread
template <int NT, typename KeyFn>
__device__ __forceinline__ void rank_key(KeyFn key, uint32_t ncand, uint32_t rank, uint32_t lo,
                                         uint32_t hi, uint32_t* h, uint32_t* sm, uint32_t* key_out,
                                         uint32_t* above_out)
{
    // [lo, hi] is the range of the keys (block_min_max)
    uint32_t need = rank, above_total = 0;
    for (;;) {
        const uint32_t width = hi - lo;
        const int shift = width < (uint32_t)kHistBins ? 0 : (32 - __clz(width)) - 11;
        const int nbins = (int)(width >> shift) + 1; // <= kHistBins
        for (int b = threadIdx.x; b < kHistBins; b += NT) h[b] = 0u;
        __syncthreads();
        for (uint32_t p = threadIdx.x; p < ncand; p += NT) {
            const uint32_t kk = key(p);
            if (kk >= lo && kk <= hi) atomicAdd(&h[(kk - lo) >> shift], 1u);
        }
        __syncthreads();
        uint32_t digit, above;
        block_find_digit<NT, kHistBins / NT>(h, nbins, need, sm, &digit, &above);
        const uint32_t inbin = h[digit];
        need -= above;
        above_total += above;
        const uint32_t nlo = lo + (digit << shift);
        const uint32_t span = shift ? ((1u << shift) - 1u) : 0u;
        const uint32_t nhi = (hi - nlo) < span ? hi : nlo + span;
        lo = nlo;
        hi = nhi;
        __syncthreads();
        if (shift == 0) break;
        if (inbin <= (uint32_t)(NT < kListCap ? NT : kListCap)) {
            // few keys left in [lo, hi]: list them (h is free now) and rank them directly
            uint32_t* list = h;          // at most kListCap keys
            uint32_t* count = sm + 40;   // one word
            if (threadIdx.x == 0) { *count = 0u; sm[41] = lo; sm[42] = 0u; }
            __syncthreads();
            for (uint32_t p = threadIdx.x; p < ncand; p += NT) {
                const uint32_t kk = key(p);
                if (kk >= lo && kk <= hi) list[atomicAdd(count, 1u)] = kk;
            }
            __syncthreads();
            const uint32_t m = *count; // == inbin
            if (threadIdx.x < m) {
                const uint32_t mine = list[threadIdx.x];
                uint32_t g = 0, e = 0;
                for (uint32_t q = 0; q < m; ++q) {
                    g += list[q] > mine;
                    e += list[q] == mine;
                }
                if (g < need && need <= g + e) { sm[41] = mine; sm[42] = g; } // same values from every such thread
            }
            __syncthreads();
            lo = sm[41];
            above_total += sm[42];
            __syncthreads();
            break;
        }
    }
    *key_out = lo;
    *above_out = above_total;
}

// Tell every reader of worker `row` where row's message enters each tile (tp[t] .. tp[t+1]),
// in the reader's own CSR position, with the reader's own weight.  Called by all threads of
// the block after tp[] is complete and visible.
// `tid` of `nthreads` threads share the work (all threads of the block by default).
__device__ __forceinline__ void publish_ranges(const Dev& dv, int row, const uint32_t* tp, int tid, int nthreads)
{
    for (int e = dv.row_ptr[row]; e < dv.row_ptr[row + 1]; ++e) {
        const int64_t reader = dv.col[e];
        const int pos = dv.rd_pos[e];
        const uint32_t wbits = __float_as_uint(dv.rd_w[e]);
        uint4* rec = dv.rec + (reader * dv.ntiles) * dv.maxdeg + pos;
        for (int64_t t = tid; t < dv.ntiles; t += nthreads) {
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


// lo: bound the ncand candidates were collected with (their rank-ncand key, roughly);
// T: key of rank k.  The key is read off a line in (log rank, key) through the two points
// (tails fall off roughly like that; a line in the rank itself sits above a convex tail and
// would keep too few), at most half an octave below the old bound.
__device__ __forceinline__ uint32_t next_bound(uint32_t lo, uint32_t T, uint32_t ncand, uint32_t k,
                                               uint32_t aim)
{
    if (ncand <= k || T < lo) return lower_bound_key(lo, 4u);
    const float span = (float)(T - lo);
    const float want = (float)k * (float)aim * (1.0f / 256.0f);
    if (want <= (float)k) return T;
    const float frac = __log2f(want / (float)k) / __log2f((float)ncand / (float)k); // 1 at rank ncand
    const float drop = span * frac;                                                // below T
    if (drop <= span) return T - (uint32_t)drop;
    float dec = drop - span;
    if (dec > (float)(4u << 21)) dec = (float)(4u << 21);
    return lo > (uint32_t)dec ? lo - (uint32_t)dec : 0u;
}

// Exclusive prefix sums, in place, of two arrays of length n (one block, NT threads).
// `carry` is two words of shared memory; totals are returned through tot_a / tot_b.
template <int NT>
__device__ __forceinline__ void block_scan_pair(uint32_t* a, uint32_t* b, int64_t n, uint32_t* sm,
                                                uint32_t* carry, uint32_t* tot_a, uint32_t* tot_b)
{
    if (threadIdx.x == 0) { carry[0] = 0u; carry[1] = 0u; }
    __syncthreads();
    for (int64_t i0 = 0; i0 < n; i0 += NT) {
        const int64_t i = i0 + threadIdx.x;
        const uint32_t va = i < n ? a[i] : 0u, vb = i < n ? b[i] : 0u;
        uint32_t ta, tb;
        const uint32_t ea = block_scan_excl<NT>(va, sm, &ta);
        const uint32_t eb = block_scan_excl<NT>(vb, sm, &tb);
        const uint32_t ca = carry[0], cb = carry[1];
        if (i < n) { a[i] = ca + ea; b[i] = cb + eb; }
        __syncthreads();
        if (threadIdx.x == 0) { carry[0] = ca + ta; carry[1] = cb + tb; }
        __syncthreads();
    }
    *tot_a = carry[0];
    *tot_b = carry[1];
}

// ---------------------------------------------------------------------------------------
// exact: one block selects straight from the dense row (three radix passes and an ordered
// compaction pass).  Slow; only for rows whose candidates could not be used.
// ---------------------------------------------------------------------------------------
template <int KIND, bool VEC, int NT>
__device__ __forceinline__ void exact_row(const Dev& dv, const StepArgs& a, int row, uint32_t* h, uint32_t* sm)
{
    const uint32_t k = (uint32_t)dv.k;
    const int64_t span = (int64_t)NT * kQuad; // coordinates per block iteration
    const int64_t nspan = (dv.d + span - 1) / span;
    uint32_t prefix = 0, pmask = 0, need = k;
    uint32_t aim_lo = 0, aim_count = 0, aim_above = 0;
    bool aim_in_bin = false;
    const uint64_t aim_want = (uint64_t)k * kAimAfterMiss / 256u;
    const uint32_t aim_rank = (uint32_t)(aim_want < (uint64_t)dv.d ? aim_want : (uint64_t)dv.d);
    for (int pass = 0; pass < 3; ++pass) {
        // digits of 11, 11 and 10 bits from the top (plain selects: arrays indexed by the pass would live on a stack)
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const int bins = pass == 2 ? 1024 : 2048;
        for (int b = threadIdx.x; b < kHistBins; b += NT) h[b] = 0u;
        __syncthreads();
        for (int64_t c = (int64_t)threadIdx.x * kQuad; c < dv.d; c += span) {
            uint32_t bits[4];
            quad_bits<KIND, VEC>(dv, a, row, c, bits);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t key = order_key<KIND>(bits[e]);
                if (c + e < dv.d && (key & pmask) == prefix)
                    atomicAdd(&h[(key >> shift) & (bins - 1)], 1u);
            }
        }
        __syncthreads();
        uint32_t digit, above;
        block_find_digit<NT, kHistBins / NT>(h, bins, need, sm, &digit, &above);
        if (KIND == SEL_TOPK && pass == 0) {
            // a second point for the next step's bound: the eighth-of-an-octave bin that holds
            // the rank the bound aims at, and how many keys lie at or above its lower edge
            uint32_t d2, a2;
            block_find_digit<NT, kHistBins / NT>(h, 2048, aim_rank, sm, &d2, &a2);
            aim_lo = d2 << 21;
            aim_count = a2 + h[d2];
            aim_in_bin = d2 == digit; // the same bin as rank k: the next pass resolves it further
            aim_above = above;
        } else if (KIND == SEL_TOPK && pass == 1 && aim_in_bin) {
            uint32_t d2, a2;
            block_find_digit<NT, kHistBins / NT>(h, 2048, aim_rank - aim_above, sm, &d2, &a2);
            aim_lo = prefix | (d2 << 10);
            aim_count = aim_above + a2 + h[d2];
        }
        need -= above;
        prefix |= digit << shift;
        pmask |= (uint32_t)(bins - 1) << shift;
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
        const uint32_t ex = block_scan_excl<NT>(__popc(gtm) | (__popc(eqm) << 16), sm, &tot);
        uint32_t g = run_gt + (ex & 0xFFFFu), q = run_eq + (ex >> 16);
        // the first thread of every tile records how many coordinates were chosen before it
        if (c % kTile == 0) {
            const int64_t t = c / kTile;
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
    publish_ranges(dv, row, tp, threadIdx.x, NT);
    if (threadIdx.x == 0) {
        dv.row_flags[row] = 0u;
        dv.row_count[row] = 0u;
        dv.row_ovf[row] = 0u;
        if (KIND == SEL_TOPK) {
            // between (rank k, key T) and (rank aim_count, key aim_lo), as after a usable step
            dv.row_lo[row] = next_bound(aim_lo, T, aim_count, k, kAimAfterMiss);
            dv.row_aim[row] = kAimAfterMiss;
        }
        atomicAdd(&dv.stats->exact_rows, 1ull);
    }
}

// Layout of the emit kernel's dynamic shared memory, fixed at choco_init from the sizes:
// slab prefix arrays, per-tile arrays and a cache of the candidate keys go to shared memory
// as far as they fit (in that order); what does not fit lives in global scratch.
//
// One block per row.  All passes over the candidates are flat (candidate p = slab * 32 + lane)
// so that their loads are independent of each other:
//   1. keys into shared memory, k-th key T by radix refinement, next bound;
//   2. per tile: number of keys above T and equal to T (atomics); per 32-candidate slab too;
//   3. prefix over tiles -> tile_ptr and the number of equal keys before each tile; prefix
//      over slabs; per tile the two prefixes at its first candidate;
//   4. every chosen candidate computes its own output position and writes itself.
// `rescue`: 0 = a row whose candidates cannot be used is selected exactly by this block;
// 1 = such a row is flagged kRowRescue instead and left to the rescue kernels that follow;
// 2 = this launch is their last stage and serves the flagged rows only.
// One block serves one row.  `dyn` is the block's dynamic shared memory (dv.emit_smem_bytes), `h`
// kHistBins words, `sm` 64 words and `s_carry` 2 words of shared memory.  `contiguous`: the row's
// candidates lie in [0, row_count) of its candidate arrays (false: in per-tile slots, which this
// algorithm does not read; the row is then treated like one whose candidates cannot be used).
template <int KIND, bool VEC, int NT>
__device__ __forceinline__ void emit_row_single(const Dev& dv, const StepArgs& a, int row, int fused, int rescue,
                                                uint32_t* dyn, uint32_t* h, uint32_t* sm, uint32_t* s_carry,
                                                bool contiguous = true)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ncand = dv.row_count[row];
    const uint32_t flags = dv.row_flags[row];
    const uint32_t k = (uint32_t)dv.k;
    __syncthreads();
    if (rescue == 2 && !(flags & kRowRescue)) return;
    if ((flags & kRowExact) || !contiguous || ncand > (uint32_t)dv.cap || ncand < k) { // the candidates cannot be used
        if (rescue == 1 && !(flags & kRowExact)) {
            // a fresh histogram would say the same for a row flagged kRowExact; any other row
            // gets new candidates from the kernels that follow
            if (threadIdx.x == 0) {
                dv.row_flags[row] = kRowRescue;
                atomicAdd(&dv.stats->rescued_rows, 1ull);
            }
            return;
        }
        exact_row<KIND, VEC, NT>(dv, a, row, h, sm);
        return;
    }
    const uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cand_pitch;
    const uint32_t* cv = dv.cand_val + (int64_t)row * dv.cand_pitch;
    const int64_t nslab = ((int64_t)ncand + 31) >> 5;

    // carve the dynamic shared memory (every piece a multiple of 16 bytes)
    uint64_t* bar = reinterpret_cast<uint64_t*>(dyn); // for the bulk copies of the candidates
    uint32_t* cursor = dyn + 4;
    const int64_t tpitch = (dv.ntiles + 3) & ~(int64_t)3;
    uint32_t *slab_g, *slab_e, *slab_gm, *slab_em, *t_gt, *t_eq, *t_sbe;
    if (dv.emit_slabs_smem) { slab_g = cursor; slab_e = cursor + dv.slab_pitch; cursor += 2 * dv.slab_pitch; }
    else { slab_g = dv.slab_a + (int64_t)row * dv.slab_pitch; slab_e = dv.slab_b + (int64_t)row * dv.slab_pitch; }
    if (dv.emit_tiles_smem) { t_gt = cursor; t_eq = cursor + tpitch; t_sbe = cursor + 2 * tpitch; cursor += 3 * tpitch; }
    else { t_gt = dv.tile_a + (int64_t)row * dv.ntiles; t_eq = dv.tile_b + (int64_t)row * dv.ntiles; t_sbe = dv.tile_c + (int64_t)row * dv.ntiles; }
    if (dv.emit_masks_smem) { slab_gm = cursor; slab_em = cursor + dv.slab_pitch; cursor += 2 * dv.slab_pitch; }
    else { slab_gm = dv.slab_c + (int64_t)row * dv.slab_pitch; slab_em = dv.slab_d + (int64_t)row * dv.slab_pitch; }
    uint32_t* sbits = cursor;                      // the candidates' value bits and
    uint32_t* sidx = cursor + dv.emit_keys_cap;    // coordinates, when they fit
    const bool cached = ncand <= (uint32_t)dv.emit_keys_cap;
    if (cached && threadIdx.x == 0) {
        // both arrays in two bulk copies: nothing is staged in registers, and all of it is in
        // flight at once (rows of the candidate arrays are 16-byte aligned, cap % 4 == 0)
        const uint32_t bytes = ((ncand + 3u) & ~3u) * (uint32_t)sizeof(uint32_t);
        mbar_init(bar, 1);
        mbar_expect_tx(bar, 2u * bytes);
        bulk_load(sbits, cv, bytes, bar);
        bulk_load(sidx, ci, bytes, bar);
    }
    // a thread's own tile segment, fetched now so that the wait overlaps the copies
    const uint32_t* so = dv.seg_off + (int64_t)row * dv.ntiles;
    const uint32_t* sc = dv.seg_cnt + (int64_t)row * dv.ntiles;
    const bool own_tile = dv.ntiles <= NT;
    uint32_t my_so = 0u, my_sc = 0u;
    if (own_tile && threadIdx.x < dv.ntiles) { my_so = __ldg(so + threadIdx.x); my_sc = __ldg(sc + threadIdx.x); }
    uint32_t klo = 0xFFFFFFFFu, khi = 0u; // range of the keys
    if (cached) {
        // thread 0 polls (bounded); the others wait at the barrier, then each thread observes
        // the completed phase itself so that the copied data is visible to it
        int ok = 1;
        if (threadIdx.x == 0) ok = mbar_wait_bounded(bar, 0, dv.stats, dv.wait_polls) ? 1 : 0;
        if (!__syncthreads_and(ok)) return; // recorded in the stats: the step's result is invalid
        (void)mbar_wait_bounded(bar, 0, dv.stats, kSpinLimit);
        for (uint32_t p = threadIdx.x; p < ncand; p += NT) {
            const uint32_t kk = order_key<KIND>(sbits[p]);
            klo = kk < klo ? kk : klo;
            khi = kk > khi ? kk : khi;
        }
    } else {
        for (uint32_t p0 = threadIdx.x; p0 < ncand; p0 += 4 * NT) {
            uint32_t bits[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t p = p0 + j * NT;
                if (p < ncand) bits[j] = __ldg(cv + p);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t p = p0 + j * NT;
                if (p < ncand) {
                    const uint32_t kk = order_key<KIND>(bits[j]);
                    klo = kk < klo ? kk : klo;
                    khi = kk > khi ? kk : khi;
                }
            }
        }
    }
    block_min_max<NT>(klo, khi, sm);
    auto bits_at = [&](uint32_t p) -> uint32_t { return cached ? sbits[p] : __ldg(cv + p); };
    auto idx_at = [&](uint32_t p) -> uint32_t { return cached ? sidx[p] : __ldg(ci + p); };
    auto key_at = [&](uint32_t p) -> uint32_t { return order_key<KIND>(bits_at(p)); };

    uint32_t T, above;
    rank_key<NT>(key_at, ncand, k, klo, khi, h, sm, &T, &above);
    const uint32_t r = k - above; // how many coordinates with key == T are kept (lowest first)

    if (KIND == SEL_TOPK) {
        // Candidate bound for the next step: only a guess (the next step verifies that it kept
        // at least k coordinates and otherwise selects exactly from the dense row).  The k
        // chosen coordinates drop to ~0, so aim the bound at today's rank 2.5 k, reading the
        // key of that rank off a straight line through (rank k, T) and (rank ncand, bound).
        if (threadIdx.x == 0) {
            uint32_t aim = dv.row_aim[row];
            aim = aim > kAimMin + kAimStep ? aim - kAimStep : kAimMin;
            dv.row_aim[row] = aim;
            dv.row_lo[row] = next_bound(dv.row_lo[row], T, ncand, k, aim);
        }
    }

    // 2. per slab of 32 candidates: which keys lie above T, which equal it (ballots), how many
    for (int64_t sl = warp; sl < nslab; sl += NT / 32) {
        const uint32_t p = (uint32_t)(sl << 5) + lane;
        bool gt = false, eq = false;
        if (p < ncand) {
            const uint32_t kk = key_at(p);
            gt = kk > T;
            eq = kk == T;
        }
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) { slab_g[sl] = __popc(bg); slab_e[sl] = __popc(be); slab_gm[sl] = bg; slab_em[sl] = be; }
    }
    __syncthreads();

    // 3. prefixes.  Slabs first: with them the number of keys above / equal to T before any
    // candidate position follows from one prefix and one ballot ...
    uint32_t tot_g, tot_e;
    block_scan_pair<NT>(slab_g, slab_e, nslab, sm, s_carry, &tot_g, &tot_e);
    auto before = [&](uint32_t pos, uint32_t& g, uint32_t& e) {
        const uint32_t s0 = pos >> 5;
        if ((int64_t)s0 < nslab) {
            const uint32_t below = (1u << (pos & 31u)) - 1u;
            g = slab_g[s0] + __popc(slab_gm[s0] & below);
            e = slab_e[s0] + __popc(slab_em[s0] & below);
        } else {
            g = tot_g;
            e = tot_e;
        }
    };
    // ... so a tile, whose candidates are consecutive, gets its two counts as differences
    for (int64_t t = threadIdx.x; t < dv.ntiles; t += NT) {
        const uint32_t cnt = own_tile ? my_sc : sc[t];
        uint32_t g0 = 0, e0 = 0, g1 = 0, e1 = 0;
        if (cnt) {
            const uint32_t first = own_tile ? my_so : so[t];
            before(first, g0, e0);
            before(first + cnt, g1, e1);
        }
        t_gt[t] = g1 - g0;
        t_eq[t] = e1 - e0;
    }
    __syncthreads();
    // tiles: t_gt <- keys above T before the tile, t_eq <- equal keys before it
    uint32_t tot_a, tot_b;
    block_scan_pair<NT>(t_gt, t_eq, dv.ntiles, sm, s_carry, &tot_a, &tot_b);
    uint32_t* tp = dv.tile_ptr + (int64_t)row * (dv.ntiles + 1);
    for (int64_t t = threadIdx.x; t < dv.ntiles; t += NT) {
        const uint32_t gb = t_gt[t], eb = t_eq[t];
        tp[t] = gb + (eb < r ? eb : r);
        // the two flat prefixes at the tile's first candidate: t_gt <- above, t_sbe <- equal
        uint32_t pg = 0, pe = 0;
        if (own_tile ? my_sc : sc[t]) before(own_tile ? my_so : so[t], pg, pe);
        t_gt[t] = pg;
        t_sbe[t] = pe;
    }
    if (threadIdx.x == 0) tp[dv.ntiles] = k;
    __syncthreads();
    // 4. every chosen candidate writes itself
    uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch;
    float* mv = dv.msg_val + (int64_t)row * dv.kpitch;
    const float* xr = a.X + (int64_t)row * dv.ld;
    const float* hr = a.Xhat + (int64_t)row * dv.ld;
    const uint32_t lt = (1u << lane) - 1u;
    // (which candidates those are is in the slabs' ballots: only they are fetched again)
    // Some of the warps do that while the others publish the range records (both are bound by
    // the latency of their scattered stores); the split follows the two amounts of work, one
    // slab per warp iteration here, 32 records per warp iteration there.
    const int nwarps = NT / 32;
    const int64_t pub_iters = (dv.ntiles * (dv.row_ptr[row + 1] - dv.row_ptr[row]) + 31) / 32;
    int kWriteWarps = (int)((nslab * nwarps + (nslab + pub_iters) / 2) / (nslab + pub_iters));
    kWriteWarps = kWriteWarps < 1 ? 1 : (kWriteWarps > nwarps - 1 ? nwarps - 1 : kWriteWarps);
    for (int64_t sl = warp; warp < kWriteWarps && sl < nslab; sl += kWriteWarps) {
        const uint32_t bg = slab_gm[sl], be = slab_em[sl];
        const bool gt = (bg >> lane) & 1u, eq = (be >> lane) & 1u;
        if (gt | eq) {
            const uint32_t p = (uint32_t)(sl << 5) + lane;
            const uint32_t id = idx_at(p);
            const uint32_t tile = id / kTile;
            const uint32_t g_in = slab_g[sl] + __popc(bg & lt) - t_gt[tile];  // above T, earlier in the tile
            const uint32_t e_in = slab_e[sl] + __popc(be & lt) - t_sbe[tile]; // equal to T, earlier in the tile
            const uint32_t eqb = t_eq[tile];                                  // equal to T, in earlier tiles
            const uint32_t room = r > eqb ? r - eqb : 0u;                     // equal keys this tile may keep
            if (gt || e_in < room) {
                const uint32_t pos = tp[tile] + g_in + (e_in < room ? e_in : room);
                mi[pos] = id;
                mv[pos] = KIND == SEL_TOPK ? __uint_as_float(bits_at(p)) : __fsub_rn(xr[id], hr[id]);
            }
        }
    }
    if (warp >= kWriteWarps) publish_ranges(dv, row, tp, threadIdx.x - kWriteWarps * 32, NT - kWriteWarps * 32);
    __syncthreads();
    if (threadIdx.x == 0) {
        dv.row_count[row] = 0u;
        dv.row_ovf[row] = 0u;
        dv.row_flags[row] = 0u;
        atomicAdd(fused ? &dv.stats->prepared_rows : &dv.stats->recompressed_rows, 1ull);
    }
}

template <int KIND, bool VEC, int NT>
__global__ void __launch_bounds__(NT) emit_kernel(Dev dv, StepArgs a, int fused, int rescue)
{
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[64];
    __shared__ uint32_t s_carry[2];
    wait_for_previous_kernel(); // the candidates come from the kernel before this one
    allow_next_kernel();
    emit_row_single<KIND, VEC, NT>(dv, a, (int)blockIdx.x, fused, rescue, dyn, h, sm, s_carry);
}

// several layers in one launch: block b serves row b % n of the table's entry b / n (top-k, one
// block per row; rows may start at any element, so the exact selection reads them element by element)
template <int NT>
__global__ void __launch_bounds__(NT)
emit_layers_kernel(const __grid_constant__ LayerTable tab, LayerSet ls, StepArgs a, int n)
{
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t sm[64];
    __shared__ uint32_t s_carry[2];
    __shared__ Dev sdev;
    const int en = (int)(blockIdx.x / (unsigned)n), row = (int)(blockIdx.x % (unsigned)n);
    load_layer_params(ls.devs + tab.layer[en], &sdev); // (set up by the host: not the previous kernel's output)
    shift_arrays(a, tab.off[en]);
    wait_for_previous_kernel(); // the candidates come from the kernel before this one
    allow_next_kernel();
    emit_row_single<SEL_TOPK, false, NT>(sdev, a, row, 1, 0, dyn, h, sm, s_carry);
}

// ---------------------------------------------------------------------------------------
// emit, several blocks per row: a thread-block cluster serves one row.
//
// The candidates of a row lie in the candidate arrays tile by tile, ascending inside a tile,
// but the tiles in the order in which their blocks of the update kernel happened to reserve
// space.  Here the tiles are cut into one run per block of the cluster, of about equal
// candidate counts, and every block gathers its run into shared memory IN TILE ORDER.  The
// concatenation of the blocks' arrays is then the row's candidate list in ascending coordinate
// order, and the message is simply its ordered compaction:
//   1. k-th key T: histogram refinement as in the one-block kernel, each block counting its own
//      keys and all blocks adding the counts up through distributed shared memory;
//   2. per 32-candidate slab the ballots of "above T" / "equal to T", prefix sums inside the
//      block, the blocks' totals exchanged: every candidate then knows how many chosen ones
//      precede it in the whole row and writes itself;
//   3. tile_ptr and the range records follow from the same prefixes at each tile's first candidate.
// Every decision that steers the control flow (usable or not, number of refinement rounds) is
// taken from values all blocks of the cluster hold alike, so they reach every cluster barrier
// together.  A row whose candidates cannot be used, or whose share per block does not fit the
// shared memory, is left to block 0, which runs the one-block algorithm above.
// ---------------------------------------------------------------------------------------
namespace cg = cooperative_groups;

constexpr int kMaxCluster = 4;
constexpr int kGroup = 8; // lanes that copy one tile's candidates

// words of dynamic shared memory the cluster algorithm needs for `cap_local` candidates per block
__host__ __device__ inline int64_t cluster_emit_words(int64_t cap_local)
{
    const int64_t spitch = ((cap_local >> 5) + 2 + 3) & ~(int64_t)3;
    return 2 * cap_local + 4 * spitch + 3 * (kSelThreads + 4) + 2 * kListCap;
}
// the same with the keys and coordinates of the block's `len` candidates in global memory
__host__ __device__ inline int64_t cluster_spill_words(int64_t len)
{
    const int64_t spitch = ((len >> 5) + 2 + 3) & ~(int64_t)3;
    return 4 * spitch + 3 * (kSelThreads + 4) + 2 * kListCap;
}

template <int KIND, bool VEC>
__global__ void __launch_bounds__(kSelThreads) emit_cluster_kernel(Dev dv, StepArgs a, int fused, int rescue, uint32_t dyn_bytes)
{
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ uint32_t h2[2][kHistBins]; // this block's histogram of the current / the previous round
    __shared__ uint32_t hsum[kHistBins];  // the cluster's
    __shared__ uint32_t sm[64];
    __shared__ uint32_t s_carry[2];
    __shared__ uint32_t xch[8];           // what this block shows the others: key range, counts
    __shared__ uint32_t part_t[kMaxCluster + 1], part_p[kMaxCluster + 1]; // first tile / candidate of each block's run
    wait_for_previous_kernel(); // the candidates come from the kernel before this one
    allow_next_kernel();
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t C = cluster.num_blocks(), rank = cluster.block_rank();
    const int row = (int)(blockIdx.x / C);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ncand = dv.row_count[row], flags = dv.row_flags[row], k = (uint32_t)dv.k;
    if (rescue == 2 && !(flags & kRowRescue)) return;
    const bool unusable = (flags & kRowExact) || ncand > (uint32_t)dv.cap || ncand < k;
    const uint32_t* so = dv.seg_off + (int64_t)row * dv.ntiles;
    const uint32_t* sc = dv.seg_cnt + (int64_t)row * dv.ntiles;
    const uint32_t ntiles = (uint32_t)dv.ntiles;

    // the runs: tile t goes to block floor(candidates before t * C / ncand)
    if (threadIdx.x <= C) {
        part_t[threadIdx.x] = threadIdx.x == 0 ? 0u : ntiles;
        part_p[threadIdx.x] = threadIdx.x == 0 ? 0u : ncand;
    }
    __syncthreads();
    if (!unusable) {
        uint32_t carry = 0;
        for (uint32_t t0 = 0; t0 < ntiles; t0 += kSelThreads) {
            const uint32_t t = t0 + threadIdx.x;
            const uint32_t cnt = t < ntiles ? sc[t] : 0u;
            uint32_t tot;
            const uint32_t ex = carry + block_scan_excl<kSelThreads>(cnt, sm, &tot);
            if (t < ntiles) {
                const uint32_t top = C - 1u;
                uint32_t mine = (uint32_t)(((uint64_t)ex * C) / ncand);
                mine = mine < top ? mine : top;
                int prev = -1;
                if (t > 0) {
                    const uint32_t pv = (uint32_t)(((uint64_t)(ex - sc[t - 1]) * C) / ncand);
                    prev = (int)(pv < top ? pv : top);
                }
                for (uint32_t c = 1; c < C; ++c)
                    if (mine >= c && prev < (int)c) { part_t[c] = t; part_p[c] = ex; }
            }
            carry += tot;
        }
        __syncthreads();
        if (threadIdx.x == 0 && carry != ncand) part_p[1] = 0xFFFFFFFFu; // inconsistent counts: do not trust the runs
        __syncthreads();
    }
    // A block keeps its run's keys and coordinates in shared memory if every block's run fits
    // there; otherwise in the row's part of two global arrays, as long as the per-slab arrays of
    // the longest run still fit (the same algorithm either way).
    const int64_t cap_local = dv.emit_cap_local;
    bool fits = !unusable;
    uint32_t longest = 0;
    for (uint32_t c = 0; c < C && fits; ++c) {
        fits = part_p[c + 1] >= part_p[c];
        const uint32_t len = part_p[c + 1] - part_p[c];
        longest = len > longest ? len : longest;
    }
    const bool in_smem = fits && (int64_t)longest <= cap_local;
    if (fits && !in_smem)
        fits = dv.spill_key != nullptr && cluster_spill_words((int64_t)longest) * 4 <= (int64_t)dyn_bytes;
    // Every block has now read the row's state; none has changed it yet.  Only behind this
    // barrier may block 0 go its own way (it rewrites the row's flags and counts), so that all
    // blocks reach the same verdict from the same values.
    cluster.sync();
    if (!fits) { // block 0 serves the row alone, with the one-block algorithm
        // (candidates the update kernel left in per-tile slots are not contiguous; those of the
        // collection kernel, fused == 0, are)
        if (rank == 0)
            emit_row_single<KIND, VEC, kSelThreads>(dv, a, row, fused, rescue, dyn, h2[0], sm, s_carry,
                                                    !(fused && dv.cand_slot != 0u));
        return;
    }

    // carve the dynamic shared memory
    const int64_t spitch = (((in_smem ? cap_local : (int64_t)longest) >> 5) + 2 + 3) & ~(int64_t)3;
    const int64_t spill_at = (int64_t)row * dv.cand_pitch + part_p[rank];
    uint32_t* keys = in_smem ? dyn : dv.spill_key + spill_at;             // value bits of this block's candidates, in tile order
    uint32_t* idxs = in_smem ? keys + cap_local : dv.spill_idx + spill_at; // their coordinates
    uint32_t* slab_g = in_smem ? idxs + cap_local : dyn;                   // per slab: keys above T (then: before the slab)
    uint32_t* slab_e = slab_g + spitch;         //           keys equal to T
    uint32_t* slab_gm = slab_e + spitch;        //           ballots of the two
    uint32_t* slab_em = slab_gm + spitch;
    uint32_t* st_a = slab_em + spitch;          // per tile of the pass: first candidate in the arrays / output position
    uint32_t* st_b = st_a + (kSelThreads + 4);  //                        candidates
    uint32_t* st_c = st_b + (kSelThreads + 4);  //                        first candidate in this block's order
    uint32_t* list_mine = st_c + (kSelThreads + 4);
    uint32_t* list_all = list_mine + kListCap;

    const uint32_t Tb = part_t[rank], Te = part_t[rank + 1];
    const uint32_t L = part_p[rank + 1] - part_p[rank];   // this block's candidates
    const uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cand_pitch;
    const uint32_t* cv = dv.cand_val + (int64_t)row * dv.cand_pitch;

    // gather: a group of kGroup lanes copies one tile's candidates
    uint32_t klo = 0xFFFFFFFFu, khi = 0u;
    {
        uint32_t carry = 0;
        for (uint32_t t0 = Tb; t0 < Te; t0 += kSelThreads) {
            const uint32_t t = t0 + threadIdx.x;
            const uint32_t cnt = t < Te ? sc[t] : 0u;
            uint32_t tot;
            const uint32_t ex = carry + block_scan_excl<kSelThreads>(cnt, sm, &tot);
            st_a[threadIdx.x] = t < Te ? so[t] : 0u;
            st_b[threadIdx.x] = cnt;
            st_c[threadIdx.x] = ex;
            __syncthreads();
            const uint32_t nt = (Te - t0) < (uint32_t)kSelThreads ? (Te - t0) : (uint32_t)kSelThreads;
            for (uint32_t i = threadIdx.x / kGroup; i < nt; i += kSelThreads / kGroup) {
                const uint32_t g = st_a[i], c = st_b[i], l = st_c[i];
                for (uint32_t j = threadIdx.x % kGroup; j < c; j += kGroup) {
                    const uint32_t bits = __ldg(cv + g + j);
                    keys[l + j] = bits;
                    idxs[l + j] = __ldg(ci + g + j);
                    const uint32_t kk = order_key<KIND>(bits);
                    klo = kk < klo ? kk : klo;
                    khi = kk > khi ? kk : khi;
                }
            }
            carry += tot;
            __syncthreads(); // the staging arrays are written again by the next pass
        }
    }
    block_min_max<kSelThreads>(klo, khi, sm);
    if (threadIdx.x == 0) { xch[0] = klo; xch[1] = khi; }
    cluster.sync();
    for (uint32_t c = 0; c < C; ++c) {
        const uint32_t* o = cluster.map_shared_rank(xch, c);
        const uint32_t a0 = o[0], a1 = o[1];
        klo = a0 < klo ? a0 : klo;
        khi = a1 > khi ? a1 : khi;
    }
    auto key_at = [&](uint32_t p) -> uint32_t { return order_key<KIND>(keys[p]); };

    // 1. the k-th key: refinement over the range the keys span, counts added up over the cluster
    uint32_t T, above_total = 0;
    {
        uint32_t need = k, lo = klo, hi = khi;
        int buf = 0;
        for (;;) {
            const uint32_t width = hi - lo;
            const int shift = width < (uint32_t)kHistBins ? 0 : (32 - __clz(width)) - 11;
            const int nbins = (int)(width >> shift) + 1; // <= kHistBins
            uint32_t* h = h2[buf];
            for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0u;
            __syncthreads();
            for (uint32_t p = threadIdx.x; p < L; p += kSelThreads) {
                const uint32_t kk = key_at(p);
                if (kk >= lo && kk <= hi) atomicAdd(&h[(kk - lo) >> shift], 1u);
            }
            cluster.sync(); // every block's counts of this round are complete
            for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) {
                uint32_t v = 0;
                for (uint32_t c = 0; c < C; ++c) v += cluster.map_shared_rank(&h2[buf][0], c)[b];
                hsum[b] = v;
            }
            __syncthreads();
            uint32_t digit, above;
            block_find_digit<kSelThreads>(hsum, nbins, need, sm, &digit, &above);
            const uint32_t inbin = hsum[digit];
            need -= above;
            above_total += above;
            const uint32_t nlo = lo + (digit << shift);
            const uint32_t span = shift ? ((1u << shift) - 1u) : 0u;
            const uint32_t nhi = (hi - nlo) < span ? hi : nlo + span;
            lo = nlo;
            hi = nhi;
            __syncthreads();
            if (shift == 0) break;
            if (inbin <= (uint32_t)kListCap) {
                // few keys left in [lo, hi]: every block lists its own, all read all lists and rank directly
                uint32_t* count = sm + 40;
                if (threadIdx.x == 0) { *count = 0u; sm[41] = lo; sm[42] = 0u; }
                __syncthreads();
                for (uint32_t p = threadIdx.x; p < L; p += kSelThreads) {
                    const uint32_t kk = key_at(p);
                    if (kk >= lo && kk <= hi) list_mine[atomicAdd(count, 1u)] = kk;
                }
                __syncthreads();
                if (threadIdx.x == 0) xch[2] = *count;
                cluster.sync();
                uint32_t m = 0;
                for (uint32_t c = 0; c < C; ++c) {
                    const uint32_t mc = cluster.map_shared_rank(xch, c)[2];
                    const uint32_t* src = cluster.map_shared_rank(list_mine, c);
                    if (m + mc <= (uint32_t)kListCap)
                        for (uint32_t q = threadIdx.x; q < mc; q += kSelThreads) list_all[m + q] = src[q];
                    m += mc;
                }
                m = m < (uint32_t)kListCap ? m : (uint32_t)kListCap; // == inbin
                __syncthreads();
                if (threadIdx.x < m) {
                    const uint32_t mine = list_all[threadIdx.x];
                    uint32_t g = 0, e = 0;
                    for (uint32_t q = 0; q < m; ++q) {
                        g += list_all[q] > mine;
                        e += list_all[q] == mine;
                    }
                    if (g < need && need <= g + e) { sm[41] = mine; sm[42] = g; } // same values from every such thread
                }
                __syncthreads();
                lo = sm[41];
                above_total += sm[42];
                __syncthreads();
                break;
            }
            buf ^= 1;
        }
        T = lo;
    }
    const uint32_t r = k - above_total; // how many coordinates with key == T are kept (lowest first)

    if (KIND == SEL_TOPK && rank == 0 && threadIdx.x == 0) {
        // candidate bound for the next step (see the one-block kernel)
        uint32_t aim = dv.row_aim[row];
        aim = aim > kAimMin + kAimStep ? aim - kAimStep : kAimMin;
        dv.row_aim[row] = aim;
        dv.row_lo[row] = next_bound(dv.row_lo[row], T, ncand, k, aim);
    }

    // 2. ballots per slab of 32 candidates, prefixes inside the block, totals over the cluster
    const int64_t nslab = ((int64_t)L + 31) >> 5;
    for (int64_t sl = warp; sl < nslab; sl += kSelThreads / 32) {
        const uint32_t p = (uint32_t)(sl << 5) + lane;
        bool gt = false, eq = false;
        if (p < L) {
            const uint32_t kk = key_at(p);
            gt = kk > T;
            eq = kk == T;
        }
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) { slab_g[sl] = __popc(bg); slab_e[sl] = __popc(be); slab_gm[sl] = bg; slab_em[sl] = be; }
    }
    __syncthreads();
    uint32_t tot_g, tot_e;
    block_scan_pair<kSelThreads>(slab_g, slab_e, nslab, sm, s_carry, &tot_g, &tot_e);
    if (threadIdx.x == 0) { xch[4] = tot_g; xch[5] = tot_e; }
    cluster.sync();
    uint32_t og = 0, oe = 0; // keys above / equal to T in the blocks before this one
    for (uint32_t c = 0; c < rank; ++c) {
        const uint32_t* o = cluster.map_shared_rank(xch, c);
        og += o[4];
        oe += o[5];
    }
    // output position of the candidate at position `pos` of this block (pos == L: of the next block's first)
    auto out_pos = [&](uint32_t pos) -> uint32_t {
        uint32_t g = tot_g, e = tot_e;
        const uint32_t s0 = pos >> 5;
        if ((int64_t)s0 < nslab) {
            const uint32_t below = (1u << (pos & 31u)) - 1u;
            g = slab_g[s0] + __popc(slab_gm[s0] & below);
            e = slab_e[s0] + __popc(slab_em[s0] & below);
        }
        e += oe;
        return og + g + (e < r ? e : r);
    };
    // every chosen candidate writes itself
    uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch;
    float* mv = dv.msg_val + (int64_t)row * dv.kpitch;
    const float* xr = a.X + (int64_t)row * dv.ld;
    const float* hr = a.Xhat + (int64_t)row * dv.ld;
    const uint32_t lt = (1u << lane) - 1u;
    for (int64_t sl = warp; sl < nslab; sl += kSelThreads / 32) {
        const uint32_t bg = slab_gm[sl], be = slab_em[sl];
        const bool gt = (bg >> lane) & 1u, eq = (be >> lane) & 1u;
        if (gt | eq) {
            const uint32_t p = (uint32_t)(sl << 5) + lane;
            const uint32_t e_before = oe + slab_e[sl] + __popc(be & lt);
            if (gt || e_before < r) {
                const uint32_t pos = og + slab_g[sl] + __popc(bg & lt) + (e_before < r ? e_before : r);
                const uint32_t id = idxs[p];
                mi[pos] = id;
                mv[pos] = KIND == SEL_TOPK ? __uint_as_float(keys[p]) : __fsub_rn(xr[id], hr[id]);
            }
        }
    }
    // 3. tile_ptr and the range records of this block's tiles
    uint32_t* tp = dv.tile_ptr + (int64_t)row * (dv.ntiles + 1);
    {
        const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
        uint32_t carry = 0;
        for (uint32_t t0 = Tb; t0 < Te; t0 += kSelThreads) {
            const uint32_t t = t0 + threadIdx.x;
            const uint32_t cnt = t < Te ? sc[t] : 0u;
            uint32_t tot;
            const uint32_t ex = carry + block_scan_excl<kSelThreads>(cnt, sm, &tot);
            // (a tile past the pass reads the position behind the pass's last candidate)
            st_a[threadIdx.x] = out_pos(ex);
            if (threadIdx.x == 0) st_a[kSelThreads] = out_pos(carry + tot);
            __syncthreads();
            if (t < Te) {
                const uint32_t first = st_a[threadIdx.x], count = st_a[threadIdx.x + 1] - first;
                tp[t] = first;
                for (int e = e0; e < e1; ++e) {
                    const int64_t reader = dv.col[e];
                    dv.rec[(reader * dv.ntiles + t) * dv.maxdeg + dv.rd_pos[e]] =
                        make_uint4((uint32_t)row, first, count, __float_as_uint(dv.rd_w[e]));
                }
            }
            carry += tot;
            __syncthreads();
        }
    }
    if (rank == C - 1 && threadIdx.x == 0) tp[dv.ntiles] = k;
    // no block may leave while another still reads its shared memory
    cluster.sync();
    if (rank == 0 && threadIdx.x == 0) {
        dv.row_count[row] = 0u;
        dv.row_ovf[row] = 0u;
        dv.row_flags[row] = 0u;
        atomicAdd(fused ? &dv.stats->prepared_rows : &dv.stats->recompressed_rows, 1ull);
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
        for (int level = 0; level < 2; ++level) { // the second round returns at once unless a bin was too full
            const dim3 g = level ? dim3((unsigned)(dv.nspans < 1024 ? dv.nspans : 1024)) : hgrid;
            if (a.vec) hist_kernel<true><<<g, kThreads, 0, st>>>(dv, a, 0, level);
            else hist_kernel<false><<<g, kThreads, 0, st>>>(dv, a, 0, level);
            bound_kernel<<<dv.n, kSelThreads, 0, st>>>(dv, 0, level);
        }
        *a.launches += 4;
    } else {
        // keep words <= hi: about k + 6 sqrt(k) + 16 of d coordinates
        const double kk = (double)dv.k;
        double frac = (kk + 6.0 * sqrt(kk) + 16.0) / (double)dv.d;
        uint32_t hi = frac >= 1.0 ? 0xFFFFFFFFu : (uint32_t)(frac * 4294967296.0);
        randk_bound_kernel<<<(dv.n + 127) / 128, 128, 0, st>>>(dv, ~hi);
        *a.launches += 1;
    }
    if (a.vec) collect_kernel<KIND, true><<<grid, kTileThreads, 0, st>>>(dv, a, 0);
    else collect_kernel<KIND, false><<<grid, kTileThreads, 0, st>>>(dv, a, 0);
    *a.launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_prepare(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? prepare_impl<SEL_TOPK>(dv, a, st)
                                   : prepare_impl<SEL_RANDK>(dv, a, st);
}

template <int KIND>
static cudaError_t emit_impl(const Dev& dv, const StepArgs& a, bool fused, int rescue, cudaStream_t st)
{
    const int vec = a.vec ? 1 : 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dv.emit_cluster > 1) {
        // several blocks per row (a thread-block cluster); shared memory for either algorithm
        auto kern = a.vec ? emit_cluster_kernel<KIND, true> : emit_cluster_kernel<KIND, false>;
        const size_t bytes = std::max<size_t>((size_t)dv.emit_smem_bytes, (size_t)cluster_emit_words(dv.emit_cap_local) * 4);
        static size_t configured[64][2] = {};
        if (dev < 0 || dev >= 64 || configured[dev][vec] < bytes) {
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) configured[dev][vec] = bytes;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)dv.n * (unsigned)dv.emit_cluster);
        cfg.blockDim = dim3(kSelThreads);
        cfg.dynamicSmemBytes = bytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[3];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)dv.emit_cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
        const HotRange hot = hot_range_of(dv);
        if (hot.base && hot.bytes > 0 && hot.ratio > 0.f) {
            attr[2].id = cudaLaunchAttributeAccessPolicyWindow;
            attr[2].val.accessPolicyWindow.base_ptr = hot.base;
            attr[2].val.accessPolicyWindow.num_bytes = hot.bytes;
            attr[2].val.accessPolicyWindow.hitRatio = hot.ratio;
            attr[2].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
            attr[2].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
            cfg.numAttrs = 3;
        }
        cfg.attrs = attr;
        e = cudaLaunchKernelEx(&cfg, kern, dv, a, fused ? 1 : 0, rescue, (uint32_t)bytes);
        if (e != cudaSuccess) return e;
        *a.launches += 1;
        return cudaGetLastError();
    }
    // short rows: small blocks, several per SM (the kernel is a chain of short phases either way)
    const int small = dv.d <= kSmallRow ? 1 : 0;
    auto kern = small ? (a.vec ? emit_kernel<KIND, true, kSelThreadsSmall> : emit_kernel<KIND, false, kSelThreadsSmall>)
                      : (a.vec ? emit_kernel<KIND, true, kSelThreads> : emit_kernel<KIND, false, kSelThreads>);
    static bool configured[64][2][2] = {};
    if (dev < 0 || dev >= 64 || !configured[dev][vec][small]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEmitSmemBudget);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev][vec][small] = true;
    }
    e = launch_overlapped(kern, dim3((unsigned)dv.n), dim3(small ? kSelThreadsSmall : kSelThreads),
                          (size_t)dv.emit_smem_bytes, st, hot_range_of(dv), dv, a, fused ? 1 : 0, rescue);
    if (e != cudaSuccess) return e;
    *a.launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_emit_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, size_t smem_bytes, bool small,
                                      const StepArgs& a, cudaStream_t st)
{
    static size_t configured[64][2] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    auto kern = small ? emit_layers_kernel<kSelThreadsSmall> : emit_layers_kernel<kSelThreads>;
    if (dev < 0 || dev >= 64 || configured[dev][small ? 1 : 0] < smem_bytes) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev][small ? 1 : 0] = smem_bytes;
    }
    return launch_overlapped(kern, dim3((unsigned)(tab.entries * n)), dim3(small ? kSelThreadsSmall : kSelThreads), smem_bytes,
                             st, HotRange{nullptr, 0, 0.f}, tab, ls, a, (int)n);
}

cudaError_t launch_select_emit(const Dev& dv, const StepArgs& a, bool fused, cudaStream_t st)
{
    return dv.kind == CHOCO_Q_TOPK ? emit_impl<SEL_TOPK>(dv, a, fused, dv.rescue ? 1 : 0, st)
                                   : emit_impl<SEL_RANDK>(dv, a, fused, 0, st);
}

cudaError_t launch_select_rescue(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    // enough blocks to fill the device when a row does need them; they return at once otherwise
    static int sms[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int nsm = (dev >= 0 && dev < 64) ? sms[dev] : 0;
    if (nsm == 0) {
        e = cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) sms[dev] = nsm;
    }
    const unsigned hblocks = (unsigned)(dv.nspans < 8 * (int64_t)nsm ? dv.nspans : 8 * (int64_t)nsm);
    const unsigned cblocks = (unsigned)(dv.ntiles < 8 * (int64_t)nsm ? dv.ntiles : 8 * (int64_t)nsm);
    for (int level = 0; level < 2; ++level) {
        if (a.vec) hist_kernel<true><<<hblocks, kThreads, 0, st>>>(dv, a, 1, level);
        else hist_kernel<false><<<hblocks, kThreads, 0, st>>>(dv, a, 1, level);
        bound_kernel<<<dv.n, kSelThreads, 0, st>>>(dv, 1, level);
    }
    if (a.vec) collect_kernel<SEL_TOPK, true><<<cblocks, kTileThreads, 0, st>>>(dv, a, 1);
    else collect_kernel<SEL_TOPK, false><<<cblocks, kTileThreads, 0, st>>>(dv, a, 1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *a.launches += 5;
    return emit_impl<SEL_TOPK>(dv, a, false, 2, st);
}

} // namespace choco
