// Update kernel for sparse Q (top_a / random_a), bulk-copy variant: Algorithm 1, the update of
// the public copies, the gossip step and the gradient step (Algorithm 2 with momentum) for one
// tile of one worker per block,
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i).
//
// The x, x^, s, g (and momentum) tiles are fetched into shared memory by asynchronous bulk
// copies that complete on an mbarrier, so no registers are tied up while they are in flight.
// A bulk copy needs 16-byte aligned addresses and sizes.  With AL (rows 16-byte aligned, d a
// multiple of 4) a tile is copied as it is; otherwise each copy starts at the 16-byte
// boundary at or below the tile's first element and ends at the one at or above its last
// (never touching a 16-byte unit that holds no element of the tile), and the tile is read
// from shared memory at the resulting offset of 0..3 elements.  Meanwhile the block reads
// the range records of its neighbours (one round trip), then all their entries that fall
// into the tile (a second one), and adds them into a shared accumulator tile: with atomic adds
// where a coordinate has one or two terms (the order cannot matter there), in CSR order where it
// has more.  With EMIT the kernel also collects the candidates of the next step's top-k
// selection from x' - x^', which it holds anyway.
#include "bulk.cuh"
#include "select.cuh"

namespace choco {

namespace {

struct Upd {
    float eta, gamma, lambda, beta;
    int nesterov; // the step goes along (g + lambda x) + beta m' instead of the new memory m'
};

template <bool HAS_G, bool HAS_M>
__device__ __forceinline__ float next_x(float x, float sn, float hn, float g, float& m, const Upd& u)
{
    const float cons = __fsub_rn(sn, hn);
    float xn = x;
    if (HAS_M) {
        const float gl = __fadd_rn(g, __fmul_rn(u.lambda, x));
        m = __fadd_rn(gl, __fmul_rn(u.beta, m));
        const float dir = u.nesterov ? __fadd_rn(gl, __fmul_rn(u.beta, m)) : m;
        xn = __fsub_rn(x, __fmul_rn(u.eta, dir));
    } else if (HAS_G) {
        xn = __fsub_rn(x, __fmul_rn(u.eta, g));
    }
    return __fadd_rn(xn, __fmul_rn(u.gamma, cons));
}

constexpr int NT = kTileThreads;
constexpr int NIT = kTileIters;
constexpr int kMaxNb = 32; // neighbours handled per batch (one lane each)
constexpr int kMaxE = 3;   // message entries a thread holds per pass

struct NbrTable {
    uint32_t lo[kMaxNb];       // first entry of neighbour r's message inside this tile
    uint32_t len[kMaxNb];      // number of such entries
    uint32_t pref[kMaxNb + 1]; // exclusive prefix of len
    uint32_t j[kMaxNb];        // the neighbour's row
    float w[kMaxNb];           // w_ij
    uint32_t self;             // position of this worker in the batch, or kMaxNb
    uint32_t pad;
};

template <bool HAS_G, bool HAS_M>
__host__ __device__ constexpr int bulk_arrays() { return 3 + (HAS_G ? 1 : 0) + (HAS_M ? 1 : 0); }

constexpr int kShiftPad = 4; // floats of slack per staged tile when it may start mid-unit

template <bool HAS_G, bool HAS_M, bool AL>
constexpr size_t bulk_smem_bytes()
{
    return (size_t)(bulk_arrays<HAS_G, HAS_M>() + 1) * kTile * sizeof(float) // tiles + acc
           + (AL ? 0 : bulk_arrays<HAS_G, HAS_M>() * kShiftPad * sizeof(float))
           + 4 * (kTile / 32) * sizeof(uint32_t)                              // touched (once, twice, more), self
           + 8                                                                // barrier
           + 2 * (NT / 32 + 1) * sizeof(uint32_t) + 8                         // scan scratch, base
           + sizeof(NbrTable);
}

// *p += v on shared memory, atomically: an IEEE single-precision add rounded to nearest that keeps
// subnormals (atomic float adds on shared memory do; those on global memory flush them to zero)
__device__ __forceinline__ void shared_add(float* p, float v)
{
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"(smem_u32(p)), "f"(v) : "memory");
}

// element offset of p inside its 16-byte unit
__device__ __forceinline__ uint32_t unit_shift(const float* p) { return (uint32_t)(((uintptr_t)p & 15u) >> 2); }

// tile: the block's tile of the row; row: the worker; d, ld: dv.d and dv.ld.  With LAYERS `dv` is
// the block's shared-memory copy of its layer's parameters, still to be filled from `dv_src`: the
// tiles are requested first (that needs d, ld and the array pointers only), the copy is made
// while they fly.
template <bool HAS_G, bool HAS_M, bool EMIT, bool AL, bool LAYERS>
__device__ __forceinline__ void update_sparse_bulk_body(const Dev& dv, const StepArgs& a, int64_t tile, int row, int64_t d,
                                                        int64_t ld, unsigned char* smem_raw, const Dev* dv_src)
{
    static_assert(NT >= kTile / 32 && NT >= kMaxNb, "one thread per mask word / neighbour");
    constexpr int kStage = kTile + (AL ? 0 : kShiftPad);
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* hs = xs + kStage;
    float* ss = hs + kStage;
    float* gs = ss + kStage;                            // used when HAS_G
    float* ms = gs + (HAS_G ? kStage : 0);              // used when HAS_M
    float* acc = ms + (HAS_M ? kStage : 0);
    uint32_t* touched = reinterpret_cast<uint32_t*>(acc + kTile);
    uint32_t* tself = touched + kTile / 32;
    uint32_t* twice = tself + kTile / 32;  // coordinates with entries of two neighbours ...
    uint32_t* more = twice + kTile / 32;   // ... of three or more
    uint64_t* bar = reinterpret_cast<uint64_t*>(more + kTile / 32);
    uint32_t(*scan)[NT / 32 + 1] = reinterpret_cast<uint32_t(*)[NT / 32 + 1]>(bar + 1);
    uint32_t* s_base = reinterpret_cast<uint32_t*>(scan) + 2 * (NT / 32 + 1);
    NbrTable* nbr = reinterpret_cast<NbrTable*>(s_base + 2);

    const int64_t c0 = tile * kTile;
    const int nvalid = (int)((d - c0) < kTile ? (d - c0) : kTile); // AL: a multiple of 4
    const int lane = threadIdx.x & 31;
    float* xr = a.X + (int64_t)row * ld + c0;
    float* hr = a.Xhat + (int64_t)row * ld + c0;
    float* sr = a.S + (int64_t)row * ld + c0;

    const float* gr = HAS_G ? a.G + (int64_t)row * ld + c0 : nullptr;
    float* mrow = HAS_M ? a.M + (int64_t)row * ld + c0 : nullptr;
    // where each staged tile's first element sits in its shared-memory buffer
    const uint32_t shx = AL ? 0u : unit_shift(xr), shh = AL ? 0u : unit_shift(hr), shs = AL ? 0u : unit_shift(sr);
    const uint32_t shg = (AL || !HAS_G) ? 0u : unit_shift(gr), shm = (AL || !HAS_M) ? 0u : unit_shift(mrow);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        auto span = [&](uint32_t sh) { return (((uint32_t)nvalid + sh) * (uint32_t)sizeof(float) + 15u) & ~15u; };
        mbar_expect_tx(bar, span(shx) + span(shh) + span(shs) + (HAS_G ? span(shg) : 0u) + (HAS_M ? span(shm) : 0u));
        bulk_load(xs, xr - shx, span(shx), bar);
        bulk_load(hs, hr - shh, span(shh), bar);
        bulk_load(ss, sr - shs, span(shs), bar);
        if (HAS_G) bulk_load(gs, gr - shg, span(shg), bar);
        if (HAS_M) bulk_load(ms, mrow - shm, span(shm), bar);
    }
    hs += shh; // the in-place x^ update below addresses the tile by coordinate
    // every array starts on an 8-byte boundary (rows of even length): pairs instead of elements
    const bool pairs = !AL && !((shx | shh | shs | shg | shm) & 1u);
#pragma unroll
    for (int it = 0; it < NIT; ++it)
        reinterpret_cast<float4*>(acc)[it * NT + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (threadIdx.x < kTile / 32) {
        touched[threadIdx.x] = 0u; tself[threadIdx.x] = 0u; twice[threadIdx.x] = 0u; more[threadIdx.x] = 0u;
    }
    if (LAYERS) load_layer_params(dv_src, const_cast<Dev*>(&dv));
    const uint4* recs = dv.rec + ((int64_t)row * dv.ntiles + tile) * dv.maxdeg;
    // Messages, range records and the candidate bound come from the kernel before this one.
    // The dense arrays requested above do not: the kernel before either ran to completion
    // before this one started, or is the emit kernel, which lets its successor start only
    // after it has itself seen the previous update complete.
    wait_for_previous_kernel();
    allow_next_kernel();
    // The candidate bound (used at the end: fetched early), as the magnitude it stands for:
    // key(v) = bits(|v|) << 1 >= lo  <=>  bits(|v|) >= ceil(lo / 2)  <=>  |v| >= the float with
    // those bits (finite floats order like their bit patterns; bits past infinity admit nothing)
    float lo_mag = 0.f;
    if (EMIT) {
        const uint32_t lo_key = __ldg(dv.row_lo + row);
        const uint32_t half = (lo_key >> 1) + (lo_key & 1u);
        lo_mag = __uint_as_float(half < 0x7F800000u ? half : 0x7F800000u);
    }
    // warp 1 builds the neighbour table of the first batch
    uint4 rc = make_uint4(0u, 0u, 0u, 0u);
    if ((threadIdx.x >> 5) == 1 && lane < dv.maxdeg) rc = __ldg(recs + lane);

    bool self_in_regs = false;  // this worker's own entries are held by threads (er == self)
    uint32_t self_lo = 0, self_len = 0;
    int er[kMaxE];
    uint32_t elc[kMaxE];
    float ev[kMaxE];
#pragma unroll
    for (int q = 0; q < kMaxE; ++q) er[q] = -1;

    for (int eb = 0; eb < dv.maxdeg; eb += kMaxNb) {
        const int nb = (dv.maxdeg - eb) < kMaxNb ? (dv.maxdeg - eb) : kMaxNb;
        if ((threadIdx.x >> 5) == 1) {
            if (eb != 0) {
                rc = make_uint4(0u, 0u, 0u, 0u);
                if (lane < nb) rc = __ldg(recs + eb + lane);
            }
            // inclusive prefix of the lengths over the lanes
            uint32_t inc = rc.z;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += t;
            }
            nbr->lo[lane] = rc.y;
            nbr->len[lane] = rc.z;
            nbr->j[lane] = rc.x;
            nbr->w[lane] = __uint_as_float(rc.w);
            nbr->pref[lane + 1] = inc;
            if (lane == 0) { nbr->pref[0] = 0u; nbr->self = kMaxNb; }
            __syncwarp();
            if (lane < nb && (int)rc.x == row && rc.z != 0u) nbr->self = (uint32_t)lane;
        }
        __syncthreads();
        const uint32_t total = nbr->pref[nb];
        const uint32_t selfr = nbr->self;
        if (selfr < (uint32_t)nb) { self_lo = nbr->lo[selfr]; self_len = nbr->len[selfr]; }
        if (dv.maxdeg <= kMaxNb && total <= (uint32_t)(NT * kMaxE)) {
            // All entries of the tile at once, each thread holding at most kMaxE of them.  The sum
            // over the neighbours starts from +0 and goes in CSR order, but with one or two terms
            // the order does not matter (0 + a is a, or +0 for a = -0; a + b = b + a): those are
            // added with shared-memory atomics (round to nearest, subnormals kept) in whatever
            // order the threads arrive.  Three bit planes count the terms per coordinate; a
            // coordinate with three or more is redone in order below.
            const int nq = (int)((total + NT - 1) / NT);
            float prod[kMaxE];
            bool third = false;
#pragma unroll
            for (int q = 0; q < kMaxE; ++q) {
                er[q] = -1;
                const uint32_t f = q * NT + threadIdx.x;
                if (q < nq && f < total) {
                    int r = 0;
                    while (nbr->pref[r + 1] <= f) ++r;
                    const uint32_t p = nbr->lo[r] + (f - nbr->pref[r]);
                    const int64_t mrow = (int64_t)nbr->j[r] * dv.kpitch;
                    er[q] = r;
                    elc[q] = __ldg(dv.msg_idx + mrow + p) - (uint32_t)c0;
                    ev[q] = __ldg(dv.msg_val + mrow + p);
                    prod[q] = __fmul_rn(nbr->w[r], ev[q]);
                }
            }
#pragma unroll
            for (int q = 0; q < kMaxE; ++q)
                if (er[q] >= 0) {
                    const uint32_t wd = elc[q] >> 5, bit = 1u << (elc[q] & 31);
                    if (atomicOr(&touched[wd], bit) & bit)
                        if (atomicOr(&twice[wd], bit) & bit) { atomicOr(&more[wd], bit); third = true; }
                    shared_add(&acc[elc[q]], prod[q]);
                }
            if (__syncthreads_or(third)) {
                // Some coordinate has three or more terms.  Its terms are ranked by neighbour: the
                // accumulator word serves as the set of neighbours with an entry there (cleared,
                // filled with one bit per neighbour, read back), then the terms are added one rank
                // per round.
                bool redo[kMaxE];
                uint32_t rank[kMaxE];
#pragma unroll
                for (int q = 0; q < kMaxE; ++q) {
                    redo[q] = er[q] >= 0 && ((more[elc[q] >> 5] >> (elc[q] & 31)) & 1u);
                    rank[q] = 0u;
                    if (redo[q]) acc[elc[q]] = 0.f; // (every thread with a term there writes the same)
                }
                __syncthreads();
                uint32_t* accw = reinterpret_cast<uint32_t*>(acc);
#pragma unroll
                for (int q = 0; q < kMaxE; ++q)
                    if (redo[q]) atomicOr(&accw[elc[q]], 1u << er[q]);
                __syncthreads();
#pragma unroll
                for (int q = 0; q < kMaxE; ++q)
                    if (redo[q]) rank[q] = (uint32_t)__popc(accw[elc[q]] & ((1u << er[q]) - 1u));
                __syncthreads();
                for (uint32_t j = 0;; ++j) {
                    bool later = false;
#pragma unroll
                    for (int q = 0; q < kMaxE; ++q)
                        if (redo[q]) {
                            if (rank[q] == j) acc[elc[q]] = __fadd_rn(j == 0u ? 0.f : acc[elc[q]], prod[q]);
                            later = later || rank[q] > j;
                        }
                    if (!__syncthreads_or(later)) break;
                }
            }
            self_in_regs = true; // this worker's own entries are among those the threads hold
        } else
        for (uint32_t f0 = 0; f0 < total; f0 += NT * kMaxE) {
#pragma unroll
            for (int q = 0; q < kMaxE; ++q) {
                const uint32_t f = f0 + q * NT + threadIdx.x;
                er[q] = -1;
                if (f < total) {
                    int r = 0;
                    while (nbr->pref[r + 1] <= f) ++r;
                    const uint32_t p = nbr->lo[r] + (f - nbr->pref[r]);
                    const int64_t mrow = (int64_t)nbr->j[r] * dv.kpitch;
                    er[q] = r;
                    elc[q] = __ldg(dv.msg_idx + mrow + p) - (uint32_t)c0;
                    ev[q] = __ldg(dv.msg_val + mrow + p);
                }
            }
            // neighbours present in this pass: [r_first, r_last]; one round per neighbour
            int r_first = 0;
            while (nbr->pref[r_first + 1] <= f0) ++r_first;
            const uint32_t f_last = (f0 + NT * kMaxE < total ? f0 + NT * kMaxE : total) - 1;
            int r_last = r_first;
            while (nbr->pref[r_last + 1] <= f_last) ++r_last;
            for (int r = r_first; r <= r_last; ++r) {
                if (nbr->len[r] == 0) continue;
                const float wr = nbr->w[r];
#pragma unroll
                for (int q = 0; q < kMaxE; ++q)
                    if (er[q] == r) {
                        acc[elc[q]] = __fadd_rn(acc[elc[q]], __fmul_rn(wr, ev[q]));
                        atomicOr(&touched[elc[q] >> 5], 1u << (elc[q] & 31));
                    }
                __syncthreads();
            }
            self_in_regs = false;
        }
        if (eb + kMaxNb < dv.maxdeg) __syncthreads(); // the table is rebuilt for the next batch
    }

    // thread 0 polls (bounded); the others wait at the barrier, then each thread observes the
    // completed phase itself so that the copied tiles are visible to it
    int ok = 1;
    if (threadIdx.x == 0) ok = mbar_wait_bounded(bar, 0, dv.stats, dv.wait_polls) ? 1 : 0;
    if (!__syncthreads_and(ok)) return; // recorded in the stats: the step's result is invalid
    if (!mbar_wait_bounded(bar, 0, dv.stats, kSpinLimit)) return;

    // x^ += q_i in place on the staged tile
    if (self_in_regs) {
        const int selfr = (int)nbr->self;
#pragma unroll
        for (int q = 0; q < kMaxE; ++q)
            if (er[q] == selfr) {
                hs[elc[q]] = __fadd_rn(hs[elc[q]], ev[q]);
                atomicOr(&tself[elc[q] >> 5], 1u << (elc[q] & 31));
            }
    } else {
        const uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch + self_lo;
        const float* mv = dv.msg_val + (int64_t)row * dv.kpitch + self_lo;
        for (uint32_t p = threadIdx.x; p < self_len; p += NT) {
            const uint32_t lc = __ldg(mi + p) - (uint32_t)c0;
            hs[lc] = __fadd_rn(hs[lc], __ldg(mv + p));
            atomicOr(&tself[lc >> 5], 1u << (lc & 31));
        }
    }
    __syncthreads();

    const Upd u = {a.eta, a.gamma, a.lambda, a.beta, dv.nesterov};
    uint32_t take = 0, cnt[NIT];
    uint32_t vbits[NIT][4];
    // a staged quad: one 128-bit read when the tile sits aligned, else element by element
    auto staged_quad = [&](const float* buf, uint32_t sh, int q4) {
        if (AL) return reinterpret_cast<const float4*>(buf)[q4];
        const float* p = buf + sh + q4 * kQuad;
        if (pairs) { // (elements past the tile's end are read from the buffer's slack and never used)
            const float2 lo2 = reinterpret_cast<const float2*>(p)[0], hi2 = reinterpret_cast<const float2*>(p)[1];
            return make_float4(lo2.x, lo2.y, hi2.x, hi2.y);
        }
        const int left = nvalid - q4 * kQuad;
        return make_float4(p[0], left > 1 ? p[1] : 0.f, left > 2 ? p[2] : 0.f, left > 3 ? p[3] : 0.f);
    };
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int q4 = it * NT + threadIdx.x;
        const int li = q4 * kQuad;
        cnt[it] = 0;
        if (li >= nvalid) continue;
        const float4 x = staged_quad(xs, shx, q4);
        const float4 h = staged_quad(hs, 0u, q4);
        const float4 s = staged_quad(ss, shs, q4);
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
        if (HAS_G) g = staged_quad(gs, shg, q4);
        if (HAS_M) m = staged_quad(ms, shm, q4);
        const uint32_t tb = (touched[li >> 5] >> (li & 31)) & 0xFu;
        const uint32_t sb = (tself[li >> 5] >> (li & 31)) & 0xFu;
        const float xv[4] = {x.x, x.y, x.z, x.w};
        const float hv[4] = {h.x, h.y, h.z, h.w};
        float sv[4] = {s.x, s.y, s.z, s.w};
        const float gv[4] = {g.x, g.y, g.z, g.w};
        float mv4[4] = {m.x, m.y, m.z, m.w};
        float xn[4];
        if (tb | sb) { // some message touched this quad: s and x^ change where flagged
            const float4 av = reinterpret_cast<const float4*>(acc)[q4];
            const float avv[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if ((tb >> e) & 1u) {
                    sv[e] = __fadd_rn(sv[e], avv[e]);
                    sr[li + e] = sv[e];
                }
                if ((sb >> e) & 1u) hr[li + e] = hv[e];
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            xn[e] = next_x<HAS_G, HAS_M>(xv[e], sv[e], hv[e], gv[e], mv4[e], u);
            if (EMIT) {
                vbits[it][e] = __float_as_uint(__fsub_rn(xn[e], hv[e]));
                if ((AL || li + e < nvalid) && fabsf(__uint_as_float(vbits[it][e])) >= lo_mag) {
                    take |= 1u << (4 * it + e);
                    ++cnt[it];
                }
            }
        }
        if (AL) {
            *reinterpret_cast<float4*>(xr + li) = make_float4(xn[0], xn[1], xn[2], xn[3]);
            if (HAS_M) *reinterpret_cast<float4*>(mrow + li) = make_float4(mv4[0], mv4[1], mv4[2], mv4[3]);
        } else if (pairs && li + kQuad <= nvalid) {
            reinterpret_cast<float2*>(xr + li)[0] = make_float2(xn[0], xn[1]);
            reinterpret_cast<float2*>(xr + li)[1] = make_float2(xn[2], xn[3]);
            if (HAS_M) {
                reinterpret_cast<float2*>(mrow + li)[0] = make_float2(mv4[0], mv4[1]);
                reinterpret_cast<float2*>(mrow + li)[1] = make_float2(mv4[2], mv4[3]);
            }
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (li + e < nvalid) {
                    xr[li + e] = xn[e];
                    if (HAS_M) mrow[li + e] = mv4[e];
                }
        }
    }

    if (EMIT) {
        uint32_t start[NIT], total;
        ordered_starts<NT, NIT, true>(cnt, scan, start, &total); // (the scratch has no other use in this kernel)
        uint32_t base;
        if (dv.cand_slot != 0u && total <= dv.cand_slot) {
            // the tile's own slot: nothing to reserve, nothing to wait for (every thread knows
            // `total`); the row's count is kept for the selection kernel by an add without a reader
            base = (uint32_t)tile * dv.cand_slot;
            if (threadIdx.x == 0) {
                if (total) atomicAdd(&dv.row_count[row], total);
                dv.seg_off[(int64_t)row * dv.ntiles + tile] = base;
                dv.seg_cnt[(int64_t)row * dv.ntiles + tile] = total;
            }
        } else {
            if (threadIdx.x == 0) {
                uint32_t b = 0u;
                bool ok = true;
                if (dv.cand_slot != 0u) { // more than a slot holds: room behind the slots
                    b = (uint32_t)dv.ntiles * dv.cand_slot + atomicAdd(&dv.row_ovf[row], total);
                    ok = (int64_t)b + total <= dv.cand_pitch;
                    // (no room left: a count above the capacity tells the selection kernel to give the candidates up)
                    atomicAdd(&dv.row_count[row], ok ? total : (uint32_t)dv.cap + 1u);
                } else {
                    b = total ? atomicAdd(&dv.row_count[row], total) : 0u;
                    ok = (int64_t)b + total <= dv.cap; // past the capacity nothing is written; the count says so
                }
                dv.seg_off[(int64_t)row * dv.ntiles + tile] = b;
                dv.seg_cnt[(int64_t)row * dv.ntiles + tile] = total;
                *s_base = ok ? b : 0xFFFFFFFFu;
            }
            __syncthreads();
            base = *s_base;
        }
        if (base == 0xFFFFFFFFu || take == 0u) return;
        uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cand_pitch + base;
        uint32_t* cv = dv.cand_val + (int64_t)row * dv.cand_pitch + base;
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const uint32_t cbase = (uint32_t)c0 + (uint32_t)(it * NT + threadIdx.x) * kQuad;
            uint32_t p = start[it];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (take & (1u << (4 * it + e))) {
                    ci[p] = cbase + e;
                    cv[p] = vbits[it][e];
                    ++p;
                }
        }
    }
}

template <bool HAS_G, bool HAS_M, bool EMIT, bool AL>
__global__ void __launch_bounds__(NT, 5) update_sparse_bulk_kernel(Dev dv, StepArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    update_sparse_bulk_body<HAS_G, HAS_M, EMIT, AL, false>(dv, a, (int64_t)blockIdx.x, (int)blockIdx.y + a.row0, dv.d, dv.ld, smem_raw,
                                                          nullptr);
}

// several layers in one launch: blockIdx.x picks (layer, tile), blockIdx.y the worker
template <bool HAS_G, bool HAS_M, bool AL>
__global__ void __launch_bounds__(NT, 5)
update_sparse_bulk_layers_kernel(const __grid_constant__ LayerTable tab, LayerSet ls, StepArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ Dev sdev;
    const int en = entry_of_block(tab, blockIdx.x);
    shift_arrays(a, tab.off[en]);
    update_sparse_bulk_body<HAS_G, HAS_M, true, AL, true>(sdev, a, (int64_t)(blockIdx.x - tab.first_block[en]), (int)blockIdx.y,
                                                         (int64_t)tab.d[en], ls.ld, smem_raw, ls.devs + tab.layer[en]);
}

template <bool HAS_G, bool HAS_M, bool AL>
cudaError_t launch_bulk_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, const StepArgs& a, cudaStream_t st)
{
    constexpr size_t smem = bulk_smem_bytes<HAS_G, HAS_M, AL>();
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    auto kern = update_sparse_bulk_layers_kernel<HAS_G, HAS_M, AL>;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    return launch_overlapped(kern, dim3(tab.first_block[tab.entries], (unsigned)n), dim3(NT), smem, st,
                             HotRange{nullptr, 0, 0.f}, tab, ls, a);
}

template <bool AL>
cudaError_t launch_terms_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, const StepArgs& a, cudaStream_t st)
{
    if (a.M) return launch_bulk_layers<true, true, AL>(tab, ls, n, a, st);
    if (a.G) return launch_bulk_layers<true, false, AL>(tab, ls, n, a, st);
    return launch_bulk_layers<false, false, AL>(tab, ls, n, a, st);
}

template <bool HAS_G, bool HAS_M, bool EMIT, bool AL>
cudaError_t launch_bulk(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    constexpr size_t smem = bulk_smem_bytes<HAS_G, HAS_M, AL>();
    // Once per device and instantiation: allow the dynamic shared memory size and ask for the
    // largest shared-memory carve-out, so that as many tiles as possible are in flight per SM.
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        auto kern = update_sparse_bulk_kernel<HAS_G, HAS_M, EMIT, AL>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const dim3 grid((unsigned)dv.ntiles, (unsigned)(a.rows > 0 ? a.rows : dv.n));
    return launch_overlapped(update_sparse_bulk_kernel<HAS_G, HAS_M, EMIT, AL>, grid, dim3(NT), smem, st,
                             hot_range_of(dv), dv, a);
}

template <bool AL>
cudaError_t launch_terms(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    if (a.M) return emit ? launch_bulk<true, true, true, AL>(dv, a, st) : launch_bulk<true, true, false, AL>(dv, a, st);
    if (a.G) return emit ? launch_bulk<true, false, true, AL>(dv, a, st) : launch_bulk<true, false, false, AL>(dv, a, st);
    return emit ? launch_bulk<false, false, true, AL>(dv, a, st) : launch_bulk<false, false, false, AL>(dv, a, st);
}

} // namespace

cudaError_t launch_update_bulk_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, const StepArgs& a, bool aligned,
                                      cudaStream_t st)
{
    return aligned ? launch_terms_layers<true>(tab, ls, n, a, st) : launch_terms_layers<false>(tab, ls, n, a, st);
}

cudaError_t launch_update_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    // a.vec: every row of every array starts on a 16-byte boundary
    return (a.vec && dv.d % 4 == 0) ? launch_terms<true>(dv, a, emit, st) : launch_terms<false>(dv, a, emit, st);
}

} // namespace choco
