// The update half of a CHOCO step (Algorithm 1, lines 6, 2 and 9; Algorithm 2 for the
// momentum variant): every worker reads its neighbours' messages back and forms
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i).
// One block owns one tile (kTile coordinates) of one row.
#include "select.cuh"

namespace choco {

struct Upd {
    float eta, gamma, lambda, beta;
};

// x' from the updated s and x^ of one coordinate
template <bool HAS_G, bool HAS_M>
__device__ __forceinline__ float next_x(float x, float sn, float hn, float g, float& m, const Upd& u)
{
    const float cons = __fsub_rn(sn, hn);
    float xn = x;
    if (HAS_M) {
        m = __fadd_rn(__fadd_rn(g, __fmul_rn(u.lambda, x)), __fmul_rn(u.beta, m));
        xn = __fsub_rn(x, __fmul_rn(u.eta, m));
    } else if (HAS_G) {
        xn = __fsub_rn(x, __fmul_rn(u.eta, g));
    }
    return __fadd_rn(xn, __fmul_rn(u.gamma, cons));
}

// ---------------------------------------------------------------------------------------
// dense Q: decode each neighbour's message on the fly
// ---------------------------------------------------------------------------------------
template <int KIND>
__device__ __forceinline__ float4 decode_quad(const Dev& dv, int j, int64_t c)
{
    if (KIND == CHOCO_Q_IDENTITY)
        return __ldg(reinterpret_cast<const float4*>(dv.msg_dense + (int64_t)j * dv.dpitch + c));
    const uint32_t word = __ldg(dv.msg_bits + (int64_t)j * dv.wpitch + (c >> 5));
    const uint32_t nib = (word >> (c & 31)) & 0xFu;
    float m[4];
    if (KIND == CHOCO_Q_SIGN) {
        const float sc = __ldg(dv.msg_scale + j);
        m[0] = m[1] = m[2] = m[3] = sc;
    } else {
        const int64_t b = dv.bucket > 0 ? c / dv.bucket : 0;
        const float nu = __ldg(dv.msg_norms + (int64_t)j * dv.npitch + b);
        const bool tail = dv.bucket > 0 && b == dv.nbuckets - 1 && (dv.d % dv.bucket) != 0;
        const float scale = __fdiv_rn(nu, __fmul_rn(tail ? dv.tau_tail : dv.tau_full, (float)dv.s));
        const uint8_t* lrow = dv.msg_levels + (int64_t)j * dv.lpitch;
        uint32_t packed, width = (uint32_t)dv.wbits;
        if (width == 8) packed = __ldg(reinterpret_cast<const uint32_t*>(lrow + c));
        else if (width == 4) packed = __ldg(reinterpret_cast<const uint16_t*>(lrow + (c >> 1)));
        else if (width == 2) packed = __ldg(lrow + (c >> 2));
        else packed = (__ldg(lrow + (c >> 3)) >> (c & 7)) & 0xFu;
        const uint32_t mask = (1u << width) - 1u;
#pragma unroll
        for (int e = 0; e < 4; ++e) m[e] = __fmul_rn(scale, (float)((packed >> (e * width)) & mask));
    }
    return make_float4(nib & 1u ? -m[0] : m[0], nib & 2u ? -m[1] : m[1], nib & 4u ? -m[2] : m[2],
                       nib & 8u ? -m[3] : m[3]);
}

template <bool VEC, int KIND, bool HAS_G, bool HAS_M>
__global__ void __launch_bounds__(kThreads) apply_dense_kernel(Dev dv, StepArgs a)
{
    const int row = blockIdx.y;
    const int64_t c0 = (int64_t)blockIdx.x * kTile;
    const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta};
    float* xr = a.X + (int64_t)row * dv.ld;
    float* hr = a.Xhat + (int64_t)row * dv.ld;
    float* sr = a.S + (int64_t)row * dv.ld;
    const float* gr = HAS_G ? a.G + (int64_t)row * dv.ld : nullptr;
    float* mr = HAS_M ? a.M + (int64_t)row * dv.ld : nullptr;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        if (c >= dv.d) continue;
        const float4 x = load_quad<VEC>(xr, c, dv.d);
        const float4 h = load_quad<VEC>(hr, c, dv.d);
        const float4 s = load_quad<VEC>(sr, c, dv.d);
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
        if (HAS_G) g = load_quad_stream<VEC>(gr, c, dv.d);
        if (HAS_M) m = load_quad<VEC>(mr, c, dv.d);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), qs = acc;
        for (int e = e0; e < e1; ++e) {
            const int j = dv.col[e];
            const float w = dv.wval[e];
            const float4 q = decode_quad<KIND>(dv, j, c);
            acc.x = __fadd_rn(acc.x, __fmul_rn(w, q.x));
            acc.y = __fadd_rn(acc.y, __fmul_rn(w, q.y));
            acc.z = __fadd_rn(acc.z, __fmul_rn(w, q.z));
            acc.w = __fadd_rn(acc.w, __fmul_rn(w, q.w));
            if (j == row) qs = q;
        }
        const float4 hn = make_float4(__fadd_rn(h.x, qs.x), __fadd_rn(h.y, qs.y),
                                      __fadd_rn(h.z, qs.z), __fadd_rn(h.w, qs.w));
        const float4 sn = make_float4(__fadd_rn(s.x, acc.x), __fadd_rn(s.y, acc.y),
                                      __fadd_rn(s.z, acc.z), __fadd_rn(s.w, acc.w));
        float4 xn;
        xn.x = next_x<HAS_G, HAS_M>(x.x, sn.x, hn.x, g.x, m.x, u);
        xn.y = next_x<HAS_G, HAS_M>(x.y, sn.y, hn.y, g.y, m.y, u);
        xn.z = next_x<HAS_G, HAS_M>(x.z, sn.z, hn.z, g.z, m.z, u);
        xn.w = next_x<HAS_G, HAS_M>(x.w, sn.w, hn.w, g.w, m.w, u);
        store_quad<VEC>(hr, c, dv.d, hn);
        store_quad<VEC>(sr, c, dv.d, sn);
        store_quad<VEC>(xr, c, dv.d, xn);
        if (HAS_M) store_quad<VEC>(mr, c, dv.d, m);
    }
}

// ---------------------------------------------------------------------------------------
// sparse Q, register-staged variant (any alignment, any d): the neighbours' (index, value)
// lists are scattered into a shared-memory tile, one neighbour after the other so that the
// additions happen in CSR order, then the tile is streamed against x, x^, s and g.  x^ and s
// are written only where a message touched them.
// ---------------------------------------------------------------------------------------
template <bool VEC, bool HAS_G, bool HAS_M>
__global__ void __launch_bounds__(kThreads) apply_sparse_kernel(Dev dv, StepArgs a)
{
    __shared__ __align__(16) float acc[kTile];
    __shared__ __align__(16) float qself[kTile];
    __shared__ uint32_t touched[kTile / 32];
    __shared__ uint32_t tself[kTile / 32];
    const int row = blockIdx.y;
    const int64_t tile = blockIdx.x;
    const int64_t c0 = tile * kTile;
    const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta};
    float* xr = a.X + (int64_t)row * dv.ld;
    float* hr = a.Xhat + (int64_t)row * dv.ld;
    float* sr = a.S + (int64_t)row * dv.ld;
    const float* gr = HAS_G ? a.G + (int64_t)row * dv.ld : nullptr;
    float* mr = HAS_M ? a.M + (int64_t)row * dv.ld : nullptr;

    // start the dense loads before touching the messages
    float4 x[kIters], h[kIters], s[kIters], g[kIters];
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        x[it] = load_quad_stream<VEC>(xr, c, dv.d);
        h[it] = load_quad_stream<VEC>(hr, c, dv.d);
        s[it] = load_quad_stream<VEC>(sr, c, dv.d);
        if (HAS_G) g[it] = load_quad_stream<VEC>(gr, c, dv.d);
        else g[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        reinterpret_cast<float4*>(acc)[it * kThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
        reinterpret_cast<float4*>(qself)[it * kThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (threadIdx.x < kTile / 32) { touched[threadIdx.x] = 0u; tself[threadIdx.x] = 0u; }
    __syncthreads();
    for (int e = e0; e < e1; ++e) {
        const int j = dv.col[e];
        const float w = dv.wval[e];
        const uint32_t* tp = dv.tile_ptr + (int64_t)j * (dv.ntiles + 1) + tile;
        const uint32_t lo = __ldg(tp), hi = __ldg(tp + 1);
        const uint32_t* mi = dv.msg_idx + (int64_t)j * dv.kpitch;
        const float* mv = dv.msg_val + (int64_t)j * dv.kpitch;
        for (uint32_t p = lo + threadIdx.x; p < hi; p += kThreads) {
            const uint32_t lc = __ldg(mi + p) - (uint32_t)c0;
            const float val = __ldg(mv + p);
            acc[lc] = __fadd_rn(acc[lc], __fmul_rn(w, val));
            atomicOr(&touched[lc >> 5], 1u << (lc & 31));
            if (j == row) {
                qself[lc] = val;
                atomicOr(&tself[lc >> 5], 1u << (lc & 31));
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int li = (it * kThreads + threadIdx.x) * kQuad;
        const int64_t c = c0 + li;
        if (c >= dv.d) continue;
        const float4 av = reinterpret_cast<const float4*>(acc)[it * kThreads + threadIdx.x];
        const float4 qv = reinterpret_cast<const float4*>(qself)[it * kThreads + threadIdx.x];
        const uint32_t tb = (touched[li >> 5] >> (li & 31)) & 0xFu;
        const uint32_t sb = (tself[li >> 5] >> (li & 31)) & 0xFu;
        float4 m = make_float4(0.f, 0.f, 0.f, 0.f);
        if (HAS_M) m = load_quad<VEC>(mr, c, dv.d);
        const float xs[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
        const float hs[4] = {h[it].x, h[it].y, h[it].z, h[it].w};
        const float ss[4] = {s[it].x, s[it].y, s[it].z, s[it].w};
        const float gs[4] = {g[it].x, g[it].y, g[it].z, g[it].w};
        const float as[4] = {av.x, av.y, av.z, av.w};
        const float qq[4] = {qv.x, qv.y, qv.z, qv.w};
        float ms[4] = {m.x, m.y, m.z, m.w};
        float xn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float hn = (sb >> e) & 1u ? __fadd_rn(hs[e], qq[e]) : hs[e];
            const float sn = (tb >> e) & 1u ? __fadd_rn(ss[e], as[e]) : ss[e];
            xn[e] = next_x<HAS_G, HAS_M>(xs[e], sn, hn, gs[e], ms[e], u);
            if (c + e < dv.d) {
                if ((sb >> e) & 1u) hr[c + e] = hn;
                if ((tb >> e) & 1u) sr[c + e] = sn;
            }
        }
        store_quad<VEC>(xr, c, dv.d, make_float4(xn[0], xn[1], xn[2], xn[3]));
        if (HAS_M) store_quad<VEC>(mr, c, dv.d, make_float4(ms[0], ms[1], ms[2], ms[3]));
    }
}

// ---------------------------------------------------------------------------------------
// sparse Q, bulk-copy variant (rows 16-byte aligned, d a multiple of 4).  The x, x^, s, g
// (and momentum) tiles are fetched into shared memory by asynchronous bulk copies that
// complete on an mbarrier, so no registers are tied up while they are in flight and the
// neighbour scatter overlaps them.  With EMIT the kernel also collects the candidates of the
// next step's top-k selection from x' - x^', which it holds anyway.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
// global -> this block's shared memory; both addresses 16-byte aligned, bytes % 16 == 0
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Wait for phase `parity` with a bound: after kSpinLimit polls the wait is recorded as timed
// out; the copies in flight are then given a second bounded grace period so that the block
// does not retire under them.  Returns false on a timeout.
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, Stats* stats)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    if ((threadIdx.x & 31) == 0) atomicAdd(&stats->timeouts, 1ull);
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) break;
        __nanosleep(256);
    }
    return false;
}

constexpr int kMaxNb = 64; // neighbours handled per batch
constexpr int kMaxE = 2;   // message entries a thread holds per batch

struct NbrTable {
    uint32_t lo[kMaxNb];       // first entry of neighbour r's message inside this tile
    uint32_t len[kMaxNb];      // number of such entries
    uint32_t pref[kMaxNb + 1]; // exclusive prefix of len
    int j[kMaxNb];             // the neighbour's row
    float w[kMaxNb];           // w_ij
    uint32_t self[2];          // this row's own range
};

template <bool HAS_G, bool HAS_M>
__host__ __device__ constexpr int bulk_arrays() { return 3 + (HAS_G ? 1 : 0) + (HAS_M ? 1 : 0); }

template <bool HAS_G, bool HAS_M>
constexpr size_t bulk_smem_bytes()
{
    return (size_t)(bulk_arrays<HAS_G, HAS_M>() + 1) * kTile * sizeof(float) // tiles + acc
           + 2 * (kTile / 32) * sizeof(uint32_t)                              // touched, self
           + 2 * 9 * sizeof(uint32_t) + 16                                    // scan scratch, barrier, base
           + sizeof(NbrTable);
}

template <bool HAS_G, bool HAS_M, bool EMIT>
__global__ void __launch_bounds__(kThreads) update_sparse_bulk_kernel(Dev dv, StepArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* hs = xs + kTile;
    float* ss = hs + kTile;
    float* gs = ss + kTile;                             // used when HAS_G
    float* ms = gs + (HAS_G ? kTile : 0);               // used when HAS_M
    float* acc = ms + (HAS_M ? kTile : 0);
    uint32_t* touched = reinterpret_cast<uint32_t*>(acc + kTile);
    uint32_t* tself = touched + kTile / 32;
    uint32_t(*scan)[9] = reinterpret_cast<uint32_t(*)[9]>(tself + kTile / 32);
    uint64_t* bar = reinterpret_cast<uint64_t*>(reinterpret_cast<uint32_t*>(scan) + 18);
    uint32_t* s_base = reinterpret_cast<uint32_t*>(bar + 1);
    NbrTable* nbr = reinterpret_cast<NbrTable*>(s_base + 2);

    const int row = blockIdx.y;
    const int64_t tile = blockIdx.x;
    const int64_t c0 = tile * kTile;
    const int nvalid = (int)((dv.d - c0) < kTile ? (dv.d - c0) : kTile); // multiple of 4
    const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta};
    float* xr = a.X + (int64_t)row * dv.ld + c0;
    float* hr = a.Xhat + (int64_t)row * dv.ld + c0;
    float* sr = a.S + (int64_t)row * dv.ld + c0;

    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t bytes = (uint32_t)nvalid * sizeof(float);
        mbar_expect_tx(bar, bytes * bulk_arrays<HAS_G, HAS_M>());
        bulk_load(xs, xr, bytes, bar);
        bulk_load(hs, hr, bytes, bar);
        bulk_load(ss, sr, bytes, bar);
        if (HAS_G) bulk_load(gs, a.G + (int64_t)row * dv.ld + c0, bytes, bar);
        if (HAS_M) bulk_load(ms, a.M + (int64_t)row * dv.ld + c0, bytes, bar);
    }
#pragma unroll
    for (int it = 0; it < kIters; ++it)
        reinterpret_cast<float4*>(acc)[it * kThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (threadIdx.x < kTile / 32) { touched[threadIdx.x] = 0u; tself[threadIdx.x] = 0u; }
    __syncthreads();

    // neighbours in CSR order: acc += w * q_j on the coordinates j's message lists in this tile
    // Up to kMaxNb neighbours at a time: first every neighbour's range in this tile (one
    // round trip), then all their entries at once (a second one), then the additions,
    // neighbour by neighbour, out of registers.
    for (int eb = e0; eb < e1; eb += kMaxNb) {
        const int nb = (e1 - eb) < kMaxNb ? (e1 - eb) : kMaxNb;
        if (threadIdx.x < nb) {
            const int j = dv.col[eb + threadIdx.x];
            const uint32_t* tp = dv.tile_ptr + (int64_t)j * (dv.ntiles + 1) + tile;
            const uint32_t lo = __ldg(tp), hi = __ldg(tp + 1);
            nbr->lo[threadIdx.x] = lo;
            nbr->len[threadIdx.x] = hi - lo;
            nbr->j[threadIdx.x] = j;
            nbr->w[threadIdx.x] = dv.wval[eb + threadIdx.x];
            if (j == row) { nbr->self[0] = lo; nbr->self[1] = hi; }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (int r = 0; r < nb; ++r) { nbr->pref[r] = run; run += nbr->len[r]; }
            nbr->pref[nb] = run;
        }
        __syncthreads();
        const uint32_t total = nbr->pref[nb];
        for (uint32_t f0 = 0; f0 < total; f0 += kThreads * kMaxE) {
            int er[kMaxE];
            uint32_t elc[kMaxE];
            float ev[kMaxE];
#pragma unroll
            for (int q = 0; q < kMaxE; ++q) {
                const uint32_t f = f0 + q * kThreads + threadIdx.x;
                er[q] = -1;
                if (f < total) {
                    int r = 0;
                    while (nbr->pref[r + 1] <= f) ++r;
                    const uint32_t p = nbr->lo[r] + (f - nbr->pref[r]);
                    const int64_t mrow = (int64_t)nbr->j[r] * dv.kpitch;
                    er[q] = r;
                    elc[q] = __ldg(dv.msg_idx + mrow + p) - (uint32_t)c0;
                    ev[q] = __fmul_rn(nbr->w[r], __ldg(dv.msg_val + mrow + p));
                }
            }
            // neighbours present in this batch of entries: [r_first, r_last]
            int r_first = 0;
            while (nbr->pref[r_first + 1] <= f0) ++r_first;
            const uint32_t f_last = (f0 + kThreads * kMaxE < total ? f0 + kThreads * kMaxE : total) - 1;
            int r_last = r_first;
            while (nbr->pref[r_last + 1] <= f_last) ++r_last;
            for (int r = r_first; r <= r_last; ++r) {
                if (nbr->len[r] == 0) continue;
#pragma unroll
                for (int q = 0; q < kMaxE; ++q)
                    if (er[q] == r) {
                        acc[elc[q]] = __fadd_rn(acc[elc[q]], ev[q]);
                        atomicOr(&touched[elc[q] >> 5], 1u << (elc[q] & 31));
                    }
                __syncthreads();
            }
        }
        __syncthreads(); // the neighbour table is reused by the next batch
    }
    const uint32_t self_lo = nbr->self[0], self_hi = nbr->self[1];

    // every thread polls (so that each sees the copied data); the verdict is made uniform
    const int arrived = __syncthreads_and(mbar_wait_bounded(bar, 0, dv.stats) ? 1 : 0);
    if (!arrived) return; // recorded in the stats: the step's result is invalid

    // x^ += q_i in place on the staged tile
    {
        const uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch;
        const float* mv = dv.msg_val + (int64_t)row * dv.kpitch;
        for (uint32_t p = self_lo + threadIdx.x; p < self_hi; p += kThreads) {
            const uint32_t lc = __ldg(mi + p) - (uint32_t)c0;
            hs[lc] = __fadd_rn(hs[lc], __ldg(mv + p));
            atomicOr(&tself[lc >> 5], 1u << (lc & 31));
        }
    }
    __syncthreads();

    const uint32_t lo_key = EMIT ? dv.row_lo[row] : 0u;
    uint32_t take = 0, cnt[kIters];
    uint32_t vbits[kIters][4];
    float* mrow = HAS_M ? a.M + (int64_t)row * dv.ld + c0 : nullptr;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int li = (it * kThreads + threadIdx.x) * kQuad;
        cnt[it] = 0;
        if (li >= nvalid) continue;
        const int q4 = it * kThreads + threadIdx.x;
        const float4 x = reinterpret_cast<const float4*>(xs)[q4];
        const float4 h = reinterpret_cast<const float4*>(hs)[q4];
        const float4 s = reinterpret_cast<const float4*>(ss)[q4];
        const float4 av = reinterpret_cast<const float4*>(acc)[q4];
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
        if (HAS_G) g = reinterpret_cast<const float4*>(gs)[q4];
        if (HAS_M) m = reinterpret_cast<const float4*>(ms)[q4];
        const uint32_t tb = (touched[li >> 5] >> (li & 31)) & 0xFu;
        const uint32_t sb = (tself[li >> 5] >> (li & 31)) & 0xFu;
        const float xv[4] = {x.x, x.y, x.z, x.w};
        const float hv[4] = {h.x, h.y, h.z, h.w};
        const float sv[4] = {s.x, s.y, s.z, s.w};
        const float gv[4] = {g.x, g.y, g.z, g.w};
        const float avv[4] = {av.x, av.y, av.z, av.w};
        float mv4[4] = {m.x, m.y, m.z, m.w};
        float xn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float sn = (tb >> e) & 1u ? __fadd_rn(sv[e], avv[e]) : sv[e];
            xn[e] = next_x<HAS_G, HAS_M>(xv[e], sn, hv[e], gv[e], mv4[e], u);
            if ((sb >> e) & 1u) hr[li + e] = hv[e];
            if ((tb >> e) & 1u) sr[li + e] = sn;
            if (EMIT) {
                vbits[it][e] = __float_as_uint(__fsub_rn(xn[e], hv[e]));
                if (order_key<SEL_TOPK>(vbits[it][e]) >= lo_key) {
                    take |= 1u << (4 * it + e);
                    ++cnt[it];
                }
            }
        }
        *reinterpret_cast<float4*>(xr + li) = make_float4(xn[0], xn[1], xn[2], xn[3]);
        if (HAS_M) *reinterpret_cast<float4*>(mrow + li) = make_float4(mv4[0], mv4[1], mv4[2], mv4[3]);
    }

    if (EMIT) {
        uint32_t start[kIters], total;
        ordered_starts(cnt, scan, start, &total);
        if (threadIdx.x == 0) {
            const uint32_t base = total ? atomicAdd(&dv.row_count[row], total) : 0u;
            dv.seg_off[(int64_t)row * dv.ntiles + tile] = base;
            dv.seg_cnt[(int64_t)row * dv.ntiles + tile] = total;
            *s_base = ((int64_t)base + total > dv.cap) ? 0xFFFFFFFFu : base;
        }
        __syncthreads();
        const uint32_t base = *s_base;
        if (base == 0xFFFFFFFFu) return;
        uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cap + base;
        uint32_t* cv = dv.cand_val + (int64_t)row * dv.cap + base;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const uint32_t cbase = (uint32_t)c0 + (uint32_t)(it * kThreads + threadIdx.x) * kQuad;
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

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------

template <bool HAS_G, bool HAS_M, bool EMIT>
static cudaError_t launch_bulk(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    constexpr size_t smem = bulk_smem_bytes<HAS_G, HAS_M>();
    if (smem > 48 * 1024) { // per device, so it is not cached in a process-wide flag
        cudaError_t e = cudaFuncSetAttribute(update_sparse_bulk_kernel<HAS_G, HAS_M, EMIT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const dim3 grid((unsigned)dv.ntiles, (unsigned)dv.n);
    update_sparse_bulk_kernel<HAS_G, HAS_M, EMIT><<<grid, kThreads, smem, st>>>(dv, a);
    return cudaSuccess;
}

template <bool VEC, bool HAS_G, bool HAS_M>
static cudaError_t apply_pick(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    const dim3 grid((unsigned)dv.ntiles, (unsigned)dv.n);
    switch (dv.kind) {
    case CHOCO_Q_TOPK:
    case CHOCO_Q_RANDK:
        if (VEC && dv.d % 4 == 0) {
            if (emit) return launch_bulk<HAS_G, HAS_M, true>(dv, a, st);
            return launch_bulk<HAS_G, HAS_M, false>(dv, a, st);
        }
        apply_sparse_kernel<VEC, HAS_G, HAS_M><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    case CHOCO_Q_SIGN:
        apply_dense_kernel<VEC, CHOCO_Q_SIGN, HAS_G, HAS_M><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    case CHOCO_Q_QSGD:
        apply_dense_kernel<VEC, CHOCO_Q_QSGD, HAS_G, HAS_M><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    default:
        apply_dense_kernel<VEC, CHOCO_Q_IDENTITY, HAS_G, HAS_M><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    }
    return cudaSuccess;
}

template <bool VEC>
static cudaError_t apply_vec(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    if (a.M) return apply_pick<VEC, true, true>(dv, a, emit, st);
    if (a.G) return apply_pick<VEC, true, false>(dv, a, emit, st);
    return apply_pick<VEC, false, false>(dv, a, emit, st);
}

bool apply_can_emit(const Dev& dv, const StepArgs& a)
{
    return dv.kind == CHOCO_Q_TOPK && a.vec && dv.d % 4 == 0;
}

cudaError_t launch_apply(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    const cudaError_t e = a.vec ? apply_vec<true>(dv, a, emit, st) : apply_vec<false>(dv, a, emit, st);
    *a.launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

} // namespace choco
