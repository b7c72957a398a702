// Update kernel for sparse Q (top_a / random_a), bulk-copy variant: Algorithm 1, lines 6, 2
// and 9 (Algorithm 2 with momentum) for one tile of one worker per block,
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i).
//
// Requirements: rows 16-byte aligned, d a multiple of 4.  The x, x^, s, g (and momentum)
// tiles are fetched into shared memory by asynchronous bulk copies that complete on an
// mbarrier, so no registers are tied up while they are in flight; warp 0 meanwhile gathers the
// neighbours' message entries that fall into the tile and is the only one that polls the
// barrier.  With EMIT the kernel also collects the candidates of the next step's top-k
// selection from x' - x^', which it holds anyway.
#include "select.cuh"

namespace choco {

namespace {

struct Upd {
    float eta, gamma, lambda, beta;
};

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

constexpr int kPrefetch = 6; // neighbours whose first 32 entries are fetched together

template <bool HAS_G, bool HAS_M>
__host__ __device__ constexpr int bulk_arrays() { return 3 + (HAS_G ? 1 : 0) + (HAS_M ? 1 : 0); }

template <int NT, bool HAS_G, bool HAS_M>
constexpr size_t bulk_smem_bytes()
{
    return (size_t)(bulk_arrays<HAS_G, HAS_M>() + 1) * kTile * sizeof(float) // tiles + acc
           + 2 * (kTile / 32) * sizeof(uint32_t)                              // touched, self
           + 8                                                                // barrier
           + 2 * (NT / 32 + 1) * sizeof(uint32_t) + 8;                        // scan scratch, base
}

template <int NT, bool HAS_G, bool HAS_M, bool EMIT>
__global__ void __launch_bounds__(NT, 5) update_sparse_bulk_kernel(Dev dv, StepArgs a)
{
    constexpr int NIT = kTile / (NT * kQuad); // quads per thread
    static_assert(NT >= kTile / 32, "one thread per mask word");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* hs = xs + kTile;
    float* ss = hs + kTile;
    float* gs = ss + kTile;                             // used when HAS_G
    float* ms = gs + (HAS_G ? kTile : 0);               // used when HAS_M
    float* acc = ms + (HAS_M ? kTile : 0);
    uint32_t* touched = reinterpret_cast<uint32_t*>(acc + kTile);
    uint32_t* tself = touched + kTile / 32;
    uint64_t* bar = reinterpret_cast<uint64_t*>(tself + kTile / 32);
    uint32_t(*scan)[NT / 32 + 1] = reinterpret_cast<uint32_t(*)[NT / 32 + 1]>(bar + 1);
    uint32_t* s_base = reinterpret_cast<uint32_t*>(scan) + 2 * (NT / 32 + 1);

    const int row = blockIdx.y;
    const int64_t tile = blockIdx.x;
    const int64_t c0 = tile * kTile;
    const int nvalid = (int)((dv.d - c0) < kTile ? (dv.d - c0) : kTile); // multiple of 4
    float* xr = a.X + (int64_t)row * dv.ld + c0;
    float* hr = a.Xhat + (int64_t)row * dv.ld + c0;
    float* sr = a.S + (int64_t)row * dv.ld + c0;

    // Thread 0 starts the tile copies; warp 0 looks up where each neighbour's message enters
    // this tile (lane r holds neighbour r of the current batch of 32) while all threads clear
    // the accumulator tile.
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        const uint32_t bytes = (uint32_t)nvalid * sizeof(float);
        mbar_expect_tx(bar, bytes * bulk_arrays<HAS_G, HAS_M>());
        bulk_load(xs, xr, bytes, bar);
        bulk_load(hs, hr, bytes, bar);
        bulk_load(ss, sr, bytes, bar);
        if (HAS_G) bulk_load(gs, a.G + (int64_t)row * dv.ld + c0, bytes, bar);
        if (HAS_M) bulk_load(ms, a.M + (int64_t)row * dv.ld + c0, bytes, bar);
    }
    const int lane = threadIdx.x & 31;
    const uint32_t lo_key = EMIT ? __ldg(dv.row_lo + row) : 0u; // needed only at the end: fetch early
    // lane r of warp 0: where neighbour r's message enters this tile (one 16-byte record)
    const uint4* recs = dv.rec + ((int64_t)row * dv.ntiles + tile) * dv.maxdeg;
    int nj = 0;
    float nw = 0.f;
    uint32_t nlo = 0, nlen = 0;
    if (threadIdx.x < 32 && lane < dv.maxdeg) {
        const uint4 rc = __ldg(recs + lane);
        nj = (int)rc.x; nlo = rc.y; nlen = rc.z; nw = __uint_as_float(rc.w);
    }
#pragma unroll
    for (int it = 0; it < NIT; ++it)
        reinterpret_cast<float4*>(acc)[it * NT + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (threadIdx.x < kTile / 32) { touched[threadIdx.x] = 0u; tself[threadIdx.x] = 0u; }
    __syncthreads();

    // Warp 0 alone adds the neighbours' entries, in CSR order; program order inside the warp
    // (plus __syncwarp between neighbours) is what orders two neighbours that hit the same
    // coordinate.  The first 32 entries of up to kPrefetch neighbours are fetched together.
    int ok = 1;
    if (threadIdx.x < 32) {
        uint32_t self_lo = 0, self_len = 0, self_idx = 0; // own entries: first 32 kept in registers
        float self_val = 0.f;
        for (int eb = 0; eb < dv.maxdeg; eb += 32) {
            if (eb != 0) {
                nlen = 0;
                if (eb + lane < dv.maxdeg) {
                    const uint4 rc = __ldg(recs + eb + lane);
                    nj = (int)rc.x; nlo = rc.y; nlen = rc.z; nw = __uint_as_float(rc.w);
                }
            }
            const int nb = (dv.maxdeg - eb) < 32 ? (dv.maxdeg - eb) : 32;
            for (int rc = 0; rc < nb; rc += kPrefetch) {
                uint32_t pidx[kPrefetch];
                float pval[kPrefetch];
#pragma unroll
                for (int q = 0; q < kPrefetch; ++q) {
                    const int r = (rc + q) & 31;
                    const int jr = __shfl_sync(0xffffffffu, nj, r);
                    const uint32_t lor = __shfl_sync(0xffffffffu, nlo, r);
                    const uint32_t lenr = __shfl_sync(0xffffffffu, nlen, r);
                    pidx[q] = 0u;
                    pval[q] = 0.f;
                    if (rc + q < nb && (uint32_t)lane < lenr) {
                        pidx[q] = __ldg(dv.msg_idx + (int64_t)jr * dv.kpitch + lor + lane);
                        pval[q] = __ldg(dv.msg_val + (int64_t)jr * dv.kpitch + lor + lane);
                    }
                }
#pragma unroll
                for (int q = 0; q < kPrefetch; ++q) {
                    if (rc + q >= nb) break;
                    const int r = rc + q;
                    const int jr = __shfl_sync(0xffffffffu, nj, r);
                    const float wr = __shfl_sync(0xffffffffu, nw, r);
                    const uint32_t lor = __shfl_sync(0xffffffffu, nlo, r);
                    const uint32_t lenr = __shfl_sync(0xffffffffu, nlen, r);
                    if (jr == row && lenr) { self_lo = lor; self_len = lenr; self_idx = pidx[q]; self_val = pval[q]; }
                    if ((uint32_t)lane < lenr) {
                        const uint32_t lc = pidx[q] - (uint32_t)c0;
                        acc[lc] = __fadd_rn(acc[lc], __fmul_rn(wr, pval[q]));
                        atomicOr(&touched[lc >> 5], 1u << (lc & 31));
                    }
                    for (uint32_t p = 32 + lane; p < lenr; p += 32) { // beyond the prefetched 32
                        const uint32_t lc = __ldg(dv.msg_idx + (int64_t)jr * dv.kpitch + lor + p) - (uint32_t)c0;
                        const float val = __ldg(dv.msg_val + (int64_t)jr * dv.kpitch + lor + p);
                        acc[lc] = __fadd_rn(acc[lc], __fmul_rn(wr, val));
                        atomicOr(&touched[lc >> 5], 1u << (lc & 31));
                    }
                    __syncwarp();
                }
            }
        }
        // wait (bounded) for the tiles, then x^ += q_i in place on the staged tile
        ok = mbar_wait_bounded(bar, 0, dv.stats) ? 1 : 0;
        if (ok) {
            if ((uint32_t)lane < self_len) {
                const uint32_t lc = self_idx - (uint32_t)c0;
                hs[lc] = __fadd_rn(hs[lc], self_val);
                atomicOr(&tself[lc >> 5], 1u << (lc & 31));
            }
            const uint32_t* mi = dv.msg_idx + (int64_t)row * dv.kpitch + self_lo;
            const float* mv = dv.msg_val + (int64_t)row * dv.kpitch + self_lo;
            for (uint32_t p = 32 + lane; p < self_len; p += 32) { // beyond the 32 kept in registers
                const uint32_t lc = __ldg(mi + p) - (uint32_t)c0;
                hs[lc] = __fadd_rn(hs[lc], __ldg(mv + p));
                atomicOr(&tself[lc >> 5], 1u << (lc & 31));
            }
        }
    }
    // the other warps wait here without polling; afterwards each thread observes the
    // completed barrier phase itself so that the copied tiles are visible to it
    if (!__syncthreads_and(ok)) return; // recorded in the stats: the step's result is invalid
    if (!mbar_wait_bounded(bar, 0, dv.stats)) return;

    const Upd u = {a.eta, a.gamma, a.lambda, a.beta};
    uint32_t take = 0, cnt[NIT];
    uint32_t vbits[NIT][4];
    float* mrow = HAS_M ? a.M + (int64_t)row * dv.ld + c0 : nullptr;
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int q4 = it * NT + threadIdx.x;
        const int li = q4 * kQuad;
        cnt[it] = 0;
        if (li >= nvalid) continue;
        const float4 x = reinterpret_cast<const float4*>(xs)[q4];
        const float4 h = reinterpret_cast<const float4*>(hs)[q4];
        const float4 s = reinterpret_cast<const float4*>(ss)[q4];
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
        if (HAS_G) g = reinterpret_cast<const float4*>(gs)[q4];
        if (HAS_M) m = reinterpret_cast<const float4*>(ms)[q4];
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
        uint32_t start[NIT], total;
        ordered_starts<NT, NIT>(cnt, scan, start, &total);
        if (threadIdx.x == 0) {
            const uint32_t base = total ? atomicAdd(&dv.row_count[row], total) : 0u;
            dv.seg_off[(int64_t)row * dv.ntiles + tile] = base;
            dv.seg_cnt[(int64_t)row * dv.ntiles + tile] = total;
            *s_base = ((int64_t)base + total > dv.cap) ? 0xFFFFFFFFu : base;
        }
        __syncthreads();
        const uint32_t base = *s_base;
        if (base == 0xFFFFFFFFu || take == 0u) return;
        uint32_t* ci = dv.cand_idx + (int64_t)row * dv.cap + base;
        uint32_t* cv = dv.cand_val + (int64_t)row * dv.cap + base;
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

template <bool HAS_G, bool HAS_M, bool EMIT>
cudaError_t launch_bulk(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    constexpr size_t smem = bulk_smem_bytes<kTileThreads, HAS_G, HAS_M>();
    // Once per device and instantiation: allow the dynamic shared memory size and ask for the
    // largest shared-memory carve-out, so that as many tiles as possible are in flight per SM.
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        auto kern = update_sparse_bulk_kernel<kTileThreads, HAS_G, HAS_M, EMIT>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const dim3 grid((unsigned)dv.ntiles, (unsigned)dv.n);
    update_sparse_bulk_kernel<kTileThreads, HAS_G, HAS_M, EMIT><<<grid, kTileThreads, smem, st>>>(dv, a);
    return cudaSuccess;
}

} // namespace

bool update_bulk_usable(const Dev& dv, const StepArgs& a)
{
    return (dv.kind == CHOCO_Q_TOPK || dv.kind == CHOCO_Q_RANDK) && a.vec && dv.d % 4 == 0;
}

cudaError_t launch_update_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    if (a.M) return emit ? launch_bulk<true, true, true>(dv, a, st) : launch_bulk<true, true, false>(dv, a, st);
    if (a.G) return emit ? launch_bulk<true, false, true>(dv, a, st) : launch_bulk<true, false, false>(dv, a, st);
    return emit ? launch_bulk<false, false, true>(dv, a, st) : launch_bulk<false, false, false>(dv, a, st);
}

} // namespace choco
