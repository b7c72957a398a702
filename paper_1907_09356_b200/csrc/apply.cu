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
// sparse Q, register-staged variant (any alignment, any d): the neighbours' (index, value)
// lists are scattered into a shared-memory tile, one neighbour after the other so that the
// additions happen in CSR order, then the tile is streamed against x, x^, s and g.  x^ and s
// are written only where a message touched them.
// ---------------------------------------------------------------------------------------
template <bool VEC, bool HAS_G, bool HAS_M>
__global__ void __launch_bounds__(kTileThreads) apply_sparse_kernel(Dev dv, StepArgs a)
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
    float4 x[kTileIters], h[kTileIters], s[kTileIters], g[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kTileThreads + threadIdx.x) * kQuad;
        x[it] = load_quad_stream<VEC>(xr, c, dv.d);
        h[it] = load_quad_stream<VEC>(hr, c, dv.d);
        s[it] = load_quad_stream<VEC>(sr, c, dv.d);
        if (HAS_G) g[it] = load_quad_stream<VEC>(gr, c, dv.d);
        else g[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
        reinterpret_cast<float4*>(acc)[it * kTileThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
        reinterpret_cast<float4*>(qself)[it * kTileThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
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
        for (uint32_t p = lo + threadIdx.x; p < hi; p += kTileThreads) {
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
    for (int it = 0; it < kTileIters; ++it) {
        const int li = (it * kTileThreads + threadIdx.x) * kQuad;
        const int64_t c = c0 + li;
        if (c >= dv.d) continue;
        const float4 av = reinterpret_cast<const float4*>(acc)[it * kTileThreads + threadIdx.x];
        const float4 qv = reinterpret_cast<const float4*>(qself)[it * kTileThreads + threadIdx.x];
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
// launchers
// ---------------------------------------------------------------------------------------

template <bool VEC, bool HAS_G, bool HAS_M>
static cudaError_t apply_pick(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    const dim3 grid((unsigned)dv.ntiles, (unsigned)dv.n);  // sparse: one block per tile
    switch (dv.kind) {
    case CHOCO_Q_TOPK:
    case CHOCO_Q_RANDK:
        if (update_bulk_usable(dv, a)) return launch_update_bulk(dv, a, emit, st);
        apply_sparse_kernel<VEC, HAS_G, HAS_M><<<grid, kTileThreads, 0, st>>>(dv, a);
        break;
    default:
        return launch_update_dense(dv, a, emit, st);
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
    if (dv.kind == CHOCO_Q_TOPK) return update_bulk_usable(dv, a);
    if (dv.kind == CHOCO_Q_RANDK) return false;
    return update_dense_can_emit(dv);
}

cudaError_t launch_apply(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    const cudaError_t e = a.vec ? apply_vec<true>(dv, a, emit, st) : apply_vec<false>(dv, a, emit, st);
    *a.launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

} // namespace choco
