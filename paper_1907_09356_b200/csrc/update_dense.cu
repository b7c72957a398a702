// Update kernel for dense Q (scaled sign, gsgd_b, identity): Algorithm 1, the update of the
// public copies, the gossip step and the gradient step (Algorithm 2 with momentum).  Every thread decodes its neighbours' packed messages for the
// four coordinates it owns and forms
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i).
// With EMIT the kernel goes on to compress x' - x^' (Appendix C), which it holds in
// registers, into the *other* message buffer: the next step's messages cost no further pass
// over X and Xhat.  (gsgd_b with one block per row needs the whole row's norm first and is
// compressed by the separate kernels instead.)
#include "common.cuh"
#include "internal.h"

namespace choco {

namespace {

// One quad per thread: all of a thread's loads are in flight at once and more warps fit per
// SM than with a loop over several quads (measured on the 32 x 25.6M workload).
constexpr int kUpdIters = 1;
constexpr int kUpdSpan = kChunk * kUpdIters;

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

// q_j for coordinates [c, c+4) out of worker j's current message
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
        const int64_t b = dv.bucket > 0 ? (c >> dv.bucket_shift) : 0; // blocks are powers of two
        const float nu = __ldg(dv.msg_norms + (int64_t)j * dv.npitch + b);
        const bool tail = b == dv.tail_bucket;
        const float scale = __fdiv_rn(nu, __fmul_rn(tail ? dv.tau_tail : dv.tau_full, (float)dv.s));
        const uint8_t* lrow = dv.msg_levels + (int64_t)j * dv.lpitch;
        uint32_t packed, width = (uint32_t)dv.wbits;
        if (width == 16) { // two 32-bit words hold the four fields
            const uint2 two = __ldg(reinterpret_cast<const uint2*>(lrow + 2 * c));
            m[0] = __fmul_rn(scale, (float)(two.x & 0xFFFFu));
            m[1] = __fmul_rn(scale, (float)(two.x >> 16));
            m[2] = __fmul_rn(scale, (float)(two.y & 0xFFFFu));
            m[3] = __fmul_rn(scale, (float)(two.y >> 16));
            return make_float4(nib & 1u ? -m[0] : m[0], nib & 2u ? -m[1] : m[1], nib & 4u ? -m[2] : m[2],
                               nib & 8u ? -m[3] : m[3]);
        }
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

__device__ __forceinline__ uint32_t sign_nibble4(const float4& v)
{
    return (uint32_t)(v.x < 0.f) | ((uint32_t)(v.y < 0.f) << 1) | ((uint32_t)(v.z < 0.f) << 2) |
           ((uint32_t)(v.w < 0.f) << 3);
}

template <bool VEC, int KIND, bool HAS_G, bool HAS_M, bool EMIT>
__global__ void __launch_bounds__(kThreads, 4) update_dense_kernel(Dev dv, StepArgs a)
{
    __shared__ float ws[kUpdIters][8];
    const int row = (int)blockIdx.y + a.row0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kUpdSpan;
    const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta, dv.nesterov};
    float* xr = a.X + (int64_t)row * dv.ld;
    float* hr = a.Xhat + (int64_t)row * dv.ld;
    float* sr = a.S + (int64_t)row * dv.ld;
    const float* gr = HAS_G ? a.G + (int64_t)row * dv.ld : nullptr;
    float* mr = HAS_M ? a.M + (int64_t)row * dv.ld : nullptr;
    float4 vn[kUpdIters]; // x' - x^': the next step's argument of Q
#pragma unroll
    for (int it = 0; it < kUpdIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        vn[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < dv.d) {
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
            if (EMIT) {
                // coordinates past d inside the last quad count as +0
                vn[it].x = __fsub_rn(xn.x, hn.x);
                if (c + 1 < dv.d) vn[it].y = __fsub_rn(xn.y, hn.y);
                if (c + 2 < dv.d) vn[it].z = __fsub_rn(xn.z, hn.z);
                if (c + 3 < dv.d) vn[it].w = __fsub_rn(xn.w, hn.w);
            }
        }
        if (EMIT) {
            const float4 v = vn[it];
            if (KIND == CHOCO_Q_IDENTITY) {
                if (c < dv.d) *reinterpret_cast<float4*>(dv.nxt_dense + (int64_t)row * dv.dpitch + c) = v;
            } else {
                float t;
                if (KIND == CHOCO_Q_SIGN) t = quad_tree(fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w));
                else t = quad_tree(__fmul_rn(v.x, v.x), __fmul_rn(v.y, v.y), __fmul_rn(v.z, v.z),
                                   __fmul_rn(v.w, v.w));
                t = warp_tree(t);
                if (lane == 0) ws[it][warp] = t;
                const uint32_t word = gather_sign_word(sign_nibble4(v), lane);
                if ((lane & 7) == 0 && c < dv.d) dv.nxt_bits[(int64_t)row * dv.wpitch + (c >> 5)] = word;
            }
        }
    }
    if (!EMIT || KIND == CHOCO_Q_IDENTITY) return;
    __syncthreads();
    if (KIND == CHOCO_Q_SIGN) {
        // per-1024 partial sums of |v|; a small kernel finishes the tree and the scale
        if (threadIdx.x < kUpdIters) {
            const int64_t chunk = (int64_t)blockIdx.x * kUpdIters + threadIdx.x;
            if (chunk < dv.nchunks) dv.partial[(int64_t)row * dv.nchunks + chunk] = tree8(ws[threadIdx.x]);
        }
        return;
    }
    // gsgd_b with blocks of dv.bucket (128..1024) coordinates: norms, dithered levels, packing
    const float sf = (float)dv.s;
    const int G = dv.bucket >> 7; // warps per block of coordinates: 1, 2, 4 or 8
#pragma unroll
    for (int it = 0; it < kUpdIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        const int w0 = warp & ~(G - 1);
        float sq;
        if (G == 1) sq = ws[it][w0];
        else if (G == 2) sq = __fadd_rn(ws[it][w0], ws[it][w0 + 1]);
        else if (G == 4) sq = __fadd_rn(__fadd_rn(ws[it][w0], ws[it][w0 + 1]),
                                        __fadd_rn(ws[it][w0 + 2], ws[it][w0 + 3]));
        else sq = tree8(ws[it]);
        const float nu = __fsqrt_rn(sq);
        const int64_t bucket = c >> dv.bucket_shift;
        if (lane == 0 && warp == w0 && bucket < dv.nbuckets)
            dv.nxt_norms[(int64_t)row * dv.npitch + bucket] = nu;
        // the dither of the message that the NEXT step applies
        const uint4 rw = coord_words(dv.seed, step_of(a) + 1, (uint32_t)row, kStreamDither, c);
        const float uu[4] = {word_to_unit(rw.x), word_to_unit(rw.y), word_to_unit(rw.z), word_to_unit(rw.w)};
        const float vv[4] = {vn[it].x, vn[it].y, vn[it].z, vn[it].w};
        uint32_t lev[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int l = 0;
            if (nu != 0.f) {
                const float r = __fdiv_rn(__fmul_rn(sf, fabsf(vv[e])), nu);
                l = (int)floorf(__fadd_rn(r, uu[e]));
                l = l > dv.s - 1 ? dv.s - 1 : l;
            }
            lev[e] = (uint32_t)l;
        }
        uint8_t* lrow = dv.nxt_levels + (int64_t)row * dv.lpitch;
        if (dv.wbits == 16) {
            if (c < dv.d)
                *reinterpret_cast<uint2*>(lrow + 2 * c) = make_uint2(lev[0] | (lev[1] << 16), lev[2] | (lev[3] << 16));
        } else if (dv.wbits == 8) {
            if (c < dv.d)
                *reinterpret_cast<uint32_t*>(lrow + c) = lev[0] | (lev[1] << 8) | (lev[2] << 16) | (lev[3] << 24);
        } else if (dv.wbits == 4) {
            if (c < dv.d)
                *reinterpret_cast<uint16_t*>(lrow + (c >> 1)) =
                    (uint16_t)(lev[0] | (lev[1] << 4) | (lev[2] << 8) | (lev[3] << 12));
        } else if (dv.wbits == 2) {
            if (c < dv.d) lrow[c >> 2] = (uint8_t)(lev[0] | (lev[1] << 2) | (lev[2] << 4) | (lev[3] << 6));
        } else {
            const uint32_t lw = gather_sign_word(lev[0] | (lev[1] << 1) | (lev[2] << 2) | (lev[3] << 3), lane);
            if ((lane & 7) == 0 && c < dv.d) *reinterpret_cast<uint32_t*>(lrow + (c >> 3)) = lw;
        }
    }
}

template <bool VEC, bool HAS_G, bool HAS_M, bool EMIT>
void pick_kind(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    const dim3 grid((unsigned)((dv.d + kUpdSpan - 1) / kUpdSpan), (unsigned)(a.rows > 0 ? a.rows : dv.n));
    switch (dv.kind) {
    case CHOCO_Q_SIGN:
        update_dense_kernel<VEC, CHOCO_Q_SIGN, HAS_G, HAS_M, EMIT><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    case CHOCO_Q_QSGD:
        update_dense_kernel<VEC, CHOCO_Q_QSGD, HAS_G, HAS_M, EMIT><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    default:
        update_dense_kernel<VEC, CHOCO_Q_IDENTITY, HAS_G, HAS_M, EMIT><<<grid, kThreads, 0, st>>>(dv, a);
        break;
    }
}

template <bool VEC, bool EMIT>
void pick_terms(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    if (a.M) pick_kind<VEC, true, true, EMIT>(dv, a, st);
    else if (a.G) pick_kind<VEC, true, false, EMIT>(dv, a, st);
    else pick_kind<VEC, false, false, EMIT>(dv, a, st);
}

} // namespace

bool update_dense_can_emit(const Dev& dv)
{
    return dv.kind == CHOCO_Q_SIGN || dv.kind == CHOCO_Q_IDENTITY ||
           (dv.kind == CHOCO_Q_QSGD && dv.bucket > 0);
}

cudaError_t launch_update_dense(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    if (update_dense_bulk_usable(dv, a)) return launch_update_dense_bulk(dv, a, emit, st);
    if (a.vec) { if (emit) pick_terms<true, true>(dv, a, st); else pick_terms<true, false>(dv, a, st); }
    else { if (emit) pick_terms<false, true>(dv, a, st); else pick_terms<false, false>(dv, a, st); }
    return cudaGetLastError();
}

} // namespace choco
