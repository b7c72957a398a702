// Dense compression operators of the paper's Appendix C ("Compression Schemes"): scaled
// sign, gsgd_b (QSGD with s = 2^(b-1) levels) and the identity, each turning the rows of
// x - x^ into the message buffers the apply kernels read back.
//
// Message layout per worker (row):
//   sign     : sign plane u32[ceil(d/32)], bit c%32 of word c/32 set iff v_c < 0, tail bits 0;
//              scale f32 = ||v||_1 / d.
//   qsgd     : block norms f32[blocks]; the same sign plane; level fields of `wbits` (1..16) bits,
//              coordinate c at bit offset c * wbits, least significant first.
//   identity : f32[d].
#include "common.cuh"
#include "internal.h"

namespace choco {

enum { NORM_L1 = 0, NORM_L2SQ = 1 };

template <bool VEC>
__device__ __forceinline__ float4 diff_quad(const Dev& dv, const StepArgs& a, int row, int64_t c)
{
    const float4 x = load_quad<VEC>(a.X + (int64_t)row * dv.ld, c, dv.d);
    const float4 h = load_quad<VEC>(a.Xhat + (int64_t)row * dv.ld, c, dv.d);
    return make_float4(__fsub_rn(x.x, h.x), __fsub_rn(x.y, h.y), __fsub_rn(x.z, h.z),
                       __fsub_rn(x.w, h.w));
}

__device__ __forceinline__ uint32_t sign_nibble(const float4& v)
{
    return (uint32_t)(v.x < 0.f) | ((uint32_t)(v.y < 0.f) << 1) | ((uint32_t)(v.z < 0.f) << 2) |
           ((uint32_t)(v.w < 0.f) << 3);
}

// ---------------------------------------------------------------------------------------
// Per-1024-coordinate partial sums of |v| (L1) or v*v (L2^2), optionally with the sign
// plane.  One block covers 4096 coordinates and writes four partials.
// ---------------------------------------------------------------------------------------
template <bool VEC, int MODE, bool PACK_SIGN>
__global__ void __launch_bounds__(kThreads) norm_partial_kernel(Dev dv, StepArgs a)
{
    __shared__ float ws[kDenseIters][8];
    const int row = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kSpan;
#pragma unroll
    for (int it = 0; it < kDenseIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        const float4 v = diff_quad<VEC>(dv, a, row, c);
        float t;
        if (MODE == NORM_L1) t = quad_tree(fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w));
        else t = quad_tree(__fmul_rn(v.x, v.x), __fmul_rn(v.y, v.y), __fmul_rn(v.z, v.z),
                           __fmul_rn(v.w, v.w));
        t = warp_tree(t);
        if (lane == 0) ws[it][warp] = t;
        if (PACK_SIGN) {
            const uint32_t word = gather_sign_word(sign_nibble(v), lane);
            if ((lane & 7) == 0 && c < dv.d) dv.msg_bits[(int64_t)row * dv.wpitch + (c >> 5)] = word;
        }
    }
    __syncthreads();
    if (threadIdx.x < kDenseIters) {
        const int64_t chunk = (int64_t)blockIdx.x * kDenseIters + threadIdx.x;
        if (chunk < dv.nchunks) dv.partial[(int64_t)row * dv.nchunks + chunk] = tree8(ws[threadIdx.x]);
    }
}

// Finish the tree over a row's partial sums.  MODE L1: scale = root / d (sign).
// MODE L2SQ: norm = sqrt(root) (QSGD with one block per row).
template <int MODE>
__device__ __forceinline__ void norm_finish_row(const Dev& dv, int row)
{
    float* src = dv.partial + (int64_t)row * dv.nchunks;
    float* dst = dv.partial2 + (int64_t)row * dv.nchunks;
    int64_t m = dv.nchunks;
    while (m > 1) {
        const int64_t half = m >> 1;
        for (int64_t j = threadIdx.x; j < half; j += blockDim.x)
            dst[j] = __fadd_rn(src[2 * j], src[2 * j + 1]);
        if ((m & 1) && threadIdx.x == 0) dst[half] = src[m - 1];
        __syncthreads();
        float* t = src; src = dst; dst = t;
        m = half + (m & 1);
    }
    if (threadIdx.x == 0) {
        if (MODE == NORM_L1) dv.msg_scale[row] = __fdiv_rn(src[0], (float)dv.d);
        else dv.msg_norms[(int64_t)row * dv.npitch] = __fsqrt_rn(src[0]);
    }
}

template <int MODE>
__global__ void __launch_bounds__(1024) norm_finish_kernel(Dev dv)
{
    norm_finish_row<MODE>(dv, (int)blockIdx.x);
}

// several layers in one launch (scaled sign: the scale of the NEXT message, whose partial sums
// the update kernel left): block b serves row b % n of the table's entry b / n
__global__ void __launch_bounds__(1024) sign_scale_layers_kernel(const __grid_constant__ LayerTable tab, LayerSet ls, int n)
{
    __shared__ Dev sdev;
    const int en = (int)(blockIdx.x / (unsigned)n), row = (int)(blockIdx.x % (unsigned)n);
    load_layer_params(ls.devs + tab.layer[en], &sdev);
    if (threadIdx.x == 0) sdev.msg_scale = sdev.nxt_scale;
    __syncthreads();
    norm_finish_row<NORM_L1>(sdev, row);
}

// ---------------------------------------------------------------------------------------
// gsgd_b: level = min(floor(s |v| / nu + u), s - 1), u from the generator's dither stream.
// BUCKET > 0: nu per block of BUCKET coordinates computed here (BUCKET in 128..1024);
// BUCKET == 0: nu of the whole row was computed by the two kernels above.
// ---------------------------------------------------------------------------------------
template <bool VEC, int WBITS, int BUCKET>
__global__ void __launch_bounds__(kThreads) qsgd_pack_kernel(Dev dv, StepArgs a)
{
    __shared__ float ws[kDenseIters][8];
    const int row = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kSpan;
    float4 v[kDenseIters];
#pragma unroll
    for (int it = 0; it < kDenseIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        v[it] = diff_quad<VEC>(dv, a, row, c);
        if constexpr (BUCKET > 0) {
            float t = quad_tree(__fmul_rn(v[it].x, v[it].x), __fmul_rn(v[it].y, v[it].y),
                                __fmul_rn(v[it].z, v[it].z), __fmul_rn(v[it].w, v[it].w));
            t = warp_tree(t);
            if (lane == 0) ws[it][warp] = t;
        }
    }
    if (BUCKET > 0) __syncthreads();
    const float sf = (float)dv.s;
#pragma unroll
    for (int it = 0; it < kDenseIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        float nu;
        int64_t bucket = 0;
        if constexpr (BUCKET > 0) {
            constexpr int G = BUCKET / 128; // warps per block of coordinates
            const int w0 = warp & ~(G - 1);
            float sq;
            if (G == 1) sq = ws[it][w0];
            else if (G == 2) sq = __fadd_rn(ws[it][w0], ws[it][w0 + 1]);
            else if (G == 4) sq = __fadd_rn(__fadd_rn(ws[it][w0], ws[it][w0 + 1]),
                                            __fadd_rn(ws[it][w0 + 2], ws[it][w0 + 3]));
            else sq = tree8(ws[it]);
            nu = __fsqrt_rn(sq);
            bucket = c / BUCKET;
            if (lane == 0 && warp == w0 && bucket < dv.nbuckets)
                dv.msg_norms[(int64_t)row * dv.npitch + bucket] = nu;
        } else {
            nu = dv.msg_norms[(int64_t)row * dv.npitch];
        }
        const uint4 rw = coord_words(dv.seed, step_of(a), (uint32_t)row, kStreamDither, c);
        const float u[4] = {word_to_unit(rw.x), word_to_unit(rw.y), word_to_unit(rw.z),
                            word_to_unit(rw.w)};
        const float vv[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
        uint32_t lev[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int l = 0;
            if (nu != 0.f) {
                const float r = __fdiv_rn(__fmul_rn(sf, fabsf(vv[e])), nu);
                l = (int)floorf(__fadd_rn(r, u[e]));
                l = l > dv.s - 1 ? dv.s - 1 : l;
            }
            lev[e] = (uint32_t)l;
        }
        const uint32_t word = gather_sign_word(sign_nibble(v[it]), lane);
        if ((lane & 7) == 0 && c < dv.d) dv.msg_bits[(int64_t)row * dv.wpitch + (c >> 5)] = word;
        uint8_t* lrow = dv.msg_levels + (int64_t)row * dv.lpitch;
        if (WBITS == 16) {
            if (c < dv.d)
                *reinterpret_cast<uint2*>(lrow + 2 * c) = make_uint2(lev[0] | (lev[1] << 16), lev[2] | (lev[3] << 16));
        } else if (WBITS == 8) {
            if (c < dv.d)
                *reinterpret_cast<uint32_t*>(lrow + c) = lev[0] | (lev[1] << 8) | (lev[2] << 16) | (lev[3] << 24);
        } else if (WBITS == 4) {
            if (c < dv.d)
                *reinterpret_cast<uint16_t*>(lrow + (c >> 1)) =
                    (uint16_t)(lev[0] | (lev[1] << 4) | (lev[2] << 8) | (lev[3] << 12));
        } else if (WBITS == 2) {
            if (c < dv.d) lrow[c >> 2] = (uint8_t)(lev[0] | (lev[1] << 2) | (lev[2] << 4) | (lev[3] << 6));
        } else {
            const uint32_t lw = gather_sign_word(lev[0] | (lev[1] << 1) | (lev[2] << 2) | (lev[3] << 3), lane);
            if ((lane & 7) == 0 && c < dv.d) *reinterpret_cast<uint32_t*>(lrow + (c >> 3)) = lw;
        }
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads) identity_kernel(Dev dv, StepArgs a)
{
    const int row = blockIdx.y;
    const int64_t c0 = (int64_t)blockIdx.x * kSpan;
#pragma unroll
    for (int it = 0; it < kDenseIters; ++it) {
        const int64_t c = c0 + (int64_t)(it * kThreads + threadIdx.x) * kQuad;
        if (c < dv.d) {
            const float4 v = diff_quad<VEC>(dv, a, row, c);
            // message rows are 16-byte aligned by construction; the pad past d is never read
            *reinterpret_cast<float4*>(dv.msg_dense + (int64_t)row * dv.dpitch + c) = v;
        }
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------

template <bool VEC, int WBITS>
static void launch_qsgd_pack(const Dev& dv, const StepArgs& a, dim3 grid, cudaStream_t st)
{
    switch (dv.bucket) {
    case 0: qsgd_pack_kernel<VEC, WBITS, 0><<<grid, kThreads, 0, st>>>(dv, a); break;
    case 128: qsgd_pack_kernel<VEC, WBITS, 128><<<grid, kThreads, 0, st>>>(dv, a); break;
    case 256: qsgd_pack_kernel<VEC, WBITS, 256><<<grid, kThreads, 0, st>>>(dv, a); break;
    case 512: qsgd_pack_kernel<VEC, WBITS, 512><<<grid, kThreads, 0, st>>>(dv, a); break;
    default: qsgd_pack_kernel<VEC, WBITS, 1024><<<grid, kThreads, 0, st>>>(dv, a); break;
    }
}

template <bool VEC>
static cudaError_t compress_impl(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    const dim3 grid((unsigned)dv.nspans, (unsigned)dv.n);
    switch (dv.kind) {
    case CHOCO_Q_SIGN:
        norm_partial_kernel<VEC, NORM_L1, true><<<grid, kThreads, 0, st>>>(dv, a);
        norm_finish_kernel<NORM_L1><<<dv.n, 1024, 0, st>>>(dv);
        *a.launches += 2;
        break;
    case CHOCO_Q_QSGD:
        if (dv.bucket == 0) {
            norm_partial_kernel<VEC, NORM_L2SQ, false><<<grid, kThreads, 0, st>>>(dv, a);
            norm_finish_kernel<NORM_L2SQ><<<dv.n, 1024, 0, st>>>(dv);
            *a.launches += 2;
        }
        switch (dv.wbits) {
        case 1: launch_qsgd_pack<VEC, 1>(dv, a, grid, st); break;
        case 2: launch_qsgd_pack<VEC, 2>(dv, a, grid, st); break;
        case 4: launch_qsgd_pack<VEC, 4>(dv, a, grid, st); break;
        case 8: launch_qsgd_pack<VEC, 8>(dv, a, grid, st); break;
        default: launch_qsgd_pack<VEC, 16>(dv, a, grid, st); break;
        }
        *a.launches += 1;
        break;
    default:
        identity_kernel<VEC><<<grid, kThreads, 0, st>>>(dv, a);
        *a.launches += 1;
        break;
    }
    return cudaGetLastError();
}

cudaError_t launch_next_sign_scale(const Dev& dv, cudaStream_t st)
{
    Dev dn = dv;
    dn.msg_scale = dv.nxt_scale;
    norm_finish_kernel<NORM_L1><<<dv.n, 1024, 0, st>>>(dn);
    return cudaGetLastError();
}

cudaError_t launch_sign_scale_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, cudaStream_t st)
{
    // small trees (layers of a launch-bound step): 128 threads each, many blocks per SM
    sign_scale_layers_kernel<<<(unsigned)(tab.entries * n), 128, 0, st>>>(tab, ls, n);
    return cudaGetLastError();
}

cudaError_t launch_compress_dense(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    return a.vec ? compress_impl<true>(dv, a, st) : compress_impl<false>(dv, a, st);
}

} // namespace choco
