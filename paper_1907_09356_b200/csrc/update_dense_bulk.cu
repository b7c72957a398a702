// Update kernel for scaled sign and bucketed gsgd_b, bulk-copy variant (rows 16-byte
// aligned, d a multiple of 4): the same arithmetic as update_dense_kernel (Algorithm 1:
// public copies, gossip step, gradient step) followed by the compression of x' - x^' for the next step, with the x, x^, s, g
// (and momentum) tiles of 2048 coordinates staged in shared memory by asynchronous bulk
// copies.  The neighbours' packed message pieces that a thread needs are small; they are
// fetched into registers while the copies are in flight.
#include "bulk.cuh"

namespace choco {

namespace {

constexpr int NT = 256;
constexpr int NIT = 2;                  // quads per thread
constexpr int kDTile = NT * kQuad * NIT; // 2048 coordinates per block
constexpr int kPre = 4;                 // neighbours whose pieces are fetched ahead

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

// The pieces of worker j's message that cover coordinates [c, c+4): the quad's four sign
// bits and (gsgd_b) its packed level fields.  The magnitude that goes with them -- the row's
// scale, or norm / (tau s) of the block -- is the same for many quads and is kept apart.
struct Piece {
    uint32_t nib;    // bit e: coordinate c + e is negative
    uint32_t packed; // level fields, wbits each (gsgd_b)
};

template <int KIND>
__device__ __forceinline__ Piece load_piece(const Dev& dv, int j, int64_t c)
{
    Piece p;
    p.nib = __ldg(dv.msg_bits + (int64_t)j * dv.wpitch + (c >> 5));
    p.packed = 0u;
    if (KIND == CHOCO_Q_QSGD) {
        const uint8_t* lrow = dv.msg_levels + (int64_t)j * dv.lpitch;
        const uint32_t width = (uint32_t)dv.wbits;
        if (width == 8) p.packed = __ldg(reinterpret_cast<const uint32_t*>(lrow + c));
        else if (width == 4) p.packed = __ldg(reinterpret_cast<const uint16_t*>(lrow + (c >> 1)));
        else if (width == 2) p.packed = __ldg(lrow + (c >> 2));
        else p.packed = (__ldg(lrow + (c >> 3)) >> (c & 7)) & 0xFu;
    }
    return p;
}

// magnitude shared by the coordinates of one block of worker j's message
template <int KIND>
__device__ __forceinline__ float load_mag(const Dev& dv, int j, int64_t bucket)
{
    if (KIND == CHOCO_Q_SIGN) return __ldg(dv.msg_scale + j);
    const float nu = __ldg(dv.msg_norms + (int64_t)j * dv.npitch + bucket);
    return __fdiv_rn(nu, __fmul_rn(bucket == dv.tail_bucket ? dv.tau_tail : dv.tau_full, (float)dv.s));
}

// small non-negative integer -> float without the conversion unit: exact below 2^23
__device__ __forceinline__ float small_uint_to_float(uint32_t v)
{
    return __fsub_rn(__uint_as_float(0x4B000000u | v), 8388608.f);
}

// mag is >= 0, so setting the sign bit negates it
__device__ __forceinline__ float with_sign(float mag, uint32_t nib, int e)
{
    return __uint_as_float(__float_as_uint(mag) | ((nib << (31 - e)) & 0x80000000u));
}

template <int KIND>
__device__ __forceinline__ float4 decode_piece(const Dev& dv, const Piece& pp, float mag, int64_t c)
{
    Piece p = pp; p.nib = (pp.nib >> (c & 31)) & 0xFu;
    float m[4];
    if (KIND == CHOCO_Q_SIGN) {
        m[0] = m[1] = m[2] = m[3] = mag;
    } else {
        const uint32_t width = (uint32_t)dv.wbits, mask = (1u << width) - 1u;
#pragma unroll
        for (int e = 0; e < 4; ++e) m[e] = __fmul_rn(mag, small_uint_to_float((p.packed >> (e * width)) & mask));
    }
    return make_float4(with_sign(m[0], p.nib, 0), with_sign(m[1], p.nib, 1), with_sign(m[2], p.nib, 2),
                       with_sign(m[3], p.nib, 3));
}

__device__ __forceinline__ uint32_t sign_nibble4(const float4& v)
{
    return (uint32_t)(v.x < 0.f) | ((uint32_t)(v.y < 0.f) << 1) | ((uint32_t)(v.z < 0.f) << 2) |
           ((uint32_t)(v.w < 0.f) << 3);
}

template <bool HAS_G, bool HAS_M>
__host__ __device__ constexpr int n_arrays() { return 3 + (HAS_G ? 1 : 0) + (HAS_M ? 1 : 0); }

template <int KIND, bool HAS_G, bool HAS_M, bool EMIT>
__global__ void __launch_bounds__(NT, 4) update_dense_bulk_kernel(Dev dv, StepArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* hs = xs + kDTile;
    float* ss = hs + kDTile;
    float* gs = ss + kDTile;                     // used when HAS_G
    float* ms = gs + (HAS_G ? kDTile : 0);       // used when HAS_M
    float* ws = ms + (HAS_M ? kDTile : 0);       // [NIT][8] warp sums
    uint64_t* bar = reinterpret_cast<uint64_t*>(ws + NIT * 8);

    const int row = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kDTile;
    const int nvalid = (int)((dv.d - c0) < kDTile ? (dv.d - c0) : kDTile); // multiple of 4
    const int e0 = dv.row_ptr[row], e1 = dv.row_ptr[row + 1];
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta};
    float* xr = a.X + (int64_t)row * dv.ld + c0;
    float* hr = a.Xhat + (int64_t)row * dv.ld + c0;
    float* sr = a.S + (int64_t)row * dv.ld + c0;
    float* mrow = HAS_M ? a.M + (int64_t)row * dv.ld + c0 : nullptr;

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        const uint32_t bytes = (uint32_t)nvalid * sizeof(float);
        mbar_expect_tx(bar, bytes * n_arrays<HAS_G, HAS_M>());
        bulk_load(xs, xr, bytes, bar);
        bulk_load(hs, hr, bytes, bar);
        bulk_load(ss, sr, bytes, bar);
        if (HAS_G) bulk_load(gs, a.G + (int64_t)row * dv.ld + c0, bytes, bar);
        if (HAS_M) bulk_load(ms, mrow, bytes, bar);
    }
    // message pieces of the first kPre neighbours, fetched while the tiles are in flight
    Piece pre[NIT][kPre];
    int prej[kPre];
    float prew[kPre], pmag[kPre];
#pragma unroll
    for (int q = 0; q < kPre; ++q) {
        prej[q] = -1;
        prew[q] = 0.f;
        pmag[q] = 0.f;
        if (e0 + q < e1) {
            prej[q] = dv.col[e0 + q];
            prew[q] = dv.wval[e0 + q];
            if (KIND == CHOCO_Q_SIGN) pmag[q] = load_mag<KIND>(dv, prej[q], 0);
        }
    }
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int li = (it * NT + threadIdx.x) * kQuad;
#pragma unroll
        for (int q = 0; q < kPre; ++q) {
            pre[it][q].nib = 0u; pre[it][q].packed = 0u;
            if (prej[q] >= 0 && li < nvalid) pre[it][q] = load_piece<KIND>(dv, prej[q], c0 + li);
        }
    }
    // gsgd_b: the 128 coordinates of a warp's quads lie in one block, so lane q fetches the
    // norm of neighbour q's block and the warp shares norm / (tau s) by shuffles later
    float nraw[NIT];
    bool ntail[NIT];
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        nraw[it] = 0.f;
        ntail[it] = false;
        if (KIND == CHOCO_Q_QSGD) {
            const int64_t bucket = (c0 + (int64_t)(it * NT + warp * 32) * kQuad) >> dv.bucket_shift;
            ntail[it] = bucket == dv.tail_bucket;
            if (lane < kPre && e0 + lane < e1 && bucket < dv.nbuckets)
                nraw[it] = __ldg(dv.msg_norms + (int64_t)dv.col[e0 + lane] * dv.npitch + bucket);
        }
    }
    // thread 0 polls (bounded); the others wait at the barrier, then each thread observes the
    // completed phase itself so that the copied tiles are visible to it
    int ok = 1;
    if (threadIdx.x == 0) ok = mbar_wait_bounded(bar, 0, dv.stats, dv.wait_polls) ? 1 : 0;
    if (!__syncthreads_and(ok)) return; // recorded in the stats: the step's result is invalid
    (void)mbar_wait_bounded(bar, 0, dv.stats, kSpinLimit);

    float4 vn[NIT]; // x' - x^': the next step's argument of Q
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int q4 = it * NT + threadIdx.x;
        const int li = q4 * kQuad;
        const int64_t c = c0 + li;
        vn[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        float lane_mag = 0.f; // lane q: norm / (tau s) of neighbour q's block
        if (KIND == CHOCO_Q_QSGD)
            lane_mag = __fdiv_rn(nraw[it], __fmul_rn(ntail[it] ? dv.tau_tail : dv.tau_full, (float)dv.s));
        float qmag[kPre];
#pragma unroll
        for (int q = 0; q < kPre; ++q)
            qmag[q] = KIND == CHOCO_Q_SIGN ? pmag[q] : __shfl_sync(0xffffffffu, lane_mag, q);
        if (li < nvalid) {
            const float4 x = reinterpret_cast<const float4*>(xs)[q4];
            const float4 h = reinterpret_cast<const float4*>(hs)[q4];
            const float4 s = reinterpret_cast<const float4*>(ss)[q4];
            float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
            if (HAS_G) g = reinterpret_cast<const float4*>(gs)[q4];
            if (HAS_M) m = reinterpret_cast<const float4*>(ms)[q4];
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), qs = acc;
#pragma unroll
            for (int q = 0; q < kPre; ++q) {
                if (prej[q] < 0) continue;
                const float4 qv = decode_piece<KIND>(dv, pre[it][q], qmag[q], c);
                acc.x = __fadd_rn(acc.x, __fmul_rn(prew[q], qv.x));
                acc.y = __fadd_rn(acc.y, __fmul_rn(prew[q], qv.y));
                acc.z = __fadd_rn(acc.z, __fmul_rn(prew[q], qv.z));
                acc.w = __fadd_rn(acc.w, __fmul_rn(prew[q], qv.w));
                if (prej[q] == row) qs = qv;
            }
            for (int e = e0 + kPre; e < e1; ++e) { // rows with more neighbours: fetched on the spot
                const int j = dv.col[e];
                const float w = dv.wval[e];
                const Piece p = load_piece<KIND>(dv, j, c);
                const float4 qv = decode_piece<KIND>(dv, p, load_mag<KIND>(dv, j, c >> dv.bucket_shift), c);
                acc.x = __fadd_rn(acc.x, __fmul_rn(w, qv.x));
                acc.y = __fadd_rn(acc.y, __fmul_rn(w, qv.y));
                acc.z = __fadd_rn(acc.z, __fmul_rn(w, qv.z));
                acc.w = __fadd_rn(acc.w, __fmul_rn(w, qv.w));
                if (j == row) qs = qv;
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
            *reinterpret_cast<float4*>(hr + li) = hn;
            *reinterpret_cast<float4*>(sr + li) = sn;
            *reinterpret_cast<float4*>(xr + li) = xn;
            if (HAS_M) *reinterpret_cast<float4*>(mrow + li) = m;
            if (EMIT)
                vn[it] = make_float4(__fsub_rn(xn.x, hn.x), __fsub_rn(xn.y, hn.y), __fsub_rn(xn.z, hn.z),
                                     __fsub_rn(xn.w, hn.w));
        }
        if (EMIT) {
            const float4 v = vn[it];
            float t;
            if (KIND == CHOCO_Q_SIGN) t = quad_tree(fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w));
            else t = quad_tree(__fmul_rn(v.x, v.x), __fmul_rn(v.y, v.y), __fmul_rn(v.z, v.z),
                               __fmul_rn(v.w, v.w));
            t = warp_tree(t);
            if (lane == 0) ws[it * 8 + warp] = t;
            const uint32_t word = gather_sign_word(sign_nibble4(v), lane);
            if ((lane & 7) == 0 && li < nvalid) dv.nxt_bits[(int64_t)row * dv.wpitch + (c >> 5)] = word;
        }
    }
    if (!EMIT) return;
    __syncthreads();
    if (KIND == CHOCO_Q_SIGN) {
        // per-1024 partial sums of |v|; a small kernel finishes the tree and the scale
        if (threadIdx.x < NIT) {
            const int64_t chunk = (int64_t)blockIdx.x * NIT + threadIdx.x;
            if (chunk < dv.nchunks) dv.partial[(int64_t)row * dv.nchunks + chunk] = tree8(ws + threadIdx.x * 8);
        }
        return;
    }
    // gsgd_b with blocks of dv.bucket (128..1024) coordinates: norms, dithered levels, packing
    const float sf = (float)dv.s;
    const int G = dv.bucket >> 7; // warps per block of coordinates: 1, 2, 4 or 8
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int li = (it * NT + threadIdx.x) * kQuad;
        const int64_t c = c0 + li;
        const float* wsi = ws + it * 8;
        const int w0 = warp & ~(G - 1);
        float sq;
        if (G == 1) sq = wsi[w0];
        else if (G == 2) sq = __fadd_rn(wsi[w0], wsi[w0 + 1]);
        else if (G == 4) sq = __fadd_rn(__fadd_rn(wsi[w0], wsi[w0 + 1]), __fadd_rn(wsi[w0 + 2], wsi[w0 + 3]));
        else sq = tree8(wsi);
        const float nu = __fsqrt_rn(sq);
        const int64_t bucket = c >> dv.bucket_shift;
        if (lane == 0 && warp == w0 && bucket < dv.nbuckets)
            dv.nxt_norms[(int64_t)row * dv.npitch + bucket] = nu;
        // the dither of the message that the NEXT step applies
        const uint4 rw = coord_words(dv.seed, step_of(a) + 1, (uint32_t)row, kStreamDither, c);
        const float uu[4] = {word_to_unit(rw.x), word_to_unit(rw.y), word_to_unit(rw.z), word_to_unit(rw.w)};
        const float vv[4] = {vn[it].x, vn[it].y, vn[it].z, vn[it].w};
        uint32_t lev[4] = {0u, 0u, 0u, 0u};
        if (nu != 0.f) { // the same for every lane of the warp
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float r = __fdiv_rn(__fmul_rn(sf, fabsf(vv[e])), nu);
                const int l = __float2int_rz(__fadd_rn(r, uu[e])); // r + u >= 0: truncation is the floor
                lev[e] = (uint32_t)(l > dv.s - 1 ? dv.s - 1 : l);
            }
        }
        uint8_t* lrow = dv.nxt_levels + (int64_t)row * dv.lpitch;
        const bool in = li < nvalid;
        if (dv.wbits == 8) {
            if (in) *reinterpret_cast<uint32_t*>(lrow + c) = lev[0] | (lev[1] << 8) | (lev[2] << 16) | (lev[3] << 24);
        } else if (dv.wbits == 4) {
            if (in) *reinterpret_cast<uint16_t*>(lrow + (c >> 1)) =
                        (uint16_t)(lev[0] | (lev[1] << 4) | (lev[2] << 8) | (lev[3] << 12));
        } else if (dv.wbits == 2) {
            if (in) lrow[c >> 2] = (uint8_t)(lev[0] | (lev[1] << 2) | (lev[2] << 4) | (lev[3] << 6));
        } else {
            const uint32_t lw = gather_sign_word(lev[0] | (lev[1] << 1) | (lev[2] << 2) | (lev[3] << 3), lane);
            if ((lane & 7) == 0 && in) *reinterpret_cast<uint32_t*>(lrow + (c >> 3)) = lw;
        }
    }
}

template <int KIND, bool HAS_G, bool HAS_M, bool EMIT>
cudaError_t launch_one(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    constexpr size_t smem = (size_t)n_arrays<HAS_G, HAS_M>() * kDTile * sizeof(float) +
                            NIT * 8 * sizeof(float) + 16;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        auto kern = update_dense_bulk_kernel<KIND, HAS_G, HAS_M, EMIT>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const dim3 grid((unsigned)((dv.d + kDTile - 1) / kDTile), (unsigned)dv.n);
    update_dense_bulk_kernel<KIND, HAS_G, HAS_M, EMIT><<<grid, NT, smem, st>>>(dv, a);
    return cudaGetLastError();
}

template <int KIND, bool EMIT>
cudaError_t launch_terms(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    if (a.M) return launch_one<KIND, true, true, EMIT>(dv, a, st);
    if (a.G) return launch_one<KIND, true, false, EMIT>(dv, a, st);
    return launch_one<KIND, false, false, EMIT>(dv, a, st);
}

} // namespace

bool update_dense_bulk_usable(const Dev& dv, const StepArgs& a)
{
    if (!(a.vec && dv.d % 4 == 0)) return false;
    return dv.kind == CHOCO_Q_SIGN || (dv.kind == CHOCO_Q_QSGD && dv.bucket > 0);
}

cudaError_t launch_update_dense_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    if (dv.kind == CHOCO_Q_SIGN)
        return emit ? launch_terms<CHOCO_Q_SIGN, true>(dv, a, st) : launch_terms<CHOCO_Q_SIGN, false>(dv, a, st);
    return emit ? launch_terms<CHOCO_Q_QSGD, true>(dv, a, st) : launch_terms<CHOCO_Q_QSGD, false>(dv, a, st);
}

} // namespace choco
