// Update kernel for scaled sign and bucketed gsgd_b: Algorithm 1's update of the public copies, gossip step and gradient step (Algorithm 2 with
// momentum) for one tile of 2048 coordinates of one worker per block,
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i),
// followed (EMIT) by the compression of x' - x^' (Appendix C) into the other message buffer,
// so that the next step's messages cost no further pass over X and Xhat.
//
// Everything a block touches moves through shared memory by asynchronous bulk copies: the x, x^,
// s, g (and momentum) tiles and, for every neighbour, the 2048-coordinate slice of its packed
// message (sign plane, level fields) are fetched with one mbarrier to wait on; the results are
// written back over the staged tiles and leave by bulk stores, as do the sign plane and the level
// fields of the next message.  No thread holds a global address or a loaded value across a wait.
// A bulk copy needs 16-byte aligned addresses and sizes.  With AL (rows 16-byte aligned, d a
// multiple of 4) a tile is copied as it is and leaves the same way; otherwise (rows that start on
// 8-byte boundaries, any d) each copy in starts at the 16-byte boundary at or below the tile's
// first element and ends at the one at or above its last, the tile is read from shared memory at
// the resulting offset of 0 or 2 elements, and the results are stored from registers (a bulk store would overwrite the neighbours of a tile that
// starts or ends inside a 16-byte unit).  The message planes are library-owned and always aligned.
//
// The per-coordinate work is kept to what the definition needs:
//   * a neighbour's contribution w_ij q_j takes only s distinct magnitudes per block of the norm,
//     fl(w fl(mag l)) for l = 0..s-1; they are tabulated once per tile (s <= 16) and a
//     coordinate's decode is a table read plus its sign bit -- the same products, the same bits;
//   * the quotient fl(fl(s |v|) / nu) of the quantiser is formed as the product with 1 / nu in
//     float64, rounded once to float32: for float32 operands that is the correctly rounded
//     quotient (the float64 product is within 2^-52 of a / nu, no quotient of two float32 numbers
//     lies within 2^-49 of the midpoint of two float32 numbers, and none is such a midpoint);
//   * floor(r + u), saturated at s - 1, is taken by clamping at s - 1/2 and adding 2^23 rounded
//     down, which leaves the integer in the low bits of the sum;
//   * the round keys of the generator depend on the seed only and come as kernel arguments.
#include "bulk.cuh"

namespace choco {

namespace {

constexpr int NT = 128;
constexpr int NIT = 4;                   // quads per thread (what a thread does once per tile weighs less that way)
constexpr int kDTile = NT * kQuad * NIT; // 2048 coordinates per block
constexpr int kWarps = NT / 32;
constexpr int kWarpSums = NIT * kWarps;  // one per 128 coordinates of the tile, in coordinate order
static_assert(kDTile == 2048 && kWarpSums == 16, "tile of 2048 coordinates: two chunks of the L1 tree, up to 16 blocks of the norm");
constexpr int kBatch = 16;               // neighbours whose message slices are staged at a time
constexpr int kTabLevels = 16;           // level magnitudes are tabulated for s <= 16

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

// shared memory -> global; both addresses 16-byte aligned, bytes % 16 == 0
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_store_commit_and_drain()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    // the staged tiles may be released once the copy engine has read them
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// order this thread's shared-memory accesses before what the copy engine does next
__device__ __forceinline__ void fence_before_bulk_copy()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// mag is >= 0, so setting the sign bit negates it; bit e of nib is coordinate e's sign
__device__ __forceinline__ float with_sign(float mag, uint32_t nib, int e)
{
    return __uint_as_float(__float_as_uint(mag) | ((nib << (31 - e)) & 0x80000000u));
}

// small non-negative integer -> float without the conversion unit: exact below 2^23
__device__ __forceinline__ float small_uint_to_float(uint32_t v)
{
    return __fsub_rn(__uint_as_float(0x4B000000u | v), 8388608.f);
}

// Philox4x32-10 with the round keys precomputed (Dev::round_key): the same words as philox4x32_10.
__device__ __forceinline__ uint4 philox_with_round_keys(uint4 ctr, const Dev& dv)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * ctr.x;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * ctr.z;
        ctr = make_uint4((uint32_t)(p1 >> 32) ^ ctr.y ^ dv.round_key[r][0], (uint32_t)p1,
                         (uint32_t)(p0 >> 32) ^ ctr.w ^ dv.round_key[r][1], (uint32_t)p0);
    }
    return ctr;
}

// Shared-memory layout, in bytes from the (128-byte aligned) base.  WBITS == 0: scaled sign.
template <int WBITS, bool HAS_G, bool HAS_M>
struct Layout {
    static constexpr int kArrays = 3 + (HAS_G ? 1 : 0) + (HAS_M ? 1 : 0);
    static constexpr int kBitsTile = kDTile / 8;               // 256 bytes of sign plane
    static constexpr int kLevTile = kDTile * WBITS / 8;        // level fields of a tile
    static constexpr int kMsgTile = kBitsTile + kLevTile;      // one neighbour's slice
    static constexpr bool kTable = WBITS >= 1 && WBITS <= 4;   // s <= 16: magnitudes tabulated
    static constexpr int kStage = kDTile + 4;                  // floats per staged tile (slack: it may start mid-unit)
    __host__ __device__ static constexpr int msg_in() { return kArrays * kStage * 4; }
    __host__ __device__ static int msg_out(int nb) { return msg_in() + nb * kMsgTile; }
    __host__ __device__ static int tables(int nb) { return msg_out(nb) + kMsgTile; }
    // per neighbour and block of the norm: 16 weighted magnitudes (or, without a table, one
    // magnitude and the weight); then the worker's own unweighted magnitudes
    __host__ __device__ static int table_floats(int nb, int nbk) { return (nb + 1) * nbk * kTabLevels; }
    __host__ __device__ static int misc(int nb, int nbk) { return tables(nb) + table_floats(nb, nbk) * 4; }
    // misc: warp sums [kWarpSums] floats, per-block reciprocal norms [16] doubles, the barrier
    __host__ __device__ static int total(int nb, int nbk) { return misc(nb, nbk) + kWarpSums * 4 + 16 * 8 + 16; }
};

// element offset of p inside its 16-byte unit
__device__ __forceinline__ uint32_t unit_shift(const float* p) { return (uint32_t)(((uintptr_t)p & 15u) >> 2); }

// four consecutive floats of a staged tile that starts `sh` (0 or 2 unless AL) elements into its
// buffer: 8-byte aligned, so two 64-bit reads
template <bool AL>
__device__ __forceinline__ float4 staged_quad(const float* buf, uint32_t sh, int q4)
{
    if (AL) return reinterpret_cast<const float4*>(buf)[q4];
    const float* p = buf + sh + q4 * kQuad;
    const float2 lo = *reinterpret_cast<const float2*>(p), hi = *reinterpret_cast<const float2*>(p + 2);
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// store the first `left` (1..4) elements of v at p (4-byte aligned)
__device__ __forceinline__ void store_some(float* p, const float4& v, int left)
{
    p[0] = v.x;
    if (left > 1) p[1] = v.y;
    if (left > 2) p[2] = v.z;
    if (left > 3) p[3] = v.w;
}

// bx: the block's tile of the row; row: the worker; d, ld: dv.d and dv.ld; nbk: blocks of the
// norm per tile (1 for sign).  With LAYERS `dv` is the block's shared-memory copy of its layer's
// parameters, still to be filled from `dv_src`: the tiles are requested first (that needs d, ld
// and the array pointers only), the copy is made while they fly.
template <int KIND, int WBITS, bool HAS_G, bool HAS_M, bool EMIT, bool AL, bool LAYERS>
__device__ __forceinline__ void update_dense_bulk_body(const Dev& dv, const StepArgs& a, int nb_stage, int nbk, int64_t bx,
                                                       int row, int64_t d, int64_t ld, unsigned char* smem_raw,
                                                       const Dev* dv_src)
{
    using L = Layout<WBITS, HAS_G, HAS_M>;
    static_assert((KIND == CHOCO_Q_SIGN) == (WBITS == 0), "sign has no level fields");
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* hs = xs + L::kStage;
    float* ss = hs + L::kStage;
    float* gs = ss + L::kStage;                     // used when HAS_G
    float* ms = gs + (HAS_G ? L::kStage : 0);       // used when HAS_M
    unsigned char* msg_in = smem_raw + L::msg_in();
    unsigned char* msg_out = smem_raw + L::msg_out(nb_stage);
    float* tab = reinterpret_cast<float*>(smem_raw + L::tables(nb_stage));
    float* tab_self = tab + nb_stage * nbk * kTabLevels;
    float* ws = reinterpret_cast<float*>(smem_raw + L::misc(nb_stage, nbk)); // [kWarpSums] sums over 128 coordinates
    double* rnu = reinterpret_cast<double*>(ws + kWarpSums);                 // [16] 1 / nu per block of the norm
    uint64_t* bar = reinterpret_cast<uint64_t*>(rnu + 16);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = bx * kDTile;
    const int nvalid = (int)((d - c0) < kDTile ? (d - c0) : kDTile); // AL: a multiple of 4
    float* xr = a.X + (int64_t)row * ld + c0;
    float* hr = a.Xhat + (int64_t)row * ld + c0;
    float* sr = a.S + (int64_t)row * ld + c0;
    float* mrow = HAS_M ? a.M + (int64_t)row * ld + c0 : nullptr;
    const float* gr = HAS_G ? a.G + (int64_t)row * ld + c0 : nullptr;
    // where each staged tile's first element sits in its shared-memory buffer
    const uint32_t shx = AL ? 0u : unit_shift(xr), shh = AL ? 0u : unit_shift(hr), shs = AL ? 0u : unit_shift(sr);
    const uint32_t shg = (AL || !HAS_G) ? 0u : unit_shift(gr), shm = (AL || !HAS_M) ? 0u : unit_shift(mrow);
    auto span = [&](uint32_t sh) { return (((uint32_t)nvalid + sh) * (uint32_t)sizeof(float) + 15u) & ~15u; };
    // sizes of the slices actually present in this tile, rounded up to whole 16-byte units (the
    // message rows are padded so that the rounded slice of the last tile stays inside the row)
    const uint32_t dense_bytes = (uint32_t)nvalid * sizeof(float);
    const uint32_t bits_bytes = ((((uint32_t)nvalid + 31u) >> 5) * 4u + 15u) & ~15u;
    const uint32_t lev_bytes = (((uint32_t)nvalid * WBITS + 7u) / 8u + 15u) & ~15u;
    const uint32_t msg_bytes = bits_bytes + (WBITS > 0 ? lev_bytes : 0u);
    const int64_t bits_off = bx * (kDTile / 32);            // words into a row's sign plane
    const int64_t lev_off = bx * L::kLevTile;               // bytes into a row's level fields

    // The barrier takes one arrival per phase, or two with LAYERS, where the tiles are requested
    // before the layer's parameters (and with them the neighbours) are known.
    const uint32_t dense_tx = span(shx) + span(shh) + span(shs) + (HAS_G ? span(shg) : 0u) + (HAS_M ? span(shm) : 0u);
    if (threadIdx.x == 0) {
        mbar_init(bar, LAYERS ? 2 : 1);
        if (LAYERS) mbar_expect_tx(bar, dense_tx);
    }
    auto request_tiles = [&]() {
        bulk_load(xs, xr - shx, span(shx), bar);
        bulk_load(hs, hr - shh, span(shh), bar);
        bulk_load(ss, sr - shs, span(shs), bar);
        if (HAS_G) bulk_load(gs, gr - shg, span(shg), bar);
        if (HAS_M) bulk_load(ms, mrow - shm, span(shm), bar);
    };
    if (LAYERS) {
        if (threadIdx.x == 0) request_tiles();
        load_layer_params(dv_src, const_cast<Dev*>(&dv));
    }
    const Upd u = {a.eta, a.gamma, a.lambda, a.beta, dv.nesterov}; // (dv is complete from here on)
    const int e0 = dv.row_ptr[row], deg = dv.row_ptr[row + 1] - e0;
    // stage the message slices of neighbours [first, first + count): lane r of warp 0 issues r's copies
    auto stage_messages = [&](int first, int count) {
        if (lane < count) {
            const int j = dv.col[e0 + first + lane];
            unsigned char* dst = msg_in + lane * L::kMsgTile;
            bulk_load(dst, dv.msg_bits + (int64_t)j * dv.wpitch + bits_off, bits_bytes, bar);
            if (WBITS > 0) bulk_load(dst + L::kBitsTile, dv.msg_levels + (int64_t)j * dv.lpitch + lev_off, lev_bytes, bar);
        }
    };
    if (warp == 0) {
        const int count = deg < nb_stage ? deg : nb_stage;
        if (lane == 0) {
            mbar_expect_tx(bar, (LAYERS ? 0u : dense_tx) + (uint32_t)count * msg_bytes);
            if (!LAYERS) request_tiles();
        }
        __syncwarp();
        stage_messages(0, count);
    }

    float acc[NIT][4], qs[NIT][4];
#pragma unroll
    for (int it = 0; it < NIT; ++it)
#pragma unroll
        for (int e = 0; e < 4; ++e) { acc[it][e] = 0.f; qs[it][e] = 0.f; }

    for (int first = 0; first < deg; first += nb_stage) {
        const int count = (deg - first) < nb_stage ? (deg - first) : nb_stage;
        if (first > 0) {
            // every thread is done with the previous batch's slices and tables
            fence_before_bulk_copy();
            __syncthreads();
            if (warp == 0) {
                if (lane == 0) {
                    mbar_expect_tx(bar, (uint32_t)count * msg_bytes);
                    if (LAYERS) mbar_arrive(bar); // the phase's second arrival
                }
                __syncwarp();
                stage_messages(first, count);
            }
        }
        // magnitudes of this batch's neighbours, while the copies fly
        int self_r = -1;
        for (int r = 0; r < count; ++r)
            if (dv.col[e0 + first + r] == row) self_r = r;
        if (KIND == CHOCO_Q_SIGN) {
            if ((int)threadIdx.x < count) {
                const int j = dv.col[e0 + first + threadIdx.x];
                const float sc = __ldg(dv.msg_scale + j);
                tab[threadIdx.x] = __fmul_rn(dv.wval[e0 + first + threadIdx.x], sc);
                if ((int)threadIdx.x == self_r) tab_self[0] = sc;
            }
        } else {
            constexpr int per = L::kTable ? kTabLevels : 2;
            for (int t = threadIdx.x; t < count * nbk * per; t += NT) {
                const int l = t % per, b = (t / per) % nbk, r = t / (per * nbk);
                const int64_t gb = (c0 >> dv.bucket_shift) + b;
                float mag = 0.f;
                const float w = dv.wval[e0 + first + r];
                if (gb < dv.nbuckets) {
                    const float nu = __ldg(dv.msg_norms + (int64_t)dv.col[e0 + first + r] * dv.npitch + gb);
                    mag = __fdiv_rn(nu, __fmul_rn(gb == dv.tail_bucket ? dv.tau_tail : dv.tau_full, (float)dv.s));
                }
                if (L::kTable) {
                    const float m = __fmul_rn(mag, (float)l);
                    tab[(r * nbk + b) * kTabLevels + l] = __fmul_rn(w, m);
                    if (r == self_r) tab_self[b * kTabLevels + l] = m;
                } else {
                    tab[(r * nbk + b) * kTabLevels + l] = l == 0 ? mag : w;
                }
            }
        }
        // thread 0 polls (bounded); the others wait at the barrier, then each thread observes the
        // completed phase itself so that the copied data is visible to it
        const uint32_t parity = (uint32_t)((first / nb_stage) & 1);
        int ok = 1;
        if (threadIdx.x == 0) ok = mbar_wait_bounded(bar, parity, dv.stats, dv.wait_polls) ? 1 : 0;
        if (!__syncthreads_and(ok)) return; // recorded in the stats: the step's result is invalid
        (void)mbar_wait_bounded(bar, parity, dv.stats, kSpinLimit);

        // neighbours in CSR order (outer loop), this thread's two quads inside
        for (int r = 0; r < count; ++r) {
            const unsigned char* slice = msg_in + r * L::kMsgTile;
            const bool self = r == self_r;
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int q4 = it * NT + threadIdx.x;
                const int li = q4 * kQuad;
                const uint32_t word = reinterpret_cast<const uint32_t*>(slice)[li >> 5];
                const uint32_t nib = (word >> (li & 31)) & 0xFu;
                float q[4];
                if (KIND == CHOCO_Q_SIGN) {
                    const float m = tab[r];
#pragma unroll
                    for (int e = 0; e < 4; ++e) q[e] = with_sign(m, nib, e);
                    if (self) {
                        const float sc = tab_self[0];
#pragma unroll
                        for (int e = 0; e < 4; ++e) qs[it][e] = with_sign(sc, nib, e);
                    }
                } else {
                    const int b = li >> dv.bucket_shift; // block of the norm: the same for the whole warp
                    const unsigned char* lev = slice + L::kBitsTile;
                    uint32_t packed, packed_hi = 0u; // the quad's four fields (16-bit fields: two words)
                    if (WBITS == 16) {
                        const uint2 two = reinterpret_cast<const uint2*>(lev)[q4];
                        packed = two.x;
                        packed_hi = two.y;
                    } else if (WBITS == 8) packed = reinterpret_cast<const uint32_t*>(lev)[q4];
                    else if (WBITS == 4) packed = reinterpret_cast<const uint16_t*>(lev)[q4];
                    else if (WBITS == 2) packed = lev[q4];
                    else packed = (uint32_t)(lev[q4 >> 1] >> (li & 4));
                    constexpr uint32_t mask = (1u << (WBITS > 0 ? WBITS : 1)) - 1u;
                    auto field = [&](int e) -> uint32_t {
                        if constexpr (WBITS == 16) return ((e < 2 ? packed : packed_hi) >> ((e & 1) * 16)) & mask;
                        else return (packed >> (e * WBITS)) & mask;
                    };
                    const float* t = tab + (r * nbk + b) * kTabLevels;
                    if (L::kTable) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) q[e] = with_sign(t[field(e)], nib, e);
                        if (self) {
                            const float* ts = tab_self + b * kTabLevels;
#pragma unroll
                            for (int e = 0; e < 4; ++e) qs[it][e] = with_sign(ts[field(e)], nib, e);
                        }
                    } else {
                        const float mag = t[0], w = t[1];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float m = __fmul_rn(mag, small_uint_to_float(field(e)));
                            if (self) qs[it][e] = with_sign(m, nib, e);
                            q[e] = with_sign(__fmul_rn(w, m), nib, e);
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[it][e] = __fadd_rn(acc[it][e], q[e]);
            }
        }
    }

    // the update itself, written back over the staged tiles
    float4 vn[NIT]; // x' - x^': the next step's argument of Q
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int q4 = it * NT + threadIdx.x;
        const int li = q4 * kQuad;
        vn[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (li < nvalid) {
            const float4 x = staged_quad<AL>(xs, shx, q4);
            const float4 h = staged_quad<AL>(hs, shh, q4);
            const float4 s = staged_quad<AL>(ss, shs, q4);
            float4 g = make_float4(0.f, 0.f, 0.f, 0.f), m = g;
            if (HAS_G) g = staged_quad<AL>(gs, shg, q4);
            if (HAS_M) m = staged_quad<AL>(ms, shm, q4);
            const float4 hn = make_float4(__fadd_rn(h.x, qs[it][0]), __fadd_rn(h.y, qs[it][1]),
                                          __fadd_rn(h.z, qs[it][2]), __fadd_rn(h.w, qs[it][3]));
            const float4 sn = make_float4(__fadd_rn(s.x, acc[it][0]), __fadd_rn(s.y, acc[it][1]),
                                          __fadd_rn(s.z, acc[it][2]), __fadd_rn(s.w, acc[it][3]));
            float4 xn;
            xn.x = next_x<HAS_G, HAS_M>(x.x, sn.x, hn.x, g.x, m.x, u);
            xn.y = next_x<HAS_G, HAS_M>(x.y, sn.y, hn.y, g.y, m.y, u);
            xn.z = next_x<HAS_G, HAS_M>(x.z, sn.z, hn.z, g.z, m.z, u);
            xn.w = next_x<HAS_G, HAS_M>(x.w, sn.w, hn.w, g.w, m.w, u);
            const int left = nvalid - li; // >= 4 except in the last quad of an unaligned row
            if (AL) {
                reinterpret_cast<float4*>(hs)[q4] = hn;
                reinterpret_cast<float4*>(ss)[q4] = sn;
                reinterpret_cast<float4*>(xs)[q4] = xn;
                if (HAS_M) reinterpret_cast<float4*>(ms)[q4] = m;
            } else {
                store_some(hr + li, hn, left);
                store_some(sr + li, sn, left);
                store_some(xr + li, xn, left);
                if (HAS_M) store_some(mrow + li, m, left);
            }
            if (EMIT) {
                // coordinates past d inside the last quad count as +0
                vn[it].x = __fsub_rn(xn.x, hn.x);
                if (AL || left > 1) vn[it].y = __fsub_rn(xn.y, hn.y);
                if (AL || left > 2) vn[it].z = __fsub_rn(xn.z, hn.z);
                if (AL || left > 3) vn[it].w = __fsub_rn(xn.w, hn.w);
            }
        }
        if (EMIT) {
            const float4 v = vn[it];
            float t;
            if (KIND == CHOCO_Q_SIGN) t = quad_tree(fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w));
            else t = quad_tree(__fmul_rn(v.x, v.x), __fmul_rn(v.y, v.y), __fmul_rn(v.z, v.z), __fmul_rn(v.w, v.w));
            t = warp_tree(t);
            if (lane == 0) ws[it * kWarps + warp] = t;
            // sign plane of the next message: this quad's four bits and its neighbour's make a byte
            const uint32_t nib = (uint32_t)(v.x < 0.f) | ((uint32_t)(v.y < 0.f) << 1) | ((uint32_t)(v.z < 0.f) << 2) |
                                 ((uint32_t)(v.w < 0.f) << 3);
            const uint32_t other = __shfl_xor_sync(0xffffffffu, nib, 1);
            if ((lane & 1) == 0) msg_out[q4 >> 1] = (unsigned char)(nib | (other << 4));
        }
    }
    fence_before_bulk_copy();
    __syncthreads();
    const bool storer = threadIdx.x == 0;
    if (storer) {
        if (AL) {
            bulk_store(xr, xs, dense_bytes);
            bulk_store(hr, hs, dense_bytes);
            bulk_store(sr, ss, dense_bytes);
            if (HAS_M) bulk_store(mrow, ms, dense_bytes);
        }
        if (EMIT) bulk_store(dv.nxt_bits + (int64_t)row * dv.wpitch + bits_off, msg_out, bits_bytes);
    }
    if (!EMIT) {
        if (storer) bulk_store_commit_and_drain();
        return;
    }
    if (KIND == CHOCO_Q_SIGN) {
        // per-1024 partial sums of |v|; a small kernel finishes the tree and the scale
        if (threadIdx.x < kDTile / kChunk) {
            const int64_t chunk = bx * (kDTile / kChunk) + threadIdx.x;
            if (chunk < dv.nchunks) dv.partial[(int64_t)row * dv.nchunks + chunk] = tree8(ws + threadIdx.x * 8);
        }
        if (storer) bulk_store_commit_and_drain();
        return;
    }
    // gsgd_b with blocks of dv.bucket (128..1024) coordinates: one thread per block of the norm
    // finishes its tree over the warp sums, stores the norm and leaves 1 / nu for the others
    const int G = dv.bucket >> 7; // warps per block of the norm: 1, 2, 4 or 8
    if ((int)threadIdx.x < nbk) {
        const float* wsi = ws + (int)threadIdx.x * G;
        float sq;
        if (G == 1) sq = wsi[0];
        else if (G == 2) sq = __fadd_rn(wsi[0], wsi[1]);
        else if (G == 4) sq = __fadd_rn(__fadd_rn(wsi[0], wsi[1]), __fadd_rn(wsi[2], wsi[3]));
        else sq = tree8(wsi);
        const float nu = __fsqrt_rn(sq);
        const int64_t gb = (c0 >> dv.bucket_shift) + threadIdx.x;
        if (gb < dv.nbuckets) dv.nxt_norms[(int64_t)row * dv.npitch + gb] = nu;
        rnu[threadIdx.x] = nu != 0.f ? 1.0 / (double)nu : 0.0; // nu = 0: every level is 0
    }
    __syncthreads();
    const float sf = (float)dv.s, top = __fsub_rn((float)dv.s, 0.5f);
    unsigned char* lev_out = msg_out + L::kBitsTile;
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int q4 = it * NT + threadIdx.x;
        const int li = q4 * kQuad;
        const double y = rnu[li >> dv.bucket_shift];
        // the dither of the message that the NEXT step applies
        const uint64_t step = step_of(a) + 1;
        const uint4 rw = philox_with_round_keys(
            make_uint4((uint32_t)((c0 + li) >> 2), (uint32_t)row, (uint32_t)step,
                       ((uint32_t)(step >> 32) << 8) | kStreamDither), dv);
        const float uu[4] = {word_to_unit(rw.x), word_to_unit(rw.y), word_to_unit(rw.z), word_to_unit(rw.w)};
        const float vv[4] = {vn[it].x, vn[it].y, vn[it].z, vn[it].w};
        uint32_t lv[4]; // 2^23 + level, as float bits
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float r = (float)((double)__fmul_rn(sf, fabsf(vv[e])) * y); // = fl(fl(s |v|) / nu)
            const float t = fminf(__fadd_rn(r, uu[e]), top);  // floor(min(t, s - 1/2)) = min(floor t, s - 1)
            lv[e] = __float_as_uint(__fadd_rd(t, 8388608.f));
        }
        constexpr uint32_t kMagic = 0x4B000000u;
        if (WBITS == 16) {
            reinterpret_cast<uint2*>(lev_out)[q4] = make_uint2((lv[1] * 65536u + lv[0]) - kMagic * 0x00010001u,
                                                               (lv[3] * 65536u + lv[2]) - kMagic * 0x00010001u);
        } else if (WBITS == 8) {
            reinterpret_cast<uint32_t*>(lev_out)[q4] =
                (((lv[3] * 256u + lv[2]) * 256u + lv[1]) * 256u + lv[0]) - kMagic * 0x01010101u;
        } else if (WBITS == 4) {
            reinterpret_cast<uint16_t*>(lev_out)[q4] =
                (uint16_t)((((lv[3] * 16u + lv[2]) * 16u + lv[1]) * 16u + lv[0]) - kMagic * 0x1111u);
        } else if (WBITS == 2) {
            lev_out[q4] = (unsigned char)((((lv[3] * 4u + lv[2]) * 4u + lv[1]) * 4u + lv[0]) - kMagic * 0x55u);
        } else {
            const uint32_t four = ((((lv[3] * 2u + lv[2]) * 2u + lv[1]) * 2u + lv[0]) - kMagic * 0xFu) & 0xFu;
            const uint32_t other = __shfl_xor_sync(0xffffffffu, four, 1);
            if ((lane & 1) == 0) lev_out[q4 >> 1] = (unsigned char)(four | (other << 4));
        }
    }
    fence_before_bulk_copy();
    __syncthreads();
    if (storer) {
        bulk_store(dv.nxt_levels + (int64_t)row * dv.lpitch + lev_off, lev_out, lev_bytes);
        bulk_store_commit_and_drain();
    }
}

// MINB: resident blocks per SM the registers are budgeted for (5: what shared memory allows, best
// for many waves of blocks; 4: more registers per thread, best when the grid is a wave or two)
template <int KIND, int WBITS, bool HAS_G, bool HAS_M, bool EMIT, bool AL, int MINB>
__global__ void __launch_bounds__(NT, MINB) update_dense_bulk_kernel(Dev dv, StepArgs a, int nb_stage)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int nbk = KIND == CHOCO_Q_QSGD ? (kDTile >> dv.bucket_shift) : 1; // blocks of the norm per tile
    update_dense_bulk_body<KIND, WBITS, HAS_G, HAS_M, EMIT, AL, false>(dv, a, nb_stage, nbk, (int64_t)blockIdx.x,
                                                                      (int)blockIdx.y + a.row0, dv.d, dv.ld, smem_raw, nullptr);
}

// several layers in one launch: blockIdx.x picks (layer, tile), blockIdx.y the worker
template <int KIND, int WBITS, bool HAS_G, bool HAS_M, bool AL>
__global__ void __launch_bounds__(NT, 5)
update_dense_bulk_layers_kernel(const __grid_constant__ LayerTable tab, LayerSet ls, StepArgs a, int nb_stage, int nbk)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ Dev sdev;
    const int en = entry_of_block(tab, blockIdx.x);
    shift_arrays(a, tab.off[en]);
    update_dense_bulk_body<KIND, WBITS, HAS_G, HAS_M, true, AL, true>(
        sdev, a, nb_stage, nbk, (int64_t)(blockIdx.x - tab.first_block[en]), (int)blockIdx.y, (int64_t)tab.d[en], ls.ld,
        smem_raw, ls.devs + tab.layer[en]);
}

// SMs of the current device (looked up once per device)
cudaError_t sm_count(int* out)
{
    static int sms[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int n = (dev >= 0 && dev < 64) ? sms[dev] : 0;
    if (n == 0) {
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) sms[dev] = n;
    }
    *out = n;
    return cudaSuccess;
}

template <typename K>
cudaError_t allow_shared_memory(K kern, size_t smem, size_t* configured)
{
    // Once per device, instantiation and size: allow the dynamic shared memory and ask for the
    // largest shared-memory carve-out, so that as many tiles as possible are in flight per SM.
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || configured[dev] < smem) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = smem;
    }
    return cudaSuccess;
}

template <int KIND, int WBITS, bool HAS_G, bool HAS_M, bool AL>
cudaError_t launch_layers_one(const Dev& proto, const LayerTable& tab, const LayerSet& ls, const StepArgs& a, cudaStream_t st)
{
    using L = Layout<WBITS, HAS_G, HAS_M>;
    const int nb_stage = proto.maxdeg < kBatch ? proto.maxdeg : kBatch;
    const int nbk = KIND == CHOCO_Q_QSGD ? (kDTile >> proto.bucket_shift) : 1;
    const size_t smem = (size_t)L::total(nb_stage, nbk);
    auto kern = update_dense_bulk_layers_kernel<KIND, WBITS, HAS_G, HAS_M, AL>;
    static size_t configured[64] = {};
    const cudaError_t e = allow_shared_memory(kern, smem, configured);
    if (e != cudaSuccess) return e;
    kern<<<dim3(tab.first_block[tab.entries], (unsigned)proto.n), NT, smem, st>>>(tab, ls, a, nb_stage, nbk);
    return cudaGetLastError();
}

template <int KIND, int WBITS, bool AL>
cudaError_t launch_layers_terms(const Dev& proto, const LayerTable& tab, const LayerSet& ls, const StepArgs& a, cudaStream_t st)
{
    if (a.M) return launch_layers_one<KIND, WBITS, true, true, AL>(proto, tab, ls, a, st);
    if (a.G) return launch_layers_one<KIND, WBITS, true, false, AL>(proto, tab, ls, a, st);
    return launch_layers_one<KIND, WBITS, false, false, AL>(proto, tab, ls, a, st);
}

template <bool AL>
cudaError_t launch_layers_kind(const Dev& proto, const LayerTable& tab, const LayerSet& ls, const StepArgs& a, cudaStream_t st)
{
    if (proto.kind == CHOCO_Q_SIGN) return launch_layers_terms<CHOCO_Q_SIGN, 0, AL>(proto, tab, ls, a, st);
    switch (proto.wbits) {
    case 1: return launch_layers_terms<CHOCO_Q_QSGD, 1, AL>(proto, tab, ls, a, st);
    case 2: return launch_layers_terms<CHOCO_Q_QSGD, 2, AL>(proto, tab, ls, a, st);
    case 4: return launch_layers_terms<CHOCO_Q_QSGD, 4, AL>(proto, tab, ls, a, st);
    case 8: return launch_layers_terms<CHOCO_Q_QSGD, 8, AL>(proto, tab, ls, a, st);
    default: return launch_layers_terms<CHOCO_Q_QSGD, 16, AL>(proto, tab, ls, a, st);
    }
}

template <int KIND, int WBITS, bool HAS_G, bool HAS_M, bool EMIT, bool AL>
cudaError_t launch_one(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    using L = Layout<WBITS, HAS_G, HAS_M>;
    const int nb_stage = dv.maxdeg < kBatch ? dv.maxdeg : kBatch;
    const int nbk = KIND == CHOCO_Q_QSGD ? (kDTile >> dv.bucket_shift) : 1;
    const size_t smem = (size_t)L::total(nb_stage, nbk);
    const dim3 grid((unsigned)((dv.d + kDTile - 1) / kDTile), (unsigned)(a.rows > 0 ? a.rows : dv.n));
    if constexpr (KIND == CHOCO_Q_SIGN) {
        // a grid of at most two waves: the time is a block's latency, not the SMs' throughput
        // (measured on 8 x 272 474: 0.0190 against 0.0206 ms per step; 32 x 272 474 prefers five)
        int nsm = 0;
        const cudaError_t es = sm_count(&nsm);
        if (es != cudaSuccess) return es;
        if ((int64_t)grid.x * grid.y <= 10 * (int64_t)nsm) {
            auto kern4 = update_dense_bulk_kernel<KIND, WBITS, HAS_G, HAS_M, EMIT, AL, 4>;
            static size_t configured4[64] = {};
            const cudaError_t e4 = allow_shared_memory(kern4, smem, configured4);
            if (e4 != cudaSuccess) return e4;
            kern4<<<grid, NT, smem, st>>>(dv, a, nb_stage);
            return cudaGetLastError();
        }
    }
    auto kern = update_dense_bulk_kernel<KIND, WBITS, HAS_G, HAS_M, EMIT, AL, 5>;
    static size_t configured[64] = {};
    const cudaError_t e = allow_shared_memory(kern, smem, configured);
    if (e != cudaSuccess) return e;
    kern<<<grid, NT, smem, st>>>(dv, a, nb_stage);
    return cudaGetLastError();
}

template <int KIND, int WBITS, bool EMIT, bool AL>
cudaError_t launch_terms(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    if (a.M) return launch_one<KIND, WBITS, true, true, EMIT, AL>(dv, a, st);
    if (a.G) return launch_one<KIND, WBITS, true, false, EMIT, AL>(dv, a, st);
    return launch_one<KIND, WBITS, false, false, EMIT, AL>(dv, a, st);
}

template <bool EMIT, bool AL>
cudaError_t launch_kind(const Dev& dv, const StepArgs& a, cudaStream_t st)
{
    if (dv.kind == CHOCO_Q_SIGN) return launch_terms<CHOCO_Q_SIGN, 0, EMIT, AL>(dv, a, st);
    switch (dv.wbits) {
    case 1: return launch_terms<CHOCO_Q_QSGD, 1, EMIT, AL>(dv, a, st);
    case 2: return launch_terms<CHOCO_Q_QSGD, 2, EMIT, AL>(dv, a, st);
    case 4: return launch_terms<CHOCO_Q_QSGD, 4, EMIT, AL>(dv, a, st);
    case 8: return launch_terms<CHOCO_Q_QSGD, 8, EMIT, AL>(dv, a, st);
    default: return launch_terms<CHOCO_Q_QSGD, 16, EMIT, AL>(dv, a, st);
    }
}

} // namespace

bool update_dense_bulk_usable(const Dev& dv, const StepArgs& a)
{
    if (!(dv.kind == CHOCO_Q_SIGN || (dv.kind == CHOCO_Q_QSGD && dv.bucket > 0))) return false;
    // every row of every array must start on an 8-byte boundary (16 with AL); rows that start
    // at an odd element go to the register kernel
    auto even = [](const void* p) { return ((uintptr_t)p & 7u) == 0; };
    return dv.ld % 2 == 0 && even(a.X) && even(a.Xhat) && even(a.S) && even(a.G) && even(a.M);
}

cudaError_t launch_update_dense_bulk_layers(const Dev& proto, const LayerTable& tab, const LayerSet& ls, const StepArgs& a,
                                            bool aligned, cudaStream_t st)
{
    return aligned ? launch_layers_kind<true>(proto, tab, ls, a, st) : launch_layers_kind<false>(proto, tab, ls, a, st);
}

cudaError_t launch_update_dense_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    // a.vec: every row of every array starts on a 16-byte boundary
    if (a.vec && dv.d % 4 == 0) return emit ? launch_kind<true, true>(dv, a, st) : launch_kind<false, true>(dv, a, st);
    return emit ? launch_kind<true, false>(dv, a, st) : launch_kind<false, false>(dv, a, st);
}

} // namespace choco
