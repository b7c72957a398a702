// Device helpers shared by the kernels of libchoco (sm_100a).
//
// Arithmetic rules every kernel follows so that results are reproducible bit for bit:
// float32, round to nearest even, no fused multiply-add (the library is compiled with
// -fmad=false), IEEE division and square root, norms summed as a pairwise tree over the
// coordinate index (level 0 = the terms, each level adds elements 2j and 2j+1, missing
// elements count as +0).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "internal.h"

namespace choco {

constexpr int kThreads = 256;            // threads per block of the streaming kernels
constexpr int kQuad = 4;                 // coordinates per thread per iteration (one 128-bit access)
constexpr int kChunk = kThreads * kQuad; // 1024 coordinates: one block iteration, one tree leaf group
constexpr int kDenseIters = 4;           // dense kernels: iterations per block
constexpr int kSpan = kChunk * kDenseIters; // dense kernels: coordinates per block (4096)
// sparse path (top-k, random-k): one block owns one tile of one row
constexpr int kTileThreads = 256;
constexpr int kTileIters = 2;            // quads per thread
constexpr int kTile = kTileThreads * kQuad * kTileIters; // 2048 coordinates

constexpr uint32_t kStreamRandK = 0;     // generator stream of the random-k selection keys
constexpr uint32_t kStreamDither = 1;    // generator stream of the QSGD dither

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  Counter = (coord / 4, worker, step low,
// (step high << 8) | stream), key = the two halves of the seed; coordinate c uses word c % 4.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) {
            key.x += 0x9E3779B9u;
            key.y += 0xBB67AE85u;
        }
        const uint32_t hi0 = __umulhi(0xD2511F53u, ctr.x);
        const uint32_t lo0 = 0xD2511F53u * ctr.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, ctr.z);
        const uint32_t lo1 = 0xCD9E8D57u * ctr.z;
        ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
    }
    return ctr;
}

__device__ __forceinline__ uint4 coord_words(uint64_t seed, uint64_t step, uint32_t worker,
                                             uint32_t stream, int64_t c)
{
    const uint4 ctr = make_uint4((uint32_t)(c >> 2), worker, (uint32_t)step,
                                 ((uint32_t)(step >> 32) << 8) | stream);
    return philox4x32_10(ctr, make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

__device__ __forceinline__ float word_to_unit(uint32_t w)
{
    return (float)(w >> 8) * 0x1p-24f; // exact: 24 bits
}

// ---------------------------------------------------------------------------------------
// Row access.  A quad is coordinates [c, c+4) with c % 4 == 0.  VEC rows (16-byte aligned
// base, pitch a multiple of 4) use one 128-bit access for full quads; other rows and the
// ragged last quad use scalar accesses.  Out-of-range coordinates read as +0.
// ---------------------------------------------------------------------------------------
template <bool VEC>
__device__ __forceinline__ float4 load_quad(const float* __restrict__ row, int64_t c, int64_t d)
{
    if (VEC && c + 4 <= d) return *reinterpret_cast<const float4*>(row + c);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < d) r.x = row[c];
    if (c + 1 < d) r.y = row[c + 1];
    if (c + 2 < d) r.z = row[c + 2];
    if (c + 3 < d) r.w = row[c + 3];
    return r;
}

// streaming variant (evict-first hint): data that is read once per step
template <bool VEC>
__device__ __forceinline__ float4 load_quad_stream(const float* __restrict__ row, int64_t c,
                                                   int64_t d)
{
    if (VEC && c + 4 <= d) return __ldcs(reinterpret_cast<const float4*>(row + c));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < d) r.x = __ldcs(row + c);
    if (c + 1 < d) r.y = __ldcs(row + c + 1);
    if (c + 2 < d) r.z = __ldcs(row + c + 2);
    if (c + 3 < d) r.w = __ldcs(row + c + 3);
    return r;
}

template <bool VEC>
__device__ __forceinline__ void store_quad(float* __restrict__ row, int64_t c, int64_t d, float4 v)
{
    if (VEC && c + 4 <= d) {
        *reinterpret_cast<float4*>(row + c) = v;
        return;
    }
    if (c < d) row[c] = v.x;
    if (c + 1 < d) row[c + 1] = v.y;
    if (c + 2 < d) row[c + 2] = v.z;
    if (c + 3 < d) row[c + 3] = v.w;
}

__device__ __forceinline__ float quad_get(const float4& q, int e)
{
    return e == 0 ? q.x : e == 1 ? q.y : e == 2 ? q.z : q.w;
}

// ---------------------------------------------------------------------------------------
// Pairwise tree pieces.  quad_tree: two levels inside a quad.  warp_tree: five more levels
// by xor-butterfly (a + b is commutative, so both lanes of a pair hold the same bits); all
// lanes end with the sum over the warp's 128 coordinates.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float quad_tree(float a, float b, float c, float d)
{
    return __fadd_rn(__fadd_rn(a, b), __fadd_rn(c, d));
}

__device__ __forceinline__ float warp_tree(float v)
{
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;
}

// Tree over the 8 warp sums of a 256-thread block (ws[0..8) in shared memory).
__device__ __forceinline__ float tree8(const float* ws)
{
    return __fadd_rn(__fadd_rn(__fadd_rn(ws[0], ws[1]), __fadd_rn(ws[2], ws[3])),
                     __fadd_rn(__fadd_rn(ws[4], ws[5]), __fadd_rn(ws[6], ws[7])));
}

// Combine four sign flags per lane (bit e = coordinate 4*lane + e is negative) of 8
// neighbouring lanes into the 32-bit word that covers coordinates [32w, 32w+32).
__device__ __forceinline__ uint32_t gather_sign_word(uint32_t nib, int lane)
{
    uint32_t w = nib << (4 * (lane & 7));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    return w;
}

// Programmatic dependent launch: a kernel launched with launch_overlapped() may be scheduled
// while the kernel before it on the stream is still draining.  It must call
// wait_for_previous_kernel() before it touches anything that kernel wrote; calling
// allow_next_kernel() lets the one after it be scheduled early in the same way.
__device__ __forceinline__ void wait_for_previous_kernel()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void allow_next_kernel()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// `hot` (optional, base == nullptr for none): a range this launch asks the L2 cache to keep
// resident (a fraction `ratio` of it) while everything else it touches streams through.  A
// per-launch attribute: nothing stays behind on the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t st, HotRange hot, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (hot.base && hot.bytes > 0 && hot.ratio > 0.f) {
        attr[1].id = cudaLaunchAttributeAccessPolicyWindow;
        attr[1].val.accessPolicyWindow.base_ptr = hot.base;
        attr[1].val.accessPolicyWindow.num_bytes = hot.bytes;
        attr[1].val.accessPolicyWindow.hitRatio = hot.ratio;
        attr[1].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        attr[1].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}


// Layered launches.  entry_of_block: the table entry whose blocks include `block`.
__device__ __forceinline__ int entry_of_block(const LayerTable& tab, uint32_t block)
{
    int lo = 0, hi = tab.entries; // first_block[lo] <= block < first_block[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tab.first_block[mid] <= block) lo = mid; else hi = mid;
    }
    return lo;
}
// Copy a layer's parameters from device memory into `sdev` (shared memory); all threads of the
// block call this, it ends with a block barrier.
__device__ __forceinline__ void load_layer_params(const Dev* src, Dev* sdev)
{
    const uint32_t* s = reinterpret_cast<const uint32_t*>(src);
    uint32_t* dst = reinterpret_cast<uint32_t*>(sdev);
    for (unsigned i = threadIdx.x; i < sizeof(Dev) / 4; i += blockDim.x) dst[i] = s[i];
    __syncthreads();
}
// advance the state arrays to a layer's first coordinate
__device__ __forceinline__ void shift_arrays(StepArgs& a, int64_t o)
{
    a.X += o;
    a.Xhat += o;
    a.S += o;
    if (a.G) a.G += o;
    if (a.M) a.M += o;
}

__device__ __forceinline__ uint32_t abs_key(float v)
{
    return __float_as_uint(v) & 0x7FFFFFFFu;
}

} // namespace choco
