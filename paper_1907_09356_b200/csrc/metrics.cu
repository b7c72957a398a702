// Consensus distance of the paper's Section 6, without the 1/n: sum_i ||x_i - xbar||^2,
// accumulated in float64.  Not part of the timed step.
#include "common.cuh"
#include "internal.h"

namespace choco {

__global__ void __launch_bounds__(256) consensus_cols_kernel(const float* X, int32_t n, int64_t d,
                                                             int64_t ld, double* scratch)
{
    __shared__ double red[256];
    const int64_t c = (int64_t)blockIdx.x * 256 + threadIdx.x;
    double acc = 0.0;
    if (c < d) {
        double mean = 0.0;
        for (int32_t i = 0; i < n; ++i) mean += (double)X[(int64_t)i * ld + c];
        mean /= (double)n;
        for (int32_t i = 0; i < n; ++i) {
            const double t = (double)X[(int64_t)i * ld + c] - mean;
            acc += t * t;
        }
    }
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) scratch[blockIdx.x] = red[0];
}

__global__ void __launch_bounds__(1024) consensus_sum_kernel(const double* scratch, int64_t m,
                                                             double* out)
{
    __shared__ double red[1024];
    double acc = 0.0;
    for (int64_t j = threadIdx.x; j < m; j += 1024) acc += scratch[j];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = red[0];
}

cudaError_t launch_consensus(const float* X, int32_t n, int64_t d, int64_t ld, double* scratch,
                             int64_t nblocks, double* out, cudaStream_t st)
{
    consensus_cols_kernel<<<(unsigned)nblocks, 256, 0, st>>>(X, n, d, ld, scratch);
    consensus_sum_kernel<<<1, 1024, 0, st>>>(scratch, nblocks, out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Consensus distance without any allocation (choco_consensus_error_noalloc).
//
// The per-block partial sums of the two kernels above normally live in memory that
// choco_init allocates.  This variant keeps them in a fixed array that is part of the loaded
// library image, so that a caller who must not allocate can still use it.
// ---------------------------------------------------------------------------------------
namespace {

constexpr int64_t kNoAllocMaxBlocks = 16384;                 // 128 KiB of float64 partials
constexpr int64_t kNoAllocMaxD = kNoAllocMaxBlocks * 256;    // 4 194 304 coordinates per worker
constexpr int kNoAllocMaxDevices = 64;

// Scratch shared by every call on a device.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels get the device address looked up below.
static __device__ __align__(256) double g_noalloc_partials[kNoAllocMaxBlocks];

// device address of g_noalloc_partials, looked up once per device
double* g_noalloc_ptr[kNoAllocMaxDevices] = {};

} // namespace
} // namespace choco

extern "C" int choco_consensus_error_noalloc(const float* X, int32_t n, int64_t d, int64_t ld,
                                             double* out_dev, void* stream)
{
    using namespace choco;
    if (!X || !out_dev || n < 1 || d < 1 || ld < d) return CHOCO_ERR_INVALID_ARG;
    if (d > kNoAllocMaxD) return CHOCO_ERR_TOO_LARGE; // the fixed scratch holds one partial per 256 columns
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return CHOCO_ERR_CUDA;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return CHOCO_ERR_TOO_LARGE;
    if (!g_noalloc_ptr[dev]) {
        // first call on this device (it is current): resolve the array's device address
        double* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_partials) != cudaSuccess || !p) return CHOCO_ERR_CUDA;
        g_noalloc_ptr[dev] = p;
    }
    double* scratch = g_noalloc_ptr[dev];
    const int64_t nblocks = (d + 255) / 256;
    cudaStream_t st = (cudaStream_t)stream;
    // every partial that the second kernel reads is written by the first one in this same
    // call, so nothing left over from an earlier call needs clearing
    consensus_cols_kernel<<<(unsigned)nblocks, 256, 0, st>>>(X, n, d, ld, scratch);
    consensus_sum_kernel<<<1, 1024, 0, st>>>(scratch, nblocks, out_dev);
    return cudaGetLastError() == cudaSuccess ? CHOCO_OK : CHOCO_ERR_CUDA;
}
