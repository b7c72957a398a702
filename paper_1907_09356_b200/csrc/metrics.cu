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

} // namespace choco
