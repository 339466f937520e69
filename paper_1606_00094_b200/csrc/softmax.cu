// Softmax over the last dimension: out[r][j] = exp(in[r][j]) / sum_i exp(in[r][i]).
// Section 2 of the paper names it, with convolution and pooling, among the operations deployment needs; it is a few
// kilobytes per image at the end of a network, so the kernel is plain: one block per row, the row cached in shared
// memory when it fits (one read of the input), maximum and sum by warp shuffles, fp32 throughout with expf.
#include <cfloat>

#include "boda_internal.h"

namespace boda {
namespace {

constexpr int kThreads = 256;
constexpr int kCacheFloats = 11 * 1024;          // 44 KB of static shared memory

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* scratch)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float w = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, w) : v + w;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                             // scratch may still be read from the previous reduction
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    v = scratch[lane & (kThreads / 32 - 1)];     // every warp reduces the 8 partial values again: same result everywhere
#pragma unroll
    for (int o = kThreads / 64; o > 0; o >>= 1) {
        const float w = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, w) : v + w;
    }
    return v;
}

__global__ void __launch_bounds__(kThreads)
softmax_rows_kernel(const float* __restrict__ in, float* __restrict__ out, int cols)
{
    __shared__ float cache[kCacheFloats];
    __shared__ float scratch[kThreads / 32];
    pdl_launch_dependents();
    const float* x = in + (size_t)blockIdx.x * cols;
    float* y = out + (size_t)blockIdx.x * cols;
    const bool cached = cols <= kCacheFloats;
    pdl_wait();
    float mx = -FLT_MAX;
    for (int j = threadIdx.x; j < cols; j += kThreads) {
        const float v = __ldg(x + j);
        if (cached) cache[j] = v;
        mx = fmaxf(mx, v);
    }
    mx = block_reduce(mx, true, scratch);
    float sum = 0.f;
    for (int j = threadIdx.x; j < cols; j += kThreads) {
        const float e = expf((cached ? cache[j] : __ldg(x + j)) - mx);
        if (cached) cache[j] = e;
        sum += e;
    }
    sum = block_reduce(sum, false, scratch);
    const float inv = 1.f / sum;
    for (int j = threadIdx.x; j < cols; j += kThreads)
        y[j] = (cached ? cache[j] : expf(__ldg(x + j) - mx)) * inv;
}

}  // namespace

int softmax_launch(const float* in, float* out, int rows, int cols, cudaStream_t stream)
{
    BODA_CUDA_TRY(launch_kernel(softmax_rows_kernel, dim3((unsigned)rows), dim3(kThreads), 0, stream, 1, in, out, cols));
    count_launch();
    return BODA_OK;
}

}  // namespace boda
