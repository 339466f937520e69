// Max-pooling (ksz x ksz window, stride, no padding, floor extent) on NCHW fp32.  Bandwidth-bound.
#include "boda_internal.h"

namespace boda {
namespace {

// A block of 256 threads takes a group of G consecutive planes (contiguous in memory, like their outputs):
// coalesced load of the whole group into shared memory, windows evaluated from there, coalesced store.
__global__ void __launch_bounds__(256)
maxpool_plane_kernel(const float* __restrict__ in, float* __restrict__ out, int NC, int H, int W, int P, int Q,
                     int ksz, int stride, int G)
{
    extern __shared__ float sm_plane[];                 // G planes of H*W floats
    pdl_launch_dependents();
    pdl_wait();
    const int HW = H * W, PQ = P * Q;
    const int g0 = blockIdx.x * G;
    const int count = min(G, NC - g0);
    const float* src = in + (size_t)g0 * HW;
    const int n_in = count * HW;
    for (int i = threadIdx.x; i < n_in; i += 256) sm_plane[i] = __ldg(src + i);
    __syncthreads();
    float* dst = out + (size_t)g0 * PQ;
    const int n_out = count * PQ;
    for (int o = threadIdx.x; o < n_out; o += 256) {
        const int pl = o / PQ;
        const int rem = o - pl * PQ;
        const int p = rem / Q;
        const int q = rem - p * Q;
        const float* w0 = sm_plane + pl * HW + (p * stride) * W + q * stride;
        float best = w0[0];
        for (int r = 0; r < ksz; ++r)
            for (int s = 0; s < ksz; ++s) best = fmaxf(best, w0[r * W + s]);
        dst[o] = best;
    }
}

// fallback for planes that do not fit shared memory: one thread per output element
__global__ void __launch_bounds__(256)
maxpool_kernel(const float* __restrict__ in, float* __restrict__ out, int NC, int H, int W, int P, int Q,
               int ksz, int stride)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)NC * P * Q;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int q = (int)(idx % Q);
        const long long t = idx / Q;
        const int p = (int)(t % P);
        const long long nc = t / P;
        const float* src = in + (nc * H + (long long)p * stride) * W + (long long)q * stride;
        float best = src[0];
        for (int r = 0; r < ksz; ++r)
            for (int s = 0; s < ksz; ++s) best = fmaxf(best, __ldg(src + r * W + s));
        out[idx] = best;
    }
}

}  // namespace

int maxpool_launch(const float* in, float* out, int N, int C, int H, int W, int ksz, int stride,
                   cudaStream_t stream)
{
    const int P = boda_conv_out_dim(H, ksz, stride, 0);
    const int Q = boda_conv_out_dim(W, ksz, stride, 0);
    const int NC = N * C;
    int G = 2048 / (H * W);
    if (G < 1) G = 1;
    const size_t smem = (size_t)G * H * W * sizeof(float);
    if (smem <= 96 * 1024) {
        static size_t attr_smem = 48 * 1024;
        if (smem > attr_smem) {
            BODA_CUDA_TRY(cudaFuncSetAttribute(maxpool_plane_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            attr_smem = smem;
        }
        const int blocks = (NC + G - 1) / G;
        BODA_CUDA_TRY(launch_kernel(maxpool_plane_kernel, dim3(blocks), dim3(256), smem, stream, 1, in, out, NC, H, W, P, Q, ksz, stride, G));
    } else {
        const long long total = (long long)NC * P * Q;
        long long blocks = (total + 255) / 256;
        if (blocks > 148LL * 16) blocks = 148LL * 16;
        BODA_CUDA_TRY(launch_kernel(maxpool_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 1, in, out, NC, H, W, P, Q, ksz, stride));
    }
    BODA_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BODA_OK;
}

}  // namespace boda
