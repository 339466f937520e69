// Max-pooling (ksz x ksz window, stride, no padding, floor extent) on NCHW fp32.  Bandwidth-bound:
// one thread per output element, consecutive threads on consecutive output columns.
#include "boda_internal.h"

namespace boda {
namespace {

__global__ void __launch_bounds__(256)
maxpool_kernel(const float* __restrict__ in, float* __restrict__ out, int NC, int H, int W, int P, int Q,
               int ksz, int stride)
{
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
    const long long total = (long long)N * C * P * Q;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    maxpool_kernel<<<(unsigned)blocks, 256, 0, stream>>>(in, out, N * C, H, W, P, Q, ksz, stride);
    count_launch();
    BODA_CUDA_TRY(cudaGetLastError());
    return BODA_OK;
}

}  // namespace boda
