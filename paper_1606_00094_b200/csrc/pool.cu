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

// ---- the same pooling on the staged activation layout of chained tensor-core layers:
// rows [(n*Hp + y)*Wp + x][Cp], channels innermost (Cp a multiple of 32), padding rows / columns / channels zero.
// Max-pooling commutes with the rounding to TF32 that the producer already applied, so values pass through as is.

// staged -> staged: one thread per output pixel and group of 4 channels (16-byte loads and stores, coalesced)
__global__ void __launch_bounds__(256)
maxpool_packed_kernel(const float* __restrict__ in, float* __restrict__ out, int N, int iHp, int iWp, int iCp, int P, int Q,
                      int ksz, int stride, int oHp, int oWp, int oCp, int Cq)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)N * P * Q * Cq;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int cq = (int)(idx % Cq);
        long long t = idx / Cq;
        const int q = (int)(t % Q); t /= Q;
        const int p = (int)(t % P);
        const int n = (int)(t / P);
        const float4* src = reinterpret_cast<const float4*>(in + (((size_t)n * iHp + (size_t)p * stride) * iWp + (size_t)q * stride) * iCp) + cq;
        float4 best = __ldg(src);
        for (int r = 0; r < ksz; ++r)
            for (int s = 0; s < ksz; ++s) {
                const float4 v = __ldg(src + ((size_t)r * iWp + s) * (iCp / 4));
                best.x = fmaxf(best.x, v.x); best.y = fmaxf(best.y, v.y); best.z = fmaxf(best.z, v.z); best.w = fmaxf(best.w, v.w);
            }
        reinterpret_cast<float4*>(out + (((size_t)n * oHp + p) * oWp + q) * oCp)[cq] = best;
    }
}

// staged -> NCHW: one thread per output element, channels fastest so that the loads coalesce
__global__ void __launch_bounds__(256)
maxpool_packed_to_nchw_kernel(const float* __restrict__ in, float* __restrict__ out, int N, int C, int iHp, int iWp, int iCp,
                              int P, int Q, int ksz, int stride)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)N * P * Q * C;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % C);
        long long t = idx / C;
        const int q = (int)(t % Q); t /= Q;
        const int p = (int)(t % P);
        const int n = (int)(t / P);
        const float* src = in + (((size_t)n * iHp + (size_t)p * stride) * iWp + (size_t)q * stride) * iCp + c;
        float best = __ldg(src);
        for (int r = 0; r < ksz; ++r)
            for (int s = 0; s < ksz; ++s) best = fmaxf(best, __ldg(src + ((size_t)r * iWp + s) * iCp));
        out[(((size_t)n * C + c) * P + p) * Q + q] = best;
    }
}

// staged -> NCHW copy (used to inspect an intermediate activation of a chain)
__global__ void __launch_bounds__(256)
unpack_to_nchw_kernel(const float* __restrict__ in, float* __restrict__ out, int N, int C, int H, int W, int Hp, int Wp, int Cp)
{
    const long long total = (long long)N * C * H * W;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int x = (int)(idx % W);
        long long t = idx / W;
        const int y = (int)(t % H); t /= H;
        const int c = (int)(t % C);
        const int n = (int)(t / C);
        out[idx] = in[(((size_t)n * Hp + y) * Wp + x) * Cp + c];
    }
}

}  // namespace

int maxpool_packed_launch(const float* in, float* out, int N, int C, int H, int W, int iHp, int iWp, int iCp, int ksz, int stride,
                          int out_packed, int oHp, int oWp, int oCp, cudaStream_t stream)
{
    const int P = boda_conv_out_dim(H, ksz, stride, 0);
    const int Q = boda_conv_out_dim(W, ksz, stride, 0);
    if (out_packed) {
        const int Cq = (iCp < oCp ? iCp : oCp) / 4;
        const long long total = (long long)N * P * Q * Cq;
        long long blocks = (total + 255) / 256;
        if (blocks > 148LL * 8) blocks = 148LL * 8;
        BODA_CUDA_TRY(launch_kernel(maxpool_packed_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 1, in, out, N, iHp, iWp, iCp,
                                    P, Q, ksz, stride, oHp, oWp, oCp, Cq));
    } else {
        const long long total = (long long)N * P * Q * C;
        long long blocks = (total + 255) / 256;
        if (blocks > 148LL * 8) blocks = 148LL * 8;
        BODA_CUDA_TRY(launch_kernel(maxpool_packed_to_nchw_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 1, in, out, N, C,
                                    iHp, iWp, iCp, P, Q, ksz, stride));
    }
    count_launch();
    return BODA_OK;
}

int unpack_to_nchw_launch(const float* in, float* out, int N, int C, int H, int W, int Hp, int Wp, int Cp, cudaStream_t stream)
{
    const long long total = (long long)N * C * H * W;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    unpack_to_nchw_kernel<<<(unsigned)blocks, 256, 0, stream>>>(in, out, N, C, H, W, Hp, Wp, Cp);
    BODA_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BODA_OK;
}

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
