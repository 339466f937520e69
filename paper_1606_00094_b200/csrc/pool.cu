// Max-pooling (ksz x ksz window, stride, no padding, floor extent) on NCHW fp32.  Bandwidth-bound.
#include <cstdlib>
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

// staged -> staged: one thread per output pixel and group of 4 channels (16-byte loads and stores, coalesced).
// KSZ / STRIDE > 0 fix the window at compile time (all its loads are then in flight together); 0 takes the run-time
// values.  Index arithmetic is 32-bit: the launcher refuses tensors of 2^31 elements or more.
template <int KSZ, int STRIDE>
__global__ void __launch_bounds__(256)
maxpool_packed_kernel(const float* __restrict__ in, float* __restrict__ out, int N, int iHp, int iWp, int iCp, int P, int Q,
                      int ksz_rt, int stride_rt, int oHp, int oWp, int oCp, int Cq)
{
    const int ksz = KSZ > 0 ? KSZ : ksz_rt, stride = STRIDE > 0 ? STRIDE : stride_rt;
    pdl_launch_dependents();
    const int total = N * P * Q * Cq;
    const int iC4 = iCp >> 2, oC4 = oCp >> 2;
    pdl_wait();
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cq = idx % Cq;
        int t = idx / Cq;
        const int q = t % Q; t /= Q;
        const int p = t % P;
        const int n = t / P;
        const float4* src = reinterpret_cast<const float4*>(in) + ((n * iHp + p * stride) * iWp + q * stride) * iC4 + cq;
        float4 best = __ldg(src);
        if constexpr (KSZ > 0) {
            float4 v[KSZ > 0 ? KSZ * KSZ : 1];
#pragma unroll
            for (int r = 0; r < KSZ; ++r)
#pragma unroll
                for (int s2 = 0; s2 < KSZ; ++s2) v[r * KSZ + s2] = __ldg(src + (r * iWp + s2) * iC4);
#pragma unroll
            for (int j = 0; j < KSZ * KSZ; ++j) {
                best.x = fmaxf(best.x, v[j].x); best.y = fmaxf(best.y, v[j].y);
                best.z = fmaxf(best.z, v[j].z); best.w = fmaxf(best.w, v[j].w);
            }
        } else {
            for (int r = 0; r < ksz; ++r)
                for (int s2 = 0; s2 < ksz; ++s2) {
                    const float4 v = __ldg(src + (r * iWp + s2) * iC4);
                    best.x = fmaxf(best.x, v.x); best.y = fmaxf(best.y, v.y); best.z = fmaxf(best.z, v.z); best.w = fmaxf(best.w, v.w);
                }
        }
        reinterpret_cast<float4*>(out)[((n * oHp + p) * oWp + q) * oC4 + cq] = best;
    }
}

// staged -> NCHW: a block takes one (image, output row) pair and 32 channels; warp w takes output columns
// w, w + 8, ... with its lanes along the channels (coalesced loads), and the block stores its 32 x 8 results through
// shared memory so that consecutive threads write consecutive columns of a channel.
template <int KSZ, int STRIDE>
__global__ void __launch_bounds__(256)
maxpool_packed_to_nchw_kernel(const float* __restrict__ in, float* __restrict__ out, int N, int C, int iHp, int iWp, int iCp,
                              int P, int Q, int ksz_rt, int stride_rt)
{
    const int ksz = KSZ > 0 ? KSZ : ksz_rt, stride = STRIDE > 0 ? STRIDE : stride_rt;
    __shared__ float tile[32][9];
    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = blockIdx.x / P, p = blockIdx.x - n * P;
    const int c0 = blockIdx.y * 32, c = c0 + lane;
    const int cn = min(32, C - c0);
    const float* row0 = in + (size_t)((n * iHp + p * stride) * iWp) * iCp + c;
    pdl_wait();
    for (int q0 = 0; q0 < Q; q0 += 8) {
        const int q = q0 + warp;
        if (q < Q && c < C) {
            const float* src = row0 + (size_t)(q * stride) * iCp;
            float best = __ldg(src);
            if constexpr (KSZ > 0) {
                float v[KSZ > 0 ? KSZ * KSZ : 1];
#pragma unroll
                for (int r = 0; r < KSZ; ++r)
#pragma unroll
                    for (int s2 = 0; s2 < KSZ; ++s2) v[r * KSZ + s2] = __ldg(src + (r * iWp + s2) * iCp);
#pragma unroll
                for (int j = 0; j < KSZ * KSZ; ++j) best = fmaxf(best, v[j]);
            } else {
                for (int r = 0; r < ksz; ++r)
                    for (int s2 = 0; s2 < ksz; ++s2) best = fmaxf(best, __ldg(src + (r * iWp + s2) * iCp));
            }
            tile[lane][warp] = best;
        }
        __syncthreads();
        const int qn = min(8, Q - q0);
        for (int j = threadIdx.x; j < cn * qn; j += 256) {
            const int ci = j / qn, qi = j - ci * qn;
            out[(((size_t)n * C + c0 + ci) * P + p) * Q + q0 + qi] = tile[ci][qi];
        }
        __syncthreads();
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
    if ((long long)N * iHp * iWp * iCp >= (1LL << 31) || (long long)N * C * H * W >= (1LL << 31)) return BODA_ERR_TOO_LARGE;
    const bool k3s2 = ksz == 3 && stride == 2;
    if (out_packed) {
        const int Cq = (iCp < oCp ? iCp : oCp) / 4;
        const long long total = (long long)N * P * Q * Cq;
        // one output item per thread: a second trip round the grid-stride loop costs another full load latency
        // (measured on the stack: 1.5 us per step against a grid capped at eight blocks per SM)
        const long long blocks = (total + 255) / 256;
        auto kernel = k3s2 ? maxpool_packed_kernel<3, 2> : maxpool_packed_kernel<0, 0>;
        BODA_CUDA_TRY(launch_kernel(kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 1, in, out, N, iHp, iWp, iCp,
                                    P, Q, ksz, stride, oHp, oWp, oCp, Cq));
    } else {
        auto kernel = k3s2 ? maxpool_packed_to_nchw_kernel<3, 2> : maxpool_packed_to_nchw_kernel<0, 0>;
        BODA_CUDA_TRY(launch_kernel(kernel, dim3((unsigned)(N * P), (unsigned)((C + 31) / 32)), dim3(256), 0, stream, 1,
                                    in, out, N, C, iHp, iWp, iCp, P, Q, ksz, stride));
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
        static DeviceSmemLimit limit(48 * 1024);
        BODA_CUDA_TRY(limit.ensure(maxpool_plane_kernel, smem));
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
