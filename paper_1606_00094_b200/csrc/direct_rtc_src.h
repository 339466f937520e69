// Source text of the run-time-compiled form of DIRECT (compiled by NVRTC in direct_rtc.cu, once per plan).
//
// Section 4 of the paper: the kernels are generated for the exact problem at run time, so that every extent is a
// literal - index arithmetic folds into constants, loops unroll, bounds tests that cannot fail disappear.  This is
// the pixel-per-thread kernel of direct_conv.cu written that way: all of N, C, H, W, K, R, S, stride, pad, ReLU, the
// output extents and the blocking (BX x BY threads per block, PY output rows and KT output channels per thread: a
// block covers BX x (BY*PY) output pixels) arrive as -D macros; the pointers are the only run-time arguments.
#pragma once

namespace boda {

static const char kDirectRtcSource[] = R"rtc(
extern "C" __global__ void __launch_bounds__(BX * BY)
boda_direct_rtc(const float* __restrict__ in, const float* __restrict__ filt, const float* __restrict__ bias,
                float* __restrict__ out)
{
    constexpr int NT = BX * BY;
    constexpr int IH = (BY * PY - 1) * STRIDE + R, IW = (BX - 1) * STRIDE + S, IWP = IW | 1;   // odd pitch: rows on different banks
    constexpr int KRED = C * R * S;
    constexpr int TILES_X = (Q + BX - 1) / BX;
    __shared__ __align__(16) float s_w[KRED * KT];          // [c][r][s][KT]
    __shared__ float s_in[C * IH * IWP];                    // [c][IH][IWP]
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tx = threadIdx.x % BX, ty = threadIdx.x / BX;
    const int bx = blockIdx.x % TILES_X, by = blockIdx.x / TILES_X;
    const int n = blockIdx.y;
    const int kg0 = blockIdx.z * KT;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // filters of this channel group: s_w[j][k] = filt[kg0 + k][j] (zeros past K); consecutive threads read consecutive j
    for (int idx = threadIdx.x; idx < KRED * KT; idx += NT) {
        const int k = idx / KRED, j = idx - k * KRED;
        s_w[j * KT + k] = (K % KT == 0 || kg0 + k < K) ? __ldg(filt + (kg0 + k) * KRED + j) : 0.f;
    }
    // input patch with its halo, zeros for the padding
    const int y0 = by * (BY * PY) * STRIDE - PAD, x0 = bx * BX * STRIDE - PAD;
    const float* img = in + (size_t)n * (C * H * W);
    for (int idx = threadIdx.x; idx < C * IH * IW; idx += NT) {
        const int c = idx / (IH * IW), rem = idx - c * (IH * IW);
        const int yy = rem / IW, xx = rem - yy * IW;
        const int y = y0 + yy, x = x0 + xx;
        const bool inside = (unsigned)y < (unsigned)H && (unsigned)x < (unsigned)W;
        s_in[(c * IH + yy) * IWP + xx] = inside ? __ldg(img + (c * H + y) * W + x) : 0.f;
    }
    __syncthreads();
    // thread (tx, ty) owns output rows ty, ty + BY, ... (PY of them): the weights of a tap are loaded once for all
    float acc[PY][KT];
#pragma unroll
    for (int i = 0; i < PY; ++i)
#pragma unroll
        for (int k = 0; k < KT; ++k) acc[i][k] = 0.f;
    const float* a_base = s_in + (ty * STRIDE) * IWP + tx * STRIDE;
#pragma unroll UNROLL_C
    for (int c = 0; c < C; ++c) {
#pragma unroll UNROLL_R
        for (int r = 0; r < R; ++r) {
#pragma unroll
            for (int s = 0; s < S; ++s) {
                float a[PY];
#pragma unroll
                for (int i = 0; i < PY; ++i) a[i] = a_base[(c * IH + i * BY * STRIDE + r) * IWP + s];
                const float4* w4 = reinterpret_cast<const float4*>(s_w + ((c * R + r) * S + s) * KT);
#pragma unroll
                for (int q4 = 0; q4 < KT / 4; ++q4) {
                    const float4 wv = w4[q4];
#pragma unroll
                    for (int i = 0; i < PY; ++i) {
                        acc[i][4 * q4] = fmaf(a[i], wv.x, acc[i][4 * q4]);
                        acc[i][4 * q4 + 1] = fmaf(a[i], wv.y, acc[i][4 * q4 + 1]);
                        acc[i][4 * q4 + 2] = fmaf(a[i], wv.z, acc[i][4 * q4 + 2]);
                        acc[i][4 * q4 + 3] = fmaf(a[i], wv.w, acc[i][4 * q4 + 3]);
                    }
                }
            }
        }
    }
    const int q = bx * BX + tx;
#pragma unroll
    for (int i = 0; i < PY; ++i) {
        const int p = by * (BY * PY) + i * BY + ty;
        if ((P % (BY * PY) == 0 || p < P) && (Q % BX == 0 || q < Q)) {
            float* o = out + ((size_t)n * K + kg0) * (P * Q) + p * Q + q;
#pragma unroll
            for (int k = 0; k < KT; ++k) {
                if (K % KT == 0 || kg0 + k < K) {
                    float v = acc[i][k] + (bias ? __ldg(bias + kg0 + k) : 0.f);
                    if (RELU) v = fmaxf(v, 0.f);
                    o[k * (P * Q)] = v;
                }
            }
        }
    }
}
)rtc";

}  // namespace boda
