// DIRECT variant: FP32 CUDA-core convolution, the general fallback (the paper's `conv`, Section 5:
// SGEMM blocking with im2col folded into the shared-memory load) and the small-input-channel path.
//
// Blocking follows the paper's SGEMM template (Section 4, Listing 1 and the parameter list after
// it): each thread owns a register tile of Mt x Nt outputs (here TM pixels x TN output channels),
// a thread block of 256 threads owns Mb*Mt x Nb*Nt = (16*TM) x (16*TN) outputs, the reduction is
// walked in chunks of Kb = 8, operands of a chunk are staged in shared memory and the inner loop
// is fully unrolled.  The gather that im2col would do is a table lookup: entry j of the table
// gives, for reduction index j = (c, r, s), the element offset inside an image and the tap, so the
// load needs no division.  Bias and ReLU are applied in registers before the store.
#include "boda_internal.h"

namespace boda {
namespace {

constexpr int kThreads = 256;
constexpr int BK = 8;

template <int TM, int TN>
__global__ void __launch_bounds__(kThreads)
direct_conv_kernel(const ConvDims d, const float* __restrict__ in, const float* __restrict__ filt,
                   const float* __restrict__ bias, float* __restrict__ out,
                   const DirectTapEntry* __restrict__ tab)
{
    constexpr int BM = 16 * TM;
    constexpr int BN = 16 * TN;
    constexpr int BNP = BN + 4;                       // padded pitch: conflict-free transposed store
    constexpr int A_PER_THREAD = (BK * BM + kThreads - 1) / kThreads;
    constexpr int B_PER_THREAD = (BK * BN + kThreads - 1) / kThreads;
    static_assert(kThreads % BM == 0 || BM % kThreads == 0, "a thread keeps one pixel for all its A loads");

    __shared__ __align__(16) float As[2][BK][BM];
    __shared__ __align__(16) float Bs[2][BK][BNP];

    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x;
    const int tx = tid & 15;                          // pixel group
    const int ty = tid >> 4;                          // channel group
    const int m0 = blockIdx.x * BM;
    const int k0 = blockIdx.y * BN;
    const int PQ = d.P * d.Q;
    const int HW = d.H * d.W;

    // ---- per-thread constants of the A (input) gather: this thread always loads pixel a_m
    const int a_ml = tid % BM;
    const int a_kk0 = tid / BM;                       // first chunk row this thread loads
    constexpr int A_KK_STEP = (kThreads >= BM) ? kThreads / BM : 1;
    int a_y0 = 0, a_x0 = 0;
    long long a_base = 0;
    bool a_ok = false;
    {
        const int m = m0 + a_ml;
        if (m < d.M) {
            const int n = m / PQ;
            const int pq = m - n * PQ;
            const int p = pq / d.Q;
            const int q = pq - p * d.Q;
            a_y0 = p * d.stride - d.pad;
            a_x0 = q * d.stride - d.pad;
            a_base = (long long)n * d.C * HW + (long long)a_y0 * d.W + a_x0;
            a_ok = true;
        }
    }
    // ---- per-thread constants of the B (filter) load
    const int b_kk = tid & (BK - 1);
    const int b_n0 = tid >> 3;                        // 0..31

    float a_pre[A_PER_THREAD];
    float b_pre[B_PER_THREAD];

    auto load_global = [&](int kred0) {
#pragma unroll
        for (int i = 0; i < A_PER_THREAD; ++i) {
            const int kk = a_kk0 + i * A_KK_STEP;
            float v = 0.f;
            if (kk < BK) {
                const DirectTapEntry e = tab[kred0 + kk];
                const int y = a_y0 + (e.rs >> 16);
                const int x = a_x0 + (e.rs & 0xffff);
                if (a_ok && (unsigned)y < (unsigned)d.H && (unsigned)x < (unsigned)d.W)
                    v = __ldg(in + a_base + e.offset);
            }
            a_pre[i] = v;
        }
#pragma unroll
        for (int i = 0; i < B_PER_THREAD; ++i) {
            const int nl = b_n0 + i * 32;
            const int k = k0 + nl;
            const int j = kred0 + b_kk;
            float v = 0.f;
            if (nl < BN && k < d.K && j < d.Kred) v = __ldg(filt + (size_t)k * d.Kred + j);
            b_pre[i] = v;
        }
    };
    auto store_shared = [&](int buf) {
#pragma unroll
        for (int i = 0; i < A_PER_THREAD; ++i) {
            const int kk = a_kk0 + i * A_KK_STEP;
            if (kk < BK) As[buf][kk][a_ml] = a_pre[i];
        }
#pragma unroll
        for (int i = 0; i < B_PER_THREAD; ++i) {
            const int nl = b_n0 + i * 32;
            if (nl < BN) Bs[buf][b_kk][nl] = b_pre[i];
        }
    };

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    const int chunks = (d.Kred + BK - 1) / BK;
    load_global(0);
    store_shared(0);
    __syncthreads();

    for (int t = 0; t < chunks; ++t) {
        const int buf = t & 1;
        if (t + 1 < chunks) load_global((t + 1) * BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
            // pixels of this thread: groups of 4 (or TM if smaller) consecutive, 64 apart
            if constexpr (TM % 4 == 0) {
#pragma unroll
                for (int g = 0; g < TM / 4; ++g) {
                    const float4 v = *reinterpret_cast<const float4*>(&As[buf][kk][g * 64 + tx * 4]);
                    a[4 * g + 0] = v.x; a[4 * g + 1] = v.y; a[4 * g + 2] = v.z; a[4 * g + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < TM; ++i) a[i] = As[buf][kk][tx * TM + i];
            }
            if constexpr (TN % 4 == 0) {
#pragma unroll
                for (int g = 0; g < TN / 4; ++g) {
                    const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][kk][ty * TN + 4 * g]);
                    b[4 * g + 0] = v.x; b[4 * g + 1] = v.y; b[4 * g + 2] = v.z; b[4 * g + 3] = v.w;
                }
            } else if constexpr (TN % 2 == 0) {
#pragma unroll
                for (int g = 0; g < TN / 2; ++g) {
                    const float2 v = *reinterpret_cast<const float2*>(&Bs[buf][kk][ty * TN + 2 * g]);
                    b[2 * g + 0] = v.x; b[2 * g + 1] = v.y;
                }
            } else {
#pragma unroll
                for (int j = 0; j < TN; ++j) b[j] = Bs[buf][kk][ty * TN + j];
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (t + 1 < chunks) store_shared(buf ^ 1);
        __syncthreads();
    }

    // ---- epilogue: bias, ReLU, NCHW store
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int ml = (TM % 4 == 0) ? ((i >> 2) * 64 + tx * 4 + (i & 3)) : (tx * TM + i);
        const int m = m0 + ml;
        if (m >= d.M) continue;
        const int n = m / PQ;
        const int pq = m - n * PQ;
        float* o = out + ((size_t)n * d.K) * PQ + pq;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int k = k0 + ty * TN + j;
            if (k < d.K) {
                float v = acc[i][j] + (bias ? __ldg(bias + k) : 0.f);
                if (d.relu) v = fmaxf(v, 0.f);
                o[(size_t)k * PQ] = v;
            }
        }
    }
}

// ---- the small-input-channel form of DIRECT (first layers: C = 3 with 3x3 ... 11x11 windows; few output channels).
// With C*R*S of a few dozen to a few hundred the GEMM blocking above spends its time on chunk hand-overs; here a
// thread owns ONE output pixel and KT output channels.  A block of 32 x 8 threads covers a 32 x 8 patch of one
// output plane: it stages the input patch with its halo (every channel, coalesced row loads, zeros for the padding)
// and the KT filters in shared memory, then walks the reduction (c, r, s) in order - one shared-memory load of the
// input per step, the KT weights as broadcast 16-byte loads, KT fused multiply-adds - and stores each output
// channel as 128-byte rows.  Such layers move more bytes than they compute (configuration 1: 11 FLOPs per byte), so
// the kernel is meant to run at memory speed.  More than KT output channels: one block per group of KT (grid.z).
// SW > 0 fixes the window width S at compile time (the inner loop then unrolls into loads at constant offsets:
// measured at run-time width, integer address arithmetic took as many issue slots as the multiply-adds, and the
// kernel was bound by instruction issue at 89 %); SW = 0 takes any width.
template <int KT, int SW>
__global__ void __launch_bounds__(256)
direct_pixel_kernel(const ConvDims d, const float* __restrict__ in, const float* __restrict__ filt,
                    const float* __restrict__ bias, float* __restrict__ out, int tiles_x, int ih, int iw, int iwp)
{
    constexpr int PY = 1;                              // output rows per thread (two were slower: half as many blocks to hide the staging latency)
    extern __shared__ __align__(16) float sm[];
    float* s_w = sm;                                   // [Kred][KT]
    float* s_in = sm + (size_t)d.Kred * KT;            // [C][ih][iwp]
    pdl_launch_dependents();
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int bx = blockIdx.x % tiles_x, by = blockIdx.x / tiles_x;
    const int n = blockIdx.y;
    const int kg0 = blockIdx.z * KT;
    pdl_wait();
    // filters of this channel group: s_w[j][k] = filt[kg0 + k][j] (zeros past K); consecutive threads read consecutive j
    for (int idx = threadIdx.x; idx < d.Kred * KT; idx += 256) {
        const int k = idx / d.Kred, j = idx - k * d.Kred;
        s_w[j * KT + k] = (kg0 + k < d.K) ? __ldg(filt + (size_t)(kg0 + k) * d.Kred + j) : 0.f;
    }
    // input patch: rows y0 .. y0 + ih - 1, columns x0 .. x0 + iw - 1 of every channel
    const int y0 = by * (8 * PY) * d.stride - d.pad, x0 = bx * 32 * d.stride - d.pad;
    const float* img = in + (size_t)n * d.C * d.H * d.W;
    for (int row = ty; row < d.C * ih; row += 8) {
        const int c = row / ih, yy = row - c * ih;
        const int y = y0 + yy;
        const bool yin = y >= 0 && y < d.H;
        const float* src = img + ((size_t)c * d.H + (yin ? y : 0)) * d.W;
        float* dst = s_in + (size_t)row * iwp;
        for (int xx = tx; xx < iw; xx += 32) {
            const int x = x0 + xx;
            dst[xx] = (yin && x >= 0 && x < d.W) ? __ldg(src + x) : 0.f;
        }
    }
    __syncthreads();
    float acc[PY][KT];
#pragma unroll
    for (int i = 0; i < PY; ++i)
#pragma unroll
        for (int k = 0; k < KT; ++k) acc[i][k] = 0.f;
    // Shared memory is addressed through 32-bit shared-space addresses and explicit ld.shared instructions, so the
    // reduction loop carries one 32-bit address per operand and nothing else.
    const uint32_t w_base = (uint32_t)__cvta_generic_to_shared(s_w);
    uint32_t a_addr = (uint32_t)__cvta_generic_to_shared(s_in) + 4u * (uint32_t)((ty * d.stride) * iwp + tx * d.stride);
    uint32_t w_addr = w_base;
    auto lds = [](uint32_t addr) { float v; asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr)); return v; };
    auto lds4 = [](uint32_t addr) {
        float4 v;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
        return v;
    };
    auto step = [&](float a0, uint32_t w) {
#pragma unroll
        for (int q = 0; q < KT / 4; ++q) {
            const float4 wv = lds4(w + 16u * q);
            acc[0][4 * q] = fmaf(a0, wv.x, acc[0][4 * q]);
            acc[0][4 * q + 1] = fmaf(a0, wv.y, acc[0][4 * q + 1]);
            acc[0][4 * q + 2] = fmaf(a0, wv.z, acc[0][4 * q + 2]);
            acc[0][4 * q + 3] = fmaf(a0, wv.w, acc[0][4 * q + 3]);
        }
    };
    const int Sw = SW > 0 ? SW : d.S;
    const int rows_total = d.C * d.R;                  // (c, r) pairs: patch row c*ih + r, consecutive filter rows
    const uint32_t row_step = 4u * (uint32_t)iwp;
    const uint32_t c_step = 4u * (uint32_t)((ih - d.R) * iwp);   // from the last window row of a channel to the first of the next
    int r = 0;
    for (int cr = 0; cr < rows_total; ++cr) {
        if constexpr (SW > 0) {
#pragma unroll
            for (int sx = 0; sx < SW; ++sx) step(lds(a_addr + 4u * sx), w_addr + (uint32_t)(sx * KT * 4));
        } else {
            for (int sx = 0; sx < Sw; ++sx) step(lds(a_addr + 4u * (uint32_t)sx), w_addr + (uint32_t)(sx * KT * 4));
        }
        w_addr += (uint32_t)(Sw * KT * 4);
        a_addr += row_step;
        if (++r == d.R) { r = 0; a_addr += c_step; }
    }
    const int q = bx * 32 + tx;
#pragma unroll
    for (int i = 0; i < PY; ++i) {
        const int p = by * (8 * PY) + ty + 8 * i;
        if (p < d.P && q < d.Q) {
            float* o = out + ((size_t)n * d.K * d.P + p) * d.Q + q;
#pragma unroll
            for (int k = 0; k < KT; ++k) {
                if (kg0 + k < d.K) {
                    float v = acc[i][k] + (bias ? __ldg(bias + kg0 + k) : 0.f);
                    if (d.relu) v = fmaxf(v, 0.f);
                    o[(size_t)(kg0 + k) * d.P * d.Q] = v;
                }
            }
        }
    }
}

// geometry of the pixel kernel for a shape; false if the patch does not fit shared memory
bool pixel_geometry(const ConvDims& d, int KT, int* ih, int* iw, int* iwp, size_t* smem)
{
    *ih = 7 * d.stride + d.R;
    *iw = 31 * d.stride + d.S;
    *iwp = *iw | 1;                                         // odd pitch: rows start on different banks
    *smem = ((size_t)d.Kred * KT + (size_t)d.C * *ih * *iwp) * sizeof(float);
    return *smem <= 200 * 1024 && d.Kred <= 4096;
}

template <int KT, int SW>
int launch_pixel_sw(const ConvDims& d, const float* in, const float* filt, const float* bias, float* out, cudaStream_t stream)
{
    int ih, iw, iwp;
    size_t smem;
    if (!pixel_geometry(d, KT, &ih, &iw, &iwp, &smem)) return BODA_ERR_UNSUPPORTED;
    static DeviceSmemLimit limit(48 * 1024);
    BODA_CUDA_TRY(limit.ensure(direct_pixel_kernel<KT, SW>, smem));
    const int tiles_x = (d.Q + 31) / 32, tiles_y = (d.P + 7) / 8;
    dim3 grid(tiles_x * tiles_y, d.N, (d.K + KT - 1) / KT);
    if (grid.y > 65535 || grid.z > 65535) return BODA_ERR_UNSUPPORTED;
    BODA_CUDA_TRY(launch_kernel(direct_pixel_kernel<KT, SW>, grid, dim3(256), smem, stream, 1, d, in, filt, bias, out, tiles_x, ih, iw, iwp));
    count_launch();
    return BODA_OK;
}

template <int KT>
int launch_pixel(const ConvDims& d, const float* in, const float* filt, const float* bias, float* out, cudaStream_t stream)
{
    switch (d.S) {
        case 3: return launch_pixel_sw<KT, 3>(d, in, filt, bias, out, stream);
        case 5: return launch_pixel_sw<KT, 5>(d, in, filt, bias, out, stream);
        case 7: return launch_pixel_sw<KT, 7>(d, in, filt, bias, out, stream);
        case 11: return launch_pixel_sw<KT, 11>(d, in, filt, bias, out, stream);
        default: return launch_pixel_sw<KT, 0>(d, in, filt, bias, out, stream);
    }
}

struct TileInfo { int TM, TN; const char* name; };
constexpr TileInfo kTiles[] = {
    {8, 8, "direct_128x128"}, {8, 6, "direct_128x96"}, {8, 4, "direct_128x64"}, {8, 2, "direct_128x32"},
    {4, 4, "direct_64x64"},   {4, 2, "direct_64x32"},  {4, 1, "direct_64x16"},  {2, 2, "direct_32x32"},
    {2, 1, "direct_32x16"},
    // pixel-per-thread form (TM = 0): TN output channels per thread
    {0, 8, "direct_pixel_k8"}, {0, 16, "direct_pixel_k16"}, {0, 32, "direct_pixel_k32"},
    // the same form compiled at run time for the exact shape (TM = -1; direct_rtc.cu)
    {-1, 4, "direct_rtc_k4"}, {-1, 8, "direct_rtc_k8"}, {-1, 16, "direct_rtc_k16"}, {-1, 32, "direct_rtc_k32"},
};
constexpr int kFirstPixelTile = 9;
constexpr int kFirstRtcTile = 12;
constexpr int kNumTiles = sizeof(kTiles) / sizeof(kTiles[0]);

template <int TM, int TN>
int launch_tile(const ConvDims& d, const float* in, const float* filt, const float* bias, float* out,
                const DirectTapEntry* tab, cudaStream_t stream)
{
    constexpr int BM = 16 * TM, BN = 16 * TN;
    dim3 grid((d.M + BM - 1) / BM, (d.K + BN - 1) / BN);
    BODA_CUDA_TRY(launch_kernel(direct_conv_kernel<TM, TN>, grid, dim3(kThreads), 0, stream, 1, d, in, filt, bias, out, tab));
    count_launch();
    return BODA_OK;
}

}  // namespace

int direct_num_tiles() { return kNumTiles; }
const char* direct_tile_name(int id) { return (id >= 0 && id < kNumTiles) ? kTiles[id].name : "?"; }

int direct_pick_tile(const ConvDims& d)
{
    // Rule of thumb in the spirit of Section 4: the widest channel tile that K fills without much
    // waste, then the tallest pixel tile that still yields about two blocks per SM.
    int best = kNumTiles - 1;
    double best_cost = 1e300;
    // small reductions with few output channels: the pixel-per-thread form, the smallest KT that covers K in one group
    // (or 32 channels per group)
    // (measured: it wins from a few ten thousand output pixels on - 19 us against 33 us for configuration 1's shape at
    // batch 256 - and loses below, where a handful of blocks cannot hide its two staging phases)
    if (d.Kred <= 512 && d.K <= 128 && d.M >= 32768) {
        const int KT = d.K <= 8 ? 8 : d.K <= 16 ? 16 : 32;
        int ih, iw, iwp;
        size_t smem;
        if (pixel_geometry(d, KT, &ih, &iw, &iwp, &smem)) return kFirstPixelTile + (KT == 8 ? 0 : KT == 16 ? 1 : 2);
    }
    for (int t = 0; t < kFirstPixelTile; ++t) {
        const int BM = 16 * kTiles[t].TM, BN = 16 * kTiles[t].TN;
        const long long gm = (d.M + BM - 1) / BM, gn = (d.K + BN - 1) / BN;
        const double padded = (double)gm * BM * gn * BN;             // FMAs issued per reduction step
        const double blocks = (double)gm * gn;
        const double waves = blocks / (148.0 * 2.0);
        const double fill = waves < 1.0 ? 1.0 / waves : (double)(long long)(waves + 0.999) / waves;
        // small register tiles pay more shared-memory traffic per FMA
        const double ldst = 1.0 + 0.5 * (1.0 / kTiles[t].TM + 1.0 / kTiles[t].TN);
        const double cost = padded * fill * ldst;
        if (cost < best_cost) { best_cost = cost; best = t; }
    }
    return best;
}

bool direct_tile_legal(const ConvDims& d, int tile_id)
{
    if (tile_id < 0 || tile_id >= kNumTiles) return false;
    if (tile_id < kFirstPixelTile) return true;
    if (tile_id >= kFirstRtcTile) {
        int bx, by, py;
        size_t sm;
        return direct_rtc_available() && direct_rtc_geometry(d, kTiles[tile_id].TN, &bx, &by, &py, &sm);
    }
    int ih, iw, iwp;
    size_t smem;
    return pixel_geometry(d, kTiles[tile_id].TN, &ih, &iw, &iwp, &smem) && d.N <= 65535 && (d.K + kTiles[tile_id].TN - 1) / kTiles[tile_id].TN <= 65535;
}

int direct_tile_rtc_kt(int tile_id) { return (tile_id >= kFirstRtcTile && tile_id < kNumTiles) ? kTiles[tile_id].TN : 0; }

int direct_rtc_pick(const ConvDims& d)
{
    // Measured on B200 (configuration 1's layer at batch 1 / 20 / 256, an 11x11 stride-4 and a 5x5 layer on 3 channels):
    // the run-time compiled kernel beats every precompiled tile where the reduction is short and the output channels
    // few.  Eight channels per thread as a rule; four where that leaves fewer than 64 blocks (more blocks hide the
    // staging latency); sixteen where 16 covers all output channels of a large layer (the input patch is staged once).
    if (d.Kred > 512 || d.K > 128 || !direct_rtc_available()) return -1;
    int bx = 32, by = 8, py = 1;
    size_t sm = 0;
    if (!direct_rtc_geometry(d, 8, &bx, &by, &py, &sm)) bx = 8, by = 4, py = 1;
    const long long blocks8 = (long long)((d.Q + bx - 1) / bx) * ((d.P + by * py - 1) / (by * py)) * d.N * ((d.K + 7) / 8);
    const int want = (d.K <= 16 && d.M >= 16384) ? 16 : blocks8 < 64 ? 4 : 8;
    const int order[3][3] = {{4, 8, 16}, {8, 4, 16}, {16, 8, 4}};
    const int* o = order[want == 4 ? 0 : want == 8 ? 1 : 2];
    for (int i = 0; i < 3; ++i)
        for (int t = kFirstRtcTile; t < kNumTiles; ++t)
            if (kTiles[t].TN == o[i] && direct_tile_legal(d, t)) return t;
    return -1;
}

int direct_table_len(const ConvDims& d) { return ((d.Kred + BK - 1) / BK) * BK; }

void direct_build_table(const ConvDims& d, DirectTapEntry* tab)
{
    const int len = direct_table_len(d);
    int j = 0;
    for (int c = 0; c < d.C; ++c)
        for (int r = 0; r < d.R; ++r)
            for (int s = 0; s < d.S; ++s, ++j) {
                tab[j].offset = c * d.H * d.W + r * d.W + s;
                tab[j].rs = (r << 16) | s;
            }
    for (; j < len; ++j) { tab[j].offset = 0; tab[j].rs = (0x4000 << 16); }
}

int direct_launch(const ConvDims& d, int tile_id, const float* in, const float* filt, const float* bias,
                  float* out, const DirectTapEntry* tab, cudaStream_t stream)
{
    switch (tile_id) {
        case 0: return launch_tile<8, 8>(d, in, filt, bias, out, tab, stream);
        case 1: return launch_tile<8, 6>(d, in, filt, bias, out, tab, stream);
        case 2: return launch_tile<8, 4>(d, in, filt, bias, out, tab, stream);
        case 3: return launch_tile<8, 2>(d, in, filt, bias, out, tab, stream);
        case 4: return launch_tile<4, 4>(d, in, filt, bias, out, tab, stream);
        case 5: return launch_tile<4, 2>(d, in, filt, bias, out, tab, stream);
        case 6: return launch_tile<4, 1>(d, in, filt, bias, out, tab, stream);
        case 7: return launch_tile<2, 2>(d, in, filt, bias, out, tab, stream);
        case 8: return launch_tile<2, 1>(d, in, filt, bias, out, tab, stream);
        case 9: return launch_pixel<8>(d, in, filt, bias, out, stream);
        case 10: return launch_pixel<16>(d, in, filt, bias, out, stream);
        case 11: return launch_pixel<32>(d, in, filt, bias, out, stream);
        default: return BODA_ERR_UNSUPPORTED;
    }
}

}  // namespace boda
