// TCONV for first layers: 3 input channels, stride 4 (the 11x11 / stride-4 layer of the AlexNet-shaped stack),
// straight from the NCHW input - no staged copy of the input at all.
//
// The paper's tconv needs "an input transformation" (Section 5).  For a stride-4 layer that transformation is the
// space-to-depth view: stride 4 on 3 channels = stride 1 on 48 channels with ceil(R/4) x ceil(S/4) taps, where
// channel (c, dy, dx) of block (yb, xb) is input pixel (4*yb + dy, 4*xb + dx) of channel c.  The other kernels read
// that view from a staged tensor a separate kernel wrote; here the CTA builds its own piece of the view in shared memory:
//
//   * A tile is 512 flat positions of the view starting at an output row of ONE image (rows_per_tile rows further
//     for every tile; the rows past that belong to the next tile and are only kept for the fused pooling).  The input
//     rows it needs - raw_rows consecutive rows of each channel - are contiguous in NCHW, so ONE bulk copy per channel
//     brings them into shared memory as they lie (source rounded down to 16 bytes; rows of 227 floats start anywhere).
//   * The four floats dx = 0..3 of a (c, dy) pair are consecutive in an input row: exactly one 16-byte piece of a
//     position's K-major row.  The eight epilogue warps, idle during the main loop, realign them: one shared-memory
//     load and one swizzled store per float, rounded to TF32.  With the channel order (c, dy, dx), chunk 0 (32
//     channels) is channels 0 and 1 and chunk 1 is channel 2: 16 channels, stored as 64-byte rows (64-byte swizzle),
//     so the padded half of the second chunk costs neither shared memory nor MMAs (6 instead of 8 MMAs per tap and
//     accumulator; the staged view padded 48 channels to 64).
//   * Chunk 1 is loaded and built while the tensor cores work on chunk 0: raw rows of channel 2 reuse the buffer of
//     channel 0, and its slab reuses the buffer of channel 1.
//
// Everything else is the halo kernel (tconv_halo.cuh): taps are MMAs whose A descriptor starts (r*Wp + s) rows into
// the slab, four 128-row accumulators with one issuing thread each, filter tiles by TMA, the same epilogues (plain,
// or fused ReLU -> max-pool).  Roles (416 threads): warp 0 = filter-tile producer; warps 1, 6, 11, 12 = MMA issuers;
// warps 2..5 and 7..10 = slab builders, then epilogue.  Waits are bounded as everywhere.
#pragma once

#include "tconv_halo.cuh"

namespace boda {
namespace first {

using namespace tc;

constexpr int kThreads = 416;
constexpr int NACC = 4;
constexpr int kStride = 4;
constexpr int kChannels = 3;
constexpr int kViewChannels = kChannels * kStride * kStride;     // 48

struct FirstParams {
    halo::HaloParams h;          // view geometry (Mflat, HpWp, Wp, S = taps per row, taps), bias, output, pooling, status
    const float* in;             // NCHW input [N][3][H][W]
    int H, W;
    int rows_per_tile;           // output rows between two tile starts
    int raw_rows;                // input rows of one channel that a tile reads
    int raw_buf_bytes;           // one raw-row buffer (also holds the 64-byte-row slab of chunk 1); multiple of 1024
    int slab_rows;               // rows of a slab: 512 + (Rb-1)*Wp + Sb-1, rounded up to 8
    int b_stages;
    long long in_floats;         // N*3*H*W
};

// global -> shared bulk copy, bytes counted on the mbarrier; addresses and size are multiples of 16 bytes
__device__ __forceinline__ void bulk_load_global(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// K-major tile with 64-byte rows (16 TF32 values), 64-byte swizzle, 8-row groups 512 bytes apart
__device__ __forceinline__ uint64_t smem_desc_k_sw64(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
tconv_first_layer_kernel(const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
                         const FirstParams p)
{
    constexpr int B_STAGE_BYTES = BN * 128;
    constexpr int ACC_COLS = BN * NACC;
    constexpr int TMEM_COLS = ACC_COLS <= 256 ? 256 : 512;
    static_assert(ACC_COLS <= 512, "accumulators exceed tensor memory");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t slab0 = smem_base;                                      // [slab_rows][128 bytes], 128-byte swizzle
    const uint32_t raw0 = slab0 + (uint32_t)p.slab_rows * 128u;            // raw rows of channel 0, later of channel 2
    const uint32_t raw1 = raw0 + (uint32_t)p.raw_buf_bytes;                // raw rows of channel 1, later slab 1
    const uint32_t slab1 = raw1;                                           // [slab_rows][64 bytes], 64-byte swizzle
    const uint32_t smem_b = raw1 + (uint32_t)p.raw_buf_bytes;
    const uint32_t bars = smem_b + (uint32_t)p.b_stages * B_STAGE_BYTES;
    const uint32_t raw_full = bars;                    // 3 x 8 bytes: channels 0, 1, 2
    const uint32_t slab_full = bars + 24;              // 2 x 8
    const uint32_t b_full = bars + 40, b_empty = b_full + 8 * halo::kMaxBStages;
    const uint32_t accum_bar = b_empty + 8 * halo::kMaxBStages;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ __align__(16) float s_bias[BN];

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n = (int)blockIdx.x / p.h.tiles_per_image;
    const int j = (int)blockIdx.x - n * p.h.tiles_per_image;
    const int row_first = p.rows_per_tile * j;                   // first output row (= first block row) of the tile
    const int f0 = n * p.h.HpWp + row_first * p.h.Wp;
    const int y0 = kStride * row_first;                          // first input row
    const int k0 = blockIdx.y * BN;
    const int taps = p.h.taps;

    pdl_launch_dependents();
    if (threadIdx.x == 64) FL_STAMP(0);
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int c = 0; c < 3; ++c) mbar_init(raw_full + 8 * c, 1);
        for (int c = 0; c < 2; ++c) mbar_init(slab_full + 8 * c, 8);            // one arrival per builder warp
        for (int s = 0; s < p.b_stages; ++s) { mbar_init(b_full + 8 * s, 1); mbar_init(b_empty + 8 * s, NACC); }
        mbar_init(accum_bar, NACC);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_b0);
        prefetch_tensormap(&map_b1);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = s_tmem_base;
    pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- filter tiles: taps of chunk 0 (32 channels, 128-byte rows), then of chunk 1 (16 channels,
            // 64-byte rows); one ring of b_stages slots of BN*128 bytes for both
            uint32_t stage = 0, par = 1;
            for (int i = 0; i < 2 * taps; ++i) {
                if (!mbar_wait(b_empty + 8 * stage, par, &s_abort, p.h.status, 52)) break;
                const bool second = i >= taps;
                const uint32_t bytes = second ? (uint32_t)(BN * 64) : (uint32_t)B_STAGE_BYTES;
                mbar_expect_tx(b_full + 8 * stage, bytes + ((i == 0 && (blockIdx.x | blockIdx.y) == 0) ? (uint32_t)p.h.tx_extra : 0u));
                if (second) tma_load_3d(smem_b + stage * B_STAGE_BYTES, &map_b1, b_full + 8 * stage, 32, k0, i - taps);
                else tma_load_3d(smem_b + stage * B_STAGE_BYTES, &map_b0, b_full + 8 * stage, 0, k0, i);
                if (++stage == (uint32_t)p.b_stages) { stage = 0; par ^= 1u; }
            }
        }
    } else if (warp == 1 || warp == 6 || warp >= 11) {
        const int acc = warp == 1 ? 0 : warp == 6 ? 1 : warp - 9;             // warps 1, 6, 11, 12: one accumulator each
        if (lane == 0) {
            // ---------------- MMA issuers
            constexpr uint32_t idesc = instr_desc_tf32<BN>();
            const uint32_t my_acc = tmem_acc + (uint32_t)(acc * BN);
            uint32_t stage = 0, par = 0;
            // Between a stage's barrier and its MMAs the four issuers are all busy with bookkeeping and the tensor pipe
            // idles, so the loops hold as little of it as possible: one loop per chunk, descriptors advanced by
            // additions (a descriptor's address field counts 16-byte units: 8 per slab row of chunk 0, 4 of chunk 1).
            bool ok = mbar_wait(slab_full, 0, &s_abort, p.h.status, 53);
            const uint32_t S = (uint32_t)p.h.S, row_step = (uint32_t)(p.h.Wp - p.h.S + 1);   // slab rows from a tap row's last tap to the next row's first
            const uint32_t nstages = (uint32_t)p.b_stages;
            uint32_t b_addr = smem_b;
            {
                uint64_t da = smem_desc_k_sw128(slab0 + (uint32_t)(acc * 128) * 128u);
                uint32_t s = 0;
                for (int i = 0; ok && i < taps; ++i) {
                    ok = mbar_wait(b_full + 8 * stage, par, &s_abort, p.h.status, 55);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t db = smem_desc_k_sw128(b_addr);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_tf32(my_acc, da + 2 * k, db + 2 * k, idesc, (i | k) ? 1u : 0u);
                    tc_commit(b_empty + 8 * stage);
                    b_addr += B_STAGE_BYTES;
                    if (++stage == nstages) { stage = 0; par ^= 1u; b_addr = smem_b; }
                    if (++s == S) { s = 0; da += 8 * row_step; } else da += 8;
                }
            }
            if (acc == 0) FL_STAMP(1);
            if (ok) ok = mbar_wait(slab_full + 8, 0, &s_abort, p.h.status, 54);
            {
                uint64_t da = smem_desc_k_sw64(slab1 + (uint32_t)(acc * 128) * 64u);
                uint32_t s = 0;
                for (int i = 0; ok && i < taps; ++i) {
                    ok = mbar_wait(b_full + 8 * stage, par, &s_abort, p.h.status, 55);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t db = smem_desc_k_sw64(b_addr);
#pragma unroll
                    for (int k = 0; k < 2; ++k) umma_tf32(my_acc, da + 2 * k, db + 2 * k, idesc, 1u);
                    tc_commit(b_empty + 8 * stage);
                    b_addr += B_STAGE_BYTES;
                    if (++stage == nstages) { stage = 0; par ^= 1u; b_addr = smem_b; }
                    if (++s == S) { s = 0; da += 4 * row_step; } else da += 4;
                }
            }
            tc_commit(accum_bar);
            if (acc == 0) FL_STAMP(6);
            if (!ok) (void)mbar_wait(accum_bar, 0, &s_abort, p.h.status, 56);
        }
    } else {
        // ---------------- slab builders (8 warps), then epilogue
        const int group = warp >= 7 ? 1 : 0;
        const int etid = threadIdx.x - (group ? 96 : 64);                  // 0 .. 255
        const int bwarp = etid >> 5;
        const int H = p.H, W = p.W;
        const int rows_avail = min(p.raw_rows, H - y0);                    // input rows that exist
        // raw rows of channel c: floats [g0, g1) of the input; the copy starts at the 16-byte boundary below g0
        auto span = [&](int c, long long& a0, long long& g1) {
            const long long g0 = ((long long)(n * kChannels + c) * H + y0) * W;
            a0 = g0 & ~3LL;
            g1 = g0 + (long long)rows_avail * W;
            return (int)(g0 - a0);
        };
        const long long in_floats16 = p.in_floats & ~3LL;                  // floats that whole 16-byte pieces cover
        auto load_raw = [&](int c, uint32_t dst, uint32_t bar) {
            long long a0, g1;
            (void)span(c, a0, g1);
            long long end = (g1 + 3) & ~3LL;
            if (end > in_floats16) end = in_floats16;                      // the tensor's last floats, if any, are fetched by hand
            const uint32_t bytes = (uint32_t)((end - a0) * 4);
            mbar_expect_tx(bar, bytes);
            bulk_load_global(dst, p.in + a0, bytes, bar);
        };
        // floats of the span past the last whole 16-byte piece of the tensor (at most 3, last image only)
        auto patch_tail = [&](int c, uint32_t dst) {
            long long a0, g1;
            (void)span(c, a0, g1);
            for (long long g = in_floats16 + etid; g < g1; g += 256)
                if (g >= a0) st_shared_f32(dst + (uint32_t)(g - a0) * 4u, __ldg(p.in + g));
        };
        if (etid == 0) {
            load_raw(0, raw0, raw_full);
            load_raw(1, raw1, raw_full + 8);
        }
        // One warp task = 8 consecutive slab rows: lane = (row, dx); per task the position is decoded once and the
        // pieces (c, dy) follow at literal offsets.  Rows of the input that do not exist (below the image) and the
        // column past its right edge read as zeros, whatever the buffer holds there.
        auto build = [&](int chunk, int mis0, int mis1) {
            const int groups = p.slab_rows >> 3;
            for (int g = bwarp; g < groups; g += 8) {
                const int i = g * 8 + (lane >> 2), dx = lane & 3;
                const int ybl = i / p.h.Wp, xb = i - ybl * p.h.Wp;
                const int x = kStride * xb + dx;
                const bool xok = x < W;
                const int yl0 = kStride * ybl;
                if (chunk == 0) {
                    const uint32_t dst = slab0 + (uint32_t)i * 128u + (uint32_t)dx * 4u;
                    float v[8];
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {                       // all eight loads first: their latencies overlap
                        const int c = jj >> 2, dy = jj & 3;                // literals after unrolling
                        const int yl = yl0 + dy;
                        const bool ok = xok && yl < rows_avail;
                        const uint32_t src = (c ? raw1 : raw0) + (uint32_t)((c ? mis1 : mis0) + yl * W + x) * 4u;
                        v[jj] = 0.f;
                        if (ok) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[jj]) : "r"(src));
                    }
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) st_shared_f32(dst + (uint32_t)((jj ^ (i & 7)) << 4), round_to_tf32(v[jj]));
                } else {
                    const uint32_t dst = slab1 + (uint32_t)i * 64u + (uint32_t)dx * 4u;
                    float v[4];
#pragma unroll
                    for (int dy = 0; dy < 4; ++dy) {
                        const int yl = yl0 + dy;
                        const bool ok = xok && yl < rows_avail;
                        const uint32_t src = raw0 + (uint32_t)(mis0 + yl * W + x) * 4u;
                        v[dy] = 0.f;
                        if (ok) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[dy]) : "r"(src));
                    }
#pragma unroll
                    for (int dy = 0; dy < 4; ++dy) st_shared_f32(dst + (uint32_t)((dy ^ ((i >> 1) & 3)) << 4), round_to_tf32(v[dy]));
                }
            }
        };
        long long a0, g1;
        const int mis_c0 = span(0, a0, g1);
        const bool tail0 = g1 > in_floats16;
        const int mis_c1 = span(1, a0, g1);
        const bool tail1 = g1 > in_floats16;
        const int mis_c2 = span(2, a0, g1);
        const bool tail2 = g1 > in_floats16;
        bool ok = true;
        if (lane == 0) ok = mbar_wait(raw_full, 0, &s_abort, p.h.status, 57) && mbar_wait(raw_full + 8, 0, &s_abort, p.h.status, 58);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        __syncwarp();
        if (tail0 || tail1) {                                   // uniform over the CTA
            if (tail0) patch_tail(0, raw0);
            if (tail1) patch_tail(1, raw1);
            asm volatile("bar.sync 2, 256;" ::: "memory");
        }
        if (etid == 0) FL_STAMP(2);
        if (ok) build(0, mis_c0, mis_c1);
        fence_proxy_async_smem();                               // the tensor core reads the slab through the asynchronous proxy
        asm volatile("bar.sync 2, 256;" ::: "memory");       // every builder is done with both raw buffers
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(slab_full) : "memory");
        if (etid == 0) FL_STAMP(3);
        if (etid == 0) load_raw(2, raw0, raw_full + 16);
        if (lane == 0) ok = ok && mbar_wait(raw_full + 16, 0, &s_abort, p.h.status, 59);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        __syncwarp();
        if (tail2) {
            patch_tail(2, raw0);
            asm volatile("bar.sync 2, 256;" ::: "memory");
        }
        if (etid == 0) FL_STAMP(4);
        if (ok) build(1, mis_c2, 0);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(slab_full + 8) : "memory");
        if (etid == 0) FL_STAMP(5);
        const uint32_t region = (uint32_t)p.slab_rows * 128u + 2u * (uint32_t)p.raw_buf_bytes + (uint32_t)p.b_stages * B_STAGE_BYTES;
        // the tile owns rows_per_tile output rows, but never positions of the next image (a small image ends inside the tile)
        halo::HaloParams h = p.h;
        h.tile_positions = min(p.h.tile_positions, p.h.HpWp - row_first * p.h.Wp);
        halo::halo_epilogue<BN, NACC>(h, smem_base, region, tmem_acc, s_bias, &s_abort, accum_bar, f0, k0, warp, lane);
        if (etid == 0) FL_STAMP(7);
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_acc, TMEM_COLS);
    }
}

// filters KCRS -> [Rb*Sb][K][48] for this kernel's view: channel (c*4 + dy)*4 + dx of block tap (rb, sb) is filter
// element (4*rb + dy, 4*sb + dx) of input channel c, zero where that lies outside the window; rounded to TF32
__global__ void __launch_bounds__(256)
pack_filters_first_layer_kernel(const float* __restrict__ filt, float* __restrict__ wp, int K, int R, int S, int Rb, int Sb)
{
    pdl_launch_dependents();
    pdl_wait();
    const int total = Rb * Sb * K * kViewChannels;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cp = idx % kViewChannels;
        const int u = idx / kViewChannels;
        const int k = u % K, tapb = u / K;
        const int rb = tapb / Sb, sb = tapb - rb * Sb;
        const int dx = cp & 3, dy = (cp >> 2) & 3, c = cp >> 4;
        const int r = rb * kStride + dy, sx = sb * kStride + dx;
        const float v = (r < R && sx < S) ? __ldg(filt + (((size_t)k * kChannels + c) * R + r) * S + sx) : 0.f;
        wp[idx] = round_to_tf32(v);
    }
}

}  // namespace first
}  // namespace boda
