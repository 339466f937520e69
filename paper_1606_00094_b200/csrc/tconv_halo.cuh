// TCONV for stride-1 layers with shared-memory reuse of the input across filter taps.
//
// The paper's tconv loads whole tiles of `in` once per workgroup and reuses them for every kernel offset,
// which cuts input traffic by about (KSZ/stride)^2 (Section 5).  Here that reuse is arranged so that the
// tensor core can read the shifted windows straight from one shared-memory slab:
//
//   The input is re-laid-out as rows of a flat matrix xs[(n*Hp + y)*Wp + x][Cp] (NHWC, channels padded to 32,
//   TF32-rounded) with Hp = H + pad, Wp = W + pad, the extra rows and columns holding zeros.  Because the
//   right-hand zero columns of one image row double as the left-hand padding of the next row (and the zero
//   rows below an image as the padding above the next image), the input pixel of output position
//   f = (n*Hp + p)*Wp + q under tap (r, s) is simply row  f - (pad*Wp + pad) + r*Wp + s  of xs.
//   A CTA owns 128*NACC consecutive flat positions f.  For each 32-channel chunk it loads ONE slab of
//   128*NACC + (R-1)*Wp + (S-1) rows (TMA tiled mode; rows before the start of xs are zero-filled) and then,
//   for every tap, issues the MMAs with the A descriptor advanced by (r*Wp + s) rows of 128 bytes.
//   Positions with p >= P or q >= Q are computed and dropped (for the AlexNet shapes: 7..16 % of the rows).
//
// NACC = 2 or 4 keeps that many 128-row accumulators in tensor memory so that every filter tile fetched from L2
// feeds 256 or 512 output rows: operand traffic per MMA cycle halves again, and again.
// Roles (416 threads): warp 0 = TMA producer, warps 1, 6, 11, 12 = MMA issuers (as many as the tile uses),
// warps 2..5 and 7..10 = epilogue.  Pipeline and bounded waits are those of the im2col kernel (igemm_tf32.cu).
#pragma once

#include "tc_ptx.cuh"

namespace boda {
namespace halo {

using namespace tc;

constexpr int kThreads = 416;      // warp 0 producer; 1, 6, 11, 12 MMA issuers; 2..5 and 7..10 epilogue
constexpr int kMaxBStages = 8;
constexpr int kASlots = 2;
constexpr int kSmemBudget = 200 * 1024;

struct HaloParams {
    int Mflat;                   // N * Hp * Wp flat output positions
    int HpWp, Wp;
    int S, taps, cchunks;
    int lead;                    // pad*Wp + pad
    int nbox, box_rows;          // slab = nbox TMA boxes of box_rows rows
    int a_slot_bytes;            // nbox * box_rows * 128, multiple of 1024
    int b_stages;
    int iters_total, iters_per_split, splits;
    const float* bias;
    OutSpec o;                   // output tensor, layout and activation
    int* status;
    int tx_extra;                // test hook: bytes added to the first stage's expected transfer size of CTA (0,0,0)
    // fused 3x3 / stride-2 max-pooling of the output (pool_rows > 0): a tile then covers output rows
    // 2*pool_rows*j .. 2*pool_rows*j + 2*pool_rows of ONE image (j = tile index within the image) and stores the
    // pool_rows pooled rows they contain; `o` describes the POOLED tensor (o.P, o.Q = pooled extent)
    int pool_rows;
    int tiles_per_image;
    // flat positions of a tile whose outputs the tile owns (128*NACC for the contiguous tiles of this kernel; fewer
    // for the row-aligned tiles of the first-layer kernel, whose last rows belong to the next tile)
    int tile_positions;
};

// output location of flat position f = (n*Hp + p)*Wp + q; positions with p >= P or q >= Q are dropped
__device__ __forceinline__ RowDst halo_row_dst(const HaloParams& p, int f, int f0)
{
    bool valid = f < p.Mflat && f - f0 < p.tile_positions;
    int n = 0, pp = 0, qq = 0;
    if (valid) {
        n = f / p.HpWp;
        const int rem = f - n * p.HpWp;
        pp = rem / p.Wp;
        qq = rem - pp * p.Wp;
        valid = pp < p.o.P && qq < p.o.Q;
    }
    return row_dst(p.o, valid, n, pp, qq);
}

template <int BN, int NACC>
struct HaloCfg {
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int ACC_COLS = BN * NACC;
    static constexpr int TMEM_COLS = ACC_COLS <= 32 ? 32 : ACC_COLS <= 64 ? 64 : ACC_COLS <= 128 ? 128 : ACC_COLS <= 256 ? 256 : 512;
    static_assert(ACC_COLS <= 512, "accumulators exceed tensor memory");
    // One thread can issue an MMA about every 70 clocks; threads in different warps, each feeding its own
    // accumulators, reach about 50 each (measured).  A reduction step of this kernel is 4 MMAs per accumulator, which
    // the tensor pipe finishes in 8*BN/4 clocks: with one issuer per accumulator the pipe, not the issue, is the limit.
    static constexpr int ISSUERS = NACC >= 4 ? 4 : NACC >= 2 ? 2 : 1;
};

#ifdef BODA_FL_PROF
// development aid (off unless the library is built with -DBODA_FL_PROF): clock stamps of CTA (0, 0)
__device__ long long g_fl_prof[16];
__device__ unsigned long long g_cta_times[2 * 512];      // per CTA: global timer (ns) at its first and last instruction
__device__ __forceinline__ unsigned long long fl_globaltimer() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define FL_CTA_TIME(which) do { const unsigned _b = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); if (_b < 512) ::boda::halo::g_cta_times[2 * _b + (which)] = ::boda::halo::fl_globaltimer(); } while (0)
#define FL_STAMP(i) do { if ((blockIdx.x | blockIdx.y) == 0) ::boda::halo::g_fl_prof[i] = clock64(); } while (0)
#else
#define FL_STAMP(i) do { } while (0)
#define FL_CTA_TIME(which) do { } while (0)
#endif

// ---- fused ReLU -> max-pool epilogue (3x3 window, stride 2, no padding, floor extent).
// The paper fuses the activation into the convolution (Section 2) and names fusion as what a BLAS call cannot do
// (Section 3); here the pooling that follows the activation is fused as well, so that the convolution's output -
// four times the bytes of the pooled tensor - is never written.  The tile's rows are whole output rows of one image
// (see HaloParams::pool_rows), so every pooling window of the pooled rows it owns lies inside the tile.
// 32 channels at a time: all accumulators' columns [32c, 32c+32) go into a shared-memory
// block [128*NACC positions][32 channels] (16-byte pieces XOR-swizzled by the position, so that thread-per-position
// writes and the window reads below are free of bank conflicts); after a barrier of the 256 epilogue threads every
// thread takes pooled (row, column, 4 channels) items, reads the nine window positions and writes the maximum -
// plus bias, after ReLU, rounded to TF32 - into the pooled tile [pool_rows * Q][BN] (or straight to an NCHW tensor).  Two blocks alternate,
// so filling block c+1 overlaps pooling block c.  At the end each pooled position leaves as one bulk copy.
// bytes of one position's 32 channels in a pooling block: 128 of data + 16 of padding, which keeps thread-per-position
// 16-byte stores and piece-per-thread window loads free of bank conflicts without any address swizzling
constexpr uint32_t kPoolRowBytes = 144;
// shared memory the fused pooling needs: two blocks and the pooled tile
__host__ __device__ constexpr long long pooled_epilogue_bytes(int nacc, int pooled_positions, int BN)
{
    return 2LL * nacc * 128 * kPoolRowBytes + (long long)pooled_positions * BN * 4;
}

template <int BN, int NACC>
__device__ __forceinline__ void halo_pooled_epilogue(const HaloParams& p, uint32_t smem_base, uint32_t tmem_acc, const float* s_bias,
                                                     int k0, int group, int quarter, int lane, int etid)
{
    static_assert(NACC == 2 || NACC == 4, "the two epilogue groups take alternate accumulators");
    constexpr int NCH = BN / 32;
    constexpr uint32_t BLOCK_BYTES = (uint32_t)NACC * 128u * kPoolRowBytes;
    const uint32_t pooled = smem_base + 2u * BLOCK_BYTES;
    const int n = (int)blockIdx.x / p.tiles_per_image;
    const int j = (int)blockIdx.x - n * p.tiles_per_image;
    const int prow0 = p.pool_rows * j;                                  // first pooled row of this tile
    const int prows = min(p.pool_rows, p.o.P - prow0);                  // pooled rows this tile owns
    const int npos = prows * p.o.Q;                                     // pooled positions this tile owns
    const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16);
    // a thread pools one 16-byte piece (4 channels) g of pooled positions t0, t0 + 32, ...: everything that depends on g
    // and on the window geometry is computed once
    const int g = etid & 7, t0 = etid >> 3;
    const uint32_t row_pitch = (uint32_t)p.Wp * kPoolRowBytes;
#pragma unroll 1
    for (int c = 0; c < NCH; ++c) {
        const uint32_t block = smem_base + (uint32_t)(c & 1) * BLOCK_BYTES;
        // The block takes the RAW accumulators: adding a per-channel bias, ReLU and rounding are all non-decreasing, so
        // they commute with the maximum and are applied to the pooled values only - a quarter of the arithmetic, which
        // is what bounds this phase (two epilogue warps per scheduler).
        auto put = [&](int acc, const uint32_t (&v)[32]) {
            const uint32_t a = block + (uint32_t)(acc * 128 + quarter * 32 + lane) * kPoolRowBytes;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                st_shared_v4(a + 16u * q, __uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]),
                             __uint_as_float(v[4 * q + 3]));
        };
        const float4 b4 = *reinterpret_cast<const float4*>(s_bias + 32 * c + 4 * g);
        const bool relu = p.o.relu != 0;
        if constexpr (NACC == 4) {
            // both of this group's accumulators are read from tensor memory before either is used: one load latency per block
            uint32_t v0[32], v1[32];
            tmem_ld_32cols(trow + group * BN + 32 * c, v0);
            tmem_ld_32cols(trow + (group + 2) * BN + 32 * c, v1);
            tmem_ld_wait();
            put(group, v0);
            put(group + 2, v1);
        } else {
            uint32_t v[32];
            tmem_ld_32cols(trow + group * BN + 32 * c, v);
            tmem_ld_wait();
            put(group, v);
        }
        if (etid == 0 && c == 0) FL_STAMP(8);
        // every thread is past its pooling of block c-1 when it arrives here, so block (c+1)&1 may be refilled after it
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (etid == 0 && c == 0) FL_STAMP(9);
        // A thread pools piece g of ONE pooled column pq for all the pooled rows of the tile, walking down the 2*prows + 1
        // output rows once: per row the maximum of the three columns 2pq .. 2pq+2, and every pooled row is the maximum of
        // three consecutive row maxima (rows 2r, 2r+1, 2r+2; row 2r+2 is also row 2(r+1) of the next pooled row).  That
        // is 3 * (2*prows + 1) window loads for prows outputs instead of 9 * prows: the pooling is bound by the
        // bandwidth of shared memory.
        for (int pq = t0; pq < p.o.Q; pq += 32) {
            uint32_t w = block + (uint32_t)(2 * pq) * kPoolRowBytes + 16u * (uint32_t)g;
            auto row_max = [&](uint32_t a) {
                float4 m = ld_shared_v4(a);
                const float4 x1 = ld_shared_v4(a + kPoolRowBytes), x2 = ld_shared_v4(a + 2u * kPoolRowBytes);
                m.x = fmaxf(m.x, fmaxf(x1.x, x2.x)); m.y = fmaxf(m.y, fmaxf(x1.y, x2.y));
                m.z = fmaxf(m.z, fmaxf(x1.z, x2.z)); m.w = fmaxf(m.w, fmaxf(x1.w, x2.w));
                return m;
            };
            float4 top = row_max(w);                                       // output row 2*pr
#pragma unroll 1
            for (int pr = 0; pr < prows; ++pr) {
                const float4 mid = row_max(w + row_pitch), bot = row_max(w + 2u * row_pitch);
                float4 m;
                m.x = fmaxf(top.x, fmaxf(mid.x, bot.x)); m.y = fmaxf(top.y, fmaxf(mid.y, bot.y));
                m.z = fmaxf(top.z, fmaxf(mid.z, bot.z)); m.w = fmaxf(top.w, fmaxf(mid.w, bot.w));
                m.x += b4.x; m.y += b4.y; m.z += b4.z; m.w += b4.w;
                if (relu) { m.x = fmaxf(m.x, 0.f); m.y = fmaxf(m.y, 0.f); m.z = fmaxf(m.z, 0.f); m.w = fmaxf(m.w, 0.f); }
                const int t = pr * p.o.Q + pq;
                if (p.o.packed) {
                    st_shared_v4(pooled + (uint32_t)(t * BN + 32 * c + 4 * g) * 4u, round_to_tf32(m.x), round_to_tf32(m.y),
                                 round_to_tf32(m.z), round_to_tf32(m.w));
                } else {
                    const int k = k0 + 32 * c + 4 * g;
                    float* dst = p.o.out + ((size_t)(n * p.o.K + k) * p.o.P + prow0 + pr) * p.o.Q + pq;
                    const float mv[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (k + e < p.o.K) dst[(size_t)e * p.o.PQ] = mv[e];
                }
                top = bot;
                w += 2u * row_pitch;
            }
        }
        if (etid == 0 && c == 0) FL_STAMP(10);
    }
    if (etid == 0) FL_STAMP(11);
    if (p.o.packed) {
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (etid == 0) FL_STAMP(12);
        const int w = min(BN, p.o.Cp - k0);
        if (w > 0) {
            // One thread issues one bulk copy, and the lanes of a warp issue theirs one after the other: copy whole
            // pooled rows where they are contiguous on both sides (the tile spans all the consumer's channels), so that
            // a tile leaves in a handful of copies instead of one per position.
            const bool rows_contiguous = w == BN && p.o.Cp == BN;
            if (rows_contiguous) {
                const bool all_contiguous = p.o.Wp == p.o.Q;
                if (all_contiguous) {
                    if (etid == 0) {
                        float* dst = p.o.out + ((size_t)(n * p.o.Hp + prow0) * p.o.Wp) * (size_t)p.o.Cp;
                        bulk_store_global(dst, pooled, (uint32_t)npos * (uint32_t)BN * 4u);
                    }
                } else if ((etid & 31) == 0 || prows > 8) {
                    // lane 0 of each of the eight warps takes rows warp, warp + 8, ...; many rows: every thread takes some
                    const int first_row = prows > 8 ? etid : etid >> 5, step = prows > 8 ? 256 : 8;
                    for (int r = first_row; r < prows; r += step) {
                        float* dst = p.o.out + ((size_t)(n * p.o.Hp + prow0 + r) * p.o.Wp) * (size_t)p.o.Cp;
                        bulk_store_global(dst, pooled + (uint32_t)(r * p.o.Q * BN) * 4u, (uint32_t)p.o.Q * (uint32_t)BN * 4u);
                    }
                }
            } else {
                for (int t = etid; t < npos; t += 256) {
                    const int pr2 = t / p.o.Q, pq2 = t - pr2 * p.o.Q;
                    float* dst = p.o.out + ((size_t)(n * p.o.Hp + prow0 + pr2) * p.o.Wp + pq2) * (size_t)p.o.Cp + k0;
                    bulk_store_global(dst, pooled + (uint32_t)(t * BN) * 4u, (uint32_t)w * 4u);
                }
            }
        }
        bulk_commit();
        if (etid == 0) FL_STAMP(13);
        bulk_wait_all();
        if (etid == 0) FL_STAMP(14);
    }
}

// ---- the epilogue of the 8 epilogue warps (2..5 and 7..10) of a CTA that owns NACC accumulators of 128 flat
// positions x BN channels: bias, ReLU, then either the fused pooling above or the plain store (NCHW, or the staged
// layout through bulk copies).  `region_bytes`: shared memory from smem_base that the idle operand buffers leave free.
template <int BN, int NACC>
__device__ __forceinline__ void halo_epilogue(const HaloParams& p, uint32_t smem_base, uint32_t region_bytes, uint32_t tmem_acc,
                                              float* s_bias, volatile int* s_abort, uint32_t accum_bar, int f0, int k0,
                                              int warp, int lane)
{
    // ---------------- epilogue: 8 warps.  Warp w may read TMEM lanes 32*(w%4) .. +31 only, so warps 2..5 and
    // 7..10 pair up on the same 32 rows: with several accumulators the two groups take alternate accumulators,
    // with one they take the two halves of its columns.
    const int quarter = warp & 3;
    const int group = warp >= 7 ? 1 : 0;
    const int row = quarter * 32 + lane;
    const int etid = threadIdx.x - (group ? 96 : 64);                  // 0 .. 255 over the epilogue threads
    for (int j = etid; j < BN; j += 256)
        s_bias[j] = (p.bias && k0 + j < p.o.K) ? __ldg(p.bias + k0 + j) : 0.f;
    if (lane == 0) (void)mbar_wait_relaxed(accum_bar, 0, s_abort, p.status, 16);   // one poller per warp
    __syncwarp();
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const bool ok = (*s_abort == 0);
    tc_fence_after();
    if (etid == 0) FL_STAMP(15);
    const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16);
    if (ok && p.pool_rows > 0) {
        if constexpr (NACC >= 2) halo_pooled_epilogue<BN, NACC>(p, smem_base, tmem_acc, s_bias, k0, group, quarter, lane, etid);
    } else if (ok && p.splits == 1) {
        constexpr int NCH = BN / 32, HALF = (NCH + 1) / 2;
        const int c_begin = (NACC == 1 && group) ? HALF : 0, c_end = (NACC == 1 && !group) ? HALF : NCH;
        // Staged layout: rows go through shared memory (the operand buffers are idle now) and leave as bulk
        // copies; every thread owns the same row slot of each of the `nbuf` tile buffers that fit, so only its
        // own earlier copy has to have been read before it overwrites a slot.
        constexpr uint32_t TILE_BYTES = 128u * out_tile_row_bytes<BN>();
        const int nbuf = (int)(region_bytes / TILE_BYTES);
        const bool bulk = p.o.packed && nbuf >= (NACC == 1 ? 1 : 2);      // with several accumulators: a buffer per group
        // Which accumulator and which tile buffer a group takes on its turn.  One accumulator: both groups share
        // it (column halves) and buffer 0.  Two: one each.  Four: with three buffers group 0 takes accumulators
        // 0 and 3 through buffer 0 and group 1 takes 1 and 2 through buffers 1 and 2, so that only one of the four
        // tiles waits for an earlier copy to leave its buffer; with two buffers each group reuses its own.
        const bool three = NACC == 4 && nbuf >= 3;
        constexpr int TURNS = NACC == 1 ? 1 : NACC / 2;
#pragma unroll 1
        for (int turn = 0; turn < TURNS; ++turn) {
            const int acc = NACC == 1 ? 0 : !three ? group + 2 * turn : group == 0 ? 3 * turn : 1 + turn;
            const int buf = NACC == 1 ? 0 : !three ? group : group == 0 ? 0 : 1 + turn;
            const bool reuse = turn > 0 && !(three && group == 1);
            const RowDst d = halo_row_dst(p, f0 + acc * 128 + row, f0);
            const uint32_t row_addr = smem_base + (uint32_t)buf * TILE_BYTES + (uint32_t)row * out_tile_row_bytes<BN>();
            if (bulk && reuse) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
#pragma unroll 1
            for (int c = c_begin; c < c_end; ++c) {
                uint32_t v[32];
                tmem_ld_32cols(trow + acc * BN + 32 * c, v);
                tmem_ld_wait();
                float y[32];
                bias_relu32(v, s_bias + 32 * c, p.o.relu != 0, y);
                if (bulk) out_tile_put32(row_addr, 32 * c, y);
                else store_row32(p.o, d, k0 + 32 * c, y);
            }
            if (bulk) {
                fence_proxy_async_smem();
                out_tile_store_row(p.o, d, k0 + 32 * c_begin, 32 * (c_end - c_begin), row_addr + 128u * (uint32_t)c_begin);
                bulk_commit();
            }
        }
        if (bulk) bulk_wait_all();
    }
}

template <int BN, int NACC>
__global__ void __launch_bounds__(kThreads, 1)
tconv_halo_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const HaloParams p)
{
    using Cfg = HaloCfg<BN, NACC>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_base + kASlots * p.a_slot_bytes;
    const uint32_t bars = smem_b + p.b_stages * Cfg::B_STAGE_BYTES;
    const uint32_t a_full = bars, a_empty = bars + 8 * kASlots;
    const uint32_t b_full = bars + 16 * kASlots, b_empty = b_full + 8 * kMaxBStages;
    const uint32_t accum_bar = b_empty + 8 * kMaxBStages;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ __align__(16) float s_bias[BN];

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    int f0 = blockIdx.x * (128 * NACC);
    if (p.pool_rows > 0) {          // tiles of whole output rows of one image (fused pooling)
        const int n = (int)blockIdx.x / p.tiles_per_image;
        f0 = n * p.HpWp + 2 * p.pool_rows * ((int)blockIdx.x - n * p.tiles_per_image) * p.Wp;
    }
    const int k0 = blockIdx.y * BN;
    const int it_begin = blockIdx.z * p.iters_per_split;
    const int it_end = min(it_begin + p.iters_per_split, p.iters_total);
    const int my_iters = it_end - it_begin;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < kASlots; ++s) { mbar_init(a_full + 8 * s, 1); mbar_init(a_empty + 8 * s, Cfg::ISSUERS); }
        for (int s = 0; s < p.b_stages; ++s) { mbar_init(b_full + 8 * s, 1); mbar_init(b_empty + 8 * s, Cfg::ISSUERS); }
        mbar_init(accum_bar, Cfg::ISSUERS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = s_tmem_base;
    pdl_wait();          // everything above overlapped the previous kernel; its results are needed from here on

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer.  One thread; ring positions, phases and addresses are advanced
            // incrementally (no division in the loop): the loop's own latency bounds the iteration rate.
            const int row0 = f0 - p.lead;                 // may be negative: those rows read as zeros
            const int chunk0 = it_begin / p.taps;
            int tap = it_begin - chunk0 * p.taps;
            int cx = chunk0 * 32;
            uint32_t a_slot = 0, a_par = 1;               // parity the producer waits for on the empty barriers
            uint32_t b_stage = 0, b_par = 1;
            uint32_t bf = b_full, be = b_empty, bdst = smem_b;
            bool need_slab = true;
            for (int i = 0; i < my_iters; ++i) {
                if (need_slab) {
                    if (!mbar_wait(a_empty + 8 * a_slot, a_par, &s_abort, p.status, 11)) break;
                    const uint32_t fb = a_full + 8 * a_slot;
                    mbar_expect_tx(fb, (uint32_t)p.a_slot_bytes);
                    const uint32_t dst = smem_a + a_slot * p.a_slot_bytes;
                    tma_load_2d(dst, &map_a, fb, cx, row0);
                    if (p.nbox > 1) tma_load_2d(dst + p.box_rows * 128, &map_a, fb, cx, row0 + p.box_rows);
                    if (p.nbox > 2) tma_load_2d(dst + 2 * p.box_rows * 128, &map_a, fb, cx, row0 + 2 * p.box_rows);
                    a_slot ^= 1u;
                    if (a_slot == 0) a_par ^= 1u;
                    need_slab = false;
                }
                if (!mbar_wait(be, b_par, &s_abort, p.status, 12)) break;
                mbar_expect_tx(bf, Cfg::B_STAGE_BYTES + ((i == 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) ? (uint32_t)p.tx_extra : 0u));
                tma_load_3d(bdst, &map_b, bf, cx, k0, tap);
                if (++b_stage == (uint32_t)p.b_stages) { b_stage = 0; b_par ^= 1u; bf = b_full; be = b_empty; bdst = smem_b; }
                else { bf += 8; be += 8; bdst += Cfg::B_STAGE_BYTES; }
                if (++tap == p.taps) { tap = 0; cx += 32; need_slab = true; }
            }
        }
    } else if (warp == 1 || warp == 6 || warp >= 11) {
        const int issuer = warp == 1 ? 0 : warp == 6 ? 1 : warp - 9;          // warps 1, 6, 11, 12
        if (lane == 0 && issuer < Cfg::ISSUERS) {
            // ---------------- MMA issuers: each feeds its own share of the accumulators
            constexpr int ACC_PER = NACC / Cfg::ISSUERS;
            const int acc0 = issuer * ACC_PER;
            constexpr uint32_t idesc = instr_desc_tf32<BN>();
            const int chunk0 = it_begin / p.taps;
            int tap = it_begin - chunk0 * p.taps;
            int s = tap % p.S;
            uint32_t a_row_off = (uint32_t)(tap / p.S) * (uint32_t)p.Wp * 128u;      // r * Wp rows
            uint32_t a_off = a_row_off + (uint32_t)s * 128u;                          // (r*Wp + s) rows of 128 bytes
            const uint32_t wp_bytes = (uint32_t)p.Wp * 128u;
            uint32_t a_slot = 0, a_par = 0, b_stage = 0, b_par = 0;
            uint32_t bf = b_full, be = b_empty;
            const uint64_t db0 = smem_desc_k_sw128(smem_b);
            uint64_t db = db0;
            uint32_t slab_addr = 0, cur_slot = 0;
            bool new_slab = true, ok = true;
            uint32_t accumulate = 0;
            for (int i = 0; i < my_iters; ++i) {
                if (new_slab) {
                    ok = mbar_wait(a_full + 8 * a_slot, a_par, &s_abort, p.status, 13);
                    if (!ok) break;
                    slab_addr = smem_a + a_slot * p.a_slot_bytes;
                    cur_slot = a_slot;
                    a_slot ^= 1u;
                    if (a_slot == 0) a_par ^= 1u;
                    new_slab = false;
                }
                ok = mbar_wait(bf, b_par, &s_abort, p.status, 14);
                if (!ok) break;
                tc_fence_after();
                // The A tile of tap (r, s) starts (r*Wp + s) rows into the slab.  The start address may sit on any
                // 128-byte row: the hardware derives every row's swizzle phase from its shared-memory address bits,
                // exactly as the TMA write did (measured: the descriptor's base-offset field must stay zero).
                const uint64_t da = smem_desc_k_sw128(slab_addr + a_off);
#pragma unroll
                for (int a = 0; a < ACC_PER; ++a) {
                    const int acc = acc0 + a;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_tf32(tmem_acc + acc * BN, da + (uint64_t)(acc * (128 * 128 / 16) + 2 * k), db + 2 * k, idesc,
                                  (k == 0) ? accumulate : 1u);
                }
                accumulate = 1u;
                tc_commit(be);
                const bool chunk_done = (tap + 1 == p.taps);
                if (chunk_done || i + 1 == my_iters) tc_commit(a_empty + 8 * cur_slot);
                if (++b_stage == (uint32_t)p.b_stages) { b_stage = 0; b_par ^= 1u; bf = b_full; be = b_empty; db = db0; }
                else { bf += 8; be += 8; db += (uint64_t)(Cfg::B_STAGE_BYTES >> 4); }
                if (chunk_done) { tap = 0; s = 0; a_row_off = 0; a_off = 0; new_slab = true; }
                else {
                    ++tap;
                    if (++s == p.S) { s = 0; a_row_off += wp_bytes; a_off = a_row_off; } else a_off += 128u;
                }
            }
            tc_commit(accum_bar);
            if (!ok) (void)mbar_wait(accum_bar, 0, &s_abort, p.status, 15);
        }
    } else {
        halo_epilogue<BN, NACC>(p, smem_base, (uint32_t)(kASlots * p.a_slot_bytes + p.b_stages * Cfg::B_STAGE_BYTES), tmem_acc,
                                s_bias, &s_abort, accum_bar, f0, k0, warp, lane);
        tc_fence_before();
    }
    __syncthreads();
    if (p.splits > 1) {
        // Split reduction through the cluster (one CTA per split), one 128-row accumulator at a time: park the
        // partial accumulator in this CTA's own shared memory (the operand buffers are idle now), synchronise the
        // cluster, sum this CTA's share of the channels over all peers and store it.
        const bool ok = (s_abort == 0);
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t rank = cluster_cta_rank();
#pragma unroll 1
        for (int acc = 0; acc < NACC; ++acc) {
            if (warp >= 2 && warp <= 5 && ok) {
                const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16) + acc * BN;
                tc_fence_after();
#pragma unroll 1
                for (int j0 = 0; j0 < BN; j0 += 32) {
                    uint32_t v[32];
                    tmem_ld_32cols(trow + j0, v);
                    tmem_ld_wait();
                    stash_row32<BN>(smem_base, row, j0, v);
                }
                tc_fence_before();
            }
            cluster_sync_all();
            if (warp >= 2 && warp <= 5 && ok)
                cluster_reduce_store<BN>(smem_base, row, rank, p.splits, halo_row_dst(p, f0 + acc * 128 + row, f0), p.o, k0, s_bias);
            cluster_sync_all();      // peers are done with this CTA's shared memory
        }
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_acc, Cfg::TMEM_COLS);
    }
}

// NCHW -> flat padded NHWC rows [(n*Hp + y)*Wp + x][Cp]; zeros in the padded rows, columns and channels;
// values rounded to TF32 (nearest, ties away).
__global__ void __launch_bounds__(256)
pack_input_halo_kernel(const float* __restrict__ in, float* __restrict__ xs, int C, int Cp, int H, int W, int Hp, int Wp)
{
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.z;
    const int f0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int HpWp = Hp * Wp;
    const float* src = in + (size_t)n * C * H * W;
    float* dst = xs + (size_t)n * HpWp * Cp;
    {
        const int f = f0 + tx;
        const int y = f / Wp, x = f - y * Wp;
        const bool inside = f < HpWp && y < H && x < W;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = c0 + ty + 8 * i;
            tile[ty + 8 * i][tx] = (inside && c < C) ? __ldg(src + ((size_t)c * H + y) * W + x) : 0.f;
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int f = f0 + ty + 8 * i, c = c0 + tx;
        if (f < HpWp) {
            uint32_t r;
            asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(tile[tx][ty + 8 * i]));
            dst[(size_t)f * Cp + c] = __uint_as_float(r);
        }
    }
}

}  // namespace halo
}  // namespace boda
