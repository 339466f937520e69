// K1CONV and TCONV: implicit-GEMM convolution on the sm_100a tensor cores (tcgen05, TF32 operands,
// fp32 accumulation in tensor memory).
//
// GEMM view (Section 3 of the paper: out = inmat * filtsmat, with inmat never materialised, Section 5):
//   M = N*P*Q output points ("pixels"), N_gemm = K output channels, reduction = (r, s, c).
// One CTA owns a 128-pixel x BN-channel output tile.  The reduction is walked tap by tap and, inside a
// tap, in chunks of 32 input channels (one 128-byte swizzled shared-memory row per pixel / channel):
//   A tile  [128 pixels][32 channels]  <- TMA im2col-mode load from the NHWC re-laid-out input; the
//            hardware walks the 128 consecutive output points of the tile across rows and images, adds
//            the tap offset (s, r) and fills out-of-image pixels with zeros (= the padding);
//   B tile  [BN channels][32 channels] <- TMA tiled load from tap-major filters [R*S][K][C].
// k1conv (kernel size 1) is the same kernel with a single tap: a plain GEMM over C.
// Roles inside the CTA (416 threads, 13 warps): warps 0, 11, 12 = producers (one elected lane each: input tile
// TMA, filter tile TMA, byte counts), warps 1 and 6 = MMA issuers (one elected lane each issues tcgen05.mma on
// alternate reduction steps into its own accumulator; tcgen05.commit releases shared-memory stages; warp 1 also
// owns the tensor-memory allocation), warps 2..5 and 7..10 = epilogue (tcgen05.ld of the accumulators, bias,
// ReLU, store or split reduction).  This is Listing 1's "load block / fma block / store block" loop with
// hardware pipelines in place of barriers.
// Every wait is bounded (4e9 SM cycles, about two seconds): on expiry the kernel records BODA_ERR_DEVICE_TIMEOUT in the
// status word, all roles leave their loops, tensor memory is released and the CTA returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "igemm_tf32.h"
#include "tc_ptx.cuh"
#include "tconv_halo.cuh"
#include "gconv_tf32.cuh"
#include "k1nchw_tf32.cuh"
#include "tconv_first_layer.cuh"

namespace boda {
namespace {

constexpr int BM = 128;          // pixels per CTA tile (UMMA M)
constexpr int BKC = 32;          // channels per reduction chunk (128 bytes of fp32)
constexpr int A_STAGE_BYTES = BM * BKC * 4;
constexpr int kIgemmThreads = 416;   // warps 0, 11, 12 producers, 1 and 6 MMA issuers, 2..5 and 7..10 epilogue

using namespace tc;


struct IgemmParams {
    int M, stride, pad, S;
    int cchunks;                 // Cp / 32
    int terms;                   // 1: TF32.  3: error-compensated TF32 (each chunk as hi*hi, lo*hi, hi*lo)
    int lo_off;                  // channel offset of the low parts in the staged operands (Cp)
    int iters_total;             // taps * cchunks * terms
    int iters_per_split;
    int splits;
    const float* bias;
    OutSpec o;                   // output tensor, layout and activation
    int* status;
    int tx_extra;                // test hook: bytes added to the first stage's expected transfer size of CTA (0,0,0)
    int b_early;                 // the staged filters were written long before this launch (bound filters): their loads need not wait for the preceding kernel
    int out_tma;                 // staged output without padding rows or columns: the tile leaves through the output tensor map
};


template <int BN> struct TileCfg {
    static constexpr int B_STAGE_BYTES = BN * BKC * 4;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
#ifndef BODA_IGEMM_DUAL_ISSUE_MAX_BN
#define BODA_IGEMM_DUAL_ISSUE_MAX_BN 192
#endif
    // MMA issuers: two for the narrower tiles, where one thread's issue cost (about 530 clocks per stage) exceeds
    // the MMA work of a stage (2*BN clocks); one for BN = 256, which is bound by the tensor pipe either way.
    // The issuers take alternate reduction steps (even / odd), so that one issues while the other's MMAs run.  Every
    // stage has one full barrier per issuer: with an odd number of stages a stage changes hands on every turn of the
    // ring, and a barrier shared by both issuers could be read one phase early by the issuer that runs ahead.
    static constexpr int ISSUERS = BN <= BODA_IGEMM_DUAL_ISSUE_MAX_BN ? 2 : 1;
    static constexpr int STAGES = (200 * 1024) / STAGE_BYTES > 8 ? 8 : (200 * 1024) / STAGE_BYTES;
    static_assert(STAGES >= 2, "both issuers need a stage");
    static constexpr int ACC_COLS = ISSUERS * BN;                                         // one accumulator per issuer
    static constexpr int TMEM_COLS = ACC_COLS <= 64 ? 64 : ACC_COLS <= 128 ? 128 : ACC_COLS <= 256 ? 256 : 512;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// output location of GEMM row m = (n, p, q)
__device__ __forceinline__ RowDst igemm_row_dst(const IgemmParams& p, int m)
{
    const bool valid = m < p.M;
    int n = 0, pp = 0, qq = 0;
    if (valid) {
        n = m / p.o.PQ;
        const int pq = m - n * p.o.PQ;
        pp = pq / p.o.Q;
        qq = pq - pp * p.o.Q;
    }
    return row_dst(p.o, valid, n, pp, qq);
}

// ------------------------------------------------------------------------------------------------
// MODE 1: the error-compensated mode (three reduction steps per channel chunk).  MODE 2: fp16 operands (a 128-byte
// row of a stage holds 64 channels, one MMA covers 16 of them; fp32 accumulation all the same).  A compile-time switch
// because the producers' loops set the pace of the main loop and every instruction in them shows in the layer's time.
enum { MODE_TF32 = 0, MODE_X3 = 1, MODE_F16 = 2 };
template <int BN, int MODE>
__global__ void __launch_bounds__(kIgemmThreads, 1)
igemm_tf32_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_o, const IgemmParams p)
{
    constexpr bool X3 = MODE == MODE_X3;
    constexpr int CH = MODE == MODE_F16 ? 64 : BKC;      // channels per reduction chunk (128 bytes)
    using Cfg = TileCfg<BN>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // swizzle atoms need 1024-byte alignment
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_base + STAGES * A_STAGE_BYTES;
    const uint32_t bars = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t full_bar = bars;                    // STAGES x 2 x 8 bytes: [stage][issuer]
    const uint32_t empty_bar = bars + 16 * STAGES;
    const uint32_t accum_bar = bars + 24 * STAGES;
    const uint32_t recv_bar = accum_bar + 8;           // split reduction: bytes pushed by the cluster peers, [chunk] (4)
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ __align__(16) float s_bias[BN];

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM;
    const int k0 = blockIdx.y * BN;
    const int it_begin = blockIdx.z * p.iters_per_split;
    const int it_end = min(it_begin + p.iters_per_split, p.iters_total);
    const int my_iters = it_end - it_begin;
    const bool exchange = split_exchange_fits(BN, p.splits, STAGES * Cfg::STAGE_BYTES);   // the same in every CTA

    pdl_launch_dependents();
    if (threadIdx.x == 0 && blockIdx.z == 0) FL_STAMP(0);
    if (threadIdx.x == 0) FL_CTA_TIME(0);
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar + 16 * s, 1); mbar_init(full_bar + 16 * s + 8, 1); mbar_init(empty_bar + 8 * s, 1); }
        mbar_init(accum_bar, Cfg::ISSUERS);           // one arrival per MMA issuer
        for (int c = 0; c < 4; ++c) mbar_init(recv_bar + 8 * c, 1);      // one per 32-channel chunk of this CTA's share
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        if (p.out_tma) prefetch_tensormap(&map_o);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = s_tmem_base;
    // Everything above overlapped the previous kernel; its results (the input) are needed from here on.  The filter
    // tiles are not its results: with bound filters their producer and the byte counts start at once, so the first
    // filter tiles (HBM-cold after a long pause) are on their way while the input is still being written.
    if (!(p.b_early && (warp == 11 || warp == 12))) pdl_wait();
    if (threadIdx.x == 0 && blockIdx.z == 0) FL_STAMP(1);

    if (warp == 0 || warp >= 11) {
        if (lane == 0) {
            // ---------------- TMA producers.  For one thread, an arrival with a byte count costs about 105 clocks, a
            // TMA issue about 125 and a successful barrier test about 45 (measured): one thread doing all of it needs
            // about 430 clocks per stage, more than the MMAs of a stage take for BN <= 192.  So three threads in three
            // warps share a stage: warp 0 loads the input tile (A), warp 11 the filter tile (B), warp 12 posts the
            // stage's byte count on its full barrier (bytes that land before the count is posted are legal: the
            // barrier's phase cannot complete before its one arrival).  Ring position, parity and addresses advance
            // incrementally: the loops hold no division.
            // Each role has its own loop with nothing in it that the role does not need: a handful of extra
            // integer instructions per stage in these loops cost a microsecond per layer (measured).
            constexpr int terms = X3 ? 3 : 1;
            const int chunk0 = it_begin / terms;
            int term = it_begin - chunk0 * terms;
            int tap = chunk0 / p.cchunks;
            int cx = (chunk0 - tap * p.cchunks) * CH;                  // first channel of the chunk
            const int cend = p.cchunks * CH;
            uint32_t stage = 0, par = 1;
            // full barrier of local reduction step i: [stage][i & 1] with two issuers, [stage][0] with one
            constexpr uint32_t FLIP = Cfg::ISSUERS == 2 ? 8u : 0u;
            uint32_t fb = full_bar, eb = empty_bar, fsel = 0;      // fb: the stage's pair of full barriers; fsel: which of them
            if (warp == 0) {
                // input tiles (A).  error-compensated mode: term 0 = hi * hi, term 1 = lo(input) * hi(filter),
                // term 2 = hi(input) * lo(filter)
                const int n0 = m0 / p.o.PQ;
                const int rem = m0 - n0 * p.o.PQ;
                const int p0 = rem / p.o.Q;
                const int q0 = rem - p0 * p.o.Q;
                const int w0 = q0 * p.stride - p.pad;
                const int h0 = p0 * p.stride - p.pad;
                const int S = p.S, lo_off = p.lo_off;
                int r = tap / S;
                int s = tap - r * S;
                uint32_t dst = smem_a;
                for (int i = 0; i < my_iters; ++i) {
                    if (!mbar_wait(eb, par, &s_abort, p.status, 1)) break;
                    tma_load_im2col_4d(dst, &map_a, fb + fsel, cx + ((X3 && term == 1) ? lo_off : 0), w0, h0, n0, (uint16_t)s, (uint16_t)r);
                    fsel ^= FLIP;
                    if (++stage == (uint32_t)STAGES) { stage = 0; par ^= 1u; fb = full_bar; eb = empty_bar; dst = smem_a; }
                    else { fb += 16; eb += 8; dst += A_STAGE_BYTES; }
                    if (!X3 || ++term == terms) {
                        term = 0;
                        cx += CH;
                        if (cx == cend) { cx = 0; if (++s == S) { s = 0; ++r; } }
                    }
                }
            } else if (warp == 11) {
                // filter tiles (B)
                const int lo_off = p.lo_off;
                uint32_t dst = smem_b;
                for (int i = 0; i < my_iters; ++i) {
                    if (!mbar_wait(eb, par, &s_abort, p.status, 6)) break;
                    tma_load_3d(dst, &map_b, fb + fsel, cx + ((X3 && term == 2) ? lo_off : 0), k0, tap);
                    fsel ^= FLIP;
                    if (++stage == (uint32_t)STAGES) { stage = 0; par ^= 1u; fb = full_bar; eb = empty_bar; dst = smem_b; }
                    else { fb += 16; eb += 8; dst += Cfg::B_STAGE_BYTES; }
                    if (!X3 || ++term == terms) {
                        term = 0;
                        cx += CH;
                        if (cx == cend) { cx = 0; ++tap; }
                    }
                }
            } else {
                // byte counts
                uint32_t bytes = Cfg::STAGE_BYTES + ((blockIdx.x | blockIdx.y | blockIdx.z) == 0 ? (uint32_t)p.tx_extra : 0u);
                for (int i = 0; i < my_iters; ++i) {
                    if (!mbar_wait(eb, par, &s_abort, p.status, 11)) break;
                    mbar_expect_tx(fb + fsel, bytes);
                    bytes = Cfg::STAGE_BYTES;
                    fsel ^= FLIP;
                    if (++stage == (uint32_t)STAGES) { stage = 0; par ^= 1u; fb = full_bar; eb = empty_bar; }
                    else { fb += 16; eb += 8; }
                }
            }
        }
    } else if (warp == 1 || warp == 6) {
        if (lane == 0 && (warp == 1 || Cfg::ISSUERS == 2)) {
            const int me = warp == 1 ? 0 : 1;
            // ---------------- MMA issuers: warp 1 takes the even reduction steps, warp 6 the odd ones.  One thread
            // needs about 430 clocks per stage (barrier test, four MMA issues, commit) - more than the MMAs take for
            // BN <= 192 - so with two issuers one issues while the other's MMAs run.  Each issuer accumulates into its
            // own TMEM accumulator (columns [0, BN) and [BN, 2*BN)); the epilogue adds the two, so the summation
            // order - and with it every output bit - is the same in every run.
            constexpr uint32_t idesc = MODE == MODE_F16 ? instr_desc_f16<BN>() : instr_desc_tf32<BN>();
            constexpr int STEP = Cfg::ISSUERS;                          // stages between two steps of one issuer
            // an issuer returns to a barrier after CYCLE of its own steps: then the barrier's phase has advanced
            constexpr int CYCLE = (STEP == 2 && STAGES % 2 == 0) ? STAGES / 2 : STAGES;
            bool ok = true;
            uint32_t par = 0;
            int stage = me, visited = 0;
            const uint32_t my_acc = tmem_acc + (uint32_t)(me * BN);
            const uint64_t da0 = smem_desc_k_sw128(smem_a), db0 = smem_desc_k_sw128(smem_b);
            uint64_t da = da0 + (uint64_t)me * (A_STAGE_BYTES >> 4), db = db0 + (uint64_t)me * (Cfg::B_STAGE_BYTES >> 4);
            uint32_t fb = full_bar + 16 * me + 8 * me, eb = empty_bar + 8 * me;
            uint32_t accumulate = 0;
            for (int i = me; i < my_iters; i += STEP) {
                ok = mbar_wait(fb, par, &s_abort, p.status, 2);
                if (!ok) break;
                if (i == 0 && blockIdx.z == 0) FL_STAMP(2);
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < BKC / 8; ++k) {     // 8 TF32 (16 fp16) values = 32 bytes = 2 descriptor units per step
                    if constexpr (MODE == MODE_F16) umma_f16(my_acc, da + 2 * k, db + 2 * k, idesc, k == 0 ? accumulate : 1u);
                    else umma_tf32(my_acc, da + 2 * k, db + 2 * k, idesc, k == 0 ? accumulate : 1u);
                }
                accumulate = 1u;
                tc_commit(eb);                          // frees the stage once these MMAs have read it
                stage += STEP;
                if (stage >= STAGES) {
                    stage -= STAGES;
                    da -= (uint64_t)(STAGES - STEP) * (A_STAGE_BYTES >> 4); db -= (uint64_t)(STAGES - STEP) * (Cfg::B_STAGE_BYTES >> 4);
                    fb -= 16 * (STAGES - STEP); eb -= 8 * (STAGES - STEP);
                } else {
                    da += (uint64_t)STEP * (A_STAGE_BYTES >> 4); db += (uint64_t)STEP * (Cfg::B_STAGE_BYTES >> 4);
                    fb += 16 * STEP; eb += 8 * STEP;
                }
                if (++visited == CYCLE) { visited = 0; par ^= 1u; }
            }
            tc_commit(accum_bar);                       // this issuer's MMAs have drained
            if (me == 0 && blockIdx.z == 0) FL_STAMP(3);
            if (!ok) (void)mbar_wait(accum_bar, 0, &s_abort, p.status, 3);
        }
    } else {
        // ---------------- epilogue: 8 warps.  Warp w may read TMEM lanes 32*(w%4) .. +31 only, so warps 2..5 and
        // 7..10 pair up on the same 32 rows and share the columns in chunks of 32: group 0 takes the even chunks of
        // a piece of work, group 1 the odd ones.  (One warp per scheduler cannot hide its own instruction latency:
        // four warps needed about 650 clocks per chunk.)
        const int quarter = warp & 3;
        const int group = warp >= 7 ? 1 : 0;
        const int row = quarter * 32 + lane;
        const int m = m0 + row;
        const int etid = threadIdx.x - (group ? 96 : 64);                  // 0 .. 255 over the epilogue threads
        // bias of this tile's channels into shared memory while the main loop runs (0 where there is none)
        for (int j = etid; j < BN; j += 256)
            s_bias[j] = (p.bias && k0 + j < p.o.K) ? __ldg(p.bias + k0 + j) : 0.f;
        if (lane == 0) (void)mbar_wait_relaxed(accum_bar, 0, &s_abort, p.status, 4);   // one poller per warp
        __syncwarp();
        // All epilogue threads meet here whatever their wait returned, then take one common decision:
        // a failed wait has raised the abort flag before returning.
        // (a barrier with an OR reduction: the decision is the same in all 256 threads even if the flag is raised
        // while they read it, so that the group barriers below are reached by everyone or by no one)
        uint32_t stop;
        asm volatile("{\n\t.reg .pred q, r;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred r, 1, 256, q;\n\tselp.u32 %0, 1, 0, r;\n\t}"
                     : "=r"(stop) : "r"((uint32_t)s_abort) : "memory");
        const bool ok = stop == 0;
        tc_fence_after();
        if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(4);
        const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16);
        const bool two_acc = Cfg::ISSUERS == 2 && my_iters >= 2;   // a single reduction step never reaches the second issuer
        // 32 accumulator columns of this thread's row (the sum of the two issuers' accumulators)
        auto load32 = [&](int j0, uint32_t (&v)[32]) {
            tmem_ld_32cols(trow + j0, v);
            if (two_acc) {
                uint32_t v2[32];
                tmem_ld_32cols(trow + BN + j0, v2);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v2[j]));
            } else {
                tmem_ld_wait();
            }
        };
        // Staged output whose rows follow one another without padding (the consumer reads it through an im2col map or
        // is a pooling layer): the tile is a box of the [rows][channels] matrix, so it leaves as tensor stores of
        // 32 rows x 32 channels (4 KB, 128-byte rows swizzled by the row like the exchange blocks).  A warp hands over
        // its own 32 rows: no barrier between warps, and 8 times fewer copies than one per half row (the copy engine
        // moved about 13 bytes per clock with 512-byte copies against 32 with large ones).
        auto store_box = [&](uint32_t chunk_block, int kc, const float (&y)[32]) {
            const uint32_t box = chunk_block + 4096u * (uint32_t)quarter;
            const uint32_t a = box + 128u * (uint32_t)lane;
#pragma unroll
            for (int g = 0; g < 8; ++g)
                st_shared_v4(a + (uint32_t)((g ^ (lane & 7)) << 4), round_to_tf32(y[4 * g]), round_to_tf32(y[4 * g + 1]),
                             round_to_tf32(y[4 * g + 2]), round_to_tf32(y[4 * g + 3]));
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && kc < p.o.Cp && m0 + 32 * quarter < p.M) {
                tma_store_2d(&map_o, box, kc, m0 + 32 * quarter);
                bulk_commit();
            }
        };
        if (p.splits == 1 && p.out_tma) {
            if (ok) {
                constexpr int NCH = BN / 32, HALF = (NCH + 1) / 2;
                const int c_begin = group ? HALF : 0, c_end = group ? NCH : HALF;
#pragma unroll 1
                for (int c = c_begin; c < c_end; ++c) {
                    uint32_t v[32];
                    load32(32 * c, v);
                    float y[32];
                    bias_relu32(v, s_bias + 32 * c, p.o.relu != 0, y);
                    store_box(smem_base + 16384u * (uint32_t)c, k0 + 32 * c, y);      // the stage buffers are idle now
                }
                if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(5);
                if (lane == 0) bulk_wait_all();
                if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(6);
            }
        } else if (p.splits == 1) {
            if (ok) {
                const RowDst d = igemm_row_dst(p, m);
                const uint32_t row_addr = smem_base + (uint32_t)row * out_tile_row_bytes<BN>();   // the stage buffers are idle now
                // group 0 takes the first half of the row's chunks, group 1 the second; in the staged layout each
                // half row leaves as one bulk copy as soon as its thread has written it
                constexpr int NCH = BN / 32, HALF = (NCH + 1) / 2;
                const int c_begin = group ? HALF : 0, c_end = group ? NCH : HALF;
#pragma unroll 1
                for (int c = c_begin; c < c_end; ++c) {
                    uint32_t v[32];
                    load32(32 * c, v);
                    float y[32];
                    bias_relu32(v, s_bias + 32 * c, p.o.relu != 0, y);
                    if (p.o.packed) out_tile_put32(row_addr, 32 * c, y);
                    else store_row32(p.o, d, k0 + 32 * c, y);
                }
                if (p.o.packed) {
                    fence_proxy_async_smem();
                    out_tile_store_row(p.o, d, k0 + 32 * c_begin, 32 * (c_end - c_begin), row_addr + 128u * (uint32_t)c_begin);
                    bulk_commit();
                    bulk_wait_all();
                }
            }
        } else if (exchange) {
            // split reduction by exchange, see split_share(): partial sums of the channels other CTAs own go into
            // send blocks, 32 channels (16 KB) at a time; as soon as a chunk is complete one thread pushes it to its
            // owner with a bulk copy, counted on the owner's barrier for that chunk, and the owner adds each chunk
            // to its own accumulator as it arrives - so writing, transfer (about 16 bytes per clock) and finishing
            // overlap.  The first push waits for the cluster barrier: every CTA's main loop has ended and its stage
            // buffers, which the blocks reuse, are free.
            cluster_arrive();
            const int rank = (int)cluster_cta_rank();
            const int per = split_share(BN, p.splits);
            const int my_w = split_width(BN, per, rank);
            const uint32_t recv_base = smem_base + 512u * (uint32_t)(per * (p.splits - 1));
            // warp 2 / warp 7 push for their group.  The whole warp takes the cluster barrier's second half together:
            // lanes of one warp waiting at different places would wait for different phases of the barrier.
            const bool push_warp = quarter == (group ? 3 : 2);
            bool waited = false;
            if (ok) {
                if (threadIdx.x == 64)
                    for (int c = 0; 32 * c < my_w; ++c) mbar_expect_tx(recv_bar + 8 * c, 16384u * (uint32_t)(p.splits - 1));
                int turn = 0;
#pragma unroll 1
                for (int dst = 0; dst < p.splits; ++dst) {
                    const int wd = split_width(BN, per, dst);
                    if (dst == rank || wd == 0) continue;
                    const uint32_t block = smem_base + 512u * (uint32_t)(per * (dst < rank ? dst : dst - 1));
                    const uint32_t slot = recv_base + 512u * (uint32_t)(wd * (rank < dst ? rank : rank - 1));
#pragma unroll 1
                    for (int c = 0; 32 * c < wd; ++c, ++turn) {
                        if ((turn & 1) != group) continue;
                        uint32_t v[32];
                        load32(dst * per + 32 * c, v);
                        xchg_put32(block + 16384u * (uint32_t)c, 32, row, 0, v);
                        fence_proxy_async_smem();
                        if (group) asm volatile("bar.sync 3, 128;" ::: "memory"); else asm volatile("bar.sync 2, 128;" ::: "memory");
                        if (push_warp) {
                            if (!waited) { cluster_wait(); waited = true; if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(6); }
                            if (lane == 0)
                                bulk_push_cluster(map_to_cta(slot + 16384u * (uint32_t)c, (uint32_t)dst), block + 16384u * (uint32_t)c, 16384u,
                                              map_to_cta(recv_bar + 8 * c, (uint32_t)dst));
                        }
                    }
                }
            }
            if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(7);
            if (!waited) cluster_wait();           // every thread takes the second half of the barrier exactly once
            if (ok && my_w > 0) {
                const RowDst d = igemm_row_dst(p, m);
#pragma unroll 1
                for (int c = group; 32 * c < my_w; c += 2) {
                    if (!mbar_wait(recv_bar + 8 * c, 0, &s_abort, p.status, 5)) break;
                    if (threadIdx.x == 64 && blockIdx.z == 0 && c == 0) FL_STAMP(8);
                    uint32_t v[32];
                    load32(rank * per + 32 * c, v);
                    float y[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) y[j] = __uint_as_float(v[j]);
                    for (int sl = 0; sl < p.splits - 1; ++sl)
                        xchg_add32(recv_base + 512u * (uint32_t)(my_w * sl) + 16384u * (uint32_t)c, 32, row, 0, y);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(y[j]);
                    bias_relu32(v, s_bias + rank * per + 32 * c, p.o.relu != 0, y);
                    // (the finished chunk goes back into the received block it was summed from: same rows, same thread)
                    if (p.out_tma) store_box(recv_base + 16384u * (uint32_t)c, k0 + rank * per + 32 * c, y);
                    else store_row32(p.o, d, k0 + rank * per + 32 * c, y);
                }
                if (p.out_tma && lane == 0) bulk_wait_all();
                if (threadIdx.x == 64 && blockIdx.z == 0) FL_STAMP(9);
            }
        } else if (ok) {
            // split reduction through remote reads (the exchange blocks do not fit), step 1: park this CTA's partial
            // accumulator in its own shared memory; the cluster-wide sum follows below.
#pragma unroll 1
            for (int j0 = 32 * group; j0 < BN; j0 += 64) {
                uint32_t v[32];
                load32(j0, v);
                stash_row32<BN>(smem_base, row, j0, v);
            }
        }
        tc_fence_before();
    }
    if (exchange && (warp < 2 || warp == 6 || warp >= 11)) {      // the other roles' half of the first cluster barrier
        cluster_arrive();
        cluster_wait();
    }
    __syncthreads();
    if (p.splits > 1) {
        if (!exchange) {
            // step 2: after the cluster barrier each CTA sums its share of the channels over all peers' shared
            // memory and stores it.
            cluster_sync_all();
            if (warp >= 2 && warp <= 5 && s_abort == 0) {
                const int row = (warp & 3) * 32 + lane;
                cluster_reduce_store<BN>(smem_base, row, cluster_cta_rank(), p.splits, igemm_row_dst(p, m0 + row), p.o, k0, s_bias);
            }
        }
        cluster_sync_all();          // nobody leaves while a peer may still read or write its shared memory
        if (threadIdx.x == 0 && blockIdx.z == 0) FL_STAMP(10);
    }
    if (threadIdx.x == 0) FL_CTA_TIME(1);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_acc, Cfg::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// Operand staging ("input transformation", Section 5): NCHW -> NHWC with channels padded to a multiple of
// 32 and values rounded to TF32 (round to nearest, ties away), so that the tensor core's truncation of the
// low mantissa bits is exact.
__device__ __forceinline__ float round_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// With `split` the row holds 2*Cp values: the TF32-rounded value hi at channel c and the rounded remainder
// lo = rna(x - hi) at channel Cp + c (error-compensated mode: x = hi + lo up to 2^-22 relative).
__global__ void __launch_bounds__(256)
pack_input_nhwc_kernel(const float* __restrict__ in, float* __restrict__ xp, int C, int Cp, int HW, int split)
{
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.z;
    const int hw0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8
    const float* src = in + (size_t)n * C * HW;
    const int Cs = split ? 2 * Cp : Cp;
    float* dst = xp + (size_t)n * HW * Cs;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, hw = hw0 + tx;
        tile[ty + 8 * i][tx] = (c < C && hw < HW) ? __ldg(src + (size_t)c * HW + hw) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int hw = hw0 + ty + 8 * i, c = c0 + tx;
        if (hw < HW) {
            const float x = tile[tx][ty + 8 * i];
            const float hi = round_tf32(x);
            dst[(size_t)hw * Cs + c] = hi;
            if (split) dst[(size_t)hw * Cs + Cp + c] = round_tf32(x - hi);
        }
    }
}

// filters KCRS -> [R*S][K][Cp], TF32-rounded, zero in the padded channels
__global__ void __launch_bounds__(256)
pack_filters_kernel(const float* __restrict__ filt, float* __restrict__ wp, int K, int C, int Cp, int RS, int split)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)RS * K * Cp;
    const int Cs = split ? 2 * Cp : Cp;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % Cp);
        const long long t = idx / Cp;
        const int k = (int)(t % K);
        const int tap = (int)(t / K);
        const float x = c < C ? __ldg(filt + ((size_t)k * C + c) * RS + tap) : 0.f;
        const float hi = round_tf32(x);
        wp[t * Cs + c] = hi;
        if (split) wp[t * Cs + Cp + c] = round_tf32(x - hi);         // see pack_input_nhwc_kernel
    }
}

// Space-to-depth staging for strided layers.  A convolution with stride t on C channels equals a stride-1
// convolution with ceil(R/t) x ceil(S/t) taps on C*t*t channels, where "channel" (dy, dx, c) of block (yb, xb)
// is pixel (yb*t + dy, xb*t + dx) of the zero-padded input and the filter taps past R or S are zeros.  It turns
// a first layer such as 11x11 stride 4 on 3 channels into a 3x3 stride-1 layer on 48 channels, which the
// tensor-core kernels can run; the paper's tconv likewise needs "an input transformation" (Section 5).
// Packed channel order: cp = (dy*C + c)*t + dx, so that the t values dx = 0..t-1 of a (dy, c) pair - which are t
// consecutive floats of one input row - stay together: for t = 4 the transform is a copy of 16-byte pieces.
// One CTA builds one block-row: it stages the t input rows of all channels in shared memory with coalesced
// reads (row pitch rounded up to 4 floats and shifted so that block 0 starts 16-byte aligned), then writes the
// [W'][Cp] row of blocks.
__global__ void __launch_bounds__(256)
pack_input_s2d_kernel(const float* __restrict__ in, float* __restrict__ xs, int C, int H, int W, int t, int pad,
                      int Hb, int Wb, int Cp)
{
    extern __shared__ __align__(16) float sm_rows[];     // [C*t rows][pitch]: element x of a row at [row*pitch + pad + x]
    pdl_launch_dependents();
    const int yb = blockIdx.x, n = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int span = Wb * t;                               // columns -pad .. span-pad-1 of the image feed this block-row
    const int pitch = (span + 3) & ~3;
    const int rows = C * t;                                // row index = dy*C + c
    pdl_wait();
    // stage: one warp per (dy, c) row, lanes along x (coalesced); zeros outside the image
    for (int row = warp; row < rows; row += nwarps) {
        const int dy = row / C, c = row - dy * C;
        const int y = yb * t + dy - pad;
        float* dstrow = sm_rows + row * pitch;
        const bool inside = y >= 0 && y < H;
        const float* src = in + (((size_t)n * C + c) * H + (inside ? y : 0)) * W - pad;
#pragma unroll 4
        for (int i = lane; i < pitch; i += 32) {
            const int x = i - pad;
            dstrow[i] = (inside && x >= 0 && x < W) ? __ldg(src + i) : 0.f;
        }
    }
    __syncthreads();
    float* dst = xs + ((size_t)n * Hb + yb) * Wb * Cp;
    if (t == 4) {
        // 16 lanes cover the 64-byte-aligned channel quads of one block: quad j < rows is (dy, c) = row j, the rest padding
        const int quads = Cp >> 2;
        for (int item = threadIdx.x; item < quads * Wb; item += blockDim.x) {
            const int j = item % quads, xb = item / quads;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (j < rows) {
                const float4 r = *reinterpret_cast<const float4*>(sm_rows + j * pitch + 4 * xb);
                v = make_float4(round_tf32(r.x), round_tf32(r.y), round_tf32(r.z), round_tf32(r.w));
            }
            *reinterpret_cast<float4*>(dst + (size_t)xb * Cp + 4 * j) = v;
        }
    } else {
        for (int item = threadIdx.x; item < Cp * Wb; item += blockDim.x) {
            const int cp = item % Cp, xb = item / Cp;
            const int row = cp / t, dx = cp - row * t;
            dst[(size_t)xb * Cp + cp] = row < rows ? round_tf32(sm_rows[row * pitch + xb * t + dx]) : 0.f;
        }
    }
}

// The same for stride 4 with the channel count a compile-time constant (first layers: C = 3).  The general kernel above
// spends most of its instructions on divisions by run-time extents and was bound by instruction issue (measured: 780
// instructions per warp for 14.6 KB of output per CTA); here a warp stages one 32-column piece of all C*4 rows at a
// time, so that the row index is a literal and the C*4 coalesced 128-byte loads of a piece are in flight together.
template <int C>
__global__ void __launch_bounds__(256)
pack_input_s2d_t4_kernel(const float* __restrict__ in, float* __restrict__ xs, int H, int W, int pad, int Hb, int Wb)
{
    constexpr int T = 4, ROWS = C * T, CP = ((C * T * T + 31) / 32) * 32, QUADS = CP / 4;
    static_assert(256 % QUADS == 0, "a block-row's 16-byte pieces are dealt to the threads without a remainder");
    extern __shared__ __align__(16) float sm_rows[];     // [ROWS][pitch]: element x of a row at [row*pitch + pad + x]
    pdl_launch_dependents();
    const int yb = blockIdx.x, n = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pitch = (Wb * T + 3) & ~3;
    const int pieces = (pitch + 31) >> 5;                  // 32-column pieces of a staged row
    const float* img = in + (size_t)n * C * H * W;
    pdl_wait();
    // A warp takes 32-column pieces warp, warp + 8, ... of ALL the rows: the row index is a literal, so (dy, c) and the
    // row's offset cost nothing, and the ROWS loads of a piece are in flight together.
    const int y_first = yb * T - pad;
    for (int piece = warp; piece < pieces; piece += 8) {
        const int i = piece * 32 + lane, x = i - pad;
        const bool xin = i < pitch && (unsigned)x < (unsigned)W;
        const float* src = img + (ptrdiff_t)y_first * W + x;
        float v[ROWS];
#pragma unroll
        for (int row = 0; row < ROWS; ++row) {
            const int dy = row / C, c = row - dy * C;      // literals after unrolling
            const bool yin = (unsigned)(y_first + dy) < (unsigned)H;
            v[row] = (xin && yin) ? __ldg(src + (c * H + dy) * W) : 0.f;      // one image's offsets fit 32 bits
        }
        if (i < pitch) {
#pragma unroll
            for (int row = 0; row < ROWS; ++row) sm_rows[row * pitch + i] = v[row];
        }
    }
    __syncthreads();
    // 16-byte piece j of a block is row j = (dy, c) of the staged rows, four consecutive floats; pieces past ROWS are padding
    float* dst = xs + ((size_t)n * Hb + yb) * Wb * CP;
    const int j = threadIdx.x % QUADS, xb0 = threadIdx.x / QUADS;
    const float* srow = sm_rows + (j < ROWS ? j : 0) * pitch + 4 * xb0;
    float* d4 = dst + xb0 * CP + 4 * j;
    for (int xb = xb0; xb < Wb; xb += 256 / QUADS, srow += 4 * (256 / QUADS), d4 += (256 / QUADS) * CP) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < ROWS) {
            const float4 r = *reinterpret_cast<const float4*>(srow);
            v = make_float4(round_tf32(r.x), round_tf32(r.y), round_tf32(r.z), round_tf32(r.w));
        }
        *reinterpret_cast<float4*>(d4) = v;
    }
}

// filters KCRS -> [Rb*Sb][K][Cp] for the space-to-depth view (zeros where the tap or channel does not exist)
__global__ void __launch_bounds__(256)
pack_filters_s2d_kernel(const float* __restrict__ filt, float* __restrict__ wp, int K, int C, int R, int S, int t,
                        int Rb, int Sb, int Cp)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)Rb * Sb * K * Cp;
    const int Cs = C * t * t;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int cp = (int)(idx % Cp);
        const long long u = idx / Cp;
        const int k = (int)(u % K);
        const int tapb = (int)(u / K);
        const int rb = tapb / Sb, sb = tapb - rb * Sb;
        float v = 0.f;
        if (cp < Cs) {
            const int g = cp / t, dx = cp - g * t;            // packed channel order (dy, c, dx), as in pack_input_s2d_kernel
            const int dy = g / C, c = g - dy * C;
            const int r = rb * t + dy, sx = sb * t + dx;
            if (r < R && sx < S) v = __ldg(filt + (((size_t)k * C + c) * R + r) * S + sx);
        }
        wp[idx] = round_tf32(v);
    }
}

// ------------------------------------------------------------------------------------------------
// Host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

int load_driver_entry_points()
{
    if (g_encode_tiled && g_encode_im2col) return BODA_OK;
    void* f1 = nullptr;
    void* f2 = nullptr;
    cudaDriverEntryPointQueryResult q1, q2;
    BODA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f1, cudaEnableDefault, &q1));
    BODA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f2, cudaEnableDefault, &q2));
    if (!f1 || !f2 || q1 != cudaDriverEntryPointSuccess || q2 != cudaDriverEntryPointSuccess) return BODA_ERR_UNSUPPORTED;
    g_encode_tiled = (EncodeTiledFn)f1;
    g_encode_im2col = (EncodeIm2colFn)f2;
    return BODA_OK;
}

// Tile table.  Ids 16..19: gather kernel (gconv_tf32.cuh; NCHW input, tconv with short reductions and k1conv).
// Ids 0..4: im2col kernel (any stride; k1conv and tconv).  Ids 5..12: halo kernel (tconv, stride 1)
// with NACC accumulators of 128 rows each (ids 5..8: 1, 9..12: 2, 13..15: 4).
// accumulators per tile: 0 = im2col kernel, 1 / 2 / 4 = halo kernel, -1 = gather kernel (gconv_tf32.cuh)
// Ids 20..22: 1x1 layers by TMA straight from NCHW (k1nchw_tf32.cuh), accumulator code -2.
// Ids 23..25: first-layer kernel (tconv_first_layer.cuh; 3 channels, stride 4, straight from NCHW), accumulator code -3.
constexpr int kTileBN[] = {64, 96, 128, 192, 256, /*halo*/ 64, 128, 192, 256, 96, 128, 192, 256, 64, 96, 128, /*gather*/ 64, 96, 128, 192,
                           /*1x1 from NCHW*/ 64, 128, 192, /*first layer*/ 64, 96, 128};
constexpr int kTileNacc[] = {0, 0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 2, 4, 4, 4, -1, -1, -1, -1, -2, -2, -2, -3, -3, -3};
constexpr int kFirstK1nTile = 20;
constexpr int kFirstGatherTile = 16;
constexpr int kNumIgemmTiles = sizeof(kTileBN) / sizeof(kTileBN[0]);
constexpr int kFirstHaloTile = 5;
constexpr int kSplitCandidates[] = {1, 2, 3, 4, 6, 8};

}  // namespace

struct IgemmPlan {
    ConvDims d;                      // the problem the kernels run (the space-to-depth view if s2d)
    ConvDims orig;                   // the layer as given
    bool s2d = false;
    int variant = 0;
    int tile_id = 0;
    int BN = 128;
    int Cp = 0;
    int terms = 1;                   // 3: error-compensated TF32, staged operands hold hi and lo parts (2*Cp channels)
    bool half = false;               // fp16 operands: staged tensors hold __half, Cp is a multiple of 64
    int Cs() const { return terms == 3 ? 2 * Cp : Cp; }
    int esize() const { return half ? 2 : 4; }            // bytes per staged operand element
    int chunk() const { return half ? 64 : BKC; }         // channels per 128-byte reduction chunk
    int splits = 1;
    int iters_total = 0, iters_per_split = 0;
    int tiles_m = 0, tiles_n = 0;
    int* d_status = nullptr;
    float* d_wp = nullptr;           // packed filters [RS][K][Cp]
    size_t wp_bytes = 0;
    const float* bound_filt = nullptr;
    size_t xp_bytes = 0, partial_bytes = 0;
    CUtensorMap map_b;
    CUtensorMap map_a;
    const void* map_a_base = nullptr;
    CUtensorMap map_o{};                  // output as a [rows][channels] matrix (im2col kernel, staged output without padding)
    const void* map_o_base = nullptr;
    // activation layouts on either side (set by igemm_plan_set_io; NCHW by default)
    int tx_extra = 0;                // test hook (BODA_TEST_TX_MISMATCH): makes one bounded wait of one CTA expire
    bool in_packed = false;          // the input already is this plan's staged layout: skip the staging kernel
    int out_packed = 0, oHp = 0, oWp = 0, oCp = 0;
    // gather kernel only
    int2* d_tab = nullptr;           // per reduction index: element offset and tap
    int gather_chunks = 0;           // ceil(C*R*S / 32)
    int sm_count = 148;
    // halo kernel only
    int nacc = 0;                    // 0: im2col kernel; 1, 2 or 4: halo kernel with that many accumulators; -1: gather kernel; -2: 1x1 from NCHW
    int Hp = 0, Wp = 0, lead = 0, slab_rows = 0, nbox = 0, box_rows = 0, a_slot_bytes = 0, b_stages = 0;
    // fused 3x3 / stride-2 max-pooling of the output (halo kernel with 2 or 4 accumulators, no split)
    int pool_rows = 0, tiles_per_image = 0, poolP = 0, poolQ = 0;
    int tiles_m_unpooled = 0;
    // first-layer kernel only (nacc == -3): view taps, tile geometry, second filter map (chunk 1: 16 channels, 64-byte rows)
    int fl_Rb = 0, fl_Sb = 0, fl_rows_per_tile = 0, fl_raw_rows = 0, fl_raw_buf = 0, fl_slab_rows = 0, fl_tiles_unpooled = 0;
    CUtensorMap map_b1;
};

// Geometry of the halo kernel for a shape and tile; false if the shape does not fit it.
static bool halo_geometry(const ConvDims& d, int BN, int nacc, IgemmPlan* p)
{
    if (d.stride != 1 || d.R * d.S < 2) return false;
    if (d.pad > d.R - 1 || d.pad > d.S - 1) return false;       // output extent must fit the padded row / image pitch
    const int Hp = d.H + d.pad, Wp = d.W + d.pad;
    const int slab_rows = 128 * nacc + (d.R - 1) * Wp + (d.S - 1);
    const int nbox = (slab_rows + 255) / 256;
    if (nbox > 3) return false;
    const int box_rows = ((((slab_rows + nbox - 1) / nbox) + 7) / 8) * 8;
    const int a_slot = nbox * box_rows * 128;
    const int b_stage = BN * 128;
    int b_stages = (halo::kSmemBudget - halo::kASlots * a_slot) / b_stage;
    if (b_stages > halo::kMaxBStages) b_stages = halo::kMaxBStages;
    if (b_stages < 2) return false;
    if ((long long)d.N * Hp * Wp > 0x7fffffffLL / 2) return false;
    if (p) {
        p->Hp = Hp; p->Wp = Wp; p->lead = d.pad * Wp + d.pad; p->slab_rows = slab_rows; p->nbox = nbox;
        p->box_rows = box_rows; p->a_slot_bytes = a_slot; p->b_stages = b_stages;
    }
    return true;
}

// Space-to-depth view of a strided layer (see pack_input_s2d_kernel); false if it does not apply.
static bool s2d_view(const ConvDims& d, ConvDims* e)
{
    const int t = d.stride;
    if (t < 2 || t > 4 || d.R * d.S < 2) return false;
    if ((size_t)d.C * t * (d.W + 2 * d.pad + t + 4) * 4 > 44 * 1024) return false;   // shared-memory staging of the pack kernel
    if ((long long)d.C * t * t > 1024) return false;
    ConvDims v = d;
    v.C = d.C * t * t;
    v.R = (d.R + t - 1) / t;
    v.S = (d.S + t - 1) / t;
    v.H = d.P - 1 + v.R;
    v.W = d.Q - 1 + v.S;
    v.stride = 1;
    v.pad = 0;
    v.Kred = v.C * v.R * v.S;
    if (e) *e = v;
    return true;
}

bool igemm_s2d_applicable(const ConvDims& d) { return s2d_view(d, nullptr); }

// Fraction of the multiply-accumulates of the space-to-depth view that are real work.
static double s2d_efficiency(const ConvDims& d)
{
    ConvDims e;
    if (!s2d_view(d, &e)) return 0.0;
    const int Cp = ((e.C + BKC - 1) / BKC) * BKC;
    return (double)d.C * d.R * d.S / ((double)Cp * e.R * e.S);
}

bool igemm_variant_legal(const ConvDims& d, int variant)
{
    if (d.R > 11 || d.S > 11 || d.stride > 8 || d.pad > 100) return false;
    if (d.P <= 0 || d.Q <= 0) return false;
    if (variant == BODA_VARIANT_K1CONV) return d.R == 1 && d.S == 1;
    if (variant == BODA_VARIANT_TCONV) return d.R * d.S >= 2;
    return false;
}

bool igemm_variant_profitable(const ConvDims& d)
{
    // Channels are padded to 32 per reduction chunk and pixels to 128 per tile: tiny C (first layers) and tiny
    // layers stay on the FP32 kernel.
    if (d.K < 16) return false;
    // tiny layers stay on the FP32 kernel (one 3 us launch beats the tensor-core kernels' fixed costs) unless the
    // reduction is long: measured on a 1x1 layer with 96 channels on 6x6 points, 16 filters: 3.7 us on the NCHW 1x1
    // kernel against 8.3 us for the FP32 kernel, whose loop over the reduction is bound by latency
    if ((long long)d.M * d.K < 128 * 64 && !(d.R * d.S == 1 && d.Kred >= 64)) return false;
    const int Cp = ((d.C + BKC - 1) / BKC) * BKC;
    // measured: staged input with C = 8 of 32 channels wins, C = 3 of 32 loses; the gather kernel needs no staged input
    // but its narrowest tile has 64 columns: with 16 filters the run-time compiled FP32 kernel wins (5x5 on 3 channels,
    // 64x64, batch 20: 12.6 against 19.1 us), so the gather rule asks for at least 32 filters
    return std::max((double)d.C / Cp, s2d_efficiency(d)) >= 0.2 ||
           (d.R * d.S >= 2 && d.K >= 32 && ((d.Kred + 31) / 32) * 32 <= gconv::kMaxKred && (long long)d.M * d.K >= 128 * 256);
}

int igemm_num_tiles() { return kNumIgemmTiles; }
int igemm_num_split_candidates() { return (int)(sizeof(kSplitCandidates) / sizeof(int)); }
int igemm_split_candidate(int i) { return kSplitCandidates[i]; }

namespace {

// Cost model (SM clocks) used when a plan is not tuned by timing; fitted to a sweep of every tile and split over
// fourteen layer shapes on B200 (its choice is within 3 % of the best measured one for each of them).
//   main loop: a stage costs the MMAs' 2*BN clocks or about 380 clocks of producer / issuer hand-shakes, whichever
//              is longer (halo kernel: 2.2*BN per accumulator, or 290 per accumulator + 390);
//   fixed:     prologue, pipeline fill and tail, about 3500 clocks (halo kernel 5000);
//   epilogue:  32 clocks per channel without a split (the SM writes about 32 bytes per clock); with a split by
//              exchange 1500 + 14 per channel sent + 20 per channel and peer received + (40 + 6 per peer) per channel
//              finished + 300 per CTA of the cluster; the remote-read fallback 60 per channel and peer;
//   waves:     CTAs over 148 SMs, and clusters over what eight GPCs of 16 SMs hold at once.
int split_share_host(int BN, int splits) { return ((((BN + splits - 1) / splits) + 31) / 32) * 32; }

double epilogue_cost(int BN, int splits, bool exchange)
{
    if (splits <= 1) return 32.0 * BN;
    const int w = split_share_host(BN, splits);
    if (exchange) return 1500.0 + 14.0 * (BN - w) + 20.0 * w * (splits - 1) + w * (40.0 + 6.0 * (splits - 1)) + 300.0 * splits;
    return 1500.0 + 22.0 * BN + 60.0 * w * splits + 300.0 * splits;
}

double wave_count(double tiles, int splits)
{
    double waves = (double)(long long)((tiles * splits + 147) / 148);
    if (splits > 1) waves = std::max(waves, (double)(long long)((tiles + 8 * (16 / splits) - 1) / (8 * (16 / splits))));
    return waves;
}

template <int BN> constexpr int stage_region_bytes() { return TileCfg<BN>::STAGES * TileCfg<BN>::STAGE_BYTES; }
int stage_region_of(int BN)
{
    return BN == 64 ? stage_region_bytes<64>() : BN == 96 ? stage_region_bytes<96>() : BN == 128 ? stage_region_bytes<128>()
         : BN == 192 ? stage_region_bytes<192>() : stage_region_bytes<256>();
}

double model_cost(const ConvDims& d, int Cp, int BN, int splits)
{
    const int iters = d.R * d.S * (Cp / BKC);
    const int ips = (iters + splits - 1) / splits;
    const int se = (iters + ips - 1) / ips;
    const long long tm = (d.M + BM - 1) / BM, tn = (d.K + BN - 1) / BN;
    const double per_iter = std::max(2.0 * BN, 380.0);
    return wave_count((double)tm * tn, se) * (ips * per_iter + 3500.0 + epilogue_cost(BN, se, split_exchange_fits(BN, se, stage_region_of(BN))));
}

double model_cost_halo(const ConvDims& d, int Cp, int BN, int nacc, int splits)
{
    const int iters = d.R * d.S * (Cp / BKC);
    const int ips = (iters + splits - 1) / splits;
    const int se = (iters + ips - 1) / ips;
    const long long mflat = (long long)d.N * (d.H + d.pad) * (d.W + d.pad);
    const long long tm = (mflat + 128 * nacc - 1) / (128 * nacc), tn = (d.K + BN - 1) / BN;
    const double per_iter = std::max(2.2 * BN * nacc, 290.0 * nacc + 390.0);
    return wave_count((double)tm * tn, se) * (ips * per_iter + 5000.0 + nacc * epilogue_cost(BN, se, false));
}

// Gather kernel: persistent over ceil(M/128) * ceil(K/BN) tiles.  Measured: a 32-index reduction step costs about
// 1250 clocks of gather work (1500 with padding, whose bounds tests ride along): neighbouring output points read
// addresses `stride` floats apart, so every load instruction of a producer warp costs L1 four wavefronts.  That is
// six to eight times the MMAs' 2*BN clocks - and still the fastest path for small-C layers with up to 7x7 windows,
// because nothing is staged (the other tensor-core paths pay about 6000 clocks for their staging kernel).
bool gather_legal(const ConvDims& d, int variant, bool x3)
{
    if ((variant != BODA_VARIANT_TCONV && variant != BODA_VARIANT_K1CONV) || x3) return false;
    const int Kp = ((d.Kred + 31) / 32) * 32;
    return Kp <= gconv::kMaxKred && d.K >= 8 && (long long)d.N * d.C * d.H * d.W < (1LL << 31);
}

double model_cost_gather(const ConvDims& d, int BN, int sm_count)
{
    const long long tiles = (long long)((d.M + BM - 1) / BM) * ((d.K + BN - 1) / BN);
    const double per_cta = (double)((tiles + sm_count - 1) / sm_count);
    const int chunks = (d.Kred + 31) / 32;
    // 1x1 layers gather whole 128-byte lines (consecutive output points are consecutive addresses): about 1000 clocks
    const double gather = d.R * d.S == 1 ? 1000.0 : d.pad ? 1500.0 : 1250.0;
    return per_cta * chunks * std::max(2.0 * BN, gather) + 4500.0 + 32.0 * BN;
}

// filters [K][C*R*S] -> [K][Kp] rounded to TF32, zeros past C*R*S: the K-major B operand of the gather kernel
__global__ void __launch_bounds__(256)
pack_filters_flat_kernel(const float* __restrict__ filt, float* __restrict__ wp, int K, int Kred, int Kp)
{
    pdl_launch_dependents();
    pdl_wait();
    const int total = K * Kp;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int k = idx / Kp, j = idx - k * Kp;
        wp[idx] = j < Kred ? round_tf32(__ldg(filt + (size_t)k * Kred + j)) : 0.f;
    }
}

template <int BN>
int launch_gather(IgemmPlan* p, const gconv::GconvParams& prm, cudaStream_t stream)
{
    using C = gconv::Cfg<BN>;
    static DeviceSmemLimit limit;
    BODA_CUDA_TRY(limit.ensure(gconv::gconv_tf32_kernel<BN>, C::SMEM_BYTES));
    const int grid = std::min(prm.tiles_total, p->sm_count);
    BODA_CUDA_TRY(launch_kernel(gconv::gconv_tf32_kernel<BN>, dim3(grid), dim3(gconv::kThreads), (size_t)C::SMEM_BYTES, stream, 1,
                                p->map_b, prm));
    count_launch();
    return BODA_OK;
}

// First-layer kernel: 3 channels, stride 4, no padding, a window of at most 12 x 12 (3 x 3 block taps); tiles of 512
// flat positions of the space-to-depth view start every 2*pr output rows of an image (pr = pooled rows a tile would own).
bool first_layer_geometry(const ConvDims& d, int variant, bool restricted, int BN, IgemmPlan* p)
{
    if (variant != BODA_VARIANT_TCONV || restricted) return false;
    if (d.C != first::kChannels || d.stride != first::kStride || d.pad != 0 || d.R * d.S < 2 || d.R > 12 || d.S > 12) return false;
    const int Rb = (d.R + 3) / 4, Sb = (d.S + 3) / 4;
    const int Hb = d.P - 1 + Rb, Wb = d.Q - 1 + Sb;
    const int pr = (512 - d.Q) / (2 * Wb);
    if (pr < 1 || d.K < 8) return false;
    const int rows_per_tile = 2 * pr;
    const int raw_rows = (rows_per_tile + Rb) * 4;
    const int slab_rows = ((512 + (Rb - 1) * Wb + (Sb - 1)) + 7) & ~7;
    const long long raw_need = (long long)raw_rows * d.W * 4 + 32;
    const int raw_buf = (int)((std::max<long long>(raw_need, (long long)slab_rows * 64) + 1023) & ~1023LL);
    const long long fixed = (long long)slab_rows * 128 + 2LL * raw_buf + 1024 + 512;
    int b_stages = (int)((232448 - fixed) / (BN * 128));
    if (b_stages > halo::kMaxBStages) b_stages = halo::kMaxBStages;
    if (b_stages < 2) return false;
    if ((long long)d.N * Hb * Wb > 0x3fffffffLL || (long long)d.N * d.C * d.H * d.W > 0x7fffffffLL) return false;
    if (p) {
        p->fl_Rb = Rb; p->fl_Sb = Sb; p->Hp = Hb; p->Wp = Wb; p->fl_rows_per_tile = rows_per_tile; p->fl_raw_rows = raw_rows;
        p->fl_raw_buf = raw_buf; p->fl_slab_rows = slab_rows; p->b_stages = b_stages;
        p->fl_tiles_unpooled = d.N * ((d.P + rows_per_tile - 1) / rows_per_tile);
    }
    return true;
}

// One kernel, nothing staged: per tap and accumulator 4 + 2 MMAs of about 57 clocks (four issuers keep the pipe busy),
// about 4000 clocks to fetch the raw rows and build the first slab, 9000 of prologue, tail and epilogue.
double model_cost_first_layer(const ConvDims& d, int BN, int sm_count)
{
    const int Rb = (d.R + 3) / 4, Sb = (d.S + 3) / 4, Wb = d.Q - 1 + Sb;
    const int pr = std::max(1, (512 - d.Q) / (2 * Wb));
    const long long tiles = (long long)d.N * ((d.P + 2 * pr - 1) / (2 * pr)) * ((d.K + BN - 1) / BN);
    const double waves = (double)((tiles + sm_count - 1) / sm_count);
    return waves * (Rb * Sb * 24.0 * std::max(57.0, 0.6 * BN) + 4000.0 + 9000.0);
}

// 1x1 from NCHW: stride 1, no padding, rows of HW floats that TMA can address (16-byte multiples), and the staged
// output layout is not offered (tiles follow images, not the flat output-point index of a consumer's tiles - the
// stores themselves would work).
bool k1n_legal(const ConvDims& d, int variant, bool x3)
{
    if (variant != BODA_VARIANT_K1CONV || x3) return false;
    if (d.R != 1 || d.S != 1 || d.stride != 1 || d.pad != 0) return false;
    return (d.H * d.W) % 4 == 0 && (long long)d.N * ((d.H * d.W + BM - 1) / BM) <= 0x7fffffffLL;
}

// One kernel, no staging: about 380 clocks per 32-channel step (or the MMAs' 2*BN), 3500 of prologue and tail,
// 32 per output channel of epilogue; tiles follow images, so an image of HW points costs ceil(HW/128) tiles.
double model_cost_k1n(const ConvDims& d, int BN, int sm_count, int splits = 1)
{
    const long long tiles = (long long)d.N * ((d.H * d.W + BM - 1) / BM) * ((d.K + BN - 1) / BN);
    const int steps = (d.C + BKC - 1) / BKC;
    if (splits > 1) {
        // one tile per CTA, clusters of `splits` CTAs; the sum through remote reads costs about 60 clocks per channel and peer
        const int ips = (steps + splits - 1) / splits;
        return wave_count((double)tiles, splits) * (ips * std::max(2.0 * BN, 410.0) + 3500.0 + epilogue_cost(BN, splits, false));
    }
    const double per_cta = (double)((tiles + sm_count - 1) / sm_count);       // persistent: epilogues hide under the next tile
    return per_cta * steps * std::max(2.0 * BN, 410.0) + 3500.0 + 32.0 * BN;
}

int encode_map_a_k1n(IgemmPlan* p, const void* in)
{
    const ConvDims& d = p->d;
    const cuuint64_t HW = (cuuint64_t)d.H * d.W;
    const cuuint64_t dims[3] = {HW, (cuuint64_t)d.C, (cuuint64_t)d.N};
    const cuuint64_t strides[2] = {HW * 4, HW * d.C * 4};
    const cuuint32_t box[3] = {32, BKC, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    // MN-major TF32 operands take the 128-byte swizzle in 32-byte pieces (the only layout the tensor core accepts for them)
    CUresult r = g_encode_tiled(&p->map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(in), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (NCHW input) failed with CUresult %d", (int)r);
        return record_cuda_error(cudaErrorInvalidValue, msg);
    }
    p->map_a_base = in;
    return BODA_OK;
}

template <int BN>
int launch_k1n(IgemmPlan* p, const k1n::K1nParams& prm, cudaStream_t stream)
{
    using C = k1n::Cfg<BN>;
    static DeviceSmemLimit limit;
    BODA_CUDA_TRY(limit.ensure(k1n::k1nchw_tf32_kernel<BN>, C::SMEM_BYTES));
    dim3 grid(std::min(prm.tiles_total, p->sm_count));
    if (prm.splits > 1) grid = dim3(prm.tiles_total, 1, prm.splits);          // one tile per CTA, a cluster per tile
    BODA_CUDA_TRY(launch_kernel(k1n::k1nchw_tf32_kernel<BN>, grid, dim3(k1n::kThreads), (size_t)C::SMEM_BYTES, stream, prm.splits,
                                p->map_a, p->map_b, prm));
    count_launch();
    return BODA_OK;
}

template <int BN>
int launch_first_layer(IgemmPlan* p, const first::FirstParams& prm, cudaStream_t stream)
{
    const int smem = p->fl_slab_rows * 128 + 2 * p->fl_raw_buf + p->b_stages * BN * 128 + 1024 + 512;
    static DeviceSmemLimit limit;
    BODA_CUDA_TRY(limit.ensure(first::tconv_first_layer_kernel<BN>, (size_t)smem));
    dim3 grid(p->tiles_m, p->tiles_n, 1);
    BODA_CUDA_TRY(launch_kernel(first::tconv_first_layer_kernel<BN>, grid, dim3(first::kThreads), (size_t)smem, stream, 1,
                                p->map_b, p->map_b1, prm));
    count_launch();
    return BODA_OK;
}

template <int BN, int NACC>
int launch_halo(IgemmPlan* p, const halo::HaloParams& prm, cudaStream_t stream)
{
    const int smem = halo::kASlots * p->a_slot_bytes + p->b_stages * BN * 128 + 1024 + 256;
    static DeviceSmemLimit limit;
    BODA_CUDA_TRY(limit.ensure(halo::tconv_halo_kernel<BN, NACC>, (size_t)smem));
    dim3 grid(p->tiles_m, p->tiles_n, p->splits);
    BODA_CUDA_TRY(launch_kernel(halo::tconv_halo_kernel<BN, NACC>, grid, dim3(halo::kThreads), (size_t)smem, stream, p->splits,
                                p->map_a, p->map_b, prm));
    count_launch();
    return BODA_OK;
}

int encode_map_a_halo(IgemmPlan* p, const void* xs)
{
    const ConvDims& d = p->d;
    const cuuint64_t dims[2] = {(cuuint64_t)p->Cp, (cuuint64_t)d.N * p->Hp * p->Wp};
    const cuuint64_t strides[1] = {(cuuint64_t)p->Cp * 4};
    const cuuint32_t box[2] = {BKC, (cuuint32_t)p->box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_tiled(&p->map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(xs), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (halo A) failed with CUresult %d", (int)r);
        return record_cuda_error(cudaErrorInvalidValue, msg);
    }
    p->map_a_base = xs;
    return BODA_OK;
}

template <int BN, int MODE>
int launch_bn_mode(IgemmPlan* p, const IgemmParams& prm, cudaStream_t stream)
{
    using Cfg = TileCfg<BN>;
    static DeviceSmemLimit limit;
    BODA_CUDA_TRY(limit.ensure(igemm_tf32_kernel<BN, MODE>, Cfg::SMEM_BYTES));
    dim3 grid(p->tiles_m, p->tiles_n, p->splits);
    BODA_CUDA_TRY(launch_kernel(igemm_tf32_kernel<BN, MODE>, grid, dim3(kIgemmThreads), (size_t)Cfg::SMEM_BYTES, stream, p->splits,
                                p->map_a, p->map_b, p->map_o, prm));
    count_launch();
    return BODA_OK;
}
template <int BN>
int launch_bn(IgemmPlan* p, const IgemmParams& prm, cudaStream_t stream)
{
    if (p->half) return launch_bn_mode<BN, MODE_F16>(p, prm, stream);
    return prm.terms == 3 ? launch_bn_mode<BN, MODE_X3>(p, prm, stream) : launch_bn_mode<BN, MODE_TF32>(p, prm, stream);
}

int encode_map_a(IgemmPlan* p, const void* xp)
{
    const ConvDims& d = p->d;
    const cuuint64_t Cs = (cuuint64_t)p->Cs(), es = (cuuint64_t)p->esize();
    const CUtensorMapDataType dtype = p->half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    const cuuint64_t dims[4] = {Cs, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    const cuuint64_t strides[3] = {Cs * es, (cuuint64_t)d.W * Cs * es, (cuuint64_t)d.H * d.W * Cs * es};
    const int lower[2] = {-d.pad, -d.pad};                                 // W, H
    const int upper[2] = {d.pad - (d.S - 1), d.pad - (d.R - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)d.stride, (cuuint32_t)d.stride, 1};
    CUresult r = g_encode_im2col(&p->map_a, dtype, 4, const_cast<void*>(xp), dims, strides,
                                 lower, upper, (cuuint32_t)p->chunk(), BM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeIm2col failed with CUresult %d", (int)r);
        return record_cuda_error(cudaErrorInvalidValue, msg);
    }
    p->map_a_base = xp;
    return BODA_OK;
}

// The staged output as a matrix [N*P*Q rows][oCp channels], boxes of 32 x 32 (what one epilogue warp hands over).
int encode_map_o(IgemmPlan* p, float* out)
{
    const ConvDims& d = p->d;
    const cuuint64_t dims[2] = {(cuuint64_t)p->oCp, (cuuint64_t)d.M};
    const cuuint64_t strides[1] = {(cuuint64_t)p->oCp * 4};
    const cuuint32_t box[2] = {32, 32}, estr[2] = {1, 1};
    CUresult r = g_encode_tiled(&p->map_o, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, out, dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (output) failed with CUresult %d", (int)r);
        return record_cuda_error(cudaErrorInvalidValue, msg);
    }
    p->map_o_base = out;
    return BODA_OK;
}

int encode_map_b(IgemmPlan* p)
{
    const ConvDims& d = p->d;
    if (p->nacc == -3) {
        // filters [Rb*Sb][K][48]: chunk 0 = channels 0..31 as 128-byte rows, chunk 1 = channels 32..47 as 64-byte rows
        const cuuint64_t fdims[3] = {(cuuint64_t)first::kViewChannels, (cuuint64_t)d.K, (cuuint64_t)(p->fl_Rb * p->fl_Sb)};
        const cuuint64_t fstrides[2] = {(cuuint64_t)first::kViewChannels * 4, (cuuint64_t)d.K * first::kViewChannels * 4};
        const cuuint32_t festr[3] = {1, 1, 1};
        const cuuint32_t box0[3] = {32, (cuuint32_t)p->BN, 1}, box1[3] = {16, (cuuint32_t)p->BN, 1};
        CUresult fr = g_encode_tiled(&p->map_b, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, p->d_wp, fdims, fstrides, box0, festr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (fr == CUDA_SUCCESS)
            fr = g_encode_tiled(&p->map_b1, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, p->d_wp, fdims, fstrides, box1, festr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (fr != CUDA_SUCCESS) {
            char msg[96];
            std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (first-layer filters) failed with CUresult %d", (int)fr);
            return record_cuda_error(cudaErrorInvalidValue, msg);
        }
        return BODA_OK;
    }
    if (p->nacc == -1) {
        const cuuint64_t Kp = (cuuint64_t)p->gather_chunks * 32;
        const cuuint64_t gdims[2] = {Kp, (cuuint64_t)d.K};
        const cuuint64_t gstrides[1] = {Kp * 4};
        const cuuint32_t gbox[2] = {BKC, (cuuint32_t)p->BN};
        const cuuint32_t gestr[2] = {1, 1};
        CUresult gr = g_encode_tiled(&p->map_b, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, p->d_wp, gdims, gstrides, gbox, gestr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (gr != CUDA_SUCCESS) {
            char msg[96];
            std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (gather B) failed with CUresult %d", (int)gr);
            return record_cuda_error(cudaErrorInvalidValue, msg);
        }
        return BODA_OK;
    }
    const cuuint64_t Cs = (cuuint64_t)p->Cs(), es = (cuuint64_t)p->esize();
    const cuuint64_t dims[3] = {Cs, (cuuint64_t)d.K, (cuuint64_t)(d.R * d.S)};
    const cuuint64_t strides[2] = {Cs * es, (cuuint64_t)d.K * Cs * es};
    const cuuint32_t box[3] = {(cuuint32_t)p->chunk(), (cuuint32_t)p->BN, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode_tiled(&p->map_b, p->half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, p->d_wp, dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return record_cuda_error(cudaErrorInvalidValue, msg);
    }
    return BODA_OK;
}

}  // namespace

int igemm_plan_create(const ConvDims& d_in, int variant, int tile_id, int split_k, int s2d, int* d_status, IgemmPlan** out, int mode,
                      size_t max_ws)
{
    // mode 1 (error-compensated TF32) and mode 2 (fp16 operands) run on the im2col kernel only, NCHW in and out
    const bool x3 = mode != 0;
    if (!igemm_variant_legal(d_in, variant)) return BODA_ERR_UNSUPPORTED;
    // strided tconv layers may run as their stride-1 space-to-depth view
    ConvDims d = d_in;
    bool use_s2d = false;
    if (x3 && s2d > 0) return BODA_ERR_UNSUPPORTED;      // the error-compensated mode runs on the im2col kernel only
    const bool force_gather = tile_id >= kFirstGatherTile && tile_id < kFirstK1nTile;
    if (force_gather && (s2d > 0 || !gather_legal(d_in, variant, x3))) return BODA_ERR_UNSUPPORTED;
    if (variant == BODA_VARIANT_TCONV && s2d != 0 && !x3 && !force_gather) {
        ConvDims e;
        const bool can = s2d_view(d_in, &e);
        if (s2d > 0 && !can) return BODA_ERR_UNSUPPORTED;
        const int Cp_in = ((d_in.C + BKC - 1) / BKC) * BKC;
        if (can && (s2d > 0 || s2d_efficiency(d_in) >= std::max(0.2, (double)d_in.C / Cp_in))) { d = e; use_s2d = true; }
    } else if (s2d > 0) {
        return BODA_ERR_UNSUPPORTED;
    }
    if (tile_id >= kNumIgemmTiles) return BODA_ERR_UNSUPPORTED;
    if (split_k < 0 || split_k > 8) return BODA_ERR_INVALID_ARG;   // one cluster (at most 8 CTAs) per output tile
    int rc = load_driver_entry_points();
    if (rc != BODA_OK) return rc;
    IgemmPlan* p = new (std::nothrow) IgemmPlan();
    if (!p) return BODA_ERR_NOMEM;
    p->d = d;
    p->orig = d_in;
    p->s2d = use_s2d;
    {
        // Test hooks, off unless the environment asks: a transfer-size mismatch that lets one bounded wait run out,
        // and a shorter limit for that wait (failure detection is tested without faulting or hanging the GPU).
        const char* mm = std::getenv("BODA_TEST_TX_MISMATCH");
        p->tx_extra = (mm && *mm == '1') ? 16 : 0;
        const char* lim = std::getenv("BODA_WAIT_LIMIT_CYCLES");
        long long cycles = lim ? std::atoll(lim) : kWaitLimitCycles;
        if (cycles < 1000000) cycles = 1000000;
        cudaError_t ce = cudaMemcpyToSymbol(c_wait_limit_cycles, &cycles, sizeof(cycles));
        if (ce != cudaSuccess) { delete p; return record_cuda_error(ce, "wait limit upload"); }
    }
    p->variant = variant;
    p->d_status = d_status;
    p->half = mode == 2;
    p->Cp = ((d.C + p->chunk() - 1) / p->chunk()) * p->chunk();
    p->terms = mode == 1 ? 3 : 1;
    p->iters_total = d.R * d.S * (p->Cp / p->chunk()) * p->terms;
    // tile and split: forced, or the minimum of the cost model
    double best = 1e300;
    int best_t = 2, best_s = 1;
    (void)cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, 0);
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (p->sm_count <= 0) p->sm_count = 148;
    }
    for (int t = 0; t < kNumIgemmTiles; ++t) {
        if (tile_id >= 0 && t != tile_id) continue;
        const int nacc = kTileNacc[t];
        if (nacc == -3) {
            if (s2d == 0 || split_k > 1 || !first_layer_geometry(d_in, variant, x3, kTileBN[t], nullptr)) continue;
            const double c = model_cost_first_layer(d_in, kTileBN[t], p->sm_count);
            if (c < best) { best = c; best_t = t; best_s = 1; }
            continue;
        }
        if (nacc == -2) {
            if (!k1n_legal(d_in, variant, x3) || s2d > 0) continue;
            for (int s : kSplitCandidates) {
                if (split_k > 0 && s != split_k) continue;
                if (s > (d_in.C + BKC - 1) / BKC) continue;
                const double c = model_cost_k1n(d_in, kTileBN[t], p->sm_count, s);
                if (c < best) { best = c; best_t = t; best_s = s; }
            }
            continue;
        }
        if (nacc < 0) {
            // the gather kernel works on the layer as given (never on a space-to-depth view) and has no split
            if (!gather_legal(d_in, variant, x3) || s2d > 0 || split_k > 1) continue;
            const double c = model_cost_gather(d_in, kTileBN[t], p->sm_count);
            if (c < best) { best = c; best_t = t; best_s = 1; }
            continue;
        }
        if (nacc > 0 && (x3 || variant != BODA_VARIANT_TCONV || !halo_geometry(d, kTileBN[t], nacc, nullptr))) continue;
        if (max_ws > 0) {
            // staged input of this tile's kernel (see xp_bytes below)
            const size_t rows = nacc > 0 ? (size_t)d.N * (d.H + d.pad) * (d.W + d.pad) : (size_t)d.N * d.H * d.W;
            if (((rows * p->Cs() * p->esize() + 1023) & ~(size_t)1023) > max_ws) continue;
        }
        for (int s : kSplitCandidates) {
            if (split_k > 0 && s != split_k) continue;
            if (s > p->iters_total) continue;
            // the input staging kernel these tiles need and the gather tiles do not: a launch, or the time to read
            // the input and write its staged copy (about 3000 bytes per clock measured on staging kernels)
            const double staging = std::max(6000.0, ((double)d_in.N * d_in.C * d_in.H * d_in.W + (double)d.N * d.H * d.W * p->Cp) * 4.0 / 3000.0);
            const double c = staging + (nacc > 0 ? model_cost_halo(d, p->Cp, kTileBN[t], nacc, s) : model_cost(d, p->Cp * p->terms / (p->half ? 2 : 1), kTileBN[t], s));
            if (c < best) { best = c; best_t = t; best_s = s; }
        }
    }
    if (best >= 1e300 && tile_id < 0) { delete p; return max_ws > 0 ? BODA_ERR_NOMEM : BODA_ERR_UNSUPPORTED; }
    if (split_k > 0) best_s = std::min(split_k, p->iters_total);
    if (tile_id >= 0) best_t = tile_id;
    p->tile_id = best_t;
    p->BN = kTileBN[best_t];
    p->nacc = kTileNacc[best_t];
    if (p->nacc == -3) {
        // ---- first-layer kernel: no staged input; filters [Rb*Sb][K][48]
        p->d = d_in;
        p->s2d = false;
        if (s2d == 0 || split_k > 1 || !first_layer_geometry(d_in, variant, x3, p->BN, p)) { delete p; return BODA_ERR_UNSUPPORTED; }
        p->Cp = 64;
        p->splits = 1;
        p->iters_total = p->iters_per_split = 2 * p->fl_Rb * p->fl_Sb;
        p->tiles_m = p->fl_tiles_unpooled;
        p->tiles_n = (d_in.K + p->BN - 1) / p->BN;
        p->xp_bytes = 0;
        p->partial_bytes = 0;
        p->wp_bytes = (size_t)p->fl_Rb * p->fl_Sb * d_in.K * first::kViewChannels * 4;
        cudaError_t fe = cudaMalloc(&p->d_wp, p->wp_bytes);
        if (fe != cudaSuccess) { igemm_plan_destroy(p); return record_cuda_error(fe, "plan allocation"); }
        rc = encode_map_b(p);
        if (rc != BODA_OK) { igemm_plan_destroy(p); return rc; }
        *out = p;
        return BODA_OK;
    }
    if (p->nacc == -2) {
        // ---- 1x1 from NCHW: no staged input; filters [K][Cp] as for the im2col kernel
        if (!k1n_legal(d_in, variant, x3) || s2d > 0) { delete p; return BODA_ERR_UNSUPPORTED; }
        p->d = d_in;
        p->s2d = false;
        p->Cp = ((d_in.C + BKC - 1) / BKC) * BKC;
        p->iters_total = p->Cp / BKC;
        {
            const int want = std::max(1, std::min(split_k > 0 ? split_k : best_s, p->iters_total));
            p->iters_per_split = (p->iters_total + want - 1) / want;
            p->splits = (p->iters_total + p->iters_per_split - 1) / p->iters_per_split;       // no empty split
        }
        p->tiles_m = d_in.N * ((d_in.H * d_in.W + BM - 1) / BM);
        p->tiles_n = (d_in.K + p->BN - 1) / p->BN;
        p->xp_bytes = 0;
        p->partial_bytes = 0;
        p->wp_bytes = (size_t)d_in.K * p->Cp * 4;
        cudaError_t ke = cudaMalloc(&p->d_wp, p->wp_bytes);
        if (ke != cudaSuccess) { igemm_plan_destroy(p); return record_cuda_error(ke, "plan allocation"); }
        rc = encode_map_b(p);
        if (rc != BODA_OK) { igemm_plan_destroy(p); return rc; }
        *out = p;
        return BODA_OK;
    }
    if (p->nacc < 0) {
        // ---- gather kernel: no staged input, filters flat [K][Kp], offset table on the device
        if (!gather_legal(d_in, variant, x3) || s2d > 0 || split_k > 1) { delete p; return BODA_ERR_UNSUPPORTED; }
        p->d = d_in;
        p->s2d = false;
        const ConvDims& g = p->d;
        p->gather_chunks = (g.Kred + 31) / 32;
        const int Kp = p->gather_chunks * 32;
        p->Cp = ((g.C + BKC - 1) / BKC) * BKC;
        p->splits = 1;
        p->iters_total = p->iters_per_split = p->gather_chunks;
        p->tiles_m = (g.M + BM - 1) / BM;
        p->tiles_n = (g.K + p->BN - 1) / p->BN;
        p->xp_bytes = 0;
        p->partial_bytes = 0;
        std::vector<int2> tab((size_t)Kp);
        for (int k = 0; k < Kp; ++k) {
            if (k < g.Kred) {
                const int c = k / (g.R * g.S), rs = k - c * g.R * g.S, r = rs / g.S, sx = rs - r * g.S;
                tab[k] = make_int2(c * g.H * g.W + r * g.W + sx, (r << 16) | sx);
            } else {
                tab[k] = make_int2(0, 0x4000 << 16);
            }
        }
        cudaError_t ge = cudaMalloc(&p->d_tab, (size_t)Kp * sizeof(int2));
        if (ge == cudaSuccess) ge = cudaMemcpy(p->d_tab, tab.data(), (size_t)Kp * sizeof(int2), cudaMemcpyHostToDevice);
        p->wp_bytes = (size_t)g.K * Kp * 4;
        if (ge == cudaSuccess) ge = cudaMalloc(&p->d_wp, p->wp_bytes);
        if (ge != cudaSuccess) { igemm_plan_destroy(p); return record_cuda_error(ge, "gather plan allocation"); }
        rc = encode_map_b(p);
        if (rc != BODA_OK) { igemm_plan_destroy(p); return rc; }
        *out = p;
        return BODA_OK;
    }
    if (p->nacc > 0 && (x3 || variant != BODA_VARIANT_TCONV || !halo_geometry(d, p->BN, p->nacc, p))) { delete p; return BODA_ERR_UNSUPPORTED; }
    p->iters_per_split = (p->iters_total + best_s - 1) / best_s;
    p->splits = (p->iters_total + p->iters_per_split - 1) / p->iters_per_split;   // no empty split
    p->tiles_n = (d.K + p->BN - 1) / p->BN;
    if (p->nacc > 0) {
        const long long mflat = (long long)d.N * p->Hp * p->Wp;
        p->tiles_m = (int)((mflat + 128 * p->nacc - 1) / (128 * p->nacc));
        p->xp_bytes = (((size_t)mflat * p->Cp * 4) + 1023) & ~(size_t)1023;
        p->partial_bytes = 0;   // split partial sums stay in shared memory (cluster reduction)
    } else {
        p->tiles_m = (d.M + BM - 1) / BM;
        p->xp_bytes = (((size_t)d.N * d.H * d.W * p->Cs() * p->esize()) + 1023) & ~(size_t)1023;
        p->partial_bytes = 0;   // split partial sums stay in shared memory (cluster reduction)
    }

    if (max_ws > 0 && p->xp_bytes > max_ws) { delete p; return BODA_ERR_NOMEM; }
    p->wp_bytes = (size_t)d.R * d.S * d.K * p->Cs() * p->esize();
    cudaError_t e = cudaMalloc(&p->d_wp, p->wp_bytes);
    if (e != cudaSuccess) { igemm_plan_destroy(p); return record_cuda_error(e, "igemm plan allocation"); }
    rc = encode_map_b(p);
    if (rc != BODA_OK) { igemm_plan_destroy(p); return rc; }
    *out = p;
    return BODA_OK;
}

void igemm_plan_destroy(IgemmPlan* p)
{
    if (!p) return;
    if (p->d_wp) cudaFree(p->d_wp);
    if (p->d_tab) cudaFree(p->d_tab);
    delete p;
}

int igemm_plan_tile(const IgemmPlan* p) { return p->tile_id; }
bool igemm_plan_writes_packed(const IgemmPlan* p) { return p->nacc != -2 && p->terms != 3 && !p->half; }
int igemm_plan_kernels_per_call(const IgemmPlan* p) { return (p->nacc < 0 || p->in_packed) ? 1 : 2; }
int igemm_plan_splits(const IgemmPlan* p) { return p->splits; }
size_t igemm_plan_workspace_bytes(const IgemmPlan* p) { return p->xp_bytes + p->partial_bytes; }

void igemm_plan_describe(const IgemmPlan* p, char* buf, size_t n)
{
    const char* view = p->s2d ? "s2d " : "";
    if (p->nacc == -3) {
        char pool[48] = "";
        if (p->pool_rows > 0) std::snprintf(pool, sizeof(pool), " +maxpool3x3s2(%d rows/tile)", p->pool_rows);
        std::snprintf(buf, n, "s2d tile=first_512x%d(id %d) taps=%dx%d rows/tile=%d stages=%d split_k=1 grid=%dx%dx1%s", p->BN, p->tile_id,
                      p->fl_Rb, p->fl_Sb, p->fl_rows_per_tile, p->b_stages, p->tiles_m, p->tiles_n, pool);
        return;
    }
    if (p->nacc == -2) {
        std::snprintf(buf, n, "tile=k1nchw_128x%d(id %d) stages=%d split_k=%d grid=%dx1x%d tiles=%d", p->BN, p->tile_id,
                      p->BN == 64 ? k1n::Cfg<64>::STAGES : p->BN == 128 ? k1n::Cfg<128>::STAGES : k1n::Cfg<192>::STAGES, p->splits,
                      p->splits > 1 ? p->tiles_m * p->tiles_n : std::min(p->tiles_m * p->tiles_n, p->sm_count), p->splits,
                      p->tiles_m * p->tiles_n);
        return;
    }
    if (p->nacc < 0) {
        const int tiles = p->tiles_m * p->tiles_n;
        std::snprintf(buf, n, "tile=gconv_128x%d(id %d) stages=%d split_k=1 grid=%dx1x1 tiles=%d", p->BN, p->tile_id,
                      p->BN <= 96 ? 5 : 4, std::min(tiles, p->sm_count), tiles);
        return;
    }
    if (p->nacc > 0) {
        char pool[48] = "";
        if (p->pool_rows > 0) std::snprintf(pool, sizeof(pool), " +maxpool3x3s2(%d rows/tile)", p->pool_rows);
        std::snprintf(buf, n, "%stile=halo_%dx%d(id %d) slab=%d stages=%d split_k=%d grid=%dx%dx%d%s", view, 128 * p->nacc, p->BN,
                      p->tile_id, p->slab_rows, p->b_stages, p->splits, p->tiles_m, p->tiles_n, p->splits, pool);
        return;
    }
    std::snprintf(buf, n, "%s%stile=igemm_128x%d(id %d) stages=%d split_k=%d grid=%dx%dx%d", view, p->half ? "f16 " : p->terms == 3 ? "x3 " : "", p->BN, p->tile_id,
                  p->BN == 64 ? TileCfg<64>::STAGES : p->BN == 96 ? TileCfg<96>::STAGES : p->BN == 128 ? TileCfg<128>::STAGES
                  : p->BN == 192 ? TileCfg<192>::STAGES : TileCfg<256>::STAGES,
                  p->splits, p->tiles_m, p->tiles_n, p->splits);
}

// fp16 operand staging (reduced-precision storage, the paper's Section 2 remark on 16-bit storage): the same two
// re-layouts with the values rounded to fp16 (nearest even) and channels padded to a multiple of 64
__global__ void __launch_bounds__(256)
pack_input_nhwc_half_kernel(const float* __restrict__ in, __half* __restrict__ xp, int C, int Cp, int HW)
{
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.z;
    const int hw0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float* src = in + (size_t)n * C * HW;
    __half* dst = xp + (size_t)n * HW * Cp;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, hw = hw0 + tx;
        tile[ty + 8 * i][tx] = (c < C && hw < HW) ? __ldg(src + (size_t)c * HW + hw) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int hw = hw0 + ty + 8 * i, c = c0 + tx;
        if (hw < HW) dst[(size_t)hw * Cp + c] = __float2half_rn(tile[tx][ty + 8 * i]);
    }
}

__global__ void __launch_bounds__(256)
pack_filters_half_kernel(const float* __restrict__ filt, __half* __restrict__ wp, int K, int C, int Cp, int RS)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)RS * K * Cp;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % Cp);
        const long long t = idx / Cp;
        const int k = (int)(t % K);
        const int tap = (int)(t / K);
        wp[idx] = __float2half_rn(c < C ? __ldg(filt + ((size_t)k * C + c) * RS + tap) : 0.f);
    }
}

// 1x1 filters with C a multiple of 4 are already [K][C] rows: the staging is a rounding copy, 16 bytes per thread
__global__ void __launch_bounds__(256)
pack_filters_1x1_kernel(const float4* __restrict__ filt, float* __restrict__ wp, int K, int C4, int Cp, int split)
{
    pdl_launch_dependents();
    pdl_wait();
    const int Cs = split ? 2 * Cp : Cp, Cp4 = Cp >> 2;
    const int total = K * Cp4;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int k = idx / Cp4, c4 = idx - k * Cp4;
        const float4 x = c4 < C4 ? __ldg(filt + (size_t)k * C4 + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 hi = make_float4(round_tf32(x.x), round_tf32(x.y), round_tf32(x.z), round_tf32(x.w));
        float* row = wp + (size_t)k * Cs;
        reinterpret_cast<float4*>(row)[c4] = hi;
        if (split)
            reinterpret_cast<float4*>(row + Cp)[c4] = make_float4(round_tf32(x.x - hi.x), round_tf32(x.y - hi.y),
                                                                  round_tf32(x.z - hi.z), round_tf32(x.w - hi.w));
    }
}

static int pack_filters(IgemmPlan* p, const float* filt, cudaStream_t stream)
{
    const ConvDims& d = p->d;
    const long long total = (long long)d.R * d.S * d.K * p->Cp;
    const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 8);
    if (p->nacc == -3) {
        const int fblocks = std::min((p->fl_Rb * p->fl_Sb * d.K * first::kViewChannels + 255) / 256, 148 * 8);
        BODA_CUDA_TRY(launch_kernel(first::pack_filters_first_layer_kernel, dim3(fblocks), dim3(256), 0, stream, 1, filt, p->d_wp,
                                    d.K, d.R, d.S, p->fl_Rb, p->fl_Sb));
    } else if (p->half) {
        BODA_CUDA_TRY(launch_kernel(pack_filters_half_kernel, dim3(blocks), dim3(256), 0, stream, 1, filt, reinterpret_cast<__half*>(p->d_wp),
                                    d.K, d.C, p->Cp, d.R * d.S));
    } else if (p->nacc == -1) {
        const int Kp = p->gather_chunks * 32;
        const int gblocks = (int)std::min<long long>(((long long)d.K * Kp + 255) / 256, 148 * 8);
        BODA_CUDA_TRY(launch_kernel(pack_filters_flat_kernel, dim3(gblocks), dim3(256), 0, stream, 1, filt, p->d_wp, d.K, d.Kred, Kp));
    } else if (p->s2d) {
        const ConvDims& o = p->orig;
        BODA_CUDA_TRY(launch_kernel(pack_filters_s2d_kernel, dim3(blocks), dim3(256), 0, stream, 1, filt, p->d_wp, o.K, o.C, o.R,
                                    o.S, o.stride, d.R, d.S, p->Cp));
    } else if (d.R * d.S == 1 && d.C % 4 == 0 && ((uintptr_t)filt & 15) == 0 && (long long)d.K * p->Cp < (1LL << 31)) {
        const int blocks4 = (int)std::min<long long>((total / 4 + 255) / 256, 148 * 8);
        BODA_CUDA_TRY(launch_kernel(pack_filters_1x1_kernel, dim3(blocks4), dim3(256), 0, stream, 1,
                                    reinterpret_cast<const float4*>(filt), p->d_wp, d.K, d.C / 4, p->Cp, p->terms == 3 ? 1 : 0));
    } else {
        BODA_CUDA_TRY(launch_kernel(pack_filters_kernel, dim3(blocks), dim3(256), 0, stream, 1, filt, p->d_wp, d.K, d.C, p->Cp,
                                    d.R * d.S, p->terms == 3 ? 1 : 0));
    }
    count_launch();
    return BODA_OK;
}

int igemm_bind_filters(IgemmPlan* p, const float* filt, cudaStream_t stream)
{
    int rc = pack_filters(p, filt, stream);
    if (rc != BODA_OK) return rc;
    // The kernels fetch bound filters without waiting for the preceding kernel in their stream (they are constants
    // by then): make sure the packing is not that predecessor.
    BODA_CUDA_TRY(cudaStreamSynchronize(stream));
    p->bound_filt = filt;
    return BODA_OK;
}

void igemm_unbind_filters(IgemmPlan* p) { p->bound_filt = nullptr; }

static OutSpec make_out_spec(const IgemmPlan* p, float* out)
{
    const ConvDims& d = p->d;
    OutSpec o;
    o.out = out;
    o.packed = p->out_packed;
    o.K = d.K; o.P = d.P; o.Q = d.Q; o.PQ = d.P * d.Q;
    if (p->pool_rows > 0) { o.P = p->poolP; o.Q = p->poolQ; o.PQ = p->poolP * p->poolQ; }   // the pooled tensor
    o.Hp = p->oHp; o.Wp = p->oWp; o.Cp = p->oCp;
    o.relu = d.relu;
    return o;
}

bool igemm_plan_input_geometry(const IgemmPlan* p, int* Hp, int* Wp, int* Cp)
{
    if (p->s2d || p->terms == 3 || p->half || p->nacc < 0) return false;   // space-to-depth staging, the hi/lo split, fp16 operands and the gather kernel read NCHW only
    if (p->nacc > 0) { *Hp = p->Hp; *Wp = p->Wp; } else { *Hp = p->d.H; *Wp = p->d.W; }
    *Cp = p->Cp;
    return true;
}

// Pooled rows per tile of the halo kernel when 3x3 / stride-2 pooling is fused into its epilogue; 0 if it cannot be:
// a tile of 128*nacc flat positions must hold 2*rows + 1 whole output rows, and two blocks of [positions][32 channels]
// plus the pooled tile must fit in the shared memory the operand buffers leave idle.
static int halo_pool_rows(const IgemmPlan* p, int ksz, int stride)
{
    const ConvDims& d = p->d;
    if (p->nacc == -3) {
        // the first-layer kernel's tiles are row-aligned already: a tile owns rows_per_tile / 2 pooled rows
        if (ksz != 3 || stride != 2 || d.P < 3 || d.Q < 3) return 0;
        const int rows = p->fl_rows_per_tile / 2, poolQ = (d.Q - 3) / 2 + 1;
        const long long region = (long long)p->fl_slab_rows * 128 + 2LL * p->fl_raw_buf + (long long)p->b_stages * p->BN * 128;
        return halo::pooled_epilogue_bytes(4, rows * poolQ, p->BN) <= region ? rows : 0;
    }
    if (p->nacc != 2 && p->nacc != 4) return 0;
    if (p->splits != 1 || ksz != 3 || stride != 2 || d.P < 3 || d.Q < 3) return 0;
    const int poolP = (d.P - 3) / 2 + 1, poolQ = (d.Q - 3) / 2 + 1;
    int rows = (128 * p->nacc - d.Q) / (2 * p->Wp);
    if (rows > poolP) rows = poolP;
    const long long region = (long long)halo::kASlots * p->a_slot_bytes + (long long)p->b_stages * p->BN * 128;
    while (rows >= 1 && halo::pooled_epilogue_bytes(p->nacc, rows * poolQ, p->BN) > region) --rows;
    return rows < 1 ? 0 : rows;
}

bool igemm_plan_can_fuse_pool(const IgemmPlan* p, int ksz, int stride) { return halo_pool_rows(p, ksz, stride) > 0; }

int igemm_plan_set_pool(IgemmPlan* p, int ksz, int stride)
{
    if (ksz == 0) {                       // back to the unfused form
        if (p->pool_rows > 0) p->tiles_m = p->nacc == -3 ? p->fl_tiles_unpooled : p->tiles_m_unpooled;
        p->pool_rows = p->tiles_per_image = p->poolP = p->poolQ = 0;
        return BODA_OK;
    }
    const int rows = halo_pool_rows(p, ksz, stride);
    if (rows <= 0) return BODA_ERR_UNSUPPORTED;
    if (p->pool_rows == 0) p->tiles_m_unpooled = p->tiles_m;
    p->pool_rows = rows;
    p->poolP = (p->d.P - 3) / 2 + 1;
    p->poolQ = (p->d.Q - 3) / 2 + 1;
    p->tiles_per_image = (p->poolP + rows - 1) / rows;
    p->tiles_m = p->d.N * p->tiles_per_image;
    return BODA_OK;
}

void igemm_plan_pooled_dims(const IgemmPlan* p, int* P, int* Q)
{
    if (p->pool_rows > 0) { *P = p->poolP; *Q = p->poolQ; } else { *P = p->d.P; *Q = p->d.Q; }
}

int igemm_plan_set_io(IgemmPlan* p, int in_packed, int out_packed, int oHp, int oWp, int oCp)
{
    if (in_packed && (p->s2d || p->nacc < 0)) return BODA_ERR_UNSUPPORTED;
    if ((in_packed || out_packed) && (p->terms == 3 || p->half)) return BODA_ERR_UNSUPPORTED;
    if (out_packed && p->nacc == -2) return BODA_ERR_UNSUPPORTED;        // that kernel's tiles follow images: NCHW output only
    const int outP = p->pool_rows > 0 ? p->poolP : p->d.P, outQ = p->pool_rows > 0 ? p->poolQ : p->d.Q;
    if (out_packed && (oCp % 32 != 0 || oCp < p->d.K || oHp < outP || oWp < outQ)) return BODA_ERR_INVALID_ARG;
    p->in_packed = in_packed != 0;
    p->out_packed = out_packed ? 1 : 0;
    p->oHp = oHp; p->oWp = oWp; p->oCp = oCp;
    p->map_o_base = nullptr;
    return BODA_OK;
}

int igemm_launch(IgemmPlan* p, const float* in, const float* filt, const float* bias, float* out, void* workspace,
                 cudaStream_t stream, cudaEvent_t after_staging)
{
    const ConvDims& d = p->d;
    const bool needs_staging = !p->in_packed && p->nacc >= 0;
    if (needs_staging && !workspace) return BODA_ERR_NOMEM;
    if (needs_staging && ((uintptr_t)workspace & 255) != 0) return BODA_ERR_INVALID_ARG;
    float* xp = p->in_packed ? const_cast<float*>(in) : (float*)workspace;
    if (filt != p->bound_filt || !filt) {
        if (!filt) return BODA_ERR_INVALID_ARG;
        int rc = pack_filters(p, filt, stream);       // unbound: re-layout on every call
        if (rc != BODA_OK) return rc;
    }
    if (p->nacc == -3) {
        if (((uintptr_t)in & 15) != 0) return BODA_ERR_INVALID_ARG;       // bulk copies start on 16-byte boundaries
        if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
        first::FirstParams fp;
        fp.h.Mflat = d.N * p->Hp * p->Wp; fp.h.HpWp = p->Hp * p->Wp; fp.h.Wp = p->Wp;
        fp.h.S = p->fl_Sb; fp.h.taps = p->fl_Rb * p->fl_Sb; fp.h.cchunks = 2; fp.h.lead = 0;
        fp.h.nbox = 0; fp.h.box_rows = 0; fp.h.a_slot_bytes = 0; fp.h.b_stages = p->b_stages;
        fp.h.iters_total = fp.h.iters_per_split = p->iters_total; fp.h.splits = 1;
        fp.h.bias = bias; fp.h.o = make_out_spec(p, out); fp.h.status = p->d_status; fp.h.tx_extra = p->tx_extra;
        fp.h.pool_rows = p->pool_rows; fp.h.tiles_per_image = p->tiles_m / d.N;
        fp.h.tile_positions = p->fl_rows_per_tile * p->Wp;
        fp.in = in; fp.H = d.H; fp.W = d.W;
        fp.rows_per_tile = p->fl_rows_per_tile; fp.raw_rows = p->fl_raw_rows; fp.raw_buf_bytes = p->fl_raw_buf;
        fp.slab_rows = p->fl_slab_rows; fp.b_stages = p->b_stages;
        fp.in_floats = (long long)d.N * d.C * d.H * d.W;
        switch (p->BN) {
            case 64: return launch_first_layer<64>(p, fp, stream);
            case 96: return launch_first_layer<96>(p, fp, stream);
            case 128: return launch_first_layer<128>(p, fp, stream);
            default: return BODA_ERR_UNSUPPORTED;
        }
    }
    if (p->nacc == -2) {
        if (p->map_a_base != in) {
            const int rc = encode_map_a_k1n(p, in);
            if (rc != BODA_OK) return rc;
        }
        if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
        k1n::K1nParams kp;
        kp.HW = d.H * d.W; kp.tiles_per_image = (kp.HW + BM - 1) / BM;
        kp.cchunks = p->Cp / BKC;
        kp.tiles_n = p->tiles_n; kp.tiles_total = p->tiles_m * p->tiles_n;
        kp.bias = bias;
        kp.o = make_out_spec(p, out);
        kp.status = p->d_status;
        kp.tx_extra = p->tx_extra;
        kp.b_early = (filt == p->bound_filt) ? 1 : 0;
        kp.splits = p->splits; kp.chunks_per_split = p->iters_per_split;
        switch (p->BN) {
            case 64: return launch_k1n<64>(p, kp, stream);
            case 128: return launch_k1n<128>(p, kp, stream);
            case 192: return launch_k1n<192>(p, kp, stream);
            default: return BODA_ERR_UNSUPPORTED;
        }
    }
    if (p->nacc < 0) {
        if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
        gconv::GconvParams gp;
        gp.in = in; gp.tab = p->d_tab; gp.bias = bias;
        gp.CHW = d.C * d.H * d.W; gp.H = d.H; gp.W = d.W; gp.R = d.R; gp.S = d.S; gp.stride = d.stride; gp.pad = d.pad;
        gp.M = d.M; gp.Kred = d.Kred; gp.nchunks = p->gather_chunks;
        gp.tiles_n = p->tiles_n; gp.tiles_total = p->tiles_m * p->tiles_n;
        gp.o = make_out_spec(p, out);
        gp.status = p->d_status;
        gp.tx_extra = p->tx_extra;
        gp.b_early = (filt == p->bound_filt) ? 1 : 0;
        switch (p->BN) {
            case 64: return launch_gather<64>(p, gp, stream);
            case 96: return launch_gather<96>(p, gp, stream);
            case 128: return launch_gather<128>(p, gp, stream);
            case 192: return launch_gather<192>(p, gp, stream);
            default: return BODA_ERR_UNSUPPORTED;
        }
    }
    if (p->s2d && !p->in_packed) {
        // both kernels read the same [N][H'][W'][Cp] layout here (the view has no padding)
        const ConvDims& o = p->orig;
        dim3 grid(d.H, d.N);
        const size_t smem = (size_t)o.C * o.stride * (((size_t)d.W * o.stride + 3) & ~(size_t)3) * 4;
        if (o.stride == 4 && o.C == 3 && p->Cp == 64)
            BODA_CUDA_TRY(launch_kernel(pack_input_s2d_t4_kernel<3>, grid, dim3(256), smem, stream, 1, in, xp, o.H, o.W, o.pad, d.H, d.W));
        else
            BODA_CUDA_TRY(launch_kernel(pack_input_s2d_kernel, grid, dim3(256), smem, stream, 1, in, xp, o.C, o.H, o.W, o.stride,
                                        o.pad, d.H, d.W, p->Cp));
        count_launch();
    }
    if (p->nacc > 0) {
        if (!p->s2d && !p->in_packed) {
            dim3 grid((p->Hp * p->Wp + 31) / 32, p->Cp / 32, d.N);
            BODA_CUDA_TRY(launch_kernel(halo::pack_input_halo_kernel, grid, dim3(256), 0, stream, 1, in, xp, d.C, p->Cp, d.H, d.W,
                                        p->Hp, p->Wp));
            count_launch();
        }
        if (p->map_a_base != xp) {
            int rc = encode_map_a_halo(p, xp);
            if (rc != BODA_OK) return rc;
        }
        if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
        halo::HaloParams hp;
        hp.Mflat = d.N * p->Hp * p->Wp; hp.HpWp = p->Hp * p->Wp; hp.Wp = p->Wp;
        hp.S = d.S; hp.taps = d.R * d.S; hp.cchunks = p->Cp / BKC; hp.lead = p->lead;
        hp.nbox = p->nbox; hp.box_rows = p->box_rows; hp.a_slot_bytes = p->a_slot_bytes; hp.b_stages = p->b_stages;
        hp.iters_total = p->iters_total; hp.iters_per_split = p->iters_per_split; hp.splits = p->splits;
        hp.bias = bias; hp.o = make_out_spec(p, out); hp.tx_extra = p->tx_extra;
        hp.status = p->d_status;
        hp.pool_rows = p->pool_rows; hp.tiles_per_image = p->tiles_per_image; hp.tile_positions = 128 * p->nacc;
        switch (p->BN * 10 + p->nacc) {
            case 641: return launch_halo<64, 1>(p, hp, stream);
            case 1281: return launch_halo<128, 1>(p, hp, stream);
            case 1921: return launch_halo<192, 1>(p, hp, stream);
            case 2561: return launch_halo<256, 1>(p, hp, stream);
            case 962: return launch_halo<96, 2>(p, hp, stream);
            case 1282: return launch_halo<128, 2>(p, hp, stream);
            case 1922: return launch_halo<192, 2>(p, hp, stream);
            case 2562: return launch_halo<256, 2>(p, hp, stream);
            case 644: return launch_halo<64, 4>(p, hp, stream);
            case 964: return launch_halo<96, 4>(p, hp, stream);
            case 1284: return launch_halo<128, 4>(p, hp, stream);
            default: return BODA_ERR_UNSUPPORTED;
        }
    }
    if (!p->s2d && !p->in_packed) {
        const int HW = d.H * d.W;
        dim3 grid((HW + 31) / 32, p->Cp / 32, d.N);
        if (p->half)
            BODA_CUDA_TRY(launch_kernel(pack_input_nhwc_half_kernel, grid, dim3(256), 0, stream, 1, in, reinterpret_cast<__half*>(xp), d.C, p->Cp, HW));
        else
            BODA_CUDA_TRY(launch_kernel(pack_input_nhwc_kernel, grid, dim3(256), 0, stream, 1, in, xp, d.C, p->Cp, HW, p->terms == 3 ? 1 : 0));
        count_launch();
    }
    if (p->map_a_base != xp) {
        int rc = encode_map_a(p, xp);
        if (rc != BODA_OK) return rc;
    }
    if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
    IgemmParams prm;
    prm.M = d.M; prm.stride = d.stride; prm.pad = d.pad; prm.S = d.S;
    prm.cchunks = p->Cp / p->chunk();
    prm.terms = p->terms;
    prm.lo_off = p->Cp;
    prm.iters_total = p->iters_total;
    prm.iters_per_split = p->iters_per_split;
    prm.splits = p->splits;
    prm.bias = bias;
    prm.o = make_out_spec(p, out);
    prm.tx_extra = p->tx_extra;
    prm.b_early = (filt == p->bound_filt) ? 1 : 0;
    prm.status = p->d_status;
    prm.out_tma = (p->out_packed && p->oHp == d.P && p->oWp == d.Q && ((uintptr_t)out & 15) == 0) ? 1 : 0;
    if (prm.out_tma && p->map_o_base != out) {
        int rc = encode_map_o(p, out);
        if (rc != BODA_OK) return rc;
    }
    switch (p->BN) {
        case 64: return launch_bn<64>(p, prm, stream);
        case 96: return launch_bn<96>(p, prm, stream);
        case 128: return launch_bn<128>(p, prm, stream);
        case 192: return launch_bn<192>(p, prm, stream);
        case 256: return launch_bn<256>(p, prm, stream);
        default: return BODA_ERR_UNSUPPORTED;
    }
}

#ifdef BODA_FL_PROF
extern "C" int boda_debug_cta_times(unsigned long long* out1024)
{
    return cudaMemcpyFromSymbol(out1024, halo::g_cta_times, sizeof(unsigned long long) * 1024) == cudaSuccess ? 0 : 3;
}
extern "C" int boda_debug_fl_prof(long long* out16)
{
    return cudaMemcpyFromSymbol(out16, halo::g_fl_prof, sizeof(long long) * 16) == cudaSuccess ? 0 : 3;
}
#endif

// ------------------------------------------------------------------------------------------------
// The same convolution with every piece of scratch (status word, re-laid-out filters and
// input, split partial sums) carved out of ONE device region handed in by the caller.  Nothing is
// allocated here; the region keeps its previous contents, so what must start at zero is cleared first.
size_t igemm_region_min_bytes(const ConvDims& d)
{
    const size_t Cp = (size_t)((d.C + BKC - 1) / BKC) * BKC;
    const size_t tiles = (size_t)((d.M + BM - 1) / BM) * (size_t)((d.K + 63) / 64);
    const size_t head = 256 + ((tiles * sizeof(int) + 255) & ~(size_t)255);
    const size_t wp = (((size_t)d.R * d.S * d.K * Cp * 4) + 1023) & ~(size_t)1023;
    const size_t xp = (((size_t)d.N * d.H * d.W * Cp * 4) + 1023) & ~(size_t)1023;
    return head + 1024 + wp + xp;
}

int igemm_run_in_region(const ConvDims& d, int variant, const float* in, const float* filt, const float* bias,
                        float* out, void* region, size_t region_bytes, cudaStream_t stream)
{
    if (!igemm_variant_legal(d, variant)) return BODA_ERR_UNSUPPORTED;
    if (!in || !filt || !out || !region || ((uintptr_t)region & 255) != 0) return BODA_ERR_INVALID_ARG;
    if (igemm_region_min_bytes(d) > region_bytes) return BODA_ERR_TOO_LARGE;
    int rc = load_driver_entry_points();
    if (rc != BODA_OK) return rc;

    IgemmPlan plan;                       // lives on the host stack for the duration of this call only
    IgemmPlan* p = &plan;
    p->d = d;
    p->orig = d;
    p->variant = variant;
    p->Cp = ((d.C + BKC - 1) / BKC) * BKC;
    p->iters_total = d.R * d.S * (p->Cp / BKC);
    p->tiles_m = (d.M + BM - 1) / BM;
    const size_t wp_bytes = (((size_t)d.R * d.S * d.K * p->Cp * 4) + 1023) & ~(size_t)1023;
    p->xp_bytes = (((size_t)d.N * d.H * d.W * p->Cp * 4) + 1023) & ~(size_t)1023;
    const size_t tiles_max = (size_t)p->tiles_m * (size_t)((d.K + 63) / 64);
    const size_t head_bytes = 256 + ((tiles_max * sizeof(int) + 255) & ~(size_t)255);
    if (head_bytes + 1024 + wp_bytes + p->xp_bytes > region_bytes) return BODA_ERR_TOO_LARGE;
    // tile and split by the cost model (split partial sums stay in shared memory: every choice fits the region)
    double best = 1e300;
    int best_t = -1, best_s = 1;
    for (int t = 0; t < kFirstHaloTile; ++t)
        for (int s : kSplitCandidates) {
            if (s > p->iters_total) continue;
            const double c = model_cost(d, p->Cp, kTileBN[t], s);
            if (c < best) { best = c; best_t = t; best_s = s; }
        }
    if (best_t < 0) return BODA_ERR_TOO_LARGE;
    p->tile_id = best_t;
    p->BN = kTileBN[best_t];
    p->iters_per_split = (p->iters_total + best_s - 1) / best_s;
    p->splits = (p->iters_total + p->iters_per_split - 1) / p->iters_per_split;
    p->tiles_n = (d.K + p->BN - 1) / p->BN;

    char* base = (char*)region;
    p->d_status = (int*)base;
    char* cur = (char*)(((uintptr_t)(base + head_bytes) + 1023) & ~(uintptr_t)1023);
    p->d_wp = (float*)cur;
    float* xp = (float*)(cur + wp_bytes);

    BODA_CUDA_TRY(cudaMemsetAsync(base, 0, head_bytes, stream));      // the status word starts at zero
    rc = encode_map_b(p);
    if (rc == BODA_OK) rc = encode_map_a(p, xp);
    if (rc == BODA_OK) rc = pack_filters(p, filt, stream);
    if (rc != BODA_OK) { p->d_wp = nullptr; return rc; }
    {
        const int HW = d.H * d.W;
        dim3 grid((HW + 31) / 32, p->Cp / 32, d.N);
        cudaError_t e = launch_kernel(pack_input_nhwc_kernel, grid, dim3(256), 0, stream, 1, in, xp, d.C, p->Cp, HW, 0);
        if (e != cudaSuccess) { p->d_wp = nullptr; return record_cuda_error(e, "pack_input_nhwc_kernel"); }
        count_launch();
    }
    IgemmParams prm;
    prm.M = d.M; prm.stride = d.stride; prm.pad = d.pad; prm.S = d.S;
    prm.cchunks = p->Cp / BKC;
    prm.terms = 1;
    prm.lo_off = 0;
    prm.iters_total = p->iters_total;
    prm.iters_per_split = p->iters_per_split;
    prm.splits = p->splits;
    prm.bias = bias;
    prm.o = make_out_spec(p, out);
    prm.b_early = 0;
    prm.out_tma = 0;
    prm.tx_extra = p->tx_extra;
    prm.status = p->d_status;
    switch (p->BN) {
        case 64: rc = launch_bn<64>(p, prm, stream); break;
        case 96: rc = launch_bn<96>(p, prm, stream); break;
        case 128: rc = launch_bn<128>(p, prm, stream); break;
        case 192: rc = launch_bn<192>(p, prm, stream); break;
        case 256: rc = launch_bn<256>(p, prm, stream); break;
        default: rc = BODA_ERR_UNSUPPORTED; break;
    }
    p->d_wp = nullptr;                    // the region is the caller's: nothing for a destructor to free
    return rc;
}

}  // namespace boda
