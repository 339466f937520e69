// TCONV for layers with few input channels (first layers such as 11x11 stride 4 on 3 channels): the input tile
// of the implicit GEMM is GATHERED from the NCHW tensor by producer warps instead of being fetched by TMA.
//
// With C = 3 a channels-innermost staged copy of the input is almost all padding (3 of 32 channels), and the
// space-to-depth view that avoids it costs a staging kernel, a 16.6 MB staged tensor and 1.59x the layer's own
// multiply-accumulates.  Here nothing is staged: the reduction index is the flattened (c, r, s) of the filter
// tensor itself - so the filters [K][C*R*S] are already the K-major B operand, only rounded to TF32 and padded to a
// multiple of 32 - and twelve producer warps build each A tile [128 output points][32 reduction indices] in shared
// memory with ordinary loads (a table gives the element offset of every reduction index; consecutive output
// points of a row read addresses `stride` floats apart, which L1 serves), round to TF32 and write the 128-byte
// swizzled layout that the tensor core's descriptor expects; a proxy fence and an mbarrier hand the stage to the
// MMA-issuing thread.  This is the paper's "no explicit inmat" (Section 3) taken literally: the patch matrix
// exists only as shared-memory tiles.
//
// The kernel is persistent: a CTA walks the tiles blockIdx.x, blockIdx.x + gridDim.x, ... with two accumulators in
// tensor memory, so that the epilogue of one tile runs under the main loop of the next.
// Roles (576 threads): warp 0 = filter-tile TMA producer (one lane), warp 1 = TMEM owner and MMA issuer (one lane),
// warps 2..5 = epilogue, warps 6..17 = gather producers in three groups of four warps (a group builds one stage;
// warp g*4 + j takes rows 32*j .. 32*j + 31).  Every wait is bounded as in the other tensor-core kernels.
#pragma once

#include "tc_ptx.cuh"

namespace boda {
namespace gconv {

using namespace tc;

constexpr int kGroups = 3;
constexpr int kFirstProducerWarp = 6;
constexpr int kThreads = 32 * (kFirstProducerWarp + 4 * kGroups);      // 576
constexpr int A_STAGE_BYTES = 128 * 128;
constexpr int kMaxKred = 1536;          // reduction indices (C*R*S rounded up to 32) the shared-memory table holds

struct GconvParams {
    const float* in;             // NCHW fp32
    const int2* tab;             // per reduction index k (padded to nchunks*32): {element offset c*H*W + r*W + s, (r << 16) | s};
                                 // indices past C*R*S carry r = 0x4000 so that the bounds test fails
    const float* bias;
    int CHW, H, W, R, S, stride, pad;
    int M;                       // N * P * Q output points
    int Kred, nchunks;           // C*R*S and ceil(C*R*S / 32)
    int tiles_n, tiles_total;    // tiles are numbered m_tile * tiles_n + n_tile
    OutSpec o;
    int* status;
    int tx_extra;                // test hook: bytes added to the expected size of the first filter tile of CTA 0
    int b_early;                 // bound filters: the filter tiles' loads need not wait for the preceding kernel
};

template <int BN> struct Cfg {
    static constexpr int STAGES = BN <= 96 ? 5 : 4;        // what fits beside the output tile and the table
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512;
    // the staged-layout output tile; the widest tile has no room for one and stores from registers instead
    static constexpr uint32_t OUT_TILE_BYTES = BN <= 128 ? 128u * out_tile_row_bytes<BN>() : 0u;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + (int)OUT_TILE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
gconv_tf32_kernel(const __grid_constant__ CUtensorMap map_b, const GconvParams p)
{
    using C = Cfg<BN>;
    constexpr int kStages = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_base + kStages * A_STAGE_BYTES;
    const uint32_t smem_out = smem_base + kStages * C::STAGE_BYTES;
    const uint32_t bars = smem_out + C::OUT_TILE_BYTES;
    const uint32_t full_bar = bars;                         // kStages: 4 producer-warp arrivals + the filter tile's byte count
    const uint32_t empty_bar = bars + 8 * kStages;          // kStages: one commit
    const uint32_t acc_full = bars + 16 * kStages;          // 2: the tile's MMAs have drained
    const uint32_t acc_empty = acc_full + 16;               // 2: the 4 epilogue warps have read the accumulator
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ __align__(16) float s_bias[BN];
    __shared__ __align__(16) int s_off[kMaxKred];           // element offset of every reduction index
    __shared__ int s_rs[kMaxKred];                          // its tap (r << 16) | s

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int my_tiles = ((int)blockIdx.x < p.tiles_total) ? (p.tiles_total - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int nchunks = p.nchunks;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar + 8 * s, 5); mbar_init(empty_bar + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), C::TMEM_COLS);
        tmem_relinquish();
    }
    // the table and the filters are the plan's own data, not a predecessor's output: read before the dependency wait
    for (int k = threadIdx.x; k < nchunks * 32; k += kThreads) {
        const int2 e = __ldg(p.tab + k);
        s_off[k] = e.x;
        s_rs[k] = e.y;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = s_tmem_base;
    if (!(p.b_early && warp == 0)) pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- filter tiles by TMA, one per stage; this arrival also carries the byte count
            uint32_t stage = 0, par = 1;
            bool first = true;
            for (int t = 0; t < my_tiles; ++t) {
                const int tile = (int)blockIdx.x + t * (int)gridDim.x;
                const int k0 = (tile % p.tiles_n) * BN;
                bool ok = true;
                for (int j = 0; j < nchunks; ++j) {
                    ok = mbar_wait(empty_bar + 8 * stage, par, &s_abort, p.status, 21);
                    if (!ok) break;
                    mbar_expect_tx(full_bar + 8 * stage, (uint32_t)C::B_STAGE_BYTES + ((first && blockIdx.x == 0) ? (uint32_t)p.tx_extra : 0u));
                    first = false;
                    tma_load_2d(smem_b + stage * C::B_STAGE_BYTES, &map_b, full_bar + 8 * stage, 32 * j, k0);
                    if (++stage == (uint32_t)kStages) { stage = 0; par ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            constexpr uint32_t idesc = instr_desc_tf32<BN>();
            const uint64_t da0 = smem_desc_k_sw128(smem_a), db0 = smem_desc_k_sw128(smem_b);
            uint32_t stage = 0, par = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const uint32_t slot = (uint32_t)t & 1u;
                // the accumulator slot is free once the epilogue of the tile two back has read it
                ok = mbar_wait(acc_empty + 8 * slot, ((uint32_t)(t >> 1) & 1u) ^ 1u, &s_abort, p.status, 22);
                if (!ok) break;
                tc_fence_after();
                const uint32_t acc = tmem_acc + slot * (uint32_t)BN;
                for (int j = 0; j < nchunks; ++j) {
                    ok = mbar_wait(full_bar + 8 * stage, par, &s_abort, p.status, 23);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t da = da0 + (uint64_t)stage * (A_STAGE_BYTES >> 4);
                    const uint64_t db = db0 + (uint64_t)stage * (C::B_STAGE_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_tf32(acc, da + 2 * k, db + 2 * k, idesc, (j | k) ? 1u : 0u);
                    tc_commit(empty_bar + 8 * stage);
                    if (++stage == (uint32_t)kStages) { stage = 0; par ^= 1u; }
                }
                if (ok) tc_commit(acc_full + 8 * slot);
            }
        }
    } else if (warp < kFirstProducerWarp) {
        // ---------------- epilogue: warps 2..5, warp w reads TMEM lanes 32*(w%4) .. +31
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t row_addr = smem_out + (uint32_t)row * out_tile_row_bytes<BN>();
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = (int)blockIdx.x + t * (int)gridDim.x;
            const int m0 = (tile / p.tiles_n) * 128, k0 = (tile % p.tiles_n) * BN;
            const uint32_t slot = (uint32_t)t & 1u;
            // bias of this tile's channels (the four warps share it; the named barrier below orders it)
            asm volatile("bar.sync 1, 128;" ::: "memory");          // the previous tile's bias reads are over
            for (int j = threadIdx.x - 64; j < BN; j += 128)
                s_bias[j] = (p.bias && k0 + j < p.o.K) ? __ldg(p.bias + k0 + j) : 0.f;
            if (lane == 0) (void)mbar_wait_relaxed(acc_full + 8 * slot, (uint32_t)(t >> 1) & 1u, &s_abort, p.status, 24);
            __syncwarp();
            // one common decision of the four warps (a barrier with an OR reduction): if any of them sees the abort
            // flag they all leave, so that nobody is left alone at the next barrier
            uint32_t stop;
            asm volatile("{\n\t.reg .pred q, r;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred r, 1, 128, q;\n\tselp.u32 %0, 1, 0, r;\n\t}"
                         : "=r"(stop) : "r"((uint32_t)s_abort) : "memory");
            if (stop) break;
            tc_fence_after();
            const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16) + slot * (uint32_t)BN;
            const int m = m0 + row;
            RowDst d;
            {
                const bool valid = m < p.M;
                int n = 0, pp = 0, qq = 0;
                if (valid) {
                    n = m / p.o.PQ;
                    const int pq = m - n * p.o.PQ;
                    pp = pq / p.o.Q;
                    qq = pq - pp * p.o.Q;
                }
                d = row_dst(p.o, valid, n, pp, qq);
            }
            const bool via_tile = C::OUT_TILE_BYTES != 0 && p.o.packed;     // staged rows leave through shared memory as bulk copies
            if (via_tile && t > 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // this row's slot is free again
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32cols(trow + 32 * c, v);
                tmem_ld_wait();
                float y[32];
                bias_relu32(v, s_bias + 32 * c, p.o.relu != 0, y);
                if (via_tile) out_tile_put32(row_addr, 32 * c, y);
                else store_row32(p.o, d, k0 + 32 * c, y);
            }
            // the accumulator has been read: hand the slot back to the issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(acc_empty + 8 * slot) : "memory");
            if (via_tile) {
                fence_proxy_async_smem();
                out_tile_store_row(p.o, d, k0, BN, row_addr);
                bulk_commit();
            }
        }
        if (C::OUT_TILE_BYTES != 0 && p.o.packed) bulk_wait_all();
    } else {
        // ---------------- gather producers: group g builds the stages of chunks g, g + 3, ... of the CTA's chunk sequence
        const int pw = warp - kFirstProducerWarp;
        const int group = pw >> 2, row = (pw & 3) * 32 + lane;
        const uint32_t sw = (uint32_t)(row & 7);
        const int total_chunks = my_tiles * nchunks;
        int cur_t = -1;
        long long base = 0;
        int y0 = 0, x0 = 0;
        bool valid = false, check_all = false;
        for (int gc = group; gc < total_chunks; gc += kGroups) {
            const int t = gc / nchunks, j = gc - t * nchunks;
            const uint32_t stage = (uint32_t)gc % (uint32_t)kStages, par = (((uint32_t)gc / (uint32_t)kStages) & 1u) ^ 1u;
            if (t != cur_t) {
                cur_t = t;
                const int tile = (int)blockIdx.x + t * (int)gridDim.x;
                const int m = (tile / p.tiles_n) * 128 + row;
                valid = m < p.M;
                if (valid) {
                    const int n = m / p.o.PQ;
                    const int pq = m - n * p.o.PQ;
                    const int pp = pq / p.o.Q, qq = pq - pp * p.o.Q;
                    y0 = pp * p.stride - p.pad;
                    x0 = qq * p.stride - p.pad;
                    base = (long long)n * p.CHW + (long long)y0 * p.W + x0;
                }
                // bounds tests are needed only where a window of this warp's 32 output points leaves the image
                const bool inside = !valid || (y0 >= 0 && y0 + p.R <= p.H && x0 >= 0 && x0 + p.S <= p.W);
                check_all = !__all_sync(0xffffffffu, inside);
            }
            const float* src = p.in + base;
            const int kk0 = 32 * j;
            float v[32];
            if (!check_all && kk0 + 32 <= p.Kred) {
                // no padding and no ragged end: every tap of a valid output point lies inside the image
                if (valid) {
#pragma unroll
                    for (int g4 = 0; g4 < 8; ++g4) {
                        const int4 off = *reinterpret_cast<const int4*>(&s_off[kk0 + 4 * g4]);
                        v[4 * g4] = __ldg(src + off.x); v[4 * g4 + 1] = __ldg(src + off.y);
                        v[4 * g4 + 2] = __ldg(src + off.z); v[4 * g4 + 3] = __ldg(src + off.w);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.f;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int rs = s_rs[kk0 + i];
                    const int y = y0 + (rs >> 16), x = x0 + (rs & 0xffff);
                    v[i] = (valid && (unsigned)y < (unsigned)p.H && (unsigned)x < (unsigned)p.W) ? __ldg(src + s_off[kk0 + i]) : 0.f;
                }
            }
            // the loads above are in flight while this waits for the stage to be free
            // one poller per warp and a warp-wide decision: no lane is left behind at the __syncwarp below
            int free_now = 0;
            if (lane == 0) free_now = mbar_wait(empty_bar + 8 * stage, par, &s_abort, p.status, 25) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, free_now, 0)) break;
            __syncwarp();     // orders the other lanes' stores below after lane 0's acquire of the empty barrier
            // 128-byte swizzle: 16-byte piece c of row `row` lives at piece c ^ (row & 7)
            const uint32_t a_row = smem_a + stage * A_STAGE_BYTES + (uint32_t)row * 128u;
#pragma unroll
            for (int g4 = 0; g4 < 8; ++g4)
                st_shared_v4(a_row + (((uint32_t)g4 ^ sw) << 4), round_to_tf32(v[4 * g4]), round_to_tf32(v[4 * g4 + 1]),
                             round_to_tf32(v[4 * g4 + 2]), round_to_tf32(v[4 * g4 + 3]));
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(full_bar + 8 * stage) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, C::TMEM_COLS);
    }
}

}  // namespace gconv
}  // namespace boda
