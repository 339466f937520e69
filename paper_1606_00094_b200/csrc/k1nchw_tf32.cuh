// K1CONV straight from NCHW: the 1x1 convolution as the per-image matrix product of Section 5 of the paper,
//   out[n][K x HW] = filt[K x C] * in[n][C x HW],
// with the input fetched by TMA from the tensor as it is - no staged copy, no gather.
//
// In NCHW the output points of one channel are contiguous and the channels are HW floats apart, so the input tile
// of the GEMM view [128 output points][32 channels] arrives "transposed": 32 rows (channels) of 128-byte pieces
// (32 output points).  The tensor core takes that as an MN-major operand: four TMA boxes of 32 channels x 32 points
// laid 4 KB apart (leading byte offset = 4096: the next 32 output points; stride byte offset = 512: the next 4
// channels), and one bit in the instruction descriptor.  MN-major TF32 operands exist in one shared-memory layout
// only: the 128-byte swizzle that permutes 32-byte pieces over 4 rows (tensor-map swizzle 128B_ATOM_32B, descriptor
// layout type 1); with the ordinary 128-byte swizzle the MMA returned zeros (measured).  The filters stay the K-major [K][Cp] operand
// of the other kernels (rounded to TF32 at bind time); the input is used as it is in memory, i.e. the tensor core
// drops the low 13 mantissa bits of each value (truncation instead of the staging kernels' round-to-nearest: up to
// 2^-10 relative per operand, inside the TF32 error bar).
// Tiles do not cross images: a tile is output points [128*t, 128*t + 128) of one image and BN output channels; points
// past HW are zero-filled by TMA and never stored.  Needs HW % 4 == 0 (TMA strides are multiples of 16 bytes).
// The kernel is persistent (at most one CTA per SM walks the tiles) with two accumulators in tensor memory, so that a
// tile's epilogue runs under the next tile's main loop.
// Roles (256 threads): warps 0 and 2 = input-tile producers (two boxes each), warp 3 = filter tile and byte count,
// warp 1 = TMEM owner and MMA issuer, warps 4..7 = epilogue.  Waits are bounded as in the other kernels.
#pragma once

#include "tc_ptx.cuh"

namespace boda {
namespace k1n {

using namespace tc;

constexpr int kThreads = 256;
constexpr int A_STAGE_BYTES = 128 * 128;
constexpr int A_BOX_BYTES = 32 * 128;

struct K1nParams {
    int HW, tiles_per_image;
    int tiles_n, tiles_total;    // tiles are numbered (image, point tile) * tiles_n + channel tile
    int cchunks;                 // ceil(C / 32)
    const float* bias;
    OutSpec o;                   // NCHW only
    int* status;
    int tx_extra;                // test hook: bytes added to the expected size of the first stage of CTA (0, 0)
    int b_early;                 // bound filters: the filter tiles' loads need not wait for the preceding kernel
    // reduction split over the CTAs of a cluster (grid.z = splits > 1: one tile per CTA, grid.x = tiles_total): CTA z
    // takes channel chunks [z*chunks_per_split, ...) and the partial sums are added through distributed shared memory
    int splits, chunks_per_split;
};

template <int BN> struct Cfg {
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES = (200 * 1024) / STAGE_BYTES > 8 ? 8 : (200 * 1024) / STAGE_BYTES;
    static constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512;      // two accumulators
    static constexpr int TMEM_COLS_ONE = BN <= 64 ? 64 : BN <= 128 ? 128 : 256;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// Shared-memory descriptor of the MN-major input tile: 128-byte rows (32 output points of one channel), 4-row groups
// 512 bytes apart along the channels, 32-point groups 4096 bytes apart along the output points, 128-byte swizzle of
// 32-byte pieces.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4)
         | ((uint64_t)(A_BOX_BYTES >> 4) << 16)    // leading byte offset: next group of 32 output points
         | ((uint64_t)(512 >> 4) << 32)            // stride byte offset: next group of 4 channels
         | (1ull << 46)                            // descriptor version of sm_100
         | (1ull << 61);                           // 128-byte swizzle of 32-byte pieces
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
k1nchw_tf32_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const K1nParams p)
{
    using C = Cfg<BN>;
    constexpr int kStages = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_base + kStages * A_STAGE_BYTES;
    const uint32_t bars = smem_base + kStages * C::STAGE_BYTES;
    const uint32_t full_bar = bars;
    const uint32_t empty_bar = bars + 8 * kStages;
    const uint32_t acc_full = bars + 16 * kStages;          // 2: the tile's MMAs have drained
    const uint32_t acc_empty = acc_full + 16;               // 2: the 4 epilogue warps have read the accumulator
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ __align__(16) float s_bias[BN];

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // persistent: this CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...; tile = (image, point tile) * tiles_n + channel tile
    const int my_tiles = ((int)blockIdx.x < p.tiles_total) ? (p.tiles_total - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int i_begin = p.splits > 1 ? (int)blockIdx.z * p.chunks_per_split : 0;
    const int steps = p.splits > 1 ? min(p.cchunks, i_begin + p.chunks_per_split) - i_begin : p.cchunks;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    // one accumulator is enough where no CTA has a second tile
    const uint32_t tmem_cols = (p.tiles_total > (int)gridDim.x) ? (uint32_t)C::TMEM_COLS : (uint32_t)C::TMEM_COLS_ONE;
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = s_tmem_base;
    // tile t of this CTA -> image, first output point, first output channel (the first tile's before the dependency wait)
    auto decode = [&](int t, int& n, int& hw0, int& k0) {
        const int tile = (int)blockIdx.x + t * (int)gridDim.x;
        const int mt = tile / p.tiles_n;
        k0 = (tile - mt * p.tiles_n) * BN;
        n = mt / p.tiles_per_image;
        hw0 = (mt - n * p.tiles_per_image) * 128;
    };
    int n, hw0, k0;
    decode(0, n, hw0, k0);
    if (!(p.b_early && warp == 3)) pdl_wait();

    if (warp == 0 || warp == 2) {
        if (lane == 0) {
            // ---------------- input tiles: boxes of 32 output points x 32 channels; warp 0 loads points 0..63, warp 2 points 64..127
            const int half = warp == 0 ? 0 : 2;
            uint32_t stage = 0, par = 1;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                if (t > 0) decode(t, n, hw0, k0);
                for (int i = 0; i < steps; ++i) {
                    ok = mbar_wait(empty_bar + 8 * stage, par, &s_abort, p.status, 41);
                    if (!ok) break;
                    const uint32_t dst = smem_a + stage * A_STAGE_BYTES + (uint32_t)half * A_BOX_BYTES;
                    tma_load_3d(dst, &map_a, full_bar + 8 * stage, hw0 + 32 * half, 32 * (i_begin + i), n);
                    tma_load_3d(dst + A_BOX_BYTES, &map_a, full_bar + 8 * stage, hw0 + 32 * half + 32, 32 * (i_begin + i), n);
                    if (++stage == (uint32_t)kStages) { stage = 0; par ^= 1u; }
                }
            }
        }
    } else if (warp == 3) {
        if (lane == 0) {
            // ---------------- filter tiles and the stage's byte count
            uint32_t stage = 0, par = 1;
            uint32_t bytes = C::STAGE_BYTES + (blockIdx.x == 0 ? (uint32_t)p.tx_extra : 0u);
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                if (t > 0) decode(t, n, hw0, k0);
                for (int i = 0; i < steps; ++i) {
                    ok = mbar_wait(empty_bar + 8 * stage, par, &s_abort, p.status, 42);
                    if (!ok) break;
                    mbar_expect_tx(full_bar + 8 * stage, bytes);
                    bytes = C::STAGE_BYTES;
                    tma_load_3d(smem_b + stage * C::B_STAGE_BYTES, &map_b, full_bar + 8 * stage, 32 * (i_begin + i), k0, 0);
                    if (++stage == (uint32_t)kStages) { stage = 0; par ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer: A is MN-major (bit 15 of the instruction descriptor), B K-major; tile t
            // accumulates in slot t & 1, so that its epilogue runs under the next tile's main loop
            constexpr uint32_t idesc = instr_desc_tf32<BN>() | (1u << 15);
            const uint64_t da0 = smem_desc_mn_sw128(smem_a), db0 = smem_desc_k_sw128(smem_b);
            uint32_t stage = 0, par = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const uint32_t slot = (uint32_t)t & 1u;
                ok = mbar_wait(acc_empty + 8 * slot, ((uint32_t)(t >> 1) & 1u) ^ 1u, &s_abort, p.status, 44);
                if (!ok) break;
                tc_fence_after();
                const uint32_t acc = tmem_acc + slot * (uint32_t)BN;
                for (int i = 0; i < steps; ++i) {
                    ok = mbar_wait(full_bar + 8 * stage, par, &s_abort, p.status, 43);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t da = da0 + (uint64_t)stage * (A_STAGE_BYTES >> 4);
                    const uint64_t db = db0 + (uint64_t)stage * (C::B_STAGE_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k)       // 8 channels per MMA: 8 rows of 128 bytes further in A, 32 bytes further in B's rows
                        umma_tf32(acc, da + (uint64_t)k * (1024 >> 4), db + 2 * k, idesc, (i | k) ? 1u : 0u);
                    tc_commit(empty_bar + 8 * stage);
                    if (++stage == (uint32_t)kStages) { stage = 0; par ^= 1u; }
                }
                if (ok) tc_commit(acc_full + 8 * slot);
            }
        }
    } else {
        // ---------------- epilogue: warps 4..7, warp w reads TMEM lanes 32*(w%4) .. +31 = output points hw0 + that
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        for (int t = 0; t < my_tiles; ++t) {
            if (t > 0) decode(t, n, hw0, k0);
            const uint32_t slot = (uint32_t)t & 1u;
            if (t > 0) asm volatile("bar.sync 1, 128;" ::: "memory");          // the previous tile's bias reads are over
            for (int j = (int)threadIdx.x - 128; j < BN; j += 128)
                s_bias[j] = (p.bias && k0 + j < p.o.K) ? __ldg(p.bias + k0 + j) : 0.f;
            if (lane == 0) (void)mbar_wait_relaxed(acc_full + 8 * slot, (uint32_t)(t >> 1) & 1u, &s_abort, p.status, 45);
            __syncwarp();
            uint32_t stop;
            asm volatile("{\n\t.reg .pred q, r;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred r, 1, 128, q;\n\tselp.u32 %0, 1, 0, r;\n\t}"
                         : "=r"(stop) : "r"((uint32_t)s_abort) : "memory");
            if (stop) break;
            tc_fence_after();
            const uint32_t trow = tmem_acc + ((uint32_t)(quarter * 32) << 16) + slot * (uint32_t)BN;
            const int hw = hw0 + row;
            const RowDst d = row_dst(p.o, hw < p.HW, n, 0, hw);
            if (p.splits > 1) {
                // split reduction, step 1: park the partial accumulator in this CTA's shared memory (the stages are idle:
                // a split CTA has one tile); the cluster-wide sum follows after the role branches
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32cols(trow + 32 * c, v);
                    tmem_ld_wait();
                    stash_row32<BN>(smem_base, row, 32 * c, v);
                }
                break;
            }
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32cols(trow + 32 * c, v);
                tmem_ld_wait();
                float y[32];
                bias_relu32(v, s_bias + 32 * c, p.o.relu != 0, y);
                store_row32(p.o, d, k0 + 32 * c, y);
            }
            // the accumulator has been read: hand the slot back to the issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(acc_empty + 8 * slot) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (p.splits > 1) {
        // step 2: every CTA of the cluster sums its share of the channels over all peers' parked accumulators in rank
        // order (the result does not depend on which CTA sums), adds the bias, applies ReLU and stores
        cluster_sync_all();
        if (warp >= 4 && s_abort == 0) {
            const int row = (warp & 3) * 32 + lane;
            const int hw = hw0 + row;
            cluster_reduce_store<BN>(smem_base, row, cluster_cta_rank(), p.splits, row_dst(p.o, hw < p.HW, n, 0, hw), p.o, k0, s_bias);
        }
        cluster_sync_all();          // nobody leaves while a peer may still read its shared memory
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, tmem_cols);
    }
}

}  // namespace k1n
}  // namespace boda
