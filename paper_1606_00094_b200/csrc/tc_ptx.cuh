// PTX wrappers shared by the tensor-core kernels: mbarrier, TMA, tcgen05 (TMEM allocation, MMA, commit, load)
// and the shared-memory / instruction descriptors of the TF32 UMMA.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "boda_internal.h"

namespace boda {
namespace tc {

constexpr long long kWaitLimitCycles = 4000000000ll;
// The limit actually used (SM cycles).  Tests shorten it through the environment variable BODA_WAIT_LIMIT_CYCLES.
__constant__ long long c_wait_limit_cycles = kWaitLimitCycles;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the CTA is aborting or the limit expired (then it raises the abort flag
// and records where it gave up).  The limit is counted on the SM's own cycle counter, which is cheap to read
// (the global nanosecond timer is not, and must stay out of the fast path): 4e9 cycles, about two seconds.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int where)
{
    long long t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 255u) == 0u) {
            if (*abort_flag) return false;
            if (spin == 256u) {
                t0 = clock64();
            } else if (clock64() - t0 > c_wait_limit_cycles) {
                *abort_flag = 1;
                if (atomicCAS(status, 0, (int)BODA_ERR_DEVICE_TIMEOUT) == 0) {
                    status[1] = KERNEL_ID_IGEMM;
                    status[2] = (int)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z));
                    status[3] = where;
                }
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int where)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, where);
}

// Bounded wait for threads that are not on the critical path (the epilogue waiting for the accumulator):
// polls rarely and sleeps in between, so that it does not compete with the producer's and the MMA issuer's
// barrier traffic.  The limit is the same number of cycles, counted in sleep quanta.
__device__ __noinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int where)
{
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > c_wait_limit_cycles) {
            *abort_flag = 1;
            if (atomicCAS(status, 0, (int)BODA_ERR_DEVICE_TIMEOUT) == 0) {
                status[1] = KERNEL_ID_IGEMM;
                status[2] = (int)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z));
                status[3] = where;
            }
            return false;
        }
        __nanosleep(200);
    }
}

__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w,
                                                   int h, int n, uint16_t off_w, uint16_t off_h)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        :: "r"(dst), "l"((uint64_t)map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        :: "r"(dst), "l"((uint64_t)map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];"
        :: "r"(dst), "l"((uint64_t)map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], TF32 operands, 128 x N x 8 per instruction
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with fp16 operands: 128 x N x 16 per instruction
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld_32cols(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled, with
// 8-row groups 1024 bytes apart (the layout both TMA loads above produce).
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4)      // start address, 16-byte units
         | (1ull << 16)                            // leading byte offset (unused for swizzled K-major)
         | ((uint64_t)(1024 >> 4) << 32)           // stride byte offset: next 8-row group
         | (1ull << 46)                            // descriptor version of sm_100
         | (2ull << 61);                           // 128-byte swizzle
}

// ---- thread-block cluster helpers (split reductions through distributed shared memory)
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared-memory address of the same variable in the CTA of the given rank of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" :: "r"(addr), "f"(v) : "memory");
}

__device__ __forceinline__ float4 ld_cluster_v4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" :: "r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
// the two halves of a cluster barrier: work placed between them overlaps the wait for the slowest CTA
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }

// ---- bulk copies out of shared memory (asynchronous proxy).  Addresses and sizes are multiples of 16 bytes.
// Writes made with ordinary stores become visible to the copy engine after this fence.
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// shared memory of this CTA -> global memory; completion is tracked by the thread's bulk group
__device__ __forceinline__ void bulk_store_global(void* gdst, uint32_t smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(gdst), "r"(smem_src), "r"(bytes) : "memory");
}
// a box of shared memory (laid out as the map's swizzle says) -> the tensor at (x, y); x * element size must be a
// multiple of 16 bytes, and elements of the box outside the tensor are not written
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t smem_src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 :: "l"(map), "r"(smem_src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// shared memory of this CTA -> shared memory of a CTA of the cluster (`dst` and `bar` are cluster addresses from
// map_to_cta); the bytes are counted on the destination CTA's mbarrier `bar`
__device__ __forceinline__ void bulk_push_cluster(uint32_t dst, uint32_t smem_src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "r"(smem_src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ float round_to_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// y[0..31] = acc[0..31] + bias[0..31], then ReLU if asked.  The bias (shared memory, 16-byte aligned, the same
// address in every lane) is read four values per load: a broadcast load costs about seven issue slots of the
// shared-memory pipe whatever its width, and one per element was a third of the epilogue's time.
__device__ __forceinline__ void bias_relu32(const uint32_t (&v)[32], const float* bias32, bool relu, float (&y)[32])
{
    const float4* b4 = reinterpret_cast<const float4*>(bias32);
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const float4 b = b4[g];
        y[4 * g] = __uint_as_float(v[4 * g]) + b.x;
        y[4 * g + 1] = __uint_as_float(v[4 * g + 1]) + b.y;
        y[4 * g + 2] = __uint_as_float(v[4 * g + 2]) + b.z;
        y[4 * g + 3] = __uint_as_float(v[4 * g + 3]) + b.w;
    }
    if (relu) {
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = fmaxf(y[j], 0.f);
    }
}

// ---- where a tensor-core kernel writes its output tile (fused bias + ReLU epilogue, Section 2 of the paper)
struct OutSpec {
    float* out;
    int packed;          // 0: NCHW [N][K][P][Q] fp32.  1: the next layer's staged input, rows [(n*Hp + p)*Wp + q][Cp]
                         //    of fp32 values rounded to TF32 (padding rows, columns and channels are never written)
    int K, P, Q, PQ;
    int Hp, Wp, Cp;      // packed geometry
    int relu;
};
struct RowDst { bool valid; size_t base; };

__device__ __forceinline__ RowDst row_dst(const OutSpec& o, bool valid, int n, int pp, int qq)
{
    RowDst d;
    d.valid = valid;
    d.base = !valid ? 0 : o.packed ? ((size_t)(n * o.Hp + pp) * o.Wp + qq) * (size_t)o.Cp
                                   : (size_t)n * o.K * o.PQ + (size_t)pp * o.Q + qq;
    return d;
}

// 32 consecutive output channels kc .. kc+31 of one output row (one row per lane; bias and ReLU already applied).
// NCHW: lane = pixel, so each of the 32 stores of a lane joins its neighbours' into one 128-byte line.
// Staged layout: see below.
__device__ __forceinline__ void store_row32(const OutSpec& o, const RowDst& d, int kc, const float (&y)[32])
{
    if (o.packed) {
        // channels are innermost: the lane's 32 values are 128 contiguous bytes; four 32-byte stores, each a whole sector
        if (d.valid && kc < o.Cp) {    // Cp is a multiple of 32; channels K..Cp-1 hold exact zeros here (zero filters, zero bias)
            float* dst = o.out + d.base + kc;
#pragma unroll
            for (int g = 0; g < 4; ++g)
                asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                             :: "l"(dst + 8 * g), "f"(round_to_tf32(y[8 * g])), "f"(round_to_tf32(y[8 * g + 1])),
                                "f"(round_to_tf32(y[8 * g + 2])), "f"(round_to_tf32(y[8 * g + 3])), "f"(round_to_tf32(y[8 * g + 4])),
                                "f"(round_to_tf32(y[8 * g + 5])), "f"(round_to_tf32(y[8 * g + 6])), "f"(round_to_tf32(y[8 * g + 7]))
                             : "memory");
        }
    } else if (d.valid) {
        float* oj = o.out + d.base + (size_t)kc * o.PQ;
        if (kc + 32 <= o.K) {
#pragma unroll
            for (int j = 0; j < 32; ++j) oj[(size_t)j * o.PQ] = y[j];
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (kc + j < o.K) oj[(size_t)j * o.PQ] = y[j];
        }
    }
}

// ---- split reduction of one 128-row accumulator over the CTAs of a cluster (one CTA per reduction split).
// Step 1: every CTA parks its partial accumulator in its own shared memory, column-major [channel][128 rows]:
// a warp (32 consecutive rows) then touches 128 contiguous bytes per channel, both when it writes here and when a
// peer reads it through distributed shared memory (remote reads want to be coalesced like global ones).
template <int BN>
__device__ __forceinline__ void stash_row32(uint32_t stash, int row, int j0, const uint32_t (&v)[32])
{
    const uint32_t a = stash + (uint32_t)(j0 * 128 + row) * 4u;
#pragma unroll
    for (int j = 0; j < 32; ++j) st_shared_f32(a + 512u * j, __uint_as_float(v[j]));
}
// Step 2 (after a cluster barrier): CTA `rank` owns a slice of the channels (a multiple of 32 wide); thread `row`
// sums its row of that slice over all CTAs in rank order - so the result does not depend on which CTA sums -
// adds the bias, applies ReLU and stores.  Remote shared memory has the latency of an L2 access, so each pass
// keeps 32 loads per peer in flight.
template <int BN>
__device__ __forceinline__ void cluster_reduce_store(uint32_t stash, int row, uint32_t rank, int splits, const RowDst& d,
                                                     const OutSpec& o, int k0, const float* s_bias)
{
    const int per = ((((BN + splits - 1) / splits) + 31) / 32) * 32;
    const int c_begin = (int)rank * per;
    const int c_end = min(BN, c_begin + per);
    uint32_t peer[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) peer[r] = r < splits ? map_to_cta(stash + (uint32_t)row * 4u, (uint32_t)r) : 0u;
#pragma unroll 1
    for (int c0 = c_begin; c0 < c_end; c0 += 32) {
        float y[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = 0.f;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if (r < splits) {
                float x[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = ld_cluster_f32(peer[r] + (uint32_t)(c0 + j) * 512u);
#pragma unroll
                for (int j = 0; j < 32; ++j) y[j] += x[j];
            }
        }
        {
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(y[j]);
            bias_relu32(v, s_bias + c0, o.relu != 0, y);
        }
        store_row32(o, d, k0 + c0, y);
    }
}

// ---- staged-layout output through shared memory: every epilogue thread lays its output row down in a row-major
// tile (row stride BN*4 + 16 bytes, which keeps the 16-byte stores of a quarter warp on distinct banks) and then
// hands that row to the copy engine as one bulk copy to global memory - 128 row copies per tile instead of
// thousands of scattered 32-byte stores.
template <int BN> __host__ __device__ constexpr uint32_t out_tile_row_bytes() { return BN * 4 + 16; }
__device__ __forceinline__ void out_tile_put32(uint32_t row_addr, int j0, const float (&y)[32])
{
    const uint32_t a = row_addr + (uint32_t)j0 * 4u;
#pragma unroll
    for (int g = 0; g < 8; ++g)
        st_shared_v4(a + 16u * g, round_to_tf32(y[4 * g]), round_to_tf32(y[4 * g + 1]), round_to_tf32(y[4 * g + 2]),
                     round_to_tf32(y[4 * g + 3]));
}
// the row's channels [k0, k0 + width) -> global; the caller commits and waits for the bulk group
__device__ __forceinline__ void out_tile_store_row(const OutSpec& o, const RowDst& d, int k0, int width, uint32_t row_addr)
{
    const int w = min(width, o.Cp - k0);
    if (d.valid && w > 0) bulk_store_global(o.out + d.base + k0, row_addr, (uint32_t)w * 4u);
}

// ---- split reduction by exchange: each CTA of the cluster owns `per` consecutive channels of the tile (the last
// owner possibly fewer) and receives the other CTAs' partial sums of those channels as one bulk copy per peer from
// shared memory to shared memory.  Exchange blocks are row-major [128 rows][w channels] with the 16-byte pieces of
// every 128-byte group XOR-swizzled by (row & 7): thread-per-row accesses then stay free of bank conflicts without
// padding, and sender and receiver use the same mapping.
__host__ __device__ constexpr int split_share(int BN, int splits) { return ((((BN + splits - 1) / splits) + 31) / 32) * 32; }
__host__ __device__ constexpr int split_width(int BN, int per, int rank)
{
    return BN - rank * per <= 0 ? 0 : (BN - rank * per < per ? BN - rank * per : per);
}
__host__ __device__ constexpr bool split_exchange_fits(int BN, int splits, int stage_region_bytes)
{
    return splits > 1 && 2 * 512 * split_share(BN, splits) * (splits - 1) <= stage_region_bytes;
}
__device__ __forceinline__ void xchg_put32(uint32_t block, int w, int row, int c0, const uint32_t (&v)[32])
{
    const uint32_t a = block + (uint32_t)(row * w + c0) * 4u;
#pragma unroll
    for (int g = 0; g < 8; ++g)
        st_shared_v4(a + (uint32_t)((g ^ (row & 7)) << 4), __uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1]),
                     __uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3]));
}
__device__ __forceinline__ void xchg_add32(uint32_t block, int w, int row, int c0, float (&y)[32])
{
    const uint32_t a = block + (uint32_t)(row * w + c0) * 4u;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const float4 t = ld_shared_v4(a + (uint32_t)((g ^ (row & 7)) << 4));
        y[4 * g] += t.x; y[4 * g + 1] += t.y; y[4 * g + 2] += t.z; y[4 * g + 3] += t.w;
    }
}

template <int BN>
__host__ __device__ constexpr uint32_t instr_desc_tf32()
{
    return (1u << 4)                   // accumulator format: fp32
         | (2u << 7) | (2u << 10)      // A and B format: TF32
         | (0u << 15) | (0u << 16)     // A and B are K-major
         | ((uint32_t)(BN >> 3) << 17) // N
         | ((uint32_t)(128 >> 4) << 24);// M = 128
}
// fp16 operands (kind::f16), fp32 accumulator
template <int BN>
__host__ __device__ constexpr uint32_t instr_desc_f16()
{
    return (1u << 4)                   // accumulator format: fp32
         | (0u << 7) | (0u << 10)      // A and B format: fp16
         | (0u << 15) | (0u << 16)     // A and B are K-major
         | ((uint32_t)(BN >> 3) << 17) // N
         | ((uint32_t)(128 >> 4) << 24);// M = 128
}

}  // namespace tc
}  // namespace boda
