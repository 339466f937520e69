// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <vector>

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "boda.h"

namespace boda {

// Device status word layout (int[4]): [0] status code, [1] where (kernel id), [2] block, [3] detail.
enum { STATUS_WORDS = 4 };
enum { KERNEL_ID_DIRECT = 1, KERNEL_ID_IGEMM = 2, KERNEL_ID_PACK = 3 };

struct ConvDims {
    int N, C, H, W, K, R, S, stride, pad, relu;
    int P, Q;
    int M;        // N*P*Q output points per channel ("pixels")
    int Kred;     // C*R*S reduction length
};

inline ConvDims make_dims(const boda_conv_shape& s) {
    ConvDims d;
    d.N = s.N; d.C = s.C; d.H = s.H; d.W = s.W; d.K = s.K; d.R = s.R; d.S = s.S;
    d.stride = s.stride; d.pad = s.pad; d.relu = s.relu ? 1 : 0;
    d.P = boda_conv_out_dim(s.H, s.R, s.stride, s.pad);
    d.Q = boda_conv_out_dim(s.W, s.S, s.stride, s.pad);
    d.M = s.N * d.P * d.Q;
    d.Kred = s.C * s.R * s.S;
    return d;
}

// Bumps the process-wide count of kernels launched by the library.
void count_launch(int n = 1);

// Records the last CUDA error text for boda_last_error_string(); returns BODA_ERR_CUDA.
int record_cuda_error(cudaError_t e, const char* what);

#define BODA_CUDA_TRY(expr)                                                  \
    do {                                                                     \
        cudaError_t _e = (expr);                                             \
        if (_e != cudaSuccess) return ::boda::record_cuda_error(_e, #expr);  \
    } while (0)

// ---- kernel launch helper
// Every kernel of the library is launched with programmatic dependent launch: it calls pdl_launch_dependents()
// at once and pdl_wait() before it first touches global memory that an earlier kernel on the stream may have
// written (or may still read), so its prologue overlaps the previous kernel's tail.  cluster_z > 1 groups the
// CTAs along grid.z into a thread-block cluster.  BODA_NO_PDL=1 in the environment turns the overlap off.
bool pdl_enabled();

template <typename Kernel, typename... Args>
cudaError_t launch_kernel(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_z, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cluster_z > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = 1;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = (unsigned)cluster_z;
        ++n;
    }
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// cudaFuncSetAttribute applies to the current device only: a kernel's dynamic shared-memory limit is raised once per
// device and kernel (one static DeviceSmemLimit per kernel instantiation), not once per process.
struct DeviceSmemLimit {
    int granted[64];
    explicit DeviceSmemLimit(int initial = 0) { for (int& v : granted) v = initial; }
    template <typename Kernel>
    cudaError_t ensure(Kernel kernel, size_t bytes)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        const bool tracked = dev >= 0 && dev < 64;
        if (tracked && (int)bytes <= granted[dev]) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e == cudaSuccess && tracked) granted[dev] = (int)bytes;
        return e;
    }
};

#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// ---- DIRECT (FP32 CUDA-core) variant -----------------------------------------------------------
// Reduction-index table entry: for flattened reduction index j = (c*R + r)*S + s the element offset
// c*H*W + r*W + s inside one image and the tap (r, s); entries past C*R*S have r = 0x4000 so that
// the bounds test fails and the element counts as padding.
struct DirectTapEntry { int offset; int rs; };

int direct_num_tiles();
const char* direct_tile_name(int tile_id);
int direct_pick_tile(const ConvDims& d);
// false for a tile that cannot run the shape (the pixel-per-thread tiles need the input patch to fit shared memory)
bool direct_tile_legal(const ConvDims& d, int tile_id);
// Length (entries) of the table the tile needs; build it on the host into `host_tab`.
int direct_table_len(const ConvDims& d);
void direct_build_table(const ConvDims& d, DirectTapEntry* host_tab);
int direct_launch(const ConvDims& d, int tile_id, const float* in, const float* filt, const float* bias,
                  float* out, const DirectTapEntry* dev_tab, cudaStream_t stream);
// Tiles compiled at run time for the exact shape (direct_rtc.cu): output channels per thread, 0 for the other tiles.
int direct_tile_rtc_kt(int tile_id);
// the run-time compiled tile that automatic selection uses for this shape, or -1 (no NVRTC, or the shape is not one
// of the small-reduction layers these tiles are for)
int direct_rtc_pick(const ConvDims& d);
// compilation alone (no GPU needed): the cubin image of the kernel for this shape and blocking
int direct_rtc_compile(const ConvDims& d, int KT, int* BX, int* BY, int* PY, size_t* smem, std::vector<char>* image);
struct DirectRtc;
bool direct_rtc_available();                     // is NVRTC there?
bool direct_rtc_geometry(const ConvDims& d, int KT, int* BX, int* BY, int* PY, size_t* smem);
int direct_rtc_create(const ConvDims& d, int KT, DirectRtc** out);    // compiles; BODA_ERR_UNSUPPORTED without NVRTC or if the shape does not fit
void direct_rtc_destroy(DirectRtc* r);
int direct_rtc_launch(DirectRtc* r, const float* in, const float* filt, const float* bias, float* out, cudaStream_t stream);
void direct_rtc_describe(const DirectRtc* r, char* buf, size_t n);

// ---- the planned forward pass with an optional event between operand staging and the main kernel
int conv_fwd_planned_ex(boda_conv_plan* plan, const float* in, const float* filt, const float* bias, float* out,
                        void* workspace, cudaStream_t stream, cudaEvent_t after_staging);
void conv_plan_out_dims(const boda_conv_plan* plan, int* N, int* K, int* P, int* Q);
// boda_conv_plan_create for a layer of a chain: with opts->tune the candidates are timed reading a staged input
// (chain_in) and writing a staged output (chain_out), the way the chain will run them
int conv_plan_create_chained(const boda_conv_shape* shape, const boda_plan_opts* opts, bool chain_in, bool chain_out,
                             int pool_ksz, int pool_stride, boda_conv_plan** plan);
// chained layers: the staged input layout a tensor-core plan reads (false: the plan reads NCHW only), and the
// switch that makes it read that layout directly / write its output in a consumer's staged layout
bool conv_plan_input_geometry(const boda_conv_plan* plan, int* Hp, int* Wp, int* Cp);
bool conv_plan_can_write_packed(const boda_conv_plan* plan);
int conv_plan_set_io(boda_conv_plan* plan, int in_packed, int out_packed, int oHp, int oWp, int oCp);
// chained layers: a max-pool that follows the convolution, fused into its epilogue (the plan then writes the pooled
// tensor); set_pool(plan, 0, 0) undoes it; call before conv_plan_set_io
bool conv_plan_can_fuse_pool(const boda_conv_plan* plan, int ksz, int stride);
int conv_plan_set_pool(boda_conv_plan* plan, int ksz, int stride);

// ---- pooling -------------------------------------------------------------------------------------
int maxpool_launch(const float* in, float* out, int N, int C, int H, int W, int ksz, int stride,
                   cudaStream_t stream);
// the same on the staged layout rows [(n*Hp + y)*Wp + x][Cp]; output staged (out_packed) or NCHW
int maxpool_packed_launch(const float* in, float* out, int N, int C, int H, int W, int iHp, int iWp, int iCp, int ksz, int stride,
                          int out_packed, int oHp, int oWp, int oCp, cudaStream_t stream);
// ---- softmax over the last dimension of [rows][cols]
int softmax_launch(const float* in, float* out, int rows, int cols, cudaStream_t stream);

int unpack_to_nchw_launch(const float* in, float* out, int N, int C, int H, int W, int Hp, int Wp, int Cp, cudaStream_t stream);

}  // namespace boda
