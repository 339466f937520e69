// boda_conv_fwd_noalloc: the tensor-core convolution for callers that cannot allocate device memory.
//
// All scratch of the kernel (re-laid-out input and filters, status word)
// lives in one file-scope device array of fixed size.  Every GPU that loads this library holds the array
// until the process exits.  Host code cannot use the array's name as a device address, so the address is
// fetched once per device with cudaGetSymbolAddress and handed to the launch code.
#include <mutex>

#include "boda_internal.h"
#include "igemm_tf32.h"

namespace {

constexpr size_t kStaticScratchBytes = BODA_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the CURRENT device; resolved on the first call for that device.
int scratch_address(void** out)
{
    int device = 0;
    BODA_CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return BODA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        int major = 0;
        BODA_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        if (major != 10) return BODA_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        BODA_CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_static_scratch));
        if (!ptr) return BODA_ERR_CUDA;
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return BODA_OK;
}

}  // namespace

extern "C" int boda_conv_fwd_noalloc(const float* in, const float* filt, const float* bias, float* out, int N, int C,
                                     int H, int W, int K, int R, int S, int stride, int pad, int relu, void* stream)
{
    if (!in || !filt || !out) return BODA_ERR_INVALID_ARG;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || R <= 0 || S <= 0 || stride < 1 || pad < 0) return BODA_ERR_INVALID_ARG;
    if (boda_conv_out_dim(H, R, stride, pad) <= 0 || boda_conv_out_dim(W, S, stride, pad) <= 0) return BODA_ERR_INVALID_ARG;
    const long long lim = 0x7fffffffLL;
    const long long P = boda_conv_out_dim(H, R, stride, pad), Q = boda_conv_out_dim(W, S, stride, pad);
    if ((long long)N * C * H * W > lim || (long long)K * C * R * S > lim || (long long)N * K * P * Q > lim)
        return BODA_ERR_TOO_LARGE;
    const boda_conv_shape shape = {N, C, H, W, K, R, S, stride, pad, relu};
    const boda::ConvDims d = boda::make_dims(shape);
    const int variant = (R == 1 && S == 1) ? BODA_VARIANT_K1CONV : BODA_VARIANT_TCONV;
    if (!boda::igemm_variant_legal(d, variant)) return BODA_ERR_UNSUPPORTED;
    if (boda::igemm_region_min_bytes(d) > kStaticScratchBytes) return BODA_ERR_TOO_LARGE;
    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != BODA_OK) return rc;
    return boda::igemm_run_in_region(d, variant, in, filt, bias, out, scratch, kStaticScratchBytes, (cudaStream_t)stream);
}
