// DIRECT compiled at run time for one exact problem (Section 4 of the paper: kernels are generated and compiled
// when the shape is known).  The source is direct_rtc_src.h; here: the NVRTC driver, the choice of blocking, the
// load of the compiled image and the launch.
//
// NVRTC is looked up with dlopen when the first such plan is made, so the library itself does not depend on it:
// where it is missing, these tiles answer BODA_ERR_UNSUPPORTED and every other path works as before.
#include <dlfcn.h>
#include <nvrtc.h>

#include <cstdio>
#include <cstdlib>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "boda_internal.h"
#include "direct_rtc_src.h"

namespace boda {

namespace {

struct NvrtcApi {
    void* handle = nullptr;
    nvrtcResult (*create)(nvrtcProgram*, const char*, const char*, int, const char* const*, const char* const*) = nullptr;
    nvrtcResult (*compile)(nvrtcProgram, int, const char* const*) = nullptr;
    nvrtcResult (*destroy)(nvrtcProgram*) = nullptr;
    nvrtcResult (*cubin_size)(nvrtcProgram, size_t*) = nullptr;
    nvrtcResult (*cubin)(nvrtcProgram, char*) = nullptr;
    nvrtcResult (*log_size)(nvrtcProgram, size_t*) = nullptr;
    nvrtcResult (*log)(nvrtcProgram, char*) = nullptr;
    bool ok = false;
};

NvrtcApi* nvrtc_api()
{
    static NvrtcApi api;
    static std::once_flag once;
    std::call_once(once, [] {
        const char* off = std::getenv("BODA_NO_RTC");        // "1": behave as if NVRTC were not installed
        if (off && *off == '1') return;
        const char* names[] = {"libnvrtc.so.12", "libnvrtc.so", "/usr/local/cuda/lib64/libnvrtc.so.12", "/usr/local/cuda/lib64/libnvrtc.so"};
        for (const char* nm : names) {
            api.handle = dlopen(nm, RTLD_NOW | RTLD_LOCAL);
            if (api.handle) break;
        }
        if (!api.handle) return;
        auto sym = [&](const char* s) { return dlsym(api.handle, s); };
        api.create = reinterpret_cast<decltype(api.create)>(sym("nvrtcCreateProgram"));
        api.compile = reinterpret_cast<decltype(api.compile)>(sym("nvrtcCompileProgram"));
        api.destroy = reinterpret_cast<decltype(api.destroy)>(sym("nvrtcDestroyProgram"));
        api.cubin_size = reinterpret_cast<decltype(api.cubin_size)>(sym("nvrtcGetCUBINSize"));
        api.cubin = reinterpret_cast<decltype(api.cubin)>(sym("nvrtcGetCUBIN"));
        api.log_size = reinterpret_cast<decltype(api.log_size)>(sym("nvrtcGetProgramLogSize"));
        api.log = reinterpret_cast<decltype(api.log)>(sym("nvrtcGetProgramLog"));
        api.ok = api.create && api.compile && api.destroy && api.cubin_size && api.cubin && api.log_size && api.log;
    });
    return &api;
}

std::string def(const char* name, long long v)
{
    char buf[64];
    std::snprintf(buf, sizeof(buf), "-D%s=%lld", name, v);
    return buf;
}

}  // namespace

struct DirectRtc {
    ConvDims d;
    int KT = 16, BX = 32, BY = 8, PY = 1;
    size_t smem = 0, cubin_bytes = 0;
    cudaLibrary_t lib = nullptr;
    cudaKernel_t kernel = nullptr;
};

// Blocking for a shape: the widest thread block (32 x 8, 16 x 8, 16 x 4, 8 x 4 threads) and the most output rows per
// thread (4, 2, 1: the weights of a tap are loaded once for all of a thread's rows) such that the input patch and the
// filters fit the 48 KB of static shared memory and the grid still has a few blocks per SM; false if nothing fits.
bool direct_rtc_geometry(const ConvDims& d, int KT, int* BX, int* BY, int* PY, size_t* smem)
{
    if (KT % 4 != 0 || KT < 4 || KT > 32) return false;
    if (d.N > 65535 || (d.K + KT - 1) / KT > 65535) return false;
    int force_py = 0;
    if (const char* e = std::getenv("BODA_RTC_ROWS_PER_THREAD")) force_py = std::atoi(e);     // measurement hook: 1, 2 or 4
    const int cand[4][2] = {{32, 8}, {16, 8}, {16, 4}, {8, 4}};
    const int pys[3] = {4, 2, 1};
    for (const auto& c : cand) {
        // no wider than the output row needs (a 13-pixel row does not want a 32-pixel patch)
        if (c[0] >= 2 * d.Q && c[0] > 8) continue;
        for (int py : pys) {
            if (force_py > 0 && py != force_py) continue;
            if (py > 1 && KT * py > 64) continue;                                  // accumulators stay in registers
            const long long blocks = (long long)((d.Q + c[0] - 1) / c[0]) * ((d.P + c[1] * py - 1) / (c[1] * py)) * d.N * ((d.K + KT - 1) / KT);
            if (force_py == 0 && py > 1 && (blocks < 8 * 148 || c[1] * py > d.P)) continue;
            const int ih = (c[1] * py - 1) * d.stride + d.R, iw = (c[0] - 1) * d.stride + d.S, iwp = iw | 1;
            const size_t bytes = ((size_t)d.Kred * KT + (size_t)d.C * ih * iwp) * sizeof(float);
            if (bytes <= 48 * 1024 - 64) { *BX = c[0]; *BY = c[1]; *PY = py; *smem = bytes; return true; }
        }
    }
    return false;
}

bool direct_rtc_available() { return nvrtc_api()->ok; }

void direct_rtc_destroy(DirectRtc* r)
{
    if (!r) return;
    if (r->lib) (void)cudaLibraryUnload(r->lib);
    delete r;
}

// Compiled images of this process, by shape and blocking: a tuner that has tried a tile and the plan that keeps it
// compile once.
struct ImageCache {
    std::mutex mu;
    std::map<std::string, std::vector<char>> images;
};
static ImageCache& image_cache() { static ImageCache c; return c; }

int direct_rtc_compile(const ConvDims& d, int KT, int* BX, int* BY, int* PY, size_t* smem, std::vector<char>* image)
{
    NvrtcApi* api = nvrtc_api();
    if (!api->ok) return BODA_ERR_UNSUPPORTED;
    if (!direct_rtc_geometry(d, KT, BX, BY, PY, smem)) return BODA_ERR_UNSUPPORTED;
    char key[160];
    std::snprintf(key, sizeof(key), "%d,%d,%d,%d,%d,%d,%d,%d,%d,%d,kt%d,%dx%dx%d", d.N, d.C, d.H, d.W, d.K, d.R, d.S, d.stride, d.pad,
                  d.relu, KT, *BX, *BY, *PY);
    {
        std::lock_guard<std::mutex> lock(image_cache().mu);
        auto it = image_cache().images.find(key);
        if (it != image_cache().images.end()) { *image = it->second; return BODA_OK; }
    }
    // full unrolling of the reduction while the kernel stays a few thousand instructions long (compilation time
    // grows faster than the body: 0.3 s for 600 instructions, 5 s for 4000); otherwise the window, or its rows, only
    const long long per_tap = (long long)KT * *PY + KT / 4 + *PY;
    const long long body = (long long)d.Kred * per_tap;
    const int unroll_c = body <= 2500 ? d.C : 1;
    const int unroll_r = (body <= 2500 || (long long)d.R * d.S * per_tap <= 2500) ? d.R : 1;
    std::vector<std::string> opts = {
        "--gpu-architecture=sm_100a", "--std=c++17", "-lineinfo",
        def("N", d.N), def("C", d.C), def("H", d.H), def("W", d.W), def("K", d.K), def("R", d.R), def("S", d.S),
        def("STRIDE", d.stride), def("PAD", d.pad), def("RELU", d.relu), def("P", d.P), def("Q", d.Q),
        def("KT", KT), def("BX", *BX), def("BY", *BY), def("PY", *PY), def("UNROLL_C", unroll_c), def("UNROLL_R", unroll_r),
    };
    std::vector<const char*> optp;
    for (const auto& o : opts) optp.push_back(o.c_str());
    nvrtcProgram prog = nullptr;
    if (api->create(&prog, kDirectRtcSource, "boda_direct_rtc.cu", 0, nullptr, nullptr) != NVRTC_SUCCESS) return BODA_ERR_CUDA;
    const nvrtcResult cr = api->compile(prog, (int)optp.size(), optp.data());
    if (cr != NVRTC_SUCCESS) {
        size_t ls = 0;
        std::string log;
        if (api->log_size(prog, &ls) == NVRTC_SUCCESS && ls > 1) { log.resize(ls); (void)api->log(prog, &log[0]); }
        (void)api->destroy(&prog);
        char msg[256];
        std::snprintf(msg, sizeof(msg), "NVRTC compilation failed (%d): %.180s", (int)cr, log.c_str());
        return record_cuda_error(cudaErrorInvalidSource, msg);
    }
    size_t nbytes = 0;
    if (api->cubin_size(prog, &nbytes) != NVRTC_SUCCESS || nbytes == 0) { (void)api->destroy(&prog); return BODA_ERR_CUDA; }
    image->resize(nbytes);
    const nvrtcResult gr = api->cubin(prog, image->data());
    (void)api->destroy(&prog);
    if (gr != NVRTC_SUCCESS) return BODA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(image_cache().mu);
    image_cache().images[key] = *image;
    return BODA_OK;
}

int direct_rtc_create(const ConvDims& d, int KT, DirectRtc** out)
{
    *out = nullptr;
    DirectRtc* r = new (std::nothrow) DirectRtc();
    if (!r) return BODA_ERR_NOMEM;
    r->d = d;
    r->KT = KT;
    std::vector<char> image;
    const int rc = direct_rtc_compile(d, KT, &r->BX, &r->BY, &r->PY, &r->smem, &image);
    if (rc != BODA_OK) { delete r; return rc; }
    r->cubin_bytes = image.size();
    cudaError_t e = cudaLibraryLoadData(&r->lib, image.data(), nullptr, nullptr, 0, nullptr, nullptr, 0);
    if (e == cudaSuccess) e = cudaLibraryGetKernel(&r->kernel, r->lib, "boda_direct_rtc");
    if (e != cudaSuccess) { direct_rtc_destroy(r); return record_cuda_error(e, "loading the run-time compiled kernel"); }
    *out = r;
    return BODA_OK;
}

int direct_rtc_launch(DirectRtc* r, const float* in, const float* filt, const float* bias, float* out, cudaStream_t stream)
{
    const ConvDims& d = r->d;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(((d.Q + r->BX - 1) / r->BX) * ((d.P + r->BY * r->PY - 1) / (r->BY * r->PY)), d.N, (d.K + r->KT - 1) / r->KT);
    cfg.blockDim = dim3(r->BX * r->BY);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    unsigned n = 0;
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    void* args[] = {(void*)&in, (void*)&filt, (void*)&bias, (void*)&out};
    BODA_CUDA_TRY(cudaLaunchKernelExC(&cfg, (const void*)r->kernel, args));
    count_launch();
    return BODA_OK;
}

void direct_rtc_describe(const DirectRtc* r, char* buf, size_t n)
{
    std::snprintf(buf, n, "rtc block=%dx%d rows=%d kt=%d smem=%zu cubin=%zu", r->BX, r->BY, r->PY, r->KT, r->smem, r->cubin_bytes);
}

}  // namespace boda
