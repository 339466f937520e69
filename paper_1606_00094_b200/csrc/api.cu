// C ABI: plans (variant selection + blocking), the forward entry points, caches and status.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <algorithm>
#include <vector>

#include "boda_internal.h"
#include "igemm_tf32.h"

namespace boda {

static thread_local std::string t_last_error;
static std::atomic<unsigned long long> g_launches{0};

bool pdl_enabled()
{
    static const bool on = []() { const char* e = std::getenv("BODA_NO_PDL"); return !(e && *e && *e != '0'); }();
    return on;
}

void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
unsigned long long launch_count() { return g_launches.load(std::memory_order_relaxed); }

int record_cuda_error(cudaError_t e, const char* what)
{
    t_last_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " in " + what;
    (void)cudaGetLastError();   // clear the sticky-less error state
    return BODA_ERR_CUDA;
}

namespace {

struct DeviceCtx {
    int device = -1;
    int cc_major = 0;
    int* d_status = nullptr;          // STATUS_WORDS ints
};

struct ShapeKey {
    int v[11];
    bool operator<(const ShapeKey& o) const { return std::memcmp(v, o.v, sizeof(v)) < 0; }
};

struct CachedEntry {
    boda_conv_plan* plan = nullptr;
    void* workspace = nullptr;
    // device staging for the host-pointer entry point
    float *s_in = nullptr, *s_filt = nullptr, *s_bias = nullptr, *s_out = nullptr;
};

std::mutex g_mutex;
std::map<int, DeviceCtx> g_ctx;
std::map<ShapeKey, CachedEntry> g_cache;

int get_ctx(int device, DeviceCtx** out)
{
    if (device < 0) BODA_CUDA_TRY(cudaGetDevice(&device));
    auto it = g_ctx.find(device);
    if (it == g_ctx.end()) {
        DeviceCtx c;
        c.device = device;
        int major = 0;
        BODA_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        c.cc_major = major;
        int prev = 0;
        BODA_CUDA_TRY(cudaGetDevice(&prev));
        BODA_CUDA_TRY(cudaSetDevice(device));
        cudaError_t e = cudaMalloc(&c.d_status, STATUS_WORDS * sizeof(int));
        if (e == cudaSuccess) e = cudaMemset(c.d_status, 0, STATUS_WORDS * sizeof(int));
        (void)cudaSetDevice(prev);
        if (e != cudaSuccess) return record_cuda_error(e, "status word allocation");
        it = g_ctx.emplace(device, c).first;
    }
    *out = &it->second;
    return BODA_OK;
}

// ---- autotune cache: a text file with one line "key tile split variant s2d" per tuned shape, named by the
// environment variable BODA_TUNE_CACHE
bool tune_cache_lookup(const char* key, int* tile, int* split, int* variant, int* s2d)
{
    const char* path = std::getenv("BODA_TUNE_CACHE");
    if (!path || !*path) return false;
    FILE* f = std::fopen(path, "r");
    if (!f) return false;
    char line[320], k[200];
    bool hit = false;
    while (std::fgets(line, sizeof(line), f)) {
        int t = 0, sp = 0, v = 0, sd = 0;
        if (std::sscanf(line, "%199s %d %d %d %d", k, &t, &sp, &v, &sd) == 5 && std::strcmp(k, key) == 0) {
            *tile = t; *split = sp; *variant = v; *s2d = sd; hit = true;
        }
    }
    std::fclose(f);
    return hit;
}

void tune_cache_store(const char* key, int tile, int split, int variant, int s2d)
{
    const char* path = std::getenv("BODA_TUNE_CACHE");
    if (!path || !*path) return;
    FILE* f = std::fopen(path, "a");
    if (!f) return;
    std::fprintf(f, "%s %d %d %d %d\n", key, tile, split, variant, s2d);
    std::fclose(f);
}

bool shape_ok(const boda_conv_shape& s)
{
    if (s.N <= 0 || s.C <= 0 || s.H <= 0 || s.W <= 0 || s.K <= 0 || s.R <= 0 || s.S <= 0) return false;
    if (s.stride < 1 || s.pad < 0) return false;
    if (s.R >= 0x4000 || s.S >= 0x4000) return false;
    if (boda_conv_out_dim(s.H, s.R, s.stride, s.pad) <= 0) return false;
    if (boda_conv_out_dim(s.W, s.S, s.stride, s.pad) <= 0) return false;
    const long long lim = 0x7fffffffLL;
    const long long P = boda_conv_out_dim(s.H, s.R, s.stride, s.pad), Q = boda_conv_out_dim(s.W, s.S, s.stride, s.pad);
    if ((long long)s.N * s.C * s.H * s.W > lim) return false;
    if ((long long)s.K * s.C * s.R * s.S > lim) return false;
    if ((long long)s.N * s.K * P * Q > lim) return false;
    return true;
}

}  // namespace
}  // namespace boda

using namespace boda;

struct boda_conv_plan {
    boda_conv_shape shape;
    ConvDims d;
    int device = 0;
    int variant = BODA_VARIANT_DIRECT;
    int tile_id = 0;
    int math = BODA_MATH_FP32;
    int* d_status = nullptr;
    DirectTapEntry* d_tab = nullptr;     // DIRECT
    DirectRtc* rtc = nullptr;            // DIRECT, tiles compiled at run time
    IgemmPlan* ig = nullptr;             // K1CONV / TCONV
    size_t ws_bytes = 0;
    bool in_packed = false;              // chained layers: the input arrives in the staged layout
};

namespace boda {

int conv_fwd_planned_ex(boda_conv_plan* p, const float* in, const float* filt, const float* bias, float* out,
                        void* workspace, cudaStream_t stream, cudaEvent_t after_staging)
{
    if (!p || !in || !out) return BODA_ERR_INVALID_ARG;
    if (p->variant == BODA_VARIANT_DIRECT) {
        if (!filt) return BODA_ERR_INVALID_ARG;
        if (after_staging) BODA_CUDA_TRY(cudaEventRecord(after_staging, stream));
        if (p->rtc) return direct_rtc_launch(p->rtc, in, filt, bias, out, stream);
        return direct_launch(p->d, p->tile_id, in, filt, bias, out, p->d_tab, stream);
    }
    if (p->ws_bytes && !workspace && !p->in_packed) return BODA_ERR_NOMEM;
    return igemm_launch(p->ig, in, filt, bias, out, workspace, stream, after_staging);
}

void conv_plan_out_dims(const boda_conv_plan* p, int* N, int* K, int* P, int* Q)
{
    *N = p->d.N; *K = p->d.K; *P = p->d.P; *Q = p->d.Q;
}

bool conv_plan_input_geometry(const boda_conv_plan* p, int* Hp, int* Wp, int* Cp)
{
    return p->ig ? igemm_plan_input_geometry(p->ig, Hp, Wp, Cp) : false;
}

bool conv_plan_can_write_packed(const boda_conv_plan* p) { return p->ig != nullptr && igemm_plan_writes_packed(p->ig); }

bool conv_plan_can_fuse_pool(const boda_conv_plan* p, int ksz, int stride)
{
    return p->ig != nullptr && p->math != BODA_MATH_TF32X3 && igemm_plan_can_fuse_pool(p->ig, ksz, stride);
}

int conv_plan_set_pool(boda_conv_plan* p, int ksz, int stride)
{
    if (!p->ig) return ksz ? BODA_ERR_UNSUPPORTED : BODA_OK;
    return igemm_plan_set_pool(p->ig, ksz, stride);
}

int conv_plan_set_io(boda_conv_plan* p, int in_packed, int out_packed, int oHp, int oWp, int oCp)
{
    if (!p->ig) return (in_packed || out_packed) ? BODA_ERR_UNSUPPORTED : BODA_OK;
    const int rc = igemm_plan_set_io(p->ig, in_packed, out_packed, oHp, oWp, oCp);
    if (rc == BODA_OK) p->in_packed = in_packed != 0;
    return rc;
}

}  // namespace boda

extern "C" {

int boda_conv_out_dim(int in_dim, int ksz, int stride, int pad)
{
    if (in_dim <= 0 || ksz <= 0 || stride <= 0 || pad < 0) return 0;
    const long long padded = (long long)in_dim + 2LL * pad;
    if (padded < ksz) return 0;
    return (int)((padded - ksz) / stride + 1);
}

void boda_plan_opts_default(boda_plan_opts* o)
{
    if (!o) return;
    o->math = BODA_MATH_AUTO;
    o->tune = 0;
    o->variant = BODA_VARIANT_AUTO;
    o->tile_id = -1;
    o->split_k = 0;
    o->device = -1;
    o->s2d = -1;
    o->max_workspace = 0;
}

int boda_conv_plan_destroy(boda_conv_plan* plan)
{
    if (!plan) return BODA_OK;
    int prev = 0;
    (void)cudaGetDevice(&prev);
    (void)cudaSetDevice(plan->device);
    if (plan->d_tab) (void)cudaFree(plan->d_tab);
    if (plan->rtc) direct_rtc_destroy(plan->rtc);
    if (plan->ig) igemm_plan_destroy(plan->ig);
    (void)cudaSetDevice(prev);
    delete plan;
    return BODA_OK;
}

static int plan_time_ms(boda_conv_plan* plan, bool chain_in, bool chain_out, int pool_ksz, int pool_stride, float* ms_out);

static int plan_build(const boda_conv_shape& shape, const boda_plan_opts& o, DeviceCtx* ctx, int variant,
                      int tile_id, int split_k, boda_conv_plan** out)
{
    boda_conv_plan* p = new (std::nothrow) boda_conv_plan();
    if (!p) return BODA_ERR_NOMEM;
    p->shape = shape;
    p->d = make_dims(shape);
    p->device = ctx->device;
    p->d_status = ctx->d_status;
    p->variant = variant;
    int rc = BODA_OK;
    if (variant == BODA_VARIANT_DIRECT) {
        p->math = BODA_MATH_FP32;
        if (tile_id >= direct_num_tiles() || (tile_id >= 0 && !direct_tile_legal(p->d, tile_id))) { delete p; return BODA_ERR_UNSUPPORTED; }
        p->tile_id = tile_id >= 0 ? tile_id : direct_pick_tile(p->d);
        const int len = direct_table_len(p->d);
        std::vector<DirectTapEntry> tab(len);
        direct_build_table(p->d, tab.data());
        cudaError_t e = cudaMalloc(&p->d_tab, len * sizeof(DirectTapEntry));
        if (e == cudaSuccess)
            e = cudaMemcpy(p->d_tab, tab.data(), len * sizeof(DirectTapEntry), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) rc = record_cuda_error(e, "tap table upload");
        if (rc == BODA_OK && tile_id < 0) {
            // short reductions with few output channels run in their run-time compiled form where NVRTC is there
            const int rt = direct_rtc_pick(p->d);
            if (rt >= 0 && direct_rtc_create(p->d, direct_tile_rtc_kt(rt), &p->rtc) == BODA_OK) p->tile_id = rt;
        } else if (rc == BODA_OK && direct_tile_rtc_kt(p->tile_id) > 0) {
            rc = direct_rtc_create(p->d, direct_tile_rtc_kt(p->tile_id), &p->rtc);
        }
        p->ws_bytes = 0;
    } else {
        p->math = o.math == BODA_MATH_TF32X3 ? BODA_MATH_TF32X3 : o.math == BODA_MATH_F16 ? BODA_MATH_F16 : BODA_MATH_TF32;
        rc = igemm_plan_create(p->d, variant, tile_id, split_k, o.s2d, ctx->d_status, &p->ig,
                               o.math == BODA_MATH_TF32X3 ? 1 : o.math == BODA_MATH_F16 ? 2 : 0, o.max_workspace);
        if (rc == BODA_OK) { p->tile_id = igemm_plan_tile(p->ig); p->ws_bytes = igemm_plan_workspace_bytes(p->ig); }
    }
    if (rc != BODA_OK) { boda_conv_plan_destroy(p); return rc; }
    *out = p;
    return BODA_OK;
}

int boda_conv_plan_create(const boda_conv_shape* shape, const boda_plan_opts* opts, boda_conv_plan** plan)
{
    return boda::conv_plan_create_chained(shape, opts, false, false, 0, 0, plan);
}

}  // extern "C"

// chain_in / chain_out: the layer will run inside a chain, its input arriving in the plan's own staged layout and its
// output leaving in a consumer's staged layout.  Only the tuner looks at them: it times every candidate the way it
// will run (no staging kernel, bulk-copy epilogue) instead of stand-alone with NCHW on both sides.  pool_ksz > 0: a
// max-pool follows the layer; candidates that can run it in their epilogue are timed that way, the others together
// with the separate pooling kernel they would need.
int boda::conv_plan_create_chained(const boda_conv_shape* shape, const boda_plan_opts* opts, bool chain_in, bool chain_out,
                                   int pool_ksz, int pool_stride, boda_conv_plan** plan)
{
    if (!shape || !plan) return BODA_ERR_INVALID_ARG;
    *plan = nullptr;
    if (!shape_ok(*shape)) return BODA_ERR_INVALID_ARG;
    boda_plan_opts o;
    boda_plan_opts_default(&o);
    if (opts) o = *opts;
    if (o.math < BODA_MATH_AUTO || o.math > BODA_MATH_F16) return BODA_ERR_INVALID_ARG;
    if (o.variant < BODA_VARIANT_AUTO || o.variant > BODA_VARIANT_TCONV) return BODA_ERR_INVALID_ARG;

    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(o.device, &ctx);
    if (rc != BODA_OK) return rc;
    if (ctx->cc_major != 10) return BODA_ERR_UNSUPPORTED;
    int prev = 0;
    BODA_CUDA_TRY(cudaGetDevice(&prev));
    BODA_CUDA_TRY(cudaSetDevice(ctx->device));

    const ConvDims d = make_dims(*shape);
    // Variant rules of Section 5: kernel size 1 -> k1conv; kernel sizes 2..11 -> tconv; else conv.
    const bool k1_legal = igemm_variant_legal(d, BODA_VARIANT_K1CONV);
    const bool t_legal = igemm_variant_legal(d, BODA_VARIANT_TCONV);
    int variant = o.variant;
    if (variant == BODA_VARIANT_AUTO) {
        if (o.math == BODA_MATH_FP32) variant = BODA_VARIANT_DIRECT;
        else if ((o.math == BODA_MATH_TF32X3 || o.math == BODA_MATH_F16) && d.K >= 16 && (k1_legal || t_legal) && o.s2d <= 0)
            variant = k1_legal ? BODA_VARIANT_K1CONV : BODA_VARIANT_TCONV;   // the mode is the caller's choice: the tensor cores if legal
        else if (k1_legal && igemm_variant_profitable(d)) variant = BODA_VARIANT_K1CONV;
        else if (t_legal && igemm_variant_profitable(d)) variant = BODA_VARIANT_TCONV;
        else variant = BODA_VARIANT_DIRECT;
    }
    if ((variant == BODA_VARIANT_K1CONV && !k1_legal) || (variant == BODA_VARIANT_TCONV && !t_legal) ||
        (variant != BODA_VARIANT_DIRECT && o.math == BODA_MATH_FP32)) {
        (void)cudaSetDevice(prev);
        return BODA_ERR_UNSUPPORTED;
    }

    if (!o.tune || o.tile_id >= 0) {
        rc = plan_build(*shape, o, ctx, variant, o.tile_id, o.split_k, plan);
        // the workspace limit ruled out every tensor-core tile: the FP32 kernel needs no workspace
        if (rc == BODA_ERR_NOMEM && o.max_workspace > 0 && o.variant == BODA_VARIANT_AUTO && o.tile_id < 0 &&
            (o.math == BODA_MATH_AUTO || o.math == BODA_MATH_TF32X3 || o.math == BODA_MATH_F16))
            rc = plan_build(*shape, o, ctx, BODA_VARIANT_DIRECT, -1, 0, plan);
    } else {
        // Automated tuning: the rule above names a variant; timing confirms or overturns it.  Every tile and split
        // of that variant is timed and, when the caller left variant and math open, so is the alternative (the FP32
        // kernel against the tensor-core variant, and a strided tconv layer with and without its space-to-depth
        // view).  The fastest plan is kept and remembered in the file named by BODA_TUNE_CACHE (if set).
        char key[160];
        // the leading number names the tile tables: entries written by a build with other tables are not matched
        constexpr int kTileTableVersion = 4;
        std::snprintf(key, sizeof(key), "t%d:%d,%d,%d,%d,%d,%d,%d,%d,%d,v%d,s%d,k%d,m%d,io%d%d", kTileTableVersion, shape->N, shape->C,
                      shape->H, shape->W, shape->K, shape->R, shape->S, shape->stride, shape->pad, o.variant, o.s2d, o.split_k, o.math,
                      chain_in ? 1 : 0, chain_out ? 1 : 0);
        if (pool_ksz > 0) std::snprintf(key + std::strlen(key), sizeof(key) - std::strlen(key), ",p%dx%d", pool_ksz, pool_stride);
        int c_tile = -1, c_split = 0, c_variant = variant, c_s2d = o.s2d;
        if (tune_cache_lookup(key, &c_tile, &c_split, &c_variant, &c_s2d)) {
            boda_plan_opts oc = o;
            oc.s2d = c_s2d;
            rc = plan_build(*shape, oc, ctx, c_variant, c_tile, c_split, plan);
            if (rc == BODA_OK) { (void)cudaSetDevice(prev); return rc; }
        }
        struct Cand { int variant, s2d; };
        std::vector<Cand> cands;
        const int tensor_variant = k1_legal ? BODA_VARIANT_K1CONV : t_legal ? BODA_VARIANT_TCONV : -1;
        const bool open_choice = o.variant == BODA_VARIANT_AUTO && o.math == BODA_MATH_AUTO;
        auto add_tensor = [&](int v) {
            if (v == BODA_VARIANT_TCONV && o.s2d < 0 && igemm_s2d_applicable(d)) { cands.push_back({v, 0}); cands.push_back({v, 1}); }
            else cands.push_back({v, o.s2d});
        };
        if (variant == BODA_VARIANT_DIRECT) {
            cands.push_back({variant, o.s2d});
            if (open_choice && tensor_variant >= 0 && d.K >= 16) add_tensor(tensor_variant);
        } else {
            add_tensor(variant);
            if (open_choice) cands.push_back({BODA_VARIANT_DIRECT, o.s2d});
        }
        boda_conv_plan* best = nullptr;
        float best_ms = 1e30f;
        int best_s2d = o.s2d;
        for (const Cand& c : cands) {
            boda_plan_opts oc = o;
            oc.s2d = c.s2d;
            const int ntiles = c.variant == BODA_VARIANT_DIRECT ? direct_num_tiles() : igemm_num_tiles();
            for (int t = 0; t < ntiles; ++t) {
                const int nsplit = c.variant == BODA_VARIANT_DIRECT ? 1 : igemm_num_split_candidates();
                for (int si = 0; si < nsplit; ++si) {
                    const int split = c.variant == BODA_VARIANT_DIRECT ? 0 : igemm_split_candidate(si);
                    if (o.split_k > 0 && split != o.split_k) continue;
                    boda_conv_plan* cand = nullptr;
                    if (plan_build(*shape, oc, ctx, c.variant, t, split, &cand) != BODA_OK) continue;
                    float ms = 0.f;
                    if (plan_time_ms(cand, chain_in, chain_out, pool_ksz, pool_stride, &ms) == BODA_OK && ms < best_ms) {
                        if (best) boda_conv_plan_destroy(best);
                        best = cand;
                        best_ms = ms;
                        best_s2d = c.s2d;
                    } else {
                        boda_conv_plan_destroy(cand);
                    }
                }
            }
        }
        if (best) {
            *plan = best;
            rc = BODA_OK;
            tune_cache_store(key, best->tile_id, best->ig ? igemm_plan_splits(best->ig) : 0, best->variant, best_s2d);
        }
        else rc = plan_build(*shape, o, ctx, variant, -1, o.split_k, plan);
    }
    (void)cudaSetDevice(prev);
    return rc;
}

extern "C" {

int boda_conv_plan_describe(const boda_conv_plan* p, char* buf, size_t n)
{
    if (!p || !buf || n == 0) return BODA_ERR_INVALID_ARG;
    static const char* vn[] = {"direct", "k1conv", "tconv"};
    if (p->variant == BODA_VARIANT_DIRECT) {
        char extra[96] = "";
        if (p->rtc) { extra[0] = ' '; direct_rtc_describe(p->rtc, extra + 1, sizeof(extra) - 1); }
        std::snprintf(buf, n, "variant=%s tile=%s(id %d)%s math=fp32 split_k=1 workspace=%zu", vn[p->variant],
                      direct_tile_name(p->tile_id), p->tile_id, extra, p->ws_bytes);
    } else {
        char tmp[160];
        igemm_plan_describe(p->ig, tmp, sizeof(tmp));
        std::snprintf(buf, n, "variant=%s %s math=%s workspace=%zu", vn[p->variant], tmp,
                      p->math == BODA_MATH_TF32X3 ? "tf32x3" : p->math == BODA_MATH_F16 ? "f16" : "tf32", p->ws_bytes);
    }
    return BODA_OK;
}

size_t boda_conv_plan_workspace_bytes(const boda_conv_plan* p) { return p ? p->ws_bytes : 0; }

int boda_conv_plan_kernels_per_call(const boda_conv_plan* p)
{
    if (!p) return 0;
    if (p->variant == BODA_VARIANT_DIRECT) return 1;
    return igemm_plan_kernels_per_call(p->ig);             // tensor-core variants: input staging (where needed) + main kernel
}

int boda_conv_plan_bind_filters(boda_conv_plan* p, const float* filt, void* stream)
{
    if (!p || !filt) return BODA_ERR_INVALID_ARG;
    if (p->variant == BODA_VARIANT_DIRECT) return BODA_OK;   // reads KCRS in place
    return igemm_bind_filters(p->ig, filt, (cudaStream_t)stream);
}

int boda_conv_fwd_planned(boda_conv_plan* p, const float* in, const float* filt, const float* bias, float* out,
                          void* workspace, void* stream)
{
    return boda::conv_fwd_planned_ex(p, in, filt, bias, out, workspace, (cudaStream_t)stream, nullptr);
}

}  // extern "C"

// Times one plan on scratch buffers (used by the tuner).  Synchronises.  chain_in / chain_out: time the plan the
// way a chain runs it - reading its own staged input layout (no staging kernel) and writing a staged output - where
// the plan's kernel can; operands hold a small non-zero constant (all-zero operands draw less power than real ones).
static int plan_time_ms(boda_conv_plan* p, bool chain_in, bool chain_out, int pool_ksz, int pool_stride, float* ms_out)
{
    const ConvDims& d = p->d;
    size_t n_in = (size_t)d.N * d.C * d.H * d.W, n_out = (size_t)d.M * d.K;
    const size_t n_f = (size_t)d.K * d.Kred;
    bool in_packed = false, out_packed = false, fused = false;
    const int oCp = ((d.K + 31) / 32) * 32;
    int outP = d.P, outQ = d.Q;                  // extent of what the convolution kernel writes
    const int poolP = pool_ksz > 0 ? boda_conv_out_dim(d.P, pool_ksz, pool_stride, 0) : 0;
    const int poolQ = pool_ksz > 0 ? boda_conv_out_dim(d.Q, pool_ksz, pool_stride, 0) : 0;
    const bool pool_after = pool_ksz > 0 && poolP > 0 && poolQ > 0;
    if (p->ig) {
        int Hp = 0, Wp = 0, Cp = 0;
        in_packed = chain_in && igemm_plan_input_geometry(p->ig, &Hp, &Wp, &Cp);
        out_packed = chain_out && igemm_plan_writes_packed(p->ig);
        if (pool_after && conv_plan_can_fuse_pool(p, pool_ksz, pool_stride) && conv_plan_set_pool(p, pool_ksz, pool_stride) == BODA_OK) {
            fused = true;
            outP = poolP; outQ = poolQ;
        }
        if (in_packed) n_in = (size_t)d.N * Hp * Wp * Cp;
        if (out_packed) n_out = (size_t)d.N * outP * outQ * oCp;
        else n_out = (size_t)d.N * d.K * outP * outQ;
        if (in_packed || out_packed) {
            const int rc_io = conv_plan_set_io(p, in_packed ? 1 : 0, out_packed ? 1 : 0, outP, outQ, oCp);
            if (rc_io != BODA_OK) { (void)conv_plan_set_pool(p, 0, 0); return rc_io; }
        }
    }
    const bool separate_pool = pool_after && !fused;
    float* pool_out = nullptr;
    // one timed call: the layer, plus the pooling kernel where the layer cannot run it itself
    auto run_once = [&](float* in_, float* f_, float* b_, float* out_, void* ws_, cudaStream_t st) -> int {
        int r = boda_conv_fwd_planned(p, in_, f_, b_, out_, ws_, st);
        if (r != BODA_OK || !separate_pool) return r;
        if (out_packed)
            return maxpool_packed_launch(out_, pool_out, d.N, d.K, d.P, d.Q, d.P, d.Q, oCp, pool_ksz, pool_stride, 1, poolP, poolQ, oCp, st);
        return maxpool_launch(out_, pool_out, d.N, d.K, d.P, d.Q, pool_ksz, pool_stride, st);
    };
    float *in = nullptr, *f = nullptr, *b = nullptr, *out = nullptr;
    void* ws = nullptr;
    int rc = BODA_OK;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaStream_t stream = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    auto cleanup = [&]() {
        if (exec) cudaGraphExecDestroy(exec); if (graph) cudaGraphDestroy(graph);
        if (stream) { cudaStreamSynchronize(stream); cudaStreamDestroy(stream); }
        if (in) cudaFree(in); if (f) cudaFree(f); if (b) cudaFree(b); if (out) cudaFree(out); if (ws) cudaFree(ws);
        if (e0) cudaEventDestroy(e0); if (e1) cudaEventDestroy(e1);
        if (pool_out) cudaFree(pool_out);
        if (in_packed || out_packed) (void)conv_plan_set_io(p, 0, 0, 0, 0, 0);
        if (fused) (void)conv_plan_set_pool(p, 0, 0);
    };
#define TRY_T(x) do { cudaError_t _e = (x); if (_e != cudaSuccess) { rc = record_cuda_error(_e, #x); cleanup(); return rc; } } while (0)
    TRY_T(cudaMalloc(&in, n_in * 4)); TRY_T(cudaMalloc(&f, n_f * 4)); TRY_T(cudaMalloc(&b, d.K * 4));
    TRY_T(cudaMalloc(&out, n_out * 4));
    if (separate_pool) TRY_T(cudaMalloc(&pool_out, (size_t)d.N * oCp * poolP * poolQ * 4));
    if (p->ws_bytes && !in_packed) TRY_T(cudaMalloc(&ws, p->ws_bytes));
    // bytes 0x3c -> the float 0.0115 (exact in TF32 after truncation or rounding alike)
    TRY_T(cudaMemset(in, 0x3c, n_in * 4)); TRY_T(cudaMemset(f, 0x3c, n_f * 4)); TRY_T(cudaMemset(b, 0, d.K * 4));
    TRY_T(cudaEventCreate(&e0)); TRY_T(cudaEventCreate(&e1));
    TRY_T(cudaStreamSynchronize(0));                    // the fills above ran on the default stream
    TRY_T(cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking));
    if (p->variant != BODA_VARIANT_DIRECT) { rc = igemm_bind_filters(p->ig, f, stream); if (rc) { cleanup(); return rc; } }
    for (int i = 0; i < 2; ++i) { rc = run_once(in, f, b, out, ws, stream); if (rc) { cleanup(); return rc; } }
    TRY_T(cudaStreamSynchronize(stream));
    // The candidates differ by a few percent, less than the host's launch cost for a small layer: the timed calls are
    // captured in a graph (device time only) and the best of three replays counts.  Without capture: plain launches.
    const int iters = 10;
    float ms = 0.f;
    bool timed = false;
    if (cudaStreamBeginCapture(stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        int crc = BODA_OK;
        for (int i = 0; i < iters && crc == BODA_OK; ++i) crc = run_once(in, f, b, out, ws, stream);
        const cudaError_t ce = cudaStreamEndCapture(stream, &graph);
        if (crc == BODA_OK && ce == cudaSuccess && graph && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
            TRY_T(cudaGraphLaunch(exec, stream));
            float best = 1e30f;
            for (int r = 0; r < 3; ++r) {
                TRY_T(cudaEventRecord(e0, stream));
                TRY_T(cudaGraphLaunch(exec, stream));
                TRY_T(cudaEventRecord(e1, stream));
                TRY_T(cudaEventSynchronize(e1));
                float t = 0.f;
                TRY_T(cudaEventElapsedTime(&t, e0, e1));
                best = std::min(best, t);
            }
            ms = best;
            timed = true;
        } else {
            (void)cudaGetLastError();
        }
    }
    if (!timed) {
        TRY_T(cudaEventRecord(e0, stream));
        for (int i = 0; i < iters; ++i) { rc = run_once(in, f, b, out, ws, stream); if (rc) { cleanup(); return rc; } }
        TRY_T(cudaEventRecord(e1, stream));
        TRY_T(cudaEventSynchronize(e1));
        TRY_T(cudaEventElapsedTime(&ms, e0, e1));
    }
    int st[STATUS_WORDS] = {0, 0, 0, 0};
    TRY_T(cudaMemcpy(st, p->d_status, sizeof(st), cudaMemcpyDeviceToHost));
    if (st[0] != 0) { (void)cudaMemset(p->d_status, 0, sizeof(st)); cleanup(); return st[0]; }
    if (p->variant != BODA_VARIANT_DIRECT) igemm_unbind_filters(p->ig);
#undef TRY_T
    cleanup();
    *ms_out = ms / iters;
    return BODA_OK;
}

extern "C" {

static int cache_lookup(const boda_conv_shape& s, bool need_staging, CachedEntry** out)
{
    int device = 0;
    BODA_CUDA_TRY(cudaGetDevice(&device));
    ShapeKey key;
    const int vals[11] = {device, s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.stride, s.pad, s.relu ? 1 : 0};
    std::memcpy(key.v, vals, sizeof(vals));
    CachedEntry* e = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        auto it = g_cache.find(key);
        if (it != g_cache.end()) e = &it->second;
    }
    if (!e) {
        boda_conv_plan* plan = nullptr;
        int rc = boda_conv_plan_create(&s, nullptr, &plan);
        if (rc != BODA_OK) return rc;
        CachedEntry ne;
        ne.plan = plan;
        if (plan->ws_bytes) {
            cudaError_t ce = cudaMalloc(&ne.workspace, plan->ws_bytes);
            if (ce != cudaSuccess) { boda_conv_plan_destroy(plan); return record_cuda_error(ce, "workspace allocation"); }
        }
        std::lock_guard<std::mutex> lock(g_mutex);
        auto ins = g_cache.emplace(key, ne);
        if (!ins.second) {   // another thread won the race
            if (ne.workspace) cudaFree(ne.workspace);
            boda_conv_plan_destroy(plan);
        }
        e = &ins.first->second;
    }
    if (need_staging && !e->s_in) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!e->s_in) {
            const ConvDims& d = e->plan->d;
            BODA_CUDA_TRY(cudaMalloc(&e->s_in, (size_t)d.N * d.C * d.H * d.W * 4));
            BODA_CUDA_TRY(cudaMalloc(&e->s_filt, (size_t)d.K * d.Kred * 4));
            BODA_CUDA_TRY(cudaMalloc(&e->s_bias, (size_t)d.K * 4));
            BODA_CUDA_TRY(cudaMalloc(&e->s_out, (size_t)d.M * d.K * 4));
        }
    }
    *out = e;
    return BODA_OK;
}

int boda_conv_fwd(const float* in, const float* filt, const float* bias, float* out, int N, int C, int H, int W,
                  int K, int R, int S, int stride, int pad, int relu, void* stream)
{
    if (!in || !filt || !out) return BODA_ERR_INVALID_ARG;
    const boda_conv_shape s = {N, C, H, W, K, R, S, stride, pad, relu};
    if (!shape_ok(s)) return BODA_ERR_INVALID_ARG;
    CachedEntry* e = nullptr;
    int rc = cache_lookup(s, false, &e);
    if (rc != BODA_OK) return rc;
    return boda_conv_fwd_planned(e->plan, in, filt, bias, out, e->workspace, stream);
}

int boda_direct_rtc_compile(const boda_conv_shape* shape, int kt, int* block_x, int* block_y, size_t* smem_bytes,
                            size_t* image_bytes)
{
    if (!shape || !shape_ok(*shape) || (kt != 4 && kt != 8 && kt != 16 && kt != 32)) return BODA_ERR_INVALID_ARG;
    const ConvDims d = make_dims(*shape);
    int bx = 0, by = 0, py = 1;
    size_t smem = 0;
    std::vector<char> image;
    const int rc = direct_rtc_compile(d, kt, &bx, &by, &py, &smem, &image);
    if (rc != BODA_OK) return rc;
    if (block_x) *block_x = bx;
    if (block_y) *block_y = by * py;
    if (smem_bytes) *smem_bytes = smem;
    if (image_bytes) *image_bytes = image.size();
    return BODA_OK;
}

int boda_sgemm(const float* A, const float* B, float* C, int M, int N, int K, void* stream)
{
    if (!A || !B || !C || M <= 0 || N <= 0 || K <= 0) return BODA_ERR_INVALID_ARG;
    // in[1][K][1][N] = B, filt[M][K][1][1] = A, out[1][M][1][N] = C
    return boda_conv_fwd(B, A, nullptr, C, 1, K, 1, N, M, 1, 1, 1, 0, 0, stream);
}

int boda_conv_fwd_host(const float* in, const float* filt, const float* bias, float* out, int N, int C, int H,
                       int W, int K, int R, int S, int stride, int pad, int relu, void* stream)
{
    if (!in || !filt || !out) return BODA_ERR_INVALID_ARG;
    const boda_conv_shape s = {N, C, H, W, K, R, S, stride, pad, relu};
    if (!shape_ok(s)) return BODA_ERR_INVALID_ARG;
    CachedEntry* e = nullptr;
    int rc = cache_lookup(s, true, &e);
    if (rc != BODA_OK) return rc;
    const ConvDims& d = e->plan->d;
    cudaStream_t st = (cudaStream_t)stream;
    BODA_CUDA_TRY(cudaMemcpyAsync(e->s_in, in, (size_t)d.N * d.C * d.H * d.W * 4, cudaMemcpyHostToDevice, st));
    BODA_CUDA_TRY(cudaMemcpyAsync(e->s_filt, filt, (size_t)d.K * d.Kred * 4, cudaMemcpyHostToDevice, st));
    if (bias) BODA_CUDA_TRY(cudaMemcpyAsync(e->s_bias, bias, (size_t)d.K * 4, cudaMemcpyHostToDevice, st));
    if (e->plan->ig) igemm_unbind_filters(e->plan->ig);   // the staged filters may have changed
    rc = boda_conv_fwd_planned(e->plan, e->s_in, e->s_filt, bias ? e->s_bias : nullptr, e->s_out, e->workspace, stream);
    if (rc != BODA_OK) return rc;
    BODA_CUDA_TRY(cudaMemcpyAsync(out, e->s_out, (size_t)d.M * d.K * 4, cudaMemcpyDeviceToHost, st));
    BODA_CUDA_TRY(cudaStreamSynchronize(st));
    return BODA_OK;
}

int boda_maxpool_fwd(const float* in, float* out, int N, int C, int H, int W, int ksz, int stride, void* stream)
{
    if (!in || !out || N <= 0 || C <= 0 || ksz <= 0 || stride <= 0) return BODA_ERR_INVALID_ARG;
    if (boda_conv_out_dim(H, ksz, stride, 0) <= 0 || boda_conv_out_dim(W, ksz, stride, 0) <= 0)
        return BODA_ERR_INVALID_ARG;
    return maxpool_launch(in, out, N, C, H, W, ksz, stride, (cudaStream_t)stream);
}

int boda_softmax_fwd(const float* in, float* out, int rows, int cols, void* stream)
{
    if (!in || !out || rows <= 0 || cols <= 0) return BODA_ERR_INVALID_ARG;
    return softmax_launch(in, out, rows, cols, (cudaStream_t)stream);
}

int boda_query_status(void* stream, int* device_status)
{
    if (!device_status) return BODA_ERR_INVALID_ARG;
    DeviceCtx* ctx = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        int rc = get_ctx(-1, &ctx);
        if (rc != BODA_OK) return rc;
    }
    BODA_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    int st[STATUS_WORDS] = {0, 0, 0, 0};
    BODA_CUDA_TRY(cudaMemcpy(st, ctx->d_status, sizeof(st), cudaMemcpyDeviceToHost));
    if (st[0] != 0) BODA_CUDA_TRY(cudaMemset(ctx->d_status, 0, sizeof(st)));
    *device_status = st[0];
    return BODA_OK;
}

int boda_clear_caches(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    for (auto& kv : g_cache) {
        CachedEntry& e = kv.second;
        if (e.workspace) cudaFree(e.workspace);
        if (e.s_in) cudaFree(e.s_in);
        if (e.s_filt) cudaFree(e.s_filt);
        if (e.s_bias) cudaFree(e.s_bias);
        if (e.s_out) cudaFree(e.s_out);
        boda_conv_plan_destroy(e.plan);
    }
    g_cache.clear();
    return BODA_OK;
}

const char* boda_status_string(int s)
{
    switch (s) {
        case BODA_OK: return "ok";
        case BODA_ERR_INVALID_ARG: return "invalid argument";
        case BODA_ERR_UNSUPPORTED: return "unsupported (device is not sm_100, or variant illegal for the shape)";
        case BODA_ERR_CUDA: return "CUDA error";
        case BODA_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case BODA_ERR_NOMEM: return "out of memory or workspace missing";
        case BODA_ERR_TOO_LARGE: return "size exceeds a fixed capacity";
        default: return "unknown status";
    }
}

const char* boda_last_error_string(void) { return t_last_error.c_str(); }

unsigned long long boda_kernel_launch_count(void) { return boda::launch_count(); }

int boda_version(void) { return 100; }

}  // extern "C"
