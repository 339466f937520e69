// boda_stack: a chain of convolution and max-pool layers (layer i+1 reads layer i's output) run as one unit.
// The stack owns the plans, the activations between layers, one workspace shared by all layers and a CUDA graph
// of the whole chain, so that a forward pass is a single graph launch with no host work between kernels.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "boda_internal.h"

using namespace boda;

struct boda_stack {
    struct Op {
        int kind = 0;                       // 0 conv, 1 max-pool
        boda_conv_shape conv{};
        int ksz = 0, stride = 0;
        boda_conv_plan* plan = nullptr;
        const float* filt = nullptr;
        const float* bias = nullptr;
        int N = 0, C = 0, H = 0, W = 0;     // input dims of this op
        int oC = 0, oH = 0, oW = 0;         // output dims
        float* out = nullptr;               // owned activation (nullptr for the last op: the caller's buffer)
        size_t out_elems = 0;               // elements of the NCHW view of the output
        // layout of the output activation: NCHW, or the consumer's staged layout rows [(n*Hp + y)*Wp + x][Cp]
        bool out_packed = false;
        int oHp = 0, oWp = 0, oCp = 0;
        bool in_packed = false;             // = out_packed of the previous op
        int iHp = 0, iWp = 0, iCp = 0;
        // a 3x3 / stride-2 max-pool that follows a convolution may run inside that convolution's epilogue: the
        // convolution is then `fused_pool` and writes the pool op's activation; the pool op is `skipped`
        bool fused_pool = false, skipped = false;
    };
    std::vector<Op> ops;
    int device = 0;
    void* workspace = nullptr;
    size_t ws_bytes = 0;
    float* staging_in = nullptr;            // device copy of a host input
    float* staging_out = nullptr;
    size_t in_elems = 0, out_elems = 0;
    // captured graphs of the chain, one per (in, out) pointer pair seen (a handful: the host path runs the
    // sub-batch stack on several slices of one buffer)
    struct Graph { const float* in; float* out; cudaGraphExec_t exec; };
    std::vector<Graph> graphs;
    cudaStream_t capture_stream = nullptr;
    // host-buffer path: the batch is copied in `host_chunks` slices on a second stream, and each slice runs through a
    // stack for the sub-batch as soon as it has arrived, so that copies and kernels overlap
    std::vector<boda_stack_op> specs;       // what the stack was created from
    std::vector<boda_plan_opts> op_opts;    // per-op plan options (empty: defaults)
    boda_stack* sub = nullptr;
    int host_chunks = 0;                    // 0: not decided yet; 1: no slicing
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t entry_event = nullptr;      // recorded on the caller's stream at entry: the copy stream waits for it
    std::vector<cudaEvent_t> chunk_events;
};

namespace {

int run_ops(boda_stack* s, const float* in, float* out, cudaStream_t stream, cudaEvent_t* events)
{
    const float* cur = in;
    const int n = (int)s->ops.size();
    for (int i = 0; i < n; ++i) {
        boda_stack::Op& op = s->ops[i];
        if (op.skipped) {                    // ran inside the preceding convolution
            if (events) for (int e = 0; e < 3; ++e) BODA_CUDA_TRY(cudaEventRecord(events[3 * i + e], stream));
            continue;
        }
        const int w = op.fused_pool ? i + 1 : i;            // the op whose activation this launch writes
        float* dst = (w == n - 1) ? out : s->ops[w].out;
        if (events) BODA_CUDA_TRY(cudaEventRecord(events[3 * i + 0], stream));
        int rc;
        if (op.kind == 0) {
            if (!op.filt) return BODA_ERR_INVALID_ARG;
            rc = conv_fwd_planned_ex(op.plan, cur, op.filt, op.bias, dst, s->workspace, stream, events ? events[3 * i + 1] : nullptr);
        } else {
            if (events) BODA_CUDA_TRY(cudaEventRecord(events[3 * i + 1], stream));
            if (op.in_packed)
                rc = maxpool_packed_launch(cur, dst, op.N, op.C, op.H, op.W, op.iHp, op.iWp, op.iCp, op.ksz, op.stride,
                                           op.out_packed ? 1 : 0, op.oHp, op.oWp, op.oCp, stream);
            else
                rc = maxpool_launch(cur, dst, op.N, op.C, op.H, op.W, op.ksz, op.stride, stream);
        }
        if (rc != BODA_OK) return rc;
        if (events) BODA_CUDA_TRY(cudaEventRecord(events[3 * i + 2], stream));
        cur = dst;
    }
    return BODA_OK;
}

void drop_graph(boda_stack* s)
{
    for (auto& g : s->graphs) cudaGraphExecDestroy(g.exec);
    s->graphs.clear();
}

int build_graph(boda_stack* s, const float* in, float* out, cudaStream_t user_stream, cudaGraphExec_t* exec_out)
{
    if (s->graphs.size() >= 8) {                         // keep the most recent ones
        cudaGraphExecDestroy(s->graphs.front().exec);
        s->graphs.erase(s->graphs.begin());
    }
    if (!s->capture_stream) BODA_CUDA_TRY(cudaStreamCreateWithFlags(&s->capture_stream, cudaStreamNonBlocking));
    // one eager pass first, on the caller's stream: per-shape set-up (kernel attributes, tensor maps) must not
    // happen inside a capture
    int rc = run_ops(s, in, out, user_stream, nullptr);
    if (rc != BODA_OK) return rc;
    BODA_CUDA_TRY(cudaStreamBeginCapture(s->capture_stream, cudaStreamCaptureModeThreadLocal));
    rc = run_ops(s, in, out, s->capture_stream, nullptr);
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(s->capture_stream, &graph);
    if (rc != BODA_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
    if (e != cudaSuccess) return record_cuda_error(e, "cudaStreamEndCapture");
    cudaGraphExec_t exec = nullptr;
    e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return record_cuda_error(e, "cudaGraphInstantiate");
    s->graphs.push_back({in, out, exec});
    *exec_out = exec;
    return BODA_OK;
}

}  // namespace

extern "C" {

int boda_stack_destroy(boda_stack* s)
{
    if (!s) return BODA_OK;
    int prev = 0;
    (void)cudaGetDevice(&prev);
    (void)cudaSetDevice(s->device);
    drop_graph(s);
    if (s->sub) boda_stack_destroy(s->sub);
    for (cudaEvent_t ev : s->chunk_events) cudaEventDestroy(ev);
    if (s->entry_event) cudaEventDestroy(s->entry_event);
    if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
    if (s->capture_stream) cudaStreamDestroy(s->capture_stream);
    for (auto& op : s->ops) {
        if (op.plan) boda_conv_plan_destroy(op.plan);
        if (op.out) cudaFree(op.out);
    }
    if (s->workspace) cudaFree(s->workspace);
    if (s->staging_in) cudaFree(s->staging_in);
    if (s->staging_out) cudaFree(s->staging_out);
    (void)cudaSetDevice(prev);
    delete s;
    return BODA_OK;
}

int boda_stack_create(const boda_stack_op* ops, int n_ops, const boda_plan_opts* opts, boda_stack** out)
{
    if (!ops || n_ops <= 0 || !out) return BODA_ERR_INVALID_ARG;
    if (!opts) return boda_stack_create_ex(ops, n_ops, nullptr, out);
    std::vector<boda_plan_opts> per_op((size_t)n_ops, *opts);
    return boda_stack_create_ex(ops, n_ops, per_op.data(), out);
}

int boda_stack_create_ex(const boda_stack_op* ops, int n_ops, const boda_plan_opts* per_op_opts, boda_stack** out)
{
    if (!ops || n_ops <= 0 || !out) return BODA_ERR_INVALID_ARG;
    *out = nullptr;
    if (ops[0].kind != BODA_STACK_CONV) return BODA_ERR_INVALID_ARG;     // the first op fixes the input dims
    boda_stack* s = new (std::nothrow) boda_stack();
    if (!s) return BODA_ERR_NOMEM;
    int device = per_op_opts ? per_op_opts[0].device : -1;
    if (device < 0) { cudaError_t e = cudaGetDevice(&device); if (e != cudaSuccess) { delete s; return record_cuda_error(e, "cudaGetDevice"); } }
    s->device = device;
    s->specs.assign(ops, ops + n_ops);
    if (per_op_opts) s->op_opts.assign(per_op_opts, per_op_opts + n_ops);
    int N = ops[0].conv.N, C = ops[0].conv.C, H = ops[0].conv.H, W = ops[0].conv.W;
    s->in_elems = (size_t)N * C * H * W;
    int rc = BODA_OK;
    for (int i = 0; i < n_ops && rc == BODA_OK; ++i) {
        boda_stack::Op op;
        op.kind = ops[i].kind;
        op.N = N; op.C = C; op.H = H; op.W = W;
        if (op.kind == BODA_STACK_CONV) {
            op.conv = ops[i].conv;
            if (op.conv.N != N || op.conv.C != C || op.conv.H != H || op.conv.W != W) { rc = BODA_ERR_INVALID_ARG; break; }
            // first by rule; layers that ask for tuning are re-planned below, once the layouts around them are known
            boda_plan_opts o;
            boda_plan_opts_default(&o);
            if (per_op_opts) o = per_op_opts[i];
            o.tune = 0;
            rc = boda_conv_plan_create(&op.conv, &o, &op.plan);
            if (rc != BODA_OK) break;
            int oN, oK, oP, oQ;
            conv_plan_out_dims(op.plan, &oN, &oK, &oP, &oQ);
            op.oC = oK; op.oH = oP; op.oW = oQ;
        } else if (op.kind == BODA_STACK_MAXPOOL) {
            op.ksz = ops[i].ksz; op.stride = ops[i].stride;
            op.oC = C;
            op.oH = boda_conv_out_dim(H, op.ksz, op.stride, 0);
            op.oW = boda_conv_out_dim(W, op.ksz, op.stride, 0);
            if (op.oH <= 0 || op.oW <= 0) { rc = BODA_ERR_INVALID_ARG; break; }
        } else { rc = BODA_ERR_INVALID_ARG; break; }
        op.out_elems = (size_t)N * op.oC * op.oH * op.oW;
        s->ops.push_back(op);
        C = op.oC; H = op.oH; W = op.oW;
    }
    // Layout of every activation between two ops: the consumer's staged layout whenever the producer can write it
    // (a tensor-core convolution, or a pool whose own input is staged) and the consumer can read it (a tensor-core
    // convolution that is not a space-to-depth view, or a pool); NCHW otherwise.  The chain's input and output are NCHW.
    const bool chain_layouts = !std::getenv("BODA_STACK_NCHW");
    const bool fuse_pools = !std::getenv("BODA_STACK_NO_POOL_FUSION");
    auto assign_layouts = [&]() {
        const int n = (int)s->ops.size();
        for (auto& op : s->ops) {
            op.in_packed = op.out_packed = op.fused_pool = op.skipped = false;
            op.oHp = op.oWp = op.oCp = op.iHp = op.iWp = op.iCp = 0;
            if (op.kind == BODA_STACK_CONV && op.plan) (void)conv_plan_set_pool(op.plan, 0, 0);
        }
        // which pools run inside the preceding convolution's epilogue
        for (int i = 0; i + 1 < n; ++i) {
            boda_stack::Op& conv = s->ops[i];
            boda_stack::Op& pool = s->ops[i + 1];
            if (fuse_pools && conv.kind == BODA_STACK_CONV && pool.kind == BODA_STACK_MAXPOOL &&
                conv_plan_can_fuse_pool(conv.plan, pool.ksz, pool.stride) && conv_plan_set_pool(conv.plan, pool.ksz, pool.stride) == BODA_OK) {
                conv.fused_pool = true;
                pool.skipped = true;
            }
        }
        // hand-over between the ops that run
        for (int i = 0; i + 1 < n; ++i) {
            boda_stack::Op& prod = s->ops[i];
            if (prod.skipped) continue;
            const int w = prod.fused_pool ? i + 1 : i;       // the op whose activation the producer writes
            if (w + 1 >= n) break;
            boda_stack::Op& cons = s->ops[w + 1];
            const bool can_write = prod.kind == BODA_STACK_CONV ? conv_plan_can_write_packed(prod.plan) : prod.in_packed;
            int Hp = cons.H, Wp = cons.W, Cp = ((cons.C + 31) / 32) * 32;
            bool can_read = true;
            if (cons.kind == BODA_STACK_CONV) can_read = conv_plan_input_geometry(cons.plan, &Hp, &Wp, &Cp);
            if (chain_layouts && can_write && can_read) {
                prod.out_packed = true; prod.oHp = Hp; prod.oWp = Wp; prod.oCp = Cp;
                cons.in_packed = true; cons.iHp = Hp; cons.iWp = Wp; cons.iCp = Cp;
                if (prod.fused_pool) { boda_stack::Op& pl = s->ops[w]; pl.out_packed = true; pl.oHp = Hp; pl.oWp = Wp; pl.oCp = Cp; }
            }
        }
    };
    if (rc == BODA_OK) assign_layouts();
    // Tuning: every layer that asks for it is planned again, its candidates timed the way the chain will run them
    // (staged input without a staging kernel, staged output through the bulk-copy epilogue) - not stand-alone with
    // NCHW on both sides, which would rank the tiles of a different kernel configuration.  A tuned plan may read
    // another staged layout than the rule's plan did, so the layouts are assigned once more afterwards.
    bool retuned = false;
    for (int i = 0; rc == BODA_OK && per_op_opts && i < (int)s->ops.size(); ++i) {
        boda_stack::Op& op = s->ops[i];
        if (op.kind != BODA_STACK_CONV || !per_op_opts[i].tune || per_op_opts[i].tile_id >= 0) continue;
        boda_conv_plan* tuned = nullptr;
        const bool pool_next = fuse_pools && i + 1 < (int)s->ops.size() && s->ops[i + 1].kind == BODA_STACK_MAXPOOL;
        rc = conv_plan_create_chained(&op.conv, &per_op_opts[i], op.in_packed, op.out_packed || (op.fused_pool && s->ops[i + 1].out_packed),
                                      pool_next ? s->ops[i + 1].ksz : 0, pool_next ? s->ops[i + 1].stride : 0, &tuned);
        if (rc != BODA_OK) break;
        boda_conv_plan_destroy(op.plan);
        op.plan = tuned;
        retuned = true;
    }
    if (rc == BODA_OK && retuned) assign_layouts();
    for (const auto& op : s->ops)
        if (op.kind == BODA_STACK_CONV && op.plan && !op.in_packed) s->ws_bytes = std::max(s->ws_bytes, boda_conv_plan_workspace_bytes(op.plan));
    for (int i = 0; rc == BODA_OK && i < (int)s->ops.size(); ++i) {
        boda_stack::Op& op = s->ops[i];
        if (op.kind == BODA_STACK_CONV) {
            rc = conv_plan_set_io(op.plan, op.in_packed ? 1 : 0, op.out_packed ? 1 : 0, op.oHp, op.oWp, op.oCp);
            if (rc != BODA_OK) break;
        }
        if (i + 1 < (int)s->ops.size() && !op.fused_pool) {   // a convolution with a fused pool writes the pool op's activation
            const size_t elems = op.out_packed ? (size_t)op.N * op.oHp * op.oWp * op.oCp : op.out_elems;
            cudaError_t e = cudaMalloc(&op.out, elems * sizeof(float));
            if (e == cudaSuccess) e = cudaMemset(op.out, 0, elems * sizeof(float));   // staged layouts: the padding stays zero
            if (e != cudaSuccess) { rc = record_cuda_error(e, "activation allocation"); break; }
        }
    }
    if (rc == BODA_OK) {
        s->out_elems = s->ops.back().out_elems;
        if (s->ws_bytes) {
            cudaError_t e = cudaMalloc(&s->workspace, s->ws_bytes);
            if (e != cudaSuccess) rc = record_cuda_error(e, "workspace allocation");
        }
    }
    if (rc != BODA_OK) { boda_stack_destroy(s); return rc; }
    *out = s;
    return BODA_OK;
}

int boda_stack_num_ops(const boda_stack* s) { return s ? (int)s->ops.size() : 0; }

int boda_stack_set_filters(boda_stack* s, int op_index, const float* filt, const float* bias, void* stream)
{
    if (!s || op_index < 0 || op_index >= (int)s->ops.size() || !filt) return BODA_ERR_INVALID_ARG;
    boda_stack::Op& op = s->ops[op_index];
    if (op.kind != BODA_STACK_CONV) return BODA_ERR_INVALID_ARG;
    const int rc = boda_conv_plan_bind_filters(op.plan, filt, stream);
    if (rc != BODA_OK) return rc;
    op.filt = filt;
    op.bias = bias;
    drop_graph(s);                       // the graph holds the old pointers
    return BODA_OK;
}

int boda_stack_out_dims(const boda_stack* s, int op_index, int* N, int* C, int* H, int* W)
{
    if (!s || op_index < 0 || op_index >= (int)s->ops.size() || !N || !C || !H || !W) return BODA_ERR_INVALID_ARG;
    const boda_stack::Op& op = s->ops[op_index];
    *N = op.N; *C = op.oC; *H = op.oH; *W = op.oW;
    return BODA_OK;
}

int boda_stack_copy_layer_output(const boda_stack* s, int op_index, float* dst_nchw, void* stream)
{
    if (!s || op_index < 0 || op_index >= (int)s->ops.size() - 1 || !dst_nchw) return BODA_ERR_INVALID_ARG;
    const boda_stack::Op& op = s->ops[op_index];
    if (op.fused_pool) return BODA_ERR_UNSUPPORTED;      // never materialised: only its pooled form exists
    if (op.out_packed)
        return unpack_to_nchw_launch(op.out, dst_nchw, op.N, op.oC, op.oH, op.oW, op.oHp, op.oWp, op.oCp, (cudaStream_t)stream);
    BODA_CUDA_TRY(cudaMemcpyAsync(dst_nchw, op.out, op.out_elems * sizeof(float), cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return BODA_OK;
}

int boda_stack_describe(const boda_stack* s, int op_index, char* buf, size_t n)
{
    if (!s || op_index < 0 || op_index >= (int)s->ops.size() || !buf || n == 0) return BODA_ERR_INVALID_ARG;
    const boda_stack::Op& op = s->ops[op_index];
    char tmp[400];
    if (op.kind == BODA_STACK_CONV) {
        const int rc = boda_conv_plan_describe(op.plan, tmp, sizeof(tmp));
        if (rc != BODA_OK) return rc;
    } else {
        std::snprintf(tmp, sizeof(tmp), "maxpool %dx%d stride %d%s", op.ksz, op.ksz, op.stride,
                      op.skipped ? " (fused into the preceding convolution's epilogue)" : "");
    }
    std::snprintf(buf, n, "%s in=%s out=%s", tmp, op.in_packed ? "staged" : "nchw", op.out_packed ? "staged" : "nchw");
    return BODA_OK;
}

int boda_stack_kernels_per_fwd(const boda_stack* s);

int boda_stack_fwd(boda_stack* s, const float* in, float* out, void* stream)
{
    if (!s || !in || !out) return BODA_ERR_INVALID_ARG;
    cudaGraphExec_t exec = nullptr;
    for (const auto& g : s->graphs)
        if (g.in == in && g.out == out) { exec = g.exec; break; }
    if (!exec) {
        const int rc = build_graph(s, in, out, (cudaStream_t)stream, &exec);
        if (rc != BODA_OK) return rc;
    }
    BODA_CUDA_TRY(cudaGraphLaunch(exec, (cudaStream_t)stream));
    count_launch(boda_stack_kernels_per_fwd(s));
    return BODA_OK;
}

int boda_stack_fwd_eager(boda_stack* s, const float* in, float* out, void* stream, void** events)
{
    if (!s || !in || !out) return BODA_ERR_INVALID_ARG;
    return run_ops(s, in, out, (cudaStream_t)stream, (cudaEvent_t*)events);
}

int boda_stack_run_op(boda_stack* s, int op_index, const float* in, float* out, void* stream)
{
    if (!s || op_index < 0 || op_index >= (int)s->ops.size()) return BODA_ERR_INVALID_ARG;
    const int n = (int)s->ops.size();
    boda_stack::Op& op = s->ops[op_index];
    if (op.skipped) return BODA_OK;                      // runs inside the preceding convolution
    const float* src = op_index == 0 ? in : s->ops[op_index - 1].out;
    const int w = op.fused_pool ? op_index + 1 : op_index;
    float* dst = w == n - 1 ? out : s->ops[w].out;
    if (!src || !dst) return BODA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (op.kind == BODA_STACK_CONV) {
        if (!op.filt) return BODA_ERR_INVALID_ARG;
        return conv_fwd_planned_ex(op.plan, src, op.filt, op.bias, dst, s->workspace, st, nullptr);
    }
    if (op.in_packed)
        return maxpool_packed_launch(src, dst, op.N, op.C, op.H, op.W, op.iHp, op.iWp, op.iCp, op.ksz, op.stride,
                                     op.out_packed ? 1 : 0, op.oHp, op.oWp, op.oCp, st);
    return maxpool_launch(src, dst, op.N, op.C, op.H, op.W, op.ksz, op.stride, st);
}

// Decides how the host path slices the batch and builds the sub-batch stack (same layers, same options, batch N/k).
static void prepare_host_slices(boda_stack* s)
{
    s->host_chunks = 1;
    const int N = s->specs[0].conv.N;
    // measured on the AlexNet-shaped stack at batch 20 (12.4 MB in): whole batch 406 us per call, two slices 305 us,
    // four 373 us, five 440 us - sub-batch kernels fill the GPU less well, so more slices cost more than they hide
    int k = (N % 2 == 0 && N >= 4) ? 2 : 1;
    if (const char* e = std::getenv("BODA_STACK_HOST_CHUNKS")) {
        const int v = std::atoi(e);
        if (v >= 1 && N % v == 0) k = v;
    }
    if (k <= 1) return;
    std::vector<boda_stack_op> specs = s->specs;
    for (auto& op : specs)
        if (op.kind == BODA_STACK_CONV) op.conv.N = N / k;
    boda_stack* sub = nullptr;
    if (boda_stack_create_ex(specs.data(), (int)specs.size(), s->op_opts.empty() ? nullptr : s->op_opts.data(), &sub) != BODA_OK) return;
    sub->host_chunks = 1;
    bool ok = cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s->entry_event, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < k; ++i) {
        cudaEvent_t ev = nullptr;
        ok = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
        if (ok) s->chunk_events.push_back(ev);
    }
    if (!ok) { boda_stack_destroy(sub); return; }
    s->sub = sub;
    s->host_chunks = k;
}

int boda_stack_fwd_host(boda_stack* s, const float* in_host, float* out_host, void* stream)
{
    if (!s || !in_host || !out_host) return BODA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    // slices of the batch start on 256-byte boundaries of the staging buffer (kernels want 16-byte aligned tensors)
    if (!s->staging_in) BODA_CUDA_TRY(cudaMalloc(&s->staging_in, (s->in_elems + 64 * 8) * sizeof(float)));
    if (!s->staging_out) BODA_CUDA_TRY(cudaMalloc(&s->staging_out, s->out_elems * sizeof(float)));
    if (s->host_chunks == 0) prepare_host_slices(s);
    if (s->host_chunks > 1) {
        // the sub-batch stack uses the same filters
        for (size_t i = 0; i < s->ops.size(); ++i) {
            const boda_stack::Op& op = s->ops[i];
            if (op.kind != BODA_STACK_CONV) continue;
            if (!op.filt) return BODA_ERR_INVALID_ARG;
            if (s->sub->ops[i].filt != op.filt || s->sub->ops[i].bias != op.bias) {
                const int rc = boda_stack_set_filters(s->sub, (int)i, op.filt, op.bias, stream);
                if (rc != BODA_OK) return rc;
            }
        }
        const int k = s->host_chunks;
        const size_t in_chunk = s->in_elems / k, out_chunk = s->out_elems / k;
        const size_t in_pitch = (in_chunk + 63) & ~(size_t)63;            // floats between slice starts in the staging buffer
        // The call is ordered on `stream`: the slices are copied on a second stream, which first waits for everything
        // the caller has queued on `stream` so far (a kernel or copy that fills in_host, for instance).
        BODA_CUDA_TRY(cudaEventRecord(s->entry_event, st));
        BODA_CUDA_TRY(cudaStreamWaitEvent(s->copy_stream, s->entry_event, 0));
        // the staging buffers are idle: every return of this function leaves both streams drained
        int rc = BODA_OK;
        cudaError_t ce = cudaSuccess;
        for (int i = 0; i < k && ce == cudaSuccess; ++i) {
            ce = cudaMemcpyAsync(s->staging_in + i * in_pitch, in_host + i * in_chunk, in_chunk * sizeof(float),
                                 cudaMemcpyHostToDevice, s->copy_stream);
            if (ce == cudaSuccess) ce = cudaEventRecord(s->chunk_events[i], s->copy_stream);
        }
        for (int i = 0; i < k && ce == cudaSuccess && rc == BODA_OK; ++i) {
            ce = cudaStreamWaitEvent(st, s->chunk_events[i], 0);
            if (ce == cudaSuccess) rc = boda_stack_fwd(s->sub, s->staging_in + i * in_pitch, s->staging_out + i * out_chunk, stream);
            if (ce != cudaSuccess || rc != BODA_OK) break;
            // a slice's result goes back while the next slice is still computing: on the copy stream (behind the
            // input copies, which are done by then) for all but the last slice
            cudaStream_t back = i + 1 < k ? s->copy_stream : st;
            if (i + 1 < k) {
                ce = cudaEventRecord(s->chunk_events[i], st);             // the slice's input event has been consumed above
                if (ce == cudaSuccess) ce = cudaStreamWaitEvent(s->copy_stream, s->chunk_events[i], 0);
            }
            if (ce == cudaSuccess)
                ce = cudaMemcpyAsync(out_host + i * out_chunk, s->staging_out + i * out_chunk, out_chunk * sizeof(float),
                                     cudaMemcpyDeviceToHost, back);
        }
        if (ce != cudaSuccess || rc != BODA_OK) {
            // no copy may still be writing the staging buffer when the caller gets the error
            (void)cudaStreamSynchronize(s->copy_stream);
            (void)cudaStreamSynchronize(st);
            return rc != BODA_OK ? rc : record_cuda_error(ce, "boda_stack_fwd_host (sliced copies)");
        }
        BODA_CUDA_TRY(cudaStreamSynchronize(s->copy_stream));
        BODA_CUDA_TRY(cudaStreamSynchronize(st));
        return BODA_OK;
    }
    BODA_CUDA_TRY(cudaMemcpyAsync(s->staging_in, in_host, s->in_elems * sizeof(float), cudaMemcpyHostToDevice, st));
    const int rc = boda_stack_fwd(s, s->staging_in, s->staging_out, stream);
    if (rc != BODA_OK) return rc;
    BODA_CUDA_TRY(cudaMemcpyAsync(out_host, s->staging_out, s->out_elems * sizeof(float), cudaMemcpyDeviceToHost, st));
    BODA_CUDA_TRY(cudaStreamSynchronize(st));
    return BODA_OK;
}

int boda_stack_kernels_per_fwd(const boda_stack* s)
{
    if (!s) return 0;
    int n = 0;
    for (const auto& op : s->ops) n += op.kind == BODA_STACK_CONV ? boda_conv_plan_kernels_per_call(op.plan) : op.skipped ? 0 : 1;
    return n;
}

}  // extern "C"
