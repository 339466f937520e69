/*
 * boda.h - C ABI of the B200 (sm_100a) convolution-forward library.
 *
 * The library computes the forward pass of one CNN convolution layer,
 *
 *     out[n][k][p][q] = act( bias[k] + sum_{c,r,s} in[n][c][p*stride+r-pad][q*stride+s-pad]
 *                                                  * filt[k][c][r][s] )
 *
 * with zero padding, P = (H + 2*pad - R)/stride + 1 (floor; Q likewise) and act = ReLU or identity.
 * This is the operation out = conv(in, filts) of Section 2 of the Boda-RTC paper (arXiv 1606.00094):
 * the window of `in` for an output point starts at (oy*stride, ox*stride) of the (padded) input and
 * spans all input channels; the output is the sum of the element-wise product of that window and
 * the filter slice of the output channel (a cross-correlation, no flip); ReLU = max(0, x) is fused
 * into the operation.  The bias, which the paper sets aside, is a per-output-channel constant added
 * before the activation.
 *
 * Conventions that hold for every entry point unless stated otherwise
 *   - Tensor pointers are DEVICE pointers to dense, row-major fp32 arrays owned by the caller:
 *       in [N][C][H][W], filt [K][C][R][S], bias [K] (NULL means no bias), out [N][K][P][Q].
 *     They must be at least 16-byte aligned; `out` must not overlap any input.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue work
 *     and return; they do not synchronise unless the comment says so.
 *   - Every function returns a boda_status (0 = success).  Nothing throws across the ABI.
 *   - The library keeps per-device caches (plans made by boda_conv_fwd, packed operands); they are
 *     protected by one mutex, so calls may come from several host threads.
 *   - Not supported, and reported as an error rather than silently mis-computed: groups, dilation,
 *     different stride or padding per spatial dimension (the paper restricts itself to scalar
 *     kernel size and stride; R != S is accepted).
 */
#ifndef BODA_H_
#define BODA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum boda_status {
    BODA_OK = 0,
    BODA_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive extent, stride < 1, pad < 0, window larger than padded input */
    BODA_ERR_UNSUPPORTED = 2,    /* device is not sm_100, or a forced variant / tile is illegal for the shape */
    BODA_ERR_CUDA = 3,           /* a CUDA runtime or driver call failed; boda_last_error_string() has the text */
    BODA_ERR_DEVICE_TIMEOUT = 4, /* a bounded wait inside a kernel expired (reported by boda_query_status) */
    BODA_ERR_NOMEM = 5,          /* device or host allocation failed, or the workspace given is too small */
    BODA_ERR_TOO_LARGE = 6       /* a size exceeds a fixed capacity stated by the entry point */
} boda_status;

/* Kernel variants.  The names follow Section 5 of the paper: `conv` (implicit-GEMM fallback, here an
 * FP32 CUDA-core kernel called DIRECT), `k1conv` (kernel size 1: a plain GEMM over input channels)
 * and `tconv` (tiled convolution for kernel sizes 2..11).  K1CONV and TCONV run on the tcgen05
 * tensor cores in TF32 with fp32 accumulation. */
enum { BODA_VARIANT_AUTO = -1, BODA_VARIANT_DIRECT = 0, BODA_VARIANT_K1CONV = 1, BODA_VARIANT_TCONV = 2 };

/* Arithmetic the plan may use. */
enum { BODA_MATH_AUTO = 0,       /* TF32 tensor cores where a tensor-core variant applies */
       BODA_MATH_FP32 = 1,       /* FP32 FMA only (DIRECT); relative L2 error vs fp64 <= 1e-5 */
       BODA_MATH_TF32 = 2,       /* TF32 operands, fp32 accumulate; relative L2 error <= 5e-3 */
       BODA_MATH_TF32X3 = 3 };   /* error-compensated TF32 on the tensor cores: every operand is split into a TF32
                                    value and a TF32 remainder, and each product is formed as hi*hi + lo*hi + hi*lo
                                    (three tensor-core products, fp32 accumulate); meets the FP32 bar (<= 1e-5) at
                                    about a third of the TF32 rate.  The paper names reduced and mixed precision as
                                    the next step (Sections 2 and 6); this is the mode for callers who need FP32
                                    accuracy from the tensor cores.  NCHW in and out only; K1CONV and TCONV (im2col
                                    kernel); where no tensor-core variant is legal the FP32 kernel runs instead. */
enum { BODA_MATH_F16 = 4 };      /* reduced-precision STORAGE (Section 2 of the paper notes that 16-bit storage suffices for
                                    inference; Section 6 lists it as the next step): input and filters are rounded to
                                    fp16 (nearest even) when they are staged, products are exact and accumulate in
                                    fp32 on the tensor cores (kind::f16, 16 channels per MMA instead of 8), output is
                                    fp32.  A precision class of its own, never chosen automatically: fp16 keeps TF32's
                                    10 mantissa bits, so the relative L2 error against the fp64 result stays <= 5e-3
                                    for operands inside fp16's range (|x| < 65504; larger values overflow to infinity,
                                    values below 6e-8 flush to zero), and <= 1e-5 against the fp64 result computed
                                    from the fp16-rounded operands.  NCHW in and out only; K1CONV and TCONV (im2col
                                    kernel); where no tensor-core variant is legal the FP32 kernel runs instead. */

typedef struct boda_conv_shape {
    int N, C, H, W;              /* input  [N][C][H][W] */
    int K, R, S;                 /* filters [K][C][R][S] */
    int stride, pad;             /* same in both spatial dimensions; zero padding */
    int relu;                    /* 0: identity, otherwise max(0, x) */
} boda_conv_shape;

typedef struct boda_plan_opts {
    int math;                    /* BODA_MATH_* */
    int tune;                    /* 0: pick variant and tile by rule; 1: time the candidates on the device (synchronises):
                                    every tile and split of the rule's variant and, where `variant` and `math` are
                                    left automatic, of the alternative variant too (FP32 kernel against tensor-core
                                    kernel, a strided TCONV layer with and without its space-to-depth view) */
    int variant;                 /* BODA_VARIANT_AUTO or a forced variant (used by tests) */
    int tile_id;                 /* -1: automatic; otherwise index into the variant's tile table (boda_conv_plan_describe
                                    prints the name).  BODA_VARIANT_DIRECT: 0..8 GEMM-blocked FP32 tiles direct_128x128 ..
                                    direct_32x16, 9..11 pixel-per-thread direct_pixel_k8/16/32, 12..15 the same compiled
                                    at run time for the exact shape direct_rtc_k4/8/16/32.  K1CONV / TCONV (pixels x
                                    channels): 0..4 igemm_128x64/96/128/192/256 (TMA im2col tiles, cluster split),
                                    5..15 halo_128/256/512xBN (TCONV stride 1 or space-to-depth view: shared-memory
                                    reuse of the input across taps), 16..19 gconv_128x64/96/128/192 (input gathered
                                    from NCHW, nothing staged; short reductions and 1x1), 20..22 k1nchw_128x64/128/192
                                    (K1CONV by TMA straight from NCHW; split_k > 1: a cluster split over the input
                                    channels), 23..25 first_512x64/96/128 (TCONV for 3 input channels, stride 4, no
                                    padding, windows up to 11x11: the space-to-depth view built in shared memory
                                    straight from NCHW, nothing staged).  A tile that cannot run the shape is refused
                                    with BODA_ERR_UNSUPPORTED. */
    int split_k;                 /* 0: automatic; otherwise the number of reduction splits of a tensor-core variant */
    int device;                  /* CUDA device ordinal; -1: the current device */
    int s2d;                     /* strided TCONV layers: -1 automatic, 0 never, 1 always run the stride-1
                                    "space-to-depth" view (stride t on C channels = stride 1 on C*t*t channels
                                    with ceil(R/t) x ceil(S/t) taps); an input transformation in the sense of
                                    Section 5 of the paper */
    size_t max_workspace;        /* 0: no limit; otherwise the largest boda_conv_plan_workspace_bytes the caller accepts:
                                    tiles that need more are not considered (a layer may then run on a kernel that
                                    stages nothing, or on the FP32 kernel); a forced variant or tile that needs more
                                    is refused with BODA_ERR_NOMEM */
} boda_plan_opts;

typedef struct boda_conv_plan boda_conv_plan;   /* opaque; created and destroyed by the library */

/* Output extent of one spatial dimension, 1 + (in + 2*pad - ksz)/stride with floor division
 * (Section 2: out_X = 1 + (in_X - KSZ)/stride on the padded input).  Returns 0 if the window does
 * not fit.  Host-only helper. */
int boda_conv_out_dim(int in_dim, int ksz, int stride, int pad);

/* Fill *opts with the defaults (automatic everything, current device). */
void boda_plan_opts_default(boda_plan_opts* opts);

/*
 * Variant selection and blocking for one layer shape: the analogue of the paper's flow
 * "operation -> variant -> blocking constants" (Section 4, Figure "codegen", and the variant rules
 * of Section 5: k1conv for kernel size 1, tconv for kernel sizes 2..11, conv otherwise).  With
 * opts->tune != 0 the legal candidates are timed on scratch buffers (ten calls captured in a CUDA graph,
 * best of three replays) and the fastest is kept (the automated tuning the paper names as future work);
 * this allocates, launches and synchronises, so it must not run while a stream is being captured.  If the
 * environment variable BODA_TUNE_CACHE names a file, tuned choices are read from and appended to it (one
 * text line "shape-and-options tile split variant s2d" per tuned shape).
 * `opts` may be NULL (defaults).  On success *plan owns device memory (index tables, packed filter
 * storage, workspace); destroy it with boda_conv_plan_destroy.
 * Errors: INVALID_ARG (bad shape), UNSUPPORTED (forced variant illegal, device not sm_100), CUDA, NOMEM.
 */
int boda_conv_plan_create(const boda_conv_shape* shape, const boda_plan_opts* opts, boda_conv_plan** plan);

/* Frees everything the plan owns.  The caller must make sure no launch that uses it is in flight. */
int boda_conv_plan_destroy(boda_conv_plan* plan);

/* Writes a NUL-terminated one-line description (variant, tile, split, math, workspace) into buf. */
int boda_conv_plan_describe(const boda_conv_plan* plan, char* buf, size_t buf_bytes);

/* Bytes of caller-provided scratch that boda_conv_fwd_planned needs (0 if none).  The scratch holds
 * the re-laid-out input (the "input transformation" that the paper's k1conv and tconv apply, Section 5). */
size_t boda_conv_plan_workspace_bytes(const boda_conv_plan* plan);

/* Kernels one boda_conv_fwd_planned call launches when the filters are bound: 1 for DIRECT and for the tensor-core
 * kernels that read NCHW themselves (gather, NCHW 1x1, first-layer kernel), 2 for the others (input staging and the
 * main kernel). */
int boda_conv_plan_kernels_per_call(const boda_conv_plan* plan);

/*
 * Optional: pre-pack the filters (and remember the bias pointer's contents are NOT copied) for a
 * tensor-core plan, so that boda_conv_fwd_planned can skip the per-call filter re-layout.  Weights
 * are constants at deployment time (Section 2 speaks of deployment / inference).  After binding,
 * the `filt` argument of boda_conv_fwd_planned is ignored when it equals the bound pointer; passing
 * a different pointer re-packs on that call.  Runs the re-layout on `stream` and waits for it (a set-up call,
 * not for the hot path): later launches may then fetch the packed filters without waiting for their predecessor
 * in the stream.  `filt` must stay unchanged while bound.
 */
int boda_conv_plan_bind_filters(boda_conv_plan* plan, const float* filt, void* stream);

/*
 * The forward pass with an explicit plan.  `workspace` must point to at least
 * boda_conv_plan_workspace_bytes(plan) bytes of device memory, 256-byte aligned (NULL if 0 bytes);
 * it may be shared between plans whose launches are ordered on one stream.  No allocation and no
 * synchronisation happen here.  The same plan must not be used from two streams at once.
 * Errors: INVALID_ARG (NULL tensor), CUDA (launch failure).
 */
int boda_conv_fwd_planned(boda_conv_plan* plan, const float* in, const float* filt, const float* bias,
                          float* out, void* workspace, void* stream);

/*
 * The forward pass in one call (the signature named by the build's specification).  Looks up, or
 * creates with default options, a plan for the shape on the current device and an internal
 * workspace, then launches on `stream`.  The first call for a shape allocates; later calls do not.
 */
int boda_conv_fwd(const float* in, const float* filt, const float* bias, float* out,
                  int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int relu,
                  void* stream);

/*
 * Same operation with HOST pointers: copies in / filt / bias to device staging buffers kept by the
 * library, runs the planned kernel(s) and copies `out` back, all on `stream`, then synchronises the
 * stream so that `out` is valid on return.  Pinned host memory makes the copies asynchronous.
 */
int boda_conv_fwd_host(const float* in_host, const float* filt_host, const float* bias_host, float* out_host,
                       int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int relu,
                       void* stream);

/*
 * Single-precision matrix product C[M][N] = A[M][K] * B[K][N], all three row-major, dense, fp32 DEVICE
 * pointers (the paper's warm-up operation: Section 4, Table 1 lists square sizes 128 ... 2048 with
 * 2*M*N*K FLOPs and 4*(M*K + K*N + M*N) bytes).  Section 5 observes that a 1x1 convolution "is" this
 * product; the library takes that literally and runs the product as the 1x1 convolution of a one-image
 * input in[1][K][1][N] = B with filters filt[M][K][1][1] = A, no bias, no ReLU, through the same plan
 * cache and kernels as boda_conv_fwd (default options: TF32 tensor cores where profitable, so the
 * TF32 error bar applies).  The first call for a size allocates; later calls do not.
 * Errors: INVALID_ARG (NULL pointer, non-positive size), plus those of boda_conv_fwd.
 */
int boda_sgemm(const float* A, const float* B, float* C, int M, int N, int K, void* stream);

/*
 * Run-time compilation (Section 4 of the paper: kernels are generated and compiled for the exact problem once its
 * sizes are known, so that every extent is a literal).  The DIRECT tiles named direct_rtc_k4 / k8 / k16 / k32
 * (tile ids 12..15 of BODA_VARIANT_DIRECT; also what automatic selection uses for layers with C*R*S <= 512 and
 * K <= 128 that stay on the FP32 kernel) are compiled by NVRTC when their plan is created: one thread per output pixel and `kt` output channels,
 * all of N, C, H, W, K, R, S, stride, pad, ReLU and the blocking as compile-time constants.  They need the NVRTC
 * shared library at run time (looked up with dlopen; without it - or with BODA_NO_RTC=1 in the environment - those
 * tiles return BODA_ERR_UNSUPPORTED and automatic selection keeps the precompiled kernels; the first plan for a
 * shape pays the compilation, 0.3 to 3 seconds) and an input patch plus filters of at most 48 KB.
 *
 * boda_direct_rtc_compile compiles the kernel for `shape` without loading or running it - it needs no GPU - and
 * reports the blocking chosen and the size of the device image.  Any of the four output pointers may be NULL.
 * Returns BODA_OK, BODA_ERR_INVALID_ARG (bad shape, kt not 4, 8, 16 or 32), BODA_ERR_UNSUPPORTED (no NVRTC, or
 * the shape does not fit), BODA_ERR_CUDA (the compiler refused the source; boda_last_error_string has its log).
 */
int boda_direct_rtc_compile(const boda_conv_shape* shape, int kt, int* block_x, int* block_y, size_t* smem_bytes,
                            size_t* image_bytes);

/*
 * The forward pass for callers that must not allocate device memory.  (The paper has no counterpart: this
 * is a property of the library, not of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework whose caching allocator
 * owns all device memory and forbids side allocations, in a real-time loop where an allocation's implicit
 * device synchronisation and unbounded latency are not acceptable, in a process whose memory budget was
 * fixed at start-up, or after start-up under a policy that freezes the address space.  boda_conv_fwd
 * allocates a plan and a workspace the first time it sees a shape; this entry point never does.
 *
 * What it does: the same operation as boda_conv_fwd, always on the tensor-core path (K1CONV for R = S = 1,
 * TCONV otherwise; TF32 operands, fp32 accumulation), with the kernel's scratch - the re-laid-out input and
 * filters and a status word - in a device array of BODA_NOALLOC_SCRATCH_BYTES that is
 * part of the library image.  Every GPU that loads the library holds that array until the process exits.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  in / filt / bias / out are device
 * pointers owned by the caller, as for boda_conv_fwd.
 *
 * Limits and rules
 *   - Shapes whose scratch does not fit (roughly 4 * (N*H*W + R*S*K) * roundup(C, 32) bytes plus a small
 *     header) are rejected with BODA_ERR_TOO_LARGE; shapes outside the tensor-core variants (R or S > 11,
 *     stride > 8) with BODA_ERR_UNSUPPORTED.  Nothing is launched in either case.
 *   - The first call on a device resolves the array's device address (cudaGetSymbolAddress), loads two
 *     driver entry points and raises the kernel's shared-memory limit.  Make that first call during
 *     start-up, before any stream capture begins.
 *   - All calls share the one array and it keeps the previous call's contents; the entry point clears the
 *     words that must start at zero itself.  Two calls whose GPU work can overlap (different streams
 *     without an ordering between them, or different host threads on unordered streams) race on the
 *     array and give wrong results: order them on one stream or with events.
 *   - A bounded wait that expires inside the kernel is recorded in the array's own header, which
 *     boda_query_status does not read; the output is then left unwritten.
 */
#define BODA_NOALLOC_SCRATCH_BYTES (32u << 20)
int boda_conv_fwd_noalloc(const float* in, const float* filt, const float* bias, float* out,
                          int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int relu,
                          void* stream);

/*
 * Max-pooling, ksz x ksz window, given stride, no padding, floor output extent; the pooling that
 * sits between the convolutions of the AlexNet-shaped stack (the paper lists pooling among the
 * deployment operations, Section 2, without analysing it).  in [N][C][H][W] -> out [N][C][P][Q],
 * device pointers.
 */
int boda_maxpool_fwd(const float* in, float* out, int N, int C, int H, int W, int ksz, int stride,
                     void* stream);

/*
 * Softmax over the last dimension, out[r][j] = exp(in[r][j]) / sum over i of exp(in[r][i]) (the third operation
 * Section 2 of the paper lists for deployment, beside convolution and pooling; it follows the classifier at the end
 * of a network).  in, out: [rows][cols] row-major fp32 DEVICE pointers, may be the same buffer; fp32 arithmetic with
 * the row maximum subtracted before exp.  Enqueues one kernel on `stream`; no allocation, no synchronisation.
 * Errors: BODA_ERR_INVALID_ARG (NULL pointer, non-positive extent), BODA_ERR_CUDA.
 */
int boda_softmax_fwd(const float* in, float* out, int rows, int cols, void* stream);

/*
 * A chain of layers run as one unit: convolutions (each followed by its bias and ReLU) and max-pools, layer
 * i+1 reading layer i's output - the shape of a CNN's convolutional trunk such as the AlexNet-shaped stack the
 * benchmark uses.  (The paper's framework runs a whole compute graph, Section 4 and Figure "Boda flow"; this is
 * the minimal form of it: a linear chain.)  The stack owns its plans, the activations between layers, one
 * workspace and a CUDA graph of the chain, so that boda_stack_fwd is one graph launch.
 * Fusion (the paper's argument for writing convolution kernels instead of calling a BLAS, Section 3): a 3x3 / stride-2
 * max-pool that follows a convolution whose kernel works on whole output rows (halo tiles of 256 or 512 positions, the
 * first-layer kernel) runs inside that kernel's epilogue; the convolution's own output is then never written, the pool
 * op launches nothing, and boda_stack_copy_layer_output returns BODA_ERR_UNSUPPORTED for that convolution.
 * BODA_STACK_NO_POOL_FUSION=1 in the environment keeps every pool a kernel of its own.  With opts->tune the layers are
 * tuned the way the chain runs them (staged input and output, the pool that follows included).
 */
enum { BODA_STACK_CONV = 0, BODA_STACK_MAXPOOL = 1 };
typedef struct boda_stack_op {
    int kind;                    /* BODA_STACK_CONV or BODA_STACK_MAXPOOL */
    boda_conv_shape conv;        /* CONV: the layer; its N, C, H, W must equal the previous op's output */
    int ksz, stride;             /* MAXPOOL: window and stride (no padding, floor extent) */
} boda_stack_op;
typedef struct boda_stack boda_stack;

/* Plans every convolution with `opts` (NULL = defaults) and allocates activations and workspace.  The first op
 * must be a convolution (it fixes the input extent).  Errors as boda_conv_plan_create, INVALID_ARG if shapes do
 * not chain. */
int boda_stack_create(const boda_stack_op* ops, int n_ops, const boda_plan_opts* opts, boda_stack** stack);
/* The same with one set of plan options per op: `per_op_opts` points to n_ops entries (those of MAXPOOL ops are
 * ignored); entry 0 also names the device.  For tests and experiments that force a tile or split per layer. */
int boda_stack_create_ex(const boda_stack_op* ops, int n_ops, const boda_plan_opts* per_op_opts, boda_stack** stack);
int boda_stack_destroy(boda_stack* stack);
int boda_stack_num_ops(const boda_stack* stack);
/* Device pointers to the filters [K][C][R][S] and bias [K] (or NULL) of convolution op `op_index`; the stack keeps
 * the pointers (the caller keeps the memory alive) and pre-packs the filters on `stream`. */
int boda_stack_set_filters(boda_stack* stack, int op_index, const float* filt, const float* bias, void* stream);
/* Output extent [N][C][H][W] of op `op_index`. */
int boda_stack_out_dims(const boda_stack* stack, int op_index, int* N, int* C, int* H, int* W);
/* Copies the activation that op `op_index` wrote in the last forward pass into dst [N][C][H][W] (device memory, the
 * extent boda_stack_out_dims reports), on `stream`.  Not for the last op, which writes the caller's buffer.
 * Between tensor-core layers the stack keeps activations in the consumer's staged layout (channels innermost,
 * zero padded, rounded to TF32 - the paper's "input transformation", written directly by the producing kernel);
 * this call converts back. */
int boda_stack_copy_layer_output(const boda_stack* stack, int op_index, float* dst, void* stream);
int boda_stack_describe(const boda_stack* stack, int op_index, char* buf, size_t buf_bytes);
/* Kernels one forward pass launches. */
int boda_stack_kernels_per_fwd(const boda_stack* stack);
/*
 * Forward pass, device pointers: in [N][C][H][W] of the first op, out = output of the last op.  The first call
 * for a given (in, out) pair runs the chain once eagerly on `stream` and captures it into a CUDA graph (this
 * allocates and must not itself be inside a stream capture); later calls with the same pointers are one
 * cudaGraphLaunch on `stream`.  Asynchronous.
 */
int boda_stack_fwd(boda_stack* stack, const float* in, float* out, void* stream);
/* Same without the graph: the kernels are launched one by one on `stream`.  `events`, if not NULL, points to
 * 3 * n_ops cudaEvent_t handles; for op i the library records events[3i] before its first kernel, events[3i+1]
 * between operand staging and the main kernel, and events[3i+2] after its last kernel (per-layer timing). */
int boda_stack_fwd_eager(boda_stack* stack, const float* in, float* out, void* stream, void** events);
/* Runs op `op_index` alone on the activations that the last forward pass left in the stack (for timing one layer
 * in place).  `in` is read only by op 0 and `out` written only by the last op; pass NULL otherwise. */
int boda_stack_run_op(boda_stack* stack, int op_index, const float* in, float* out, void* stream);
/* Forward pass with HOST buffers: copies `in_host` to the device, runs the chain, copies the result into
 * `out_host` and synchronises `stream`.  The call is ordered on `stream`: `in_host` is not read before the work
 * queued on `stream` so far has finished (the copies run on a second stream that first waits for it).  On an
 * error return no copy is still in flight.  Pinned host memory makes the copies asynchronous.  Batch items are
 * independent (Section 2 of the paper), so for even N >= 4 the batch is copied in two slices (BODA_STACK_HOST_CHUNKS=k: k slices) on a second
 * stream and each slice runs, as soon as it has arrived, through a stack of the same layers planned for the
 * sub-batch (created on the first call; same filters; BODA_STACK_HOST_CHUNKS=1 in the environment keeps the batch
 * whole): host-to-device copies and kernels overlap.  Results meet the same error bars as boda_stack_fwd but need
 * not be bitwise equal to it (the sub-batch plans may sum in another order). */
int boda_stack_fwd_host(boda_stack* stack, const float* in_host, float* out_host, void* stream);

/*
 * Reads the device-side status word of the current device: kernels never trap or spin for ever;
 * a bounded wait that expires records BODA_ERR_DEVICE_TIMEOUT there and the kernel returns.
 * Synchronises `stream`, copies the word to *device_status (BODA_OK if nothing was recorded) and
 * clears it.
 */
int boda_query_status(void* stream, int* device_status);

/* Releases the per-device caches made by boda_conv_fwd / boda_conv_fwd_host (plans, workspaces). */
int boda_clear_caches(void);

const char* boda_status_string(int status);

/* Text of the last CUDA error seen by the calling thread ("" if none). */
const char* boda_last_error_string(void);

/* Number of kernels this library has launched in this process so far (all devices, all threads).
 * A counter for benchmarks and tests that want to state how much of the work ran in these kernels. */
unsigned long long boda_kernel_launch_count(void);

/* Library version, e.g. 100 for 0.1.0. */
int boda_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BODA_H_ */
