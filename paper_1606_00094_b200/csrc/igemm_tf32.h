// Tensor-core (tcgen05, TF32) implicit-GEMM variants K1CONV and TCONV: host-side interface.
#pragma once

#include "boda_internal.h"

namespace boda {

struct IgemmPlan;

bool igemm_variant_legal(const ConvDims& d, int variant);
// Rule used by automatic selection: is the tensor-core path expected to beat DIRECT for this shape?
bool igemm_variant_profitable(const ConvDims& d);
int igemm_num_tiles();
int igemm_num_split_candidates();
int igemm_split_candidate(int i);

// s2d: -1 automatic, 0 never, 1 force the space-to-depth view of a strided tconv layer.
// mode: 0 TF32; 1 error-compensated TF32 (three tensor-core products per FP32 product); 2 fp16 operands (fp32
// accumulate).  Modes 1 and 2: im2col kernel only, NCHW in and out.
// max_ws: 0, or the largest workspace (staged input) the caller accepts; BODA_ERR_NOMEM if no tile fits it.
int igemm_plan_create(const ConvDims& d, int variant, int tile_id, int split_k, int s2d, int* d_status, IgemmPlan** out,
                      int mode = 0, size_t max_ws = 0);
bool igemm_s2d_applicable(const ConvDims& d);
void igemm_plan_destroy(IgemmPlan* p);
int igemm_plan_tile(const IgemmPlan* p);
bool igemm_plan_writes_packed(const IgemmPlan* p);       // can the plan write a consumer's staged layout?
int igemm_plan_kernels_per_call(const IgemmPlan* p);     // 1, or 2 where an input staging kernel runs first
int igemm_plan_splits(const IgemmPlan* p);
size_t igemm_plan_workspace_bytes(const IgemmPlan* p);
void igemm_plan_describe(const IgemmPlan* p, char* buf, size_t n);
int igemm_bind_filters(IgemmPlan* p, const float* filt, cudaStream_t stream);
void igemm_unbind_filters(IgemmPlan* p);
// after_staging (may be null): event recorded on the stream between the operand-staging kernels and the main kernel
int igemm_launch(IgemmPlan* p, const float* in, const float* filt, const float* bias, float* out, void* workspace,
                 cudaStream_t stream, cudaEvent_t after_staging = nullptr);

// Activation layouts for chained layers.  igemm_plan_input_geometry: the staged input layout this plan reads,
// rows [(n*Hp + y)*Wp + x][Cp] (false if the plan cannot take a staged input).  igemm_plan_set_io: in_packed =
// the `in` pointer of igemm_launch already is that layout (no staging kernel, no workspace); out_packed = write
// the output as rows [(n*oHp + p)*oWp + q][oCp] rounded to TF32 instead of NCHW.
bool igemm_plan_input_geometry(const IgemmPlan* p, int* Hp, int* Wp, int* Cp);
int igemm_plan_set_io(IgemmPlan* p, int in_packed, int out_packed, int oHp, int oWp, int oCp);

// Fused ReLU -> 3x3 / stride-2 max-pooling in the epilogue (halo tiles with 2 or 4 accumulators, no split): the plan
// then writes the POOLED tensor (out_packed geometry and NCHW extents refer to it).  set_pool(p, 0, 0) undoes it.
// Call set_pool before set_io.
bool igemm_plan_can_fuse_pool(const IgemmPlan* p, int ksz, int stride);
int igemm_plan_set_pool(IgemmPlan* p, int ksz, int stride);
void igemm_plan_pooled_dims(const IgemmPlan* p, int* P, int* Q);

// Scratch-in-a-caller-region form (allocates nothing): bytes needed at least, and the run itself.
size_t igemm_region_min_bytes(const ConvDims& d);
int igemm_run_in_region(const ConvDims& d, int variant, const float* in, const float* filt, const float* bias,
                        float* out, void* region, size_t region_bytes, cudaStream_t stream);

}  // namespace boda
