#include "igemm_tf32.h"
namespace boda {
bool igemm_variant_legal(const ConvDims&, int) { return false; }
bool igemm_variant_profitable(const ConvDims&) { return false; }
int igemm_num_tiles() { return 0; }
int igemm_num_split_candidates() { return 0; }
int igemm_split_candidate(int) { return 1; }
int igemm_plan_create(const ConvDims&, int, int, int, int*, IgemmPlan**) { return BODA_ERR_UNSUPPORTED; }
void igemm_plan_destroy(IgemmPlan*) {}
int igemm_plan_tile(const IgemmPlan*) { return 0; }
size_t igemm_plan_workspace_bytes(const IgemmPlan*) { return 0; }
void igemm_plan_describe(const IgemmPlan*, char* b, size_t n) { if (n) b[0] = 0; }
int igemm_bind_filters(IgemmPlan*, const float*, cudaStream_t) { return BODA_ERR_UNSUPPORTED; }
void igemm_unbind_filters(IgemmPlan*) {}
int igemm_launch(IgemmPlan*, const float*, const float*, const float*, float*, void*, cudaStream_t) { return BODA_ERR_UNSUPPORTED; }
}
