// Tensor-core input projection (placeholder until the tcgen05 kernel lands).
#include "common.cuh"
#include <cstdio>
namespace lstm {
int proj_tc_plan(ProjTcPlan *, const __nv_bfloat16 *, const __nv_bfloat16 *, int, int, int, int, int, char *err, int errlen)
{
    snprintf(err, errlen, "tensor-core projection not built");
    return 1;
}
cudaError_t launch_proj_tc(const ProjTcPlan &, const float *, float *, int *, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t proj_tc_prepare() { return cudaSuccess; }
}  // namespace lstm
