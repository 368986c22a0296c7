// MLP sample gradient (placeholder until the tensor-core path lands).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <string>

#include "rfast_internal.h"

namespace rfast {

struct MlpPlan { int unused; };

int mlp_plan_create(int, int, int, int, int, int, int64_t, int, const float*, MlpPlan** out,
                    size_t* dev_bytes, std::string& err) {
    *out = nullptr;
    *dev_bytes = 0;
    err = "MLP objective is not available in this build";
    return RFAST_EINVAL;
}
void mlp_plan_destroy(MlpPlan* plan) { delete plan; }
int mlp_grad_launch(MlpPlan*, const GradArgs&, const __nv_bfloat16*, const int*, int, cudaStream_t,
                    int64_t*, std::string& err) {
    err = "MLP objective is not available in this build";
    return RFAST_EINVAL;
}

}  // namespace rfast
