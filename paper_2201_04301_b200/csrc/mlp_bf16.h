// bf16 tensor-core path of the MLP gradients (tcgen05 + TMA); see mlp_bf16.cu.
#pragma once
#include "mlp.h"

namespace gcada {
const char* mlp_bf16_supported(const std::vector<int>& dims);
cudaError_t mlp_bf16_plan_create(MlpPlan* plan, cudaStream_t st, std::vector<void*>* owned, const char** why);
cudaError_t mlp_bf16_launch(const Params& P, const MlpPlan& plan, cudaStream_t st, int* n_launches);
// Work that has to follow the selection kernel: keeps the selected groups' uploads (as factors) and forms
// the aggregate of Eq. (3) in Params::agg_hi.
cudaError_t mlp_bf16_launch_post(const Params& P, const MlpPlan& plan, cudaStream_t st, int* n_launches);
cudaError_t mlp_bf16_group_gradient(const Params& P, const MlpPlan& plan, int g, float* row, cudaStream_t st);
}  // namespace gcada
