#include "mlp_bf16.h"
namespace gcada {
const char* mlp_bf16_supported(const std::vector<int>&) { return "the bf16 MLP path is not built yet"; }
cudaError_t mlp_bf16_plan_create(MlpPlan*, cudaStream_t, std::vector<void*>*, const char** why) {
  *why = "the bf16 MLP path is not built yet";
  return cudaSuccess;
}
cudaError_t mlp_bf16_launch(const Params&, const MlpPlan&, cudaStream_t, int* n) {
  *n = 0;
  return cudaErrorNotSupported;
}
}  // namespace gcada
