// Launch plan and launcher declarations of the MLP gradient path.
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "common.cuh"

namespace gcada {

struct MlpPlan {
  int n_layers = 0;
  int launches_per_iter = 0;
  int compute = 0;
  int dims[16] = {0};
  long long w_off[16] = {0};  // offset of W_l inside theta
  long long b_off[16] = {0};  // offset of b_l inside theta
  // workspaces (device)
  void* xb = nullptr;         // gathered minibatch rows
  int* yb = nullptr;          // gathered labels
  float* act[16] = {nullptr}; // act[l]: [2][G*B][dims[l]] post-activation of layer l (l >= 1)
  float* dz[16] = {nullptr};  // dz[l]: [2][G*B][dims[l]] gradient w.r.t. pre-activation of layer l
  int sm_count = 0;
};

// nullptr if the architecture is supported, else the reason.
const char* mlp_supported(const std::vector<int>& dims, int compute);
// Allocates workspaces (appended to *owned; zeroed on `st`).  *why non-empty = unsupported shape.
cudaError_t mlp_plan_create(const std::vector<int>& dims, int compute, int G, int B, int D, long long p_pad,
                            int sm_count, cudaStream_t st, MlpPlan* plan, std::vector<void*>* owned,
                            const char** why);
// Enqueues the dual-point forward/backward of every group; writes P.fresh and P.stale.
cudaError_t launch_grad_mlp(const Params& P, const MlpPlan& plan, cudaStream_t st, int* n_launches);

}  // namespace gcada
