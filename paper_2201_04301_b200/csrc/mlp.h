// Launch plan and launcher declarations of the MLP gradient path.
#pragma once
#include <cuda_runtime.h>

#include <utility>
#include <vector>

#include "common.cuh"

namespace gcada {

constexpr int MLP_MAX_LAYERS = 15;

struct MlpPlan {
  int n_layers = 0;           // L
  int launches_per_iter = 0;
  int skip_launches = 0;      // kernels before the update when only the selected groups compute (rule PS)
  int post_launches = 0;      // kernels that follow the selection kernel (bf16 path: upload + aggregate)
  int compute = 0;            // 0 fp32, 1 bf16 operands
  int inspect = 0;            // set by the caller before the plan is created: both gradients of every group
                              // are kept (GCADA_OPT_KEEP_STALE); decides which partial sums of the norm exist
  int G = 0, B = 0, D = 0;
  long long p_pad = 0;
  int dims[MLP_MAX_LAYERS + 1] = {0};
  long long w_off[MLP_MAX_LAYERS + 1] = {0};  // offset of W_l inside theta (l = 1..L)
  long long b_off[MLP_MAX_LAYERS + 1] = {0};  // offset of b_l inside theta
  int sm_count = 0;
  // fp32 workspaces (device)
  float* xb = nullptr;                        // [G*B][dims[0]] gathered minibatch rows
  int* yb = nullptr;                          // [G*B] gathered class ids
  float* act[MLP_MAX_LAYERS + 1] = {nullptr}; // act[l], 1 <= l < L: [2][G*B][dims[l]] after ReLU; act[L]: class scores
  float* dz[MLP_MAX_LAYERS + 1] = {nullptr};  // dz[l], 1 <= l <= L: [2][G*B][dims[l]] gradient w.r.t. z_l
  // fp32 path: the weight and bias gradients of the layers above the first do not feed the back-propagation
  // chain, so they are enqueued on a second stream between a fork and a join event (branches of the graph
  // when the iteration is captured)
  cudaStream_t side = nullptr;
  cudaEvent_t ev_dz[MLP_MAX_LAYERS + 1] = {nullptr};  // ev_dz[l]: dz_l is complete (on the main stream)
  cudaEvent_t ev_join = nullptr;
  void* bf16_impl = nullptr;                  // opaque state of the bf16 tensor-core path
  std::vector<std::pair<void*, size_t>> state;  // device buffers that carry state across iterations (checkpoints)
  int norm_parts = 0;                         // > 0: the gradient kernels themselves deliver this many partial sums
                                              // of ||fresh_g - stale_g||^2 per group in Params::lhs_part
};

// nullptr if the architecture is supported, else the reason.
const char* mlp_supported(const std::vector<int>& dims, int compute);
// Allocates workspaces (appended to *owned; zeroed on `st`).  *why non-empty = unsupported shape.
cudaError_t mlp_plan_create(const std::vector<int>& dims, int compute, int G, int B, int D, long long p_pad,
                            int sm_count, cudaStream_t st, MlpPlan* plan, std::vector<void*>* owned,
                            const char** why);
// Destroys the plan's stream and events (device buffers belong to the caller's `owned` list).
void mlp_plan_release(MlpPlan* plan);
// Enqueues the dual-point forward/backward of every group; writes each group's fresh-gradient row and P.stale.
cudaError_t launch_grad_mlp(const Params& P, const MlpPlan& plan, cudaStream_t st, int* n_launches);
// Work that must follow the selection kernel (none for the fp32 path; bf16: the selected groups' uploads
// are kept and the aggregate of Eq. (3) is formed).
cudaError_t launch_grad_mlp_post(const Params& P, const MlpPlan& plan, cudaStream_t st, int* n_launches);
// bf16 path without kept per-group gradients: group g's last uploaded gradient rebuilt into `row` (device).
cudaError_t mlp_group_gradient(const Params& P, const MlpPlan& plan, int g, float* row, cudaStream_t st);

// Reporting aid (not a step of Algorithm 1): the mean softmax cross-entropy of the CURRENT iterate (the fp32
// master parameters, fp32 arithmetic, whatever the model's compute type) over rows [first, first + n) of the
// resident training set, into out[0] (device).  The rows are pushed through the fp32 tile kernels in slabs of
// MLP_EVAL_SLAB rows; `buf` are two device buffers of MLP_EVAL_SLAB * (widest layer, input included) floats,
// `ones` MLP_EVAL_SLAB / 64 bytes of value 1, `part` 1024 doubles.
constexpr int MLP_EVAL_SLAB = 4096;
struct MlpEvalScratch {
  float* buf[2] = {nullptr, nullptr};
  unsigned char* ones = nullptr;
  double* part = nullptr;
};
cudaError_t mlp_eval_loss(const Params& P, const MlpPlan& plan, long long first, long long n, const MlpEvalScratch& sc,
                          double* out, cudaStream_t st);

}  // namespace gcada
