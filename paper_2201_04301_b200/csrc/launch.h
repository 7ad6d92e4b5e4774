// Host-side launch plans and launcher declarations shared by the translation
// units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#include "common.cuh"

namespace gcada {

struct LinearPlan {
  bool small;       // d <= 256: warp-per-row kernel, else the row-ring kernel
  int cpl;          // small: columns per lane
  int cpt, threads, R, nslot;  // large: 16-byte chunks per thread, CTA size, rows per batch, ring slots
  int ctas_per_sm;  // large: resident CTAs per SM the shape is sized for
  bool full;        // large: a row is exactly threads*cpt 16-byte chunks
  size_t smem_bytes;
  int n_cta;
  int maxseg;       // partial slots per CTA
};

// Chooses the kernel and its shape; false (with *why) if the shape is not supported.
bool plan_linear(int d, long long ld, const void* X, int G, int B, int sm_count, size_t smem_optin,
                 LinearPlan* plan, const char** why);
// One-time function attributes (dynamic shared memory size); call before the first launch.
cudaError_t prepare_grad_linear(const LinearPlan& plan, bool quad);
// pdl (here and below): the launch carries the programmatic-dependent-launch attribute (see pdl_wait)
cudaError_t launch_grad_linear(const Params& P, const LinearPlan& plan, bool quad, cudaStream_t st, bool pdl = false);

struct TailPlan {
  int select_cols4_per_block;  // float4 columns per block of the selection kernel
  int select_blocks_x;         // blocks per group
  int update_blocks;
  int direct_blocks;  // blocks of update_direct_kernel (a few per SM; each walks the columns with the grid's stride)
  int ps_blocks;               // column blocks of ps_lhs_kernel
};
void plan_tail(long long p_pad, int G, int sm_count, TailPlan* plan);
// Rule PS only: the printed left side of Eq. (9) for every group (run before the selection kernel).
cudaError_t launch_ps_lhs(const Params& P, const TailPlan& plan, cudaStream_t st, bool pdl = false);
// what: 0 = reduce the gradient partial sums and schedule, 1 = schedule only, 2 = reduce only (skip mode).
cudaError_t launch_select(const Params& P, const TailPlan& plan, cudaStream_t st, int what = 0, bool pdl = false);
cudaError_t launch_update(const Params& P, const TailPlan& plan, cudaStream_t st, bool pdl = false);

// Narrow linear models, free-running default rule: any number of iterations in one launch of a single
// thread-block cluster (see linear_cluster.cu).
struct ClusterPlan {
  bool usable = false;
  int cpl = 1, rr = 8, n_cta = 1;
  size_t smem_bytes = 0;
};
bool plan_linear_cluster(int d, int G, int M, int D, int B, long long p_pad, size_t smem_optin, ClusterPlan* plan);
cudaError_t launch_linear_cluster(const Params& P, const ClusterPlan& plan, bool quad, int n_iters, cudaStream_t st);
// Same launch shape, nothing but the per-iteration cluster barrier (measurement aid).
cudaError_t launch_linear_cluster_empty(const ClusterPlan& plan, int n_iters, cudaStream_t st);

// Mean loss of a logistic / quadratic model over rows [first, first + n) of the resident training set at
// `theta` (device, d floats); result in scratch[0].  `scratch` holds eval_loss_scratch_doubles() doubles.
int eval_loss_scratch_doubles();
cudaError_t launch_eval_loss_linear(const Params& P, const float* theta, bool quad, long long first, long long n,
                                    double* scratch, cudaStream_t st);

}  // namespace gcada
