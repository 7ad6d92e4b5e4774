// Objective value for reporting: the mean per-sample loss (Eq. 1 restricted to
// a range of rows) of a logistic or quadratic model at a given iterate.  Not
// part of an iteration of Algorithm 1; used to draw loss-versus-wall-clock
// curves such as those of Section VI.
#include "common.cuh"
#include "launch.h"

namespace gcada {

namespace {

constexpr int EVAL_BLOCKS = 592;  // partial sums (4 per SM on a 148-SM part; any grid size is correct)

// One warp per row (grid-stride); lane l owns columns l, l+32, ...; everything in double.
__global__ void __launch_bounds__(256) eval_loss_kernel(const float* __restrict__ X, const float* __restrict__ y,
                                                        long long ld, int d, long long first, long long n,
                                                        const float* __restrict__ theta, int quad, double* part) {
  __shared__ double scratch[40];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double local = 0.0;
  for (long long r = (long long)blockIdx.x * 8 + warp; r < n; r += (long long)gridDim.x * 8) {
    const float* x = X + (first + r) * ld;
    double z = 0.0;
    for (int c = lane; c < d; c += 32) z += (double)x[c] * (double)theta[c];
    z = warp_sum(z);
    if (lane == 0) {
      const double yy = (double)y[first + r];
      if (quad) {
        const double e = z - yy;
        local += 0.5 * e * e;
      } else {
        // ln(1 + e^z) - y z, written so that neither branch overflows
        local += fmax(z, 0.0) + log1p(exp(-fabs(z))) - yy * z;
      }
    }
  }
  const double tot = block_sum(local, scratch);
  if (threadIdx.x == 0) part[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(256) eval_finish_kernel(const double* part, int n_part, long long n, double* out) {
  __shared__ double scratch[40];
  double s = 0.0;
  for (int i = threadIdx.x; i < n_part; i += 256) s += part[i];
  s = block_sum(s, scratch);
  if (threadIdx.x == 0) out[0] = s / (double)n;
}

}  // namespace

int eval_loss_scratch_doubles() { return EVAL_BLOCKS + 1; }

cudaError_t launch_eval_loss_linear(const Params& P, const float* theta, bool quad, long long first, long long n,
                                    double* scratch, cudaStream_t st) {
  eval_loss_kernel<<<EVAL_BLOCKS, 256, 0, st>>>(reinterpret_cast<const float*>(P.X), reinterpret_cast<const float*>(P.y),
                                                P.ld, P.d, first, n, theta, quad ? 1 : 0, scratch + 1);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  eval_finish_kernel<<<1, 256, 0, st>>>(scratch + 1, EVAL_BLOCKS, n, scratch);
  return cudaGetLastError();
}

}  // namespace gcada
