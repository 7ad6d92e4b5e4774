// Shared device-side declarations of the G-CADA step library: the state that
// lives in device memory, the parameter block handed to every kernel, the
// counter-based generator and a few reduction helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gcada {

// Device error words (DevState::err).
enum { DEV_OK = 0, DEV_ERR_COPY_TIMEOUT = 1, DEV_ERR_BOUNDS = 2, DEV_ERR_CHAIN = 3 };
// What a failed index check was about to store to (DevState::err_info with DEV_ERR_BOUNDS).
enum { CHK_PARTIAL = 1, CHK_LHS_PART = 2, CHK_HIST = 3, CHK_SEL_LIST = 4, CHK_GRAD_ROW = 5, CHK_FACTOR = 6 };

// Mutable run state kept in device memory so that a captured graph can be
// replayed without changing kernel arguments.
struct DevState {
  long long k;                    // iteration about to run
  unsigned long long uploads;     // sum of selection masks
  unsigned long long comm;        // (M_G + 1) * uploads, Eq. (5)/(19)
  unsigned long long comp;        // M_G * uploads, Eq. (6)/(22)
  double wall;                    // simulated wall-clock, Eq. (4) summed
  double last_dt;                 // its last increment
  double rhs;                     // right side of Eq. (9), last iteration
  int err;                        // DEV_*
  int err_info;
  unsigned int ticket_select;     // "last block done" counters
  unsigned int ticket_update;
  unsigned int ticket_aux;
  unsigned int pad_;
  long long k_chain;              // k as it was when the running chain of iterations began (a chain = the
                                  // iterations captured in one graph; see Params::k_off)
};

// How a per-group gradient is spread over partial-sum slots by the linear
// (logistic / quadratic) gradient kernels: CTA c owns the rows
// [c*R/n, (c+1)*R/n) of the G*B minibatch rows and writes one slot per group
// it touches, slot = c*maxseg + (g - first group of c).
struct PartialMap {
  int n_cta;      // 0 = gradients are already whole (one "slot" per group); -1 = whole, and lhs_part already
                  // holds `maxseg` partial sums of the innovation norm per group (nothing left to reduce)
  int maxseg;
  int rows_per_group;  // B
};

// Element counts of the buffers that kernels address with computed positions.  The library built with
// -DGCADA_DEBUG checks every such position against them before it stores (see GCADA_INDEX_OK).
struct Limits {
  long long partial_slots;  // slots of 2 * p_pad floats in Params::partial
  long long lhs_parts;      // doubles in Params::lhs_part
  long long hist_bytes;     // bytes in Params::hist
  long long grad_rows;      // rows of p_pad floats in Params::gbuf
};

struct Params {
  DevState* st;
  Limits lim;
  // problem
  int G, M, M_G, D, B;
  long long n_g;        // shard rows per group
  long long p, p_pad;   // parameters; padded row stride of every p-vector (multiple of 4)
  int d;                // features (linear models)
  long long ld;         // row stride of X in elements
  const void* X;
  const void* y;
  int identity_batch;   // 1: minibatch of group g = rows g*B .. of X (host-fed step)
  // constants
  double c;
  const double* c_d;    // [D] per-lag constants of the right side of Eq. (9), or null: c_d = c as printed
  float alpha, beta1, beta2, omb1, omb2, eps;
  double alpha_d;       // alpha in double, for the step-size schedule
  int sched_kind;       // 0: alpha^k = alpha; 1: alpha / (1 + k/a)^b; 2: alpha * b^floor(k/a)
  double sched_a, sched_b;
  int delay_law;        // 0: shift - ln(1-u)/rate; 1: Pareto shift*(1-u)^(-1/rate); 2: uniform shift + u/rate
  float scale;          // 1/B (mean) or 1 (sum)
  uint32_t seed_lo, seed_hi;
  double shift, inv_rate;
  // state vectors (stride p_pad)
  float* theta_ring;    // (D+1) iterates; slot j mod (D+1) holds theta^j
  float* h;
  float* vhat;
  float* agg_hi;        // lazily aggregated gradient, Eq. (3), as an unevaluated sum hi + lo
  float* agg_lo;
  int agg_direct;       // 1: agg_hi already holds this iteration's aggregate when the update kernel runs (it was
                        // formed from the stored factors of the last uploads); nothing is folded in from gbuf
  // Two gradient buffers per group: buffer cur[g] holds the group's last uploaded gradient, the other one
  // receives this iteration's fresh gradient; selecting the group flips cur[g], so nothing is copied.
  float* gbuf;          // [2][G] rows of p_pad floats (null when per-group gradients are not materialised)
  unsigned char* cur;   // [G]
  float* stale;         // [G] gradient at the stale iterate (optional, may be null)
  float* partial;       // [slots][2] partial sums of (fresh, stale)
  PartialMap pm;
  // scheduler
  int* tau;             // [G] age of information
  double* lhs;          // [G]
  double* t_g;          // [G]
  double* s_ring;       // [D] squared step norms, slot j mod D holds ||theta^{j+1}-theta^j||^2
  double* lhs_part;     // [G][nblk_select]
  double* upd_part;     // [nblk_update]
  unsigned char* mask_cur;  // [G]
  unsigned char* hist;      // [hist_cap][G]
  long long hist_cap;
  const unsigned char* forced;  // [n][G] or null
  long long forced_base;        // iteration of forced row 0
  // rule PS (the left side of Eq. (9) as printed): L_g^2 ||theta^k - theta^{k-tau_g}||^2
  const double* ps_L2;          // [G] squared smoothness constants, or null (rule INNOV)
  double* ps_lhs;               // [G] the printed left side, written by ps_lhs_kernel
  double* ps_part;              // [D][blocks] partial sums of ||theta^k - theta^{k-d}||^2
  int* age_order;               // [G] the groups sorted by age of information (stable), rewritten at the start of
                                // every iteration of the bf16 MLP path: tiles of groups of equal age read the
                                // same slot of the weight ring, so they are scheduled next to each other
  int* sel_list;                // [G] groups selected this iteration, ascending (written with the mask)
  int* sel_count;               // [1] how many
  // Iterations captured back to back in one graph form a chain; iteration number k_off of the chain runs
  // iteration st->k_chain + k_off (st->k_chain is rewritten by the update kernel of the chain's last iteration
  // only, so it can be read while the previous iteration is still running).  pdl = 1: the linear models'
  // gradient and selection kernels of the chain carry the programmatic-dependent-launch attribute, and the
  // wide models' gradient kernel starts the copies of its first rows (they depend on the draw, not on the
  // iterate) before it waits for the previous iteration's update to finish.
  int k_off, chain_last, pdl;
  int skip_unselected;          // 1: the selection of this iteration is already in mask_cur and the gradient
                                // kernels work on the selected groups only (rule PS: Algorithm 1 as printed,
                                // workers of unselected groups compute nothing)
};

// Programmatic dependent launch.  Every kernel of an iteration calls pdl_wait() before it reads or writes
// anything that another kernel writes: when launched with the attribute it returns once the previous kernel
// of the stream has finished and its writes are visible, otherwise at once.  pdl_launch_dependents() lets the
// next kernel's blocks become resident (and sit in their own pdl_wait) as soon as every block of this one has
// started.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KA, typename... A>
inline cudaError_t launch_k(void (*kern)(KA...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                            A&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KA>(args)...);
}

// Index check of the debug library: true if 0 <= idx < limit; otherwise the run's error word is raised (first
// failure wins; err_info says which buffer) and the caller skips the access - nothing traps, the context stays
// usable and every getter then reports the failure.  Compiles to `true` in the ordinary library.
#ifdef GCADA_DEBUG
__device__ __forceinline__ bool index_ok(DevState* st, long long idx, long long limit, int what) {
  if (idx >= 0 && idx < limit) return true;
  if (atomicCAS(&st->err, (int)DEV_OK, (int)DEV_ERR_BOUNDS) == (int)DEV_OK) st->err_info = what;
  return false;
}
#define GCADA_INDEX_OK(st, idx, limit, what) gcada::index_ok((st), (long long)(idx), (long long)(limit), (what))
#else
#define GCADA_INDEX_OK(st, idx, limit, what) true
#endif

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, ctr.x), lo0 = 0xD2511F53u * ctr.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, ctr.z), lo1 = 0xCD9E8D57u * ctr.z;
    ctr = make_uint4(hi1 ^ ctr.y ^ k0, lo1, hi0 ^ ctr.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return ctr;
}

__device__ __forceinline__ uint32_t philox_word(uint32_t a, uint32_t b, uint32_t k, uint32_t stream,
                                                uint32_t k0, uint32_t k1) {
  const uint4 o = philox4x32_10(make_uint4(a >> 2, b, k, stream), k0, k1);
  const uint32_t s = a & 3u;
  return s == 0 ? o.x : (s == 1 ? o.y : (s == 2 ? o.z : o.w));
}

// Global row of draw j of group g at iteration k (Section II-A: a minibatch
// drawn at random from the group's shard; uniform with replacement).
__device__ __forceinline__ long long batch_row(const Params& P, uint32_t k, int g, int j) {
  if (P.identity_batch) return (long long)g * P.B + j;
  const uint32_t w = philox_word((uint32_t)j, (uint32_t)g, k, 0u, P.seed_lo, P.seed_hi);
  return (long long)g * P.n_g + (long long)(((unsigned long long)w * (unsigned long long)P.n_g) >> 32);
}

// Row that receives group g's gradient at theta^k BEFORE this iteration's selection has flipped cur[g].
__device__ __forceinline__ float* fresh_row(const Params& P, int g) {
  return P.gbuf + ((long long)(1 - P.cur[g]) * P.G + g) * P.p_pad;
}
// Row holding the last uploaded gradient of group g (for a group selected this iteration, after the flip,
// that is its fresh gradient) and the other row (for such a group: the gradient it replaces).
__device__ __forceinline__ float* last_row(const Params& P, int g) {
  return P.gbuf + ((long long)P.cur[g] * P.G + g) * P.p_pad;
}
__device__ __forceinline__ float* other_row(const Params& P, int g) {
  return P.gbuf + ((long long)(1 - P.cur[g]) * P.G + g) * P.p_pad;
}

// Groups the gradient kernels work on: all of them (identity, returns P.G), or - in skip mode - the
// ones selected this iteration, ascending, in list[] (shared memory, SKIP_MAX_GROUPS ints).  Called by
// every thread of the block; contains block-wide barriers.
constexpr int SKIP_MAX_GROUPS = 1024;
__device__ __forceinline__ int build_group_list(const Params& P, int* list, int* count_sm) {
  if (!P.skip_unselected) return P.G;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int cnt = 0;
    for (int g0 = 0; g0 < P.G; g0 += 32) {
      const int gg = g0 + lane;
      const bool s = gg < P.G && P.mask_cur[gg] != 0;
      const unsigned int b = __ballot_sync(0xffffffffu, s);
      if (s) list[cnt + __popc(b & ((1u << lane) - 1u))] = gg;
      cnt += __popc(b);
    }
    if (lane == 0) *count_sm = cnt;
  }
  __syncthreads();
  return *count_sm;
}

// Computing time of worker m at iteration k (Section II-B).
__device__ __forceinline__ double worker_time(const Params& P, uint32_t k, int m) {
  const uint32_t w = philox_word((uint32_t)m, 0u, k, 1u, P.seed_lo, P.seed_hi);
  const double u = ((double)w + 0.5) * 2.3283064365386963e-10;  // 2^-32
  if (P.delay_law == 1) return P.shift * exp(-log1p(-u) * P.inv_rate);
  if (P.delay_law == 2) return P.shift + u * P.inv_rate;
  return P.shift - log1p(-u) * P.inv_rate;
}

// Step size alpha^k of Eq. (8c).
__device__ __forceinline__ float step_size(const Params& P, long long k) {
  if (P.sched_kind == 1) return (float)(P.alpha_d / pow(1.0 + (double)k / P.sched_a, P.sched_b));
  if (P.sched_kind == 2) return (float)(P.alpha_d * pow(P.sched_b, (double)(k / (long long)P.sched_a)));
  return P.alpha;
}

// ---------------------------------------------------------------------------
// Reductions with a fixed order (bitwise reproducible).
// ---------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over a block of up to 1024 threads; result valid in every thread.
// `scratch` holds at least 33 doubles of shared memory.
__device__ __forceinline__ double block_sum(double v, double* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  if (w == 0) {
    double t = lane < nw ? scratch[lane] : 0.0;
    t = warp_sum(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

}  // namespace gcada
