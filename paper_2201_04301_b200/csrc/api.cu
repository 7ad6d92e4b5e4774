// Host side of the C ABI declared in include/gcada.h: context, device state,
// launch plans, CUDA-graph replay of the per-iteration kernel chain.
#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <string>
#include <vector>

#include "../../include/gcada.h"
#include "common.cuh"
#include "launch.h"
#include "mlp.h"

using namespace gcada;

namespace {
thread_local std::string g_create_error;
constexpr int GRAPH_CHAIN = 16;  // iterations per replayed graph
constexpr int TIMING_CAP = 512;  // iterations whose phase times are kept
}  // namespace

struct gcada_ctx {
  int device = 0;
  int sm_count = 0;
  size_t smem_optin = 0;
  cudaStream_t stream = nullptr;
  // model
  int kind = 0, compute = 0;
  std::vector<int> dims;
  long long p = 0, p_pad = 0;
  // algorithm
  int M = 0, M_G = 0, G = 0, D = 0;
  double c = 0, alpha = 0, beta1 = 0, beta2 = 0, eps = 0;
  unsigned long long seed = 0;
  double shift = 1.0, rate = 1.0;
  int rule = 0, reduction = 0, keep_stale = 0, use_graph = 1, persistent = 1;
  ClusterPlan cluster{};
  long long hist_cap = 65536;
  // data
  const void* X = nullptr;
  const void* y = nullptr;
  long long N = 0, ld = 0;
  int B = 0;
  bool have_data = false, have_theta = false, ready = false;
  long long k_host = 0;  // iterations enqueued since set_theta
  unsigned long long launches = 0;
  // device memory
  std::vector<void*> owned;
  std::vector<double> L2;  // squared smoothness constants (rule PS)
  std::vector<double> c_d; // per-lag constants of Eq. (9)'s right side (empty: c for every lag)
  int sched_kind = 0;
  double sched_a = 1.0, sched_b = 0.0;
  int delay_law = 0;
  DevState* st = nullptr;
  Params P{};
  LinearPlan lin{};
  TailPlan tail{};
  MlpPlan mlp{};
  unsigned char* forced_dev = nullptr;
  size_t forced_cap = 0;
  void* stage_x = nullptr;
  void* stage_y = nullptr;
  long long stage_ld = 0;
  std::vector<std::pair<void*, size_t>> state;  // device buffers a checkpoint holds (besides the plan's)
  double* eval_scratch = nullptr;
  MlpEvalScratch mlp_eval{};
  float* row_scratch = nullptr;  // one p-vector for getters that rebuild a group's gradient on demand
  // graphs (free-running resident-data mode only)
  cudaGraphExec_t graph1 = nullptr, graphN = nullptr;
  // optional per-phase timing
  int timing = 0;
  std::vector<cudaEvent_t> events;  // TIMING_CAP * 5
  long long timed = 0;              // timed iterations so far
  bool capturing = false;
  std::string err;
};

namespace {

gcada_status fail(gcada_ctx* ctx, gcada_status s, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx)
    ctx->err = buf;
  else
    g_create_error = buf;
  return s;
}

#define CK(call)                                                                                  \
  do {                                                                                            \
    cudaError_t e_ = (call);                                                                      \
    if (e_ != cudaSuccess)                                                                        \
      return fail(ctx, e_ == cudaErrorMemoryAllocation ? GCADA_ENOMEM : GCADA_ECUDA, "%s: %s", #call, \
                  cudaGetErrorString(e_));                                                        \
  } while (0)

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) cudaSetDevice(dev);
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

void drop_graphs(gcada_ctx* ctx) {
  if (ctx->graph1) cudaGraphExecDestroy(ctx->graph1);
  if (ctx->graphN) cudaGraphExecDestroy(ctx->graphN);
  ctx->graph1 = ctx->graphN = nullptr;
}

void free_all(gcada_ctx* ctx) {
  drop_graphs(ctx);
  mlp_plan_release(&ctx->mlp);
  for (cudaEvent_t e : ctx->events)
    if (e) cudaEventDestroy(e);
  ctx->events.clear();
  ctx->timed = 0;
  for (void* q : ctx->owned) cudaFree(q);
  ctx->owned.clear();
  if (ctx->forced_dev) cudaFree(ctx->forced_dev);
  ctx->forced_dev = nullptr;
  ctx->forced_cap = 0;
  if (ctx->stage_x) cudaFree(ctx->stage_x);
  if (ctx->stage_y) cudaFree(ctx->stage_y);
  ctx->stage_x = ctx->stage_y = nullptr;
  ctx->row_scratch = nullptr;  // was in `owned`
  ctx->eval_scratch = nullptr;
  ctx->mlp_eval = MlpEvalScratch{};
  ctx->state.clear();
  ctx->st = nullptr;
  ctx->ready = false;
}

template <class T>
gcada_status dev_alloc(gcada_ctx* ctx, T** out, size_t count) {
  void* q = nullptr;
  const size_t bytes = (count ? count : 1) * sizeof(T);
  CK(cudaMalloc(&q, bytes));
  ctx->owned.push_back(q);
  CK(cudaMemsetAsync(q, 0, bytes, ctx->stream));
  *out = reinterpret_cast<T*>(q);
  return GCADA_OK;
}

#define TRY(expr)                        \
  do {                                   \
    gcada_status s_ = (expr);            \
    if (s_ != GCADA_OK) return s_;       \
  } while (0)

bool is_linear(const gcada_ctx* ctx) { return ctx->kind != GCADA_MODEL_MLP; }
// bf16 MLP: the aggregate is formed from the stored factors of the last uploads; per-group gradient
// vectors exist only when they are kept for inspection
bool factored(const gcada_ctx* ctx) { return !is_linear(ctx) && ctx->compute == GCADA_COMPUTE_BF16; }

// (Re)build device state and plans once model, data shape and theta^0 are known.
gcada_status make_ready(gcada_ctx* ctx, const float* theta0, int on_device) {
  free_all(ctx);
  Params& P = ctx->P;
  P = Params{};
  P.G = ctx->G;
  P.M = ctx->M;
  P.M_G = ctx->M_G;
  P.D = ctx->D;
  P.p = ctx->p;
  P.p_pad = ctx->p_pad;
  P.d = ctx->dims[0];
  P.c = ctx->c;
  P.alpha = (float)ctx->alpha;
  P.alpha_d = ctx->alpha;
  P.sched_kind = ctx->sched_kind;
  P.sched_a = ctx->sched_a;
  P.sched_b = ctx->sched_b;
  P.beta1 = (float)ctx->beta1;
  P.beta2 = (float)ctx->beta2;
  P.omb1 = (float)(1.0 - ctx->beta1);
  P.omb2 = (float)(1.0 - ctx->beta2);
  P.eps = (float)ctx->eps;
  P.hist_cap = ctx->hist_cap;
  const long long pp = ctx->p_pad;
  const int G = ctx->G, D = ctx->D;
  TRY(dev_alloc(ctx, &ctx->st, 1));
  P.st = ctx->st;
  TRY(dev_alloc(ctx, &P.theta_ring, (size_t)(D + 1) * pp));
  TRY(dev_alloc(ctx, &P.h, (size_t)pp));
  TRY(dev_alloc(ctx, &P.vhat, (size_t)pp));
  TRY(dev_alloc(ctx, &P.agg_hi, (size_t)pp));
  TRY(dev_alloc(ctx, &P.agg_lo, (size_t)pp));
  P.agg_direct = factored(ctx) ? 1 : 0;
  if (!factored(ctx) || ctx->keep_stale) TRY(dev_alloc(ctx, &P.gbuf, (size_t)2 * G * pp));
  TRY(dev_alloc(ctx, &P.cur, (size_t)G));
  // the fp32 MLP kernels hand over both gradients; the others keep the stale one only on request
  if (ctx->keep_stale || (!is_linear(ctx) && ctx->compute == GCADA_COMPUTE_FP32))
    TRY(dev_alloc(ctx, &P.stale, (size_t)G * pp));
  TRY(dev_alloc(ctx, &P.tau, (size_t)G));
  TRY(dev_alloc(ctx, &P.lhs, (size_t)G));
  TRY(dev_alloc(ctx, &P.t_g, (size_t)G));
  TRY(dev_alloc(ctx, &P.s_ring, (size_t)D));
  TRY(dev_alloc(ctx, &P.mask_cur, (size_t)G));
  TRY(dev_alloc(ctx, &P.sel_list, (size_t)G));
  TRY(dev_alloc(ctx, &P.age_order, (size_t)G));
  TRY(dev_alloc(ctx, &P.sel_count, (size_t)1));
  TRY(dev_alloc(ctx, &P.hist, (size_t)ctx->hist_cap * G));
  plan_tail(pp, G, ctx->sm_count, &ctx->tail);
  TRY(dev_alloc(ctx, &P.lhs_part, (size_t)G * ctx->tail.select_blocks_x));
  P.lim.lhs_parts = (long long)G * ctx->tail.select_blocks_x;
  P.lim.hist_bytes = ctx->hist_cap * G;
  P.lim.grad_rows = P.gbuf ? 2LL * G : 0;
  TRY(dev_alloc(ctx, &P.upd_part, (size_t)ctx->tail.update_blocks));
  // everything an iteration inherits from earlier ones
  {
    auto& S = ctx->state;
    S.emplace_back(ctx->st, sizeof(DevState));
    S.emplace_back(P.theta_ring, sizeof(float) * (size_t)(D + 1) * pp);
    S.emplace_back(P.h, sizeof(float) * (size_t)pp);
    S.emplace_back(P.vhat, sizeof(float) * (size_t)pp);
    S.emplace_back(P.agg_hi, sizeof(float) * (size_t)pp);
    S.emplace_back(P.agg_lo, sizeof(float) * (size_t)pp);
    if (P.gbuf) S.emplace_back(P.gbuf, sizeof(float) * (size_t)2 * G * pp);
    S.emplace_back(P.cur, (size_t)G);
    S.emplace_back(P.tau, sizeof(int) * (size_t)G);
    S.emplace_back(P.s_ring, sizeof(double) * (size_t)D);
    S.emplace_back(P.mask_cur, (size_t)G);
    S.emplace_back(P.hist, (size_t)ctx->hist_cap * G);
    S.emplace_back(P.lhs, sizeof(double) * (size_t)G);
    S.emplace_back(P.t_g, sizeof(double) * (size_t)G);
  }
  // tau_g^0 = D: the first iteration selects every group
  {
    std::vector<int> tau0(G, D);
    CK(cudaMemcpyAsync(P.tau, tau0.data(), sizeof(int) * G, cudaMemcpyHostToDevice, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
  }
  CK(cudaMemcpyAsync(P.theta_ring, theta0, sizeof(float) * ctx->p,
                     on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  ctx->k_host = 0;
  ctx->have_theta = true;
  return GCADA_OK;
}

// Things that depend on the data shape (batch size, X pointer).
gcada_status make_plans(gcada_ctx* ctx) {
  if (ctx->ready) return GCADA_OK;
  Params& P = ctx->P;
  P.B = ctx->B;
  P.scale = ctx->reduction == 0 ? (float)(1.0 / ctx->B) : 1.0f;
  P.seed_lo = (uint32_t)(ctx->seed & 0xffffffffu);
  P.seed_hi = (uint32_t)(ctx->seed >> 32);
  P.shift = ctx->shift;
  P.inv_rate = 1.0 / ctx->rate;
  P.delay_law = ctx->delay_law;
  P.c_d = nullptr;
  if (!ctx->c_d.empty()) {
    double* cd = nullptr;
    TRY(dev_alloc(ctx, &cd, (size_t)ctx->D));
    CK(cudaMemcpyAsync(cd, ctx->c_d.data(), sizeof(double) * ctx->D, cudaMemcpyHostToDevice, ctx->stream));
    P.c_d = cd;
  }
  P.X = ctx->X;
  P.y = ctx->y;
  P.ld = ctx->ld;
  P.n_g = ctx->have_data ? ctx->N / ctx->G : 1;
  if (is_linear(ctx)) {
    const char* why = "";
    // the plan must also hold for the staging buffer of host-fed steps
    const void* xa = ctx->have_data ? ctx->X : nullptr;
    const long long ld = ctx->have_data ? ctx->ld : ((ctx->dims[0] + 3) / 4) * 4;
    if (!plan_linear(ctx->dims[0], ld, xa, ctx->G, ctx->B, ctx->sm_count, ctx->smem_optin, &ctx->lin,
                     &why))
      return fail(ctx, GCADA_EINVAL, "%s", why);
    CK(prepare_grad_linear(ctx->lin, ctx->kind == GCADA_MODEL_QUADRATIC));
    // narrow models with few groups: whole iterations inside one thread-block cluster
    ctx->cluster.usable = false;
    if (ctx->persistent && ctx->have_data && ctx->rule == 0 && !ctx->keep_stale)
      plan_linear_cluster(ctx->dims[0], ctx->G, ctx->M, ctx->D, ctx->B, ctx->p_pad, ctx->smem_optin, &ctx->cluster);
    P.pm.n_cta = ctx->lin.n_cta;
    P.pm.maxseg = ctx->lin.maxseg;
    P.pm.rows_per_group = ctx->B;
    TRY(dev_alloc(ctx, &P.partial, (size_t)ctx->lin.n_cta * ctx->lin.maxseg * 2 * ctx->p_pad));
    P.lim.partial_slots = (long long)ctx->lin.n_cta * ctx->lin.maxseg;
  } else {
    P.pm.n_cta = 0;
    P.pm.maxseg = 0;
    P.pm.rows_per_group = ctx->B;
    const char* why = "";
    std::vector<void*> bufs;
    ctx->mlp.inspect = ctx->keep_stale;
    cudaError_t e = mlp_plan_create(ctx->dims, ctx->compute, ctx->G, ctx->B, ctx->D, ctx->p_pad, ctx->sm_count,
                                    ctx->stream, &ctx->mlp, &bufs, &why);
    for (void* q : bufs) ctx->owned.push_back(q);
    if (e != cudaSuccess) return fail(ctx, e == cudaErrorMemoryAllocation ? GCADA_ENOMEM : GCADA_ECUDA, "MLP plan: %s (%s)", why, cudaGetErrorString(e));
    if (why[0]) return fail(ctx, GCADA_EINVAL, "%s", why);
    if (ctx->mlp.norm_parts > 0) {  // the gradient kernels deliver the innovation-norm partial sums themselves
      P.pm.n_cta = -1;
      P.pm.maxseg = ctx->mlp.norm_parts;
      TRY(dev_alloc(ctx, &P.lhs_part, (size_t)ctx->G * ctx->mlp.norm_parts));
      P.lim.lhs_parts = (long long)ctx->G * ctx->mlp.norm_parts;
    }
  }
  if (ctx->rule == 1) {
    double* l2 = nullptr;
    TRY(dev_alloc(ctx, &l2, (size_t)ctx->G));
    CK(cudaMemcpyAsync(l2, ctx->L2.data(), sizeof(double) * ctx->G, cudaMemcpyHostToDevice, ctx->stream));
    P.ps_L2 = l2;
    // the printed test needs no gradient: only the selected groups compute (Algorithm 1's own order).  The
    // MLPs do so unless per-group gradients are kept for inspection.
    P.skip_unselected = ((is_linear(ctx) && ctx->G <= SKIP_MAX_GROUPS) || (!is_linear(ctx) && !ctx->keep_stale)) ? 1 : 0;
    TRY(dev_alloc(ctx, &P.ps_lhs, (size_t)ctx->G));
    TRY(dev_alloc(ctx, &P.ps_part, (size_t)ctx->D * ctx->tail.ps_blocks));
  } else {
    P.ps_L2 = nullptr;
    P.skip_unselected = 0;
  }
  P.k_off = 0;  // outside a captured chain every iteration is a chain of its own
  P.chain_last = 1;
  P.pdl = 0;
  CK(cudaStreamSynchronize(ctx->stream));
  ctx->ready = true;
  return GCADA_OK;
}

gcada_status enqueue_iteration(gcada_ctx* ctx, const Params& P) {
  cudaEvent_t* ev = nullptr;
  if (ctx->timing && !ctx->capturing) {
    if (ctx->events.empty()) {
      ctx->events.resize((size_t)TIMING_CAP * 5, nullptr);
      for (auto& e : ctx->events) CK(cudaEventCreate(&e));
    }
    ev = &ctx->events[(size_t)(ctx->timed % TIMING_CAP) * 5];
    CK(cudaEventRecord(ev[0], ctx->stream));
  }
  if (P.skip_unselected) {
    // Rule PS on a linear model, Algorithm 1 in its printed order: the server decides first (no gradient
    // is needed for the printed test), then only the selected groups compute.
    CK(launch_ps_lhs(P, ctx->tail, ctx->stream));
    CK(launch_select(P, ctx->tail, ctx->stream, 1));
    if (ev) CK(cudaEventRecord(ev[1], ctx->stream));  // reported as "selection" below via the phase map
    if (is_linear(ctx)) {
      CK(launch_grad_linear(P, ctx->lin, ctx->kind == GCADA_MODEL_QUADRATIC, ctx->stream));
      CK(launch_select(P, ctx->tail, ctx->stream, 2));
      if (ev) CK(cudaEventRecord(ev[2], ctx->stream));
      ctx->launches += 5;
    } else {
      int n = 0, m = 0;
      CK(launch_grad_mlp(P, ctx->mlp, ctx->stream, &n));
      if (ev) CK(cudaEventRecord(ev[2], ctx->stream));
      CK(launch_grad_mlp_post(P, ctx->mlp, ctx->stream, &m));
      ctx->launches += (unsigned long long)(3 + n + m);
    }
    if (ev) CK(cudaEventRecord(ev[3], ctx->stream));
    CK(launch_update(P, ctx->tail, ctx->stream));
    if (ev) {
      CK(cudaEventRecord(ev[4], ctx->stream));
      ctx->timed += 1;
    }
    return GCADA_OK;
  }
  // Inside a captured chain the linear models' gradient and selection kernels are launched programmatically
  // dependent.  The selection kernel's blocks become resident while the gradient kernel drains; the update
  // kernel, launched in the ordinary way, lets the next iteration's gradient kernel start at once, which
  // computes its draw and starts copying its first rows while the update runs.  Measured on the d = 4096
  // workload (us per iteration, same GPU): plain launches 107.2, this arrangement 102.7; with the update
  // kernel programmatically dependent too, so that the copies also run under the selection kernel, 104.7
  // (the selection's chain of dependent loads queues behind them); every kernel releasing its dependents at
  // its start 109.8.
  const bool pdl = P.pdl != 0 && is_linear(ctx);
  if (is_linear(ctx)) {
    CK(launch_grad_linear(P, ctx->lin, ctx->kind == GCADA_MODEL_QUADRATIC, ctx->stream, pdl && P.k_off > 0));
    ctx->launches += 1;
  } else {
    int n = 0;
    CK(launch_grad_mlp(P, ctx->mlp, ctx->stream, &n));
    ctx->launches += (unsigned long long)n;
  }
  if (ev) CK(cudaEventRecord(ev[1], ctx->stream));
  if (P.ps_L2) {
    CK(launch_ps_lhs(P, ctx->tail, ctx->stream, pdl));
    ctx->launches += 1;
  }
  CK(launch_select(P, ctx->tail, ctx->stream, 0, pdl));
  if (ev) CK(cudaEventRecord(ev[2], ctx->stream));
  if (!is_linear(ctx)) {  // bf16 MLP: the uploads are kept and the aggregate is formed (counted with the update phase)
    int n = 0;
    CK(launch_grad_mlp_post(P, ctx->mlp, ctx->stream, &n));
    ctx->launches += (unsigned long long)n;
  }
  if (ev) CK(cudaEventRecord(ev[3], ctx->stream));
  CK(launch_update(P, ctx->tail, ctx->stream, false));
  if (ev) {
    CK(cudaEventRecord(ev[4], ctx->stream));
    ctx->timed += 1;
  }
  ctx->launches += 2;
  return GCADA_OK;
}

gcada_status capture_graph(gcada_ctx* ctx, int iters, cudaGraph_t* out) {
  cudaGraph_t graph = nullptr;
  const unsigned long long before = ctx->launches;
  CK(cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
  gcada_status s = GCADA_OK;
  ctx->capturing = true;
  for (int i = 0; i < iters && s == GCADA_OK; ++i) {
    Params Q = ctx->P;
    Q.k_off = i;
    Q.chain_last = i == iters - 1;
    Q.pdl = Q.skip_unselected ? 0 : 1;
    s = enqueue_iteration(ctx, Q);
  }
  ctx->capturing = false;
  cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph);
  ctx->launches = before;
  if (s != GCADA_OK) {
    if (graph) cudaGraphDestroy(graph);
    return s;
  }
  CK(e);
  *out = graph;
  return GCADA_OK;
}

gcada_status capture(gcada_ctx* ctx, int iters, cudaGraphExec_t* out) {
  cudaGraph_t graph = nullptr;
  TRY(capture_graph(ctx, iters, &graph));
  cudaError_t e = cudaGraphInstantiate(out, graph, 0);
  cudaGraphDestroy(graph);
  CK(e);
  return GCADA_OK;
}

// A kernel that does nothing, for gcada_time_empty_chain.
__global__ void empty_kernel() {}

int kernels_per_iteration(const gcada_ctx* ctx) {
  if (is_linear(ctx)) return ctx->P.skip_unselected ? 5 : 3 + (ctx->rule == 1 ? 1 : 0);
  if (ctx->P.skip_unselected) return 3 + ctx->mlp.skip_launches + ctx->mlp.post_launches;
  return 2 + ctx->mlp.launches_per_iter + ctx->mlp.post_launches + (ctx->rule == 1 ? 1 : 0);
}

gcada_status check_runnable(gcada_ctx* ctx, bool need_data) {
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  if (need_data && !ctx->have_data) return fail(ctx, GCADA_ESTATE, "gcada_set_data has not been called");
  if (ctx->B <= 0) return fail(ctx, GCADA_ESTATE, "no minibatch size: call gcada_set_data or gcada_set_batch");
  if (ctx->rule != 0 && ctx->L2.empty())
    return fail(ctx, GCADA_ESTATE, "rule PS needs the smoothness constants: call gcada_set_smoothness");
  return GCADA_OK;
}

// Device row holding group g's fresh gradient of the last iteration (what = 0) or its last uploaded
// gradient (what = 1), given host copies of cur[] and of the last selection mask.
const float* group_row(const gcada_ctx* ctx, int what, int g, const std::vector<unsigned char>& cur,
                       const std::vector<unsigned char>& mask) {
  int buf = cur[g];
  if (what == 0 && !mask[g]) buf = 1 - buf;  // an unselected group's fresh gradient sits in the other row
  return ctx->P.gbuf + ((long long)buf * ctx->G + g) * ctx->p_pad;
}

// Device pointer to group g's row for a getter.  Where per-group gradients are not materialised (bf16 MLP
// without GCADA_OPT_KEEP_STALE) the last uploaded gradient is rebuilt from its stored factors into a
// scratch row; the fresh gradient of a group is then only available as its last upload.
gcada_status group_row_dev(gcada_ctx* ctx, int what, int g, const std::vector<unsigned char>& cur,
                           const std::vector<unsigned char>& mask, const float** out) {
  if (ctx->P.gbuf) {
    *out = group_row(ctx, what, g, cur, mask);
    return GCADA_OK;
  }
  if (!ctx->ready) return fail(ctx, GCADA_ESTATE, "no iteration has run yet");
  if (!ctx->row_scratch) {
    TRY(dev_alloc(ctx, &ctx->row_scratch, (size_t)ctx->p_pad));
  }
  CK(cudaMemsetAsync(ctx->row_scratch, 0, sizeof(float) * (size_t)ctx->p_pad, ctx->stream));
  CK(mlp_group_gradient(ctx->P, ctx->mlp, g, ctx->row_scratch, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  *out = ctx->row_scratch;
  return GCADA_OK;
}

gcada_status read_state(gcada_ctx* ctx, DevState* out) {
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaMemcpy(out, ctx->st, sizeof(DevState), cudaMemcpyDeviceToHost));
  if (out->err == DEV_ERR_COPY_TIMEOUT)
    return fail(ctx, GCADA_ETIMEOUT, "device-side error %d: a bounded wait on an asynchronous copy or a pipeline barrier gave up",
                out->err);
  if (out->err == DEV_ERR_BOUNDS)
    return fail(ctx, GCADA_ECUDA, "device-side error %d: an index check of the debug library failed (buffer %d); the store was skipped",
                out->err, out->err_info);
  if (out->err == DEV_ERR_CHAIN)
    return fail(ctx, GCADA_ECUDA, "device-side error %d: a gradient kernel started inside a chain of iterations found the iteration counter elsewhere than the chain's bookkeeping",
                out->err);
  if (out->err != DEV_OK) return fail(ctx, GCADA_ECUDA, "device-side error %d", out->err);
  return GCADA_OK;
}

}  // namespace

extern "C" {

gcada_status gcada_create(const gcada_model* model, int M, int M_G, int D, double c, double alpha, double beta1,
                          double beta2, double eps, gcada_ctx** out) {
  gcada_ctx* ctx = nullptr;
  if (!out) return fail(ctx, GCADA_EINVAL, "out is NULL");
  *out = nullptr;
  if (!model || !model->dims) return fail(ctx, GCADA_EINVAL, "model is NULL");
  if (M <= 0 || M_G <= 0 || M % M_G != 0) return fail(ctx, GCADA_EINVAL, "need M > 0, M_G > 0 and M divisible by M_G");
  if (D < 1) return fail(ctx, GCADA_EINVAL, "need D >= 1");
  if (!(c >= 0) || !(alpha > 0) || !(beta1 > 0 && beta1 < 1) || !(beta2 > 0 && beta2 < 1) || !(eps > 0))
    return fail(ctx, GCADA_EINVAL, "need c >= 0, alpha > 0, 0 < beta1, beta2 < 1, eps > 0");
  if (M / M_G > 65535) return fail(ctx, GCADA_EINVAL, "at most 65535 groups");
  if (model->kind == GCADA_MODEL_MLP && M / M_G > 32767) return fail(ctx, GCADA_EINVAL, "at most 32767 groups for an MLP");
  long long p = 0;
  if (model->kind == GCADA_MODEL_LOGISTIC || model->kind == GCADA_MODEL_QUADRATIC) {
    if (model->n_dims != 1 || model->dims[0] < 1 || model->dims[0] > 4096)
      return fail(ctx, GCADA_EINVAL, "logistic / quadratic models need n_dims == 1 and 1 <= d <= 4096");
    if (model->compute != GCADA_COMPUTE_FP32) return fail(ctx, GCADA_EINVAL, "linear models compute in fp32");
    p = model->dims[0];
  } else if (model->kind == GCADA_MODEL_MLP) {
    if (model->n_dims < 2) return fail(ctx, GCADA_EINVAL, "an MLP needs n_dims >= 2");
    for (int l = 0; l < model->n_dims; ++l)
      if (model->dims[l] < 1) return fail(ctx, GCADA_EINVAL, "layer sizes must be positive");
    for (int l = 1; l < model->n_dims; ++l) p += (long long)model->dims[l] * model->dims[l - 1] + model->dims[l];
    if (model->compute != GCADA_COMPUTE_FP32 && model->compute != GCADA_COMPUTE_BF16)
      return fail(ctx, GCADA_EINVAL, "unknown compute type");
    const char* why = mlp_supported(std::vector<int>(model->dims, model->dims + model->n_dims), model->compute);
    if (why) return fail(ctx, GCADA_EINVAL, "%s", why);
  } else {
    return fail(ctx, GCADA_EINVAL, "unknown model kind %d", model->kind);
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(ctx, GCADA_ECUDA, "no usable CUDA device: %s", cudaGetErrorString(e));
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess) return fail(ctx, GCADA_ECUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(e));
  if (prop.major < 10)
    return fail(ctx, GCADA_ECUDA, "this library is built for sm_100a only; device is sm_%d%d", prop.major, prop.minor);
  ctx = new (std::nothrow) gcada_ctx();
  if (!ctx) return fail(nullptr, GCADA_ENOMEM, "out of host memory");
  ctx->device = dev;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->smem_optin = prop.sharedMemPerBlockOptin;
  ctx->kind = model->kind;
  ctx->compute = model->compute;
  ctx->dims.assign(model->dims, model->dims + model->n_dims);
  ctx->p = p;
  ctx->p_pad = (p + 31) / 32 * 32;
  ctx->M = M;
  ctx->M_G = M_G;
  ctx->G = M / M_G;
  ctx->D = D;
  ctx->c = c;
  ctx->alpha = alpha;
  ctx->beta1 = beta1;
  ctx->beta2 = beta2;
  ctx->eps = eps;
  *out = ctx;
  return GCADA_OK;
}

gcada_status gcada_set_stream(gcada_ctx* ctx, void* cuda_stream) {
  if (!ctx) return GCADA_EINVAL;
  DeviceGuard dg(ctx->device);
  if (ctx->st) CK(cudaStreamSynchronize(ctx->stream));
  ctx->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_data(gcada_ctx* ctx, const void* X_dev, const void* y_dev, long long N, long long ld_x,
                            int batch) {
  if (!ctx) return GCADA_EINVAL;
  if (!X_dev || !y_dev) return fail(ctx, GCADA_EINVAL, "X_dev / y_dev is NULL");
  if (batch <= 0) return fail(ctx, GCADA_EINVAL, "batch must be positive");
  if (ld_x < ctx->dims[0]) return fail(ctx, GCADA_EINVAL, "ld_x is smaller than the feature count");
  if (N / ctx->G <= 0) return fail(ctx, GCADA_EINVAL, "fewer rows than groups");
  if (N / ctx->G > 0xffffffffLL) return fail(ctx, GCADA_EINVAL, "shards of more than 2^32 rows are not supported");
  if (is_linear(ctx) && ctx->dims[0] > 256 && ((ld_x & 3) != 0 || (reinterpret_cast<uintptr_t>(X_dev) & 15) != 0))
    return fail(ctx, GCADA_EINVAL, "for d > 256 X_dev must be 16-byte aligned and ld_x a multiple of 4");
  DeviceGuard dg(ctx->device);
  if (ctx->st) CK(cudaStreamSynchronize(ctx->stream));
  const bool shape_changed = batch != ctx->B;
  ctx->X = X_dev;
  ctx->y = y_dev;
  ctx->N = N;
  ctx->ld = ld_x;
  ctx->B = batch;
  ctx->have_data = true;
  drop_graphs(ctx);
  if (ctx->ready && !shape_changed) {
    ctx->P.X = X_dev;
    ctx->P.y = y_dev;
    ctx->P.ld = ld_x;
    ctx->P.n_g = N / ctx->G;
  } else if (ctx->ready) {
    return fail(ctx, GCADA_ESTATE, "the minibatch size cannot change once stepping has begun; call gcada_set_theta to restart");
  }
  return GCADA_OK;
}

gcada_status gcada_set_batch(gcada_ctx* ctx, int batch) {
  if (!ctx) return GCADA_EINVAL;
  if (batch <= 0) return fail(ctx, GCADA_EINVAL, "batch must be positive");
  if (ctx->ready && batch != ctx->B)
    return fail(ctx, GCADA_ESTATE, "the minibatch size cannot change once stepping has begun; call gcada_set_theta to restart");
  ctx->B = batch;
  return GCADA_OK;
}

gcada_status gcada_set_theta(gcada_ctx* ctx, const float* theta0, long long p, int on_device) {
  if (!ctx) return GCADA_EINVAL;
  if (!theta0) return fail(ctx, GCADA_EINVAL, "theta0 is NULL");
  if (p != ctx->p) return fail(ctx, GCADA_EINVAL, "p = %lld but the model has %lld parameters", p, ctx->p);
  DeviceGuard dg(ctx->device);
  if (ctx->st) CK(cudaStreamSynchronize(ctx->stream));
  return make_ready(ctx, theta0, on_device);
}

gcada_status gcada_set_seed(gcada_ctx* ctx, unsigned long long seed) {
  if (!ctx) return GCADA_EINVAL;
  ctx->seed = seed;
  ctx->P.seed_lo = (uint32_t)(seed & 0xffffffffu);
  ctx->P.seed_hi = (uint32_t)(seed >> 32);
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_delay_model(gcada_ctx* ctx, double shift, double rate) {
  if (!ctx) return GCADA_EINVAL;
  if (!(shift >= 0) || !(rate > 0)) return fail(ctx, GCADA_EINVAL, "need shift >= 0 and rate > 0");
  ctx->shift = shift;
  ctx->rate = rate;
  ctx->P.shift = shift;
  ctx->P.inv_rate = 1.0 / rate;
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_delay_law(gcada_ctx* ctx, int law) {
  if (!ctx) return GCADA_EINVAL;
  if (law < 0 || law > 2) return fail(ctx, GCADA_EINVAL, "unknown delay law %d", law);
  ctx->delay_law = law;
  ctx->P.delay_law = law;
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_lag_weights(gcada_ctx* ctx, const double* c_d, int D) {
  if (!ctx) return GCADA_EINVAL;
  if (ctx->k_host > 0) return fail(ctx, GCADA_ESTATE, "the lag weights are fixed once stepping has begun");
  if (!c_d) {
    ctx->c_d.clear();
  } else {
    if (D != ctx->D) return fail(ctx, GCADA_EINVAL, "need D = %d lag weights", ctx->D);
    for (int d = 0; d < D; ++d)
      if (!(c_d[d] >= 0)) return fail(ctx, GCADA_EINVAL, "lag weights must be non-negative");
    ctx->c_d.assign(c_d, c_d + D);
  }
  ctx->ready = false;  // the device copy is made with the plans
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_step_schedule(gcada_ctx* ctx, int kind, double a, double b) {
  if (!ctx) return GCADA_EINVAL;
  if (kind == GCADA_SCHEDULE_CONST) {
    a = 1.0;
    b = 0.0;
  } else if (kind == GCADA_SCHEDULE_POLY) {
    if (!(a > 0) || !(b >= 0)) return fail(ctx, GCADA_EINVAL, "polynomial decay needs a > 0 and b >= 0");
  } else if (kind == GCADA_SCHEDULE_STEP) {
    if (!(a >= 1) || a != (double)(long long)a || !(b > 0)) return fail(ctx, GCADA_EINVAL, "step decay needs an integer a >= 1 and b > 0");
  } else {
    return fail(ctx, GCADA_EINVAL, "unknown schedule %d", kind);
  }
  ctx->sched_kind = kind;
  ctx->sched_a = a;
  ctx->sched_b = b;
  ctx->P.sched_kind = kind;
  ctx->P.sched_a = a;
  ctx->P.sched_b = b;
  drop_graphs(ctx);
  return GCADA_OK;
}

gcada_status gcada_set_option(gcada_ctx* ctx, int key, double value) {
  if (!ctx) return GCADA_EINVAL;
  if (key == GCADA_OPT_TIMING) {
    ctx->timing = value != 0;
    ctx->timed = 0;
    return GCADA_OK;
  }
  if (ctx->k_host > 0 && key != GCADA_OPT_GRAPH)
    return fail(ctx, GCADA_ESTATE, "options are fixed once stepping has begun; call gcada_set_theta to restart");
  switch (key) {
    case GCADA_OPT_RULE:
      if (value != 0 && value != 1) return fail(ctx, GCADA_EINVAL, "rule must be 0 (INNOV) or 1 (PS)");
      ctx->rule = (int)value;
      break;
    case GCADA_OPT_REDUCTION:
      if (value != 0 && value != 1) return fail(ctx, GCADA_EINVAL, "reduction must be 0 (mean) or 1 (sum)");
      ctx->reduction = (int)value;
      break;
    case GCADA_OPT_HISTORY:
      if (!(value >= 1) || value > 1e9) return fail(ctx, GCADA_EINVAL, "history must be in [1, 1e9]");
      ctx->hist_cap = (long long)value;
      break;
    case GCADA_OPT_KEEP_STALE:
      ctx->keep_stale = value != 0;
      break;
    case GCADA_OPT_PERSISTENT:
      ctx->persistent = value != 0;
      break;
    case GCADA_OPT_GRAPH:
      ctx->use_graph = value != 0;
      drop_graphs(ctx);
      return GCADA_OK;
    default:
      return fail(ctx, GCADA_EINVAL, "unknown option %d", key);
  }
  // options change buffer shapes: rebuild lazily at the next set_theta
  if (ctx->have_theta) {
    DeviceGuard dg(ctx->device);
    std::vector<float> th((size_t)ctx->p);
    CK(cudaStreamSynchronize(ctx->stream));
    CK(cudaMemcpy(th.data(), ctx->P.theta_ring, sizeof(float) * ctx->p, cudaMemcpyDeviceToHost));
    return make_ready(ctx, th.data(), 0);
  }
  return GCADA_OK;
}

gcada_status gcada_set_smoothness(gcada_ctx* ctx, const double* L, int G) {
  if (!ctx) return GCADA_EINVAL;
  if (!L || G != ctx->G) return fail(ctx, GCADA_EINVAL, "need G = %d smoothness constants", ctx->G);
  for (int g = 0; g < G; ++g)
    if (!(L[g] >= 0)) return fail(ctx, GCADA_EINVAL, "smoothness constants must be non-negative");
  if (ctx->k_host > 0) return fail(ctx, GCADA_ESTATE, "the smoothness constants are fixed once stepping has begun");
  ctx->L2.resize(G);
  for (int g = 0; g < G; ++g) ctx->L2[g] = L[g] * L[g];
  ctx->ready = false;  // the device copy is made with the plans
  drop_graphs(ctx);
  return GCADA_OK;
}

static gcada_status run_iterations(gcada_ctx* ctx, int n_iters, const unsigned char* mask) {
  TRY(check_runnable(ctx, true));
  if (n_iters < 0) return fail(ctx, GCADA_EINVAL, "n_iters is negative");
  if (n_iters == 0) return GCADA_OK;
  DeviceGuard dg(ctx->device);
  TRY(make_plans(ctx));
  Params P = ctx->P;
  if (mask) {
    const size_t bytes = (size_t)n_iters * ctx->G;
    CK(cudaStreamSynchronize(ctx->stream));
    if (bytes > ctx->forced_cap) {
      if (ctx->forced_dev) CK(cudaFree(ctx->forced_dev));
      ctx->forced_dev = nullptr;
      ctx->forced_cap = 0;
      CK(cudaMalloc(reinterpret_cast<void**>(&ctx->forced_dev), bytes));
      ctx->forced_cap = bytes;
    }
    CK(cudaMemcpy(ctx->forced_dev, mask, bytes, cudaMemcpyHostToDevice));
    P.forced = ctx->forced_dev;
    P.forced_base = ctx->k_host;
    for (int i = 0; i < n_iters; ++i) TRY(enqueue_iteration(ctx, P));
    ctx->k_host += n_iters;
    return GCADA_OK;
  }
  int left = n_iters;
  if (is_linear(ctx) && ctx->cluster.usable && !ctx->timing) {
    cudaError_t e = launch_linear_cluster(ctx->P, ctx->cluster, ctx->kind == GCADA_MODEL_QUADRATIC, n_iters, ctx->stream);
    if (e == cudaSuccess) {
      ctx->launches += 1;
      ctx->k_host += n_iters;
      return GCADA_OK;
    }
    cudaGetLastError();            // this device does not take the cluster launch: the kernel chain does the work
    ctx->cluster.usable = false;
  }
  if (ctx->use_graph && ctx->stream != nullptr && !ctx->timing) {
    // both graphs are captured, instantiated and uploaded by the first free-running step, whatever its
    // length, so that no later call pays for a capture
    if (!ctx->graph1) {
      TRY(capture(ctx, 1, &ctx->graph1));
      CK(cudaGraphUpload(ctx->graph1, ctx->stream));
    }
    if (!ctx->graphN) {
      TRY(capture(ctx, GRAPH_CHAIN, &ctx->graphN));
      CK(cudaGraphUpload(ctx->graphN, ctx->stream));
    }
    const int kpi = kernels_per_iteration(ctx);
    while (left >= GRAPH_CHAIN && ctx->graphN) {
      CK(cudaGraphLaunch(ctx->graphN, ctx->stream));
      ctx->launches += (unsigned long long)kpi * GRAPH_CHAIN;
      left -= GRAPH_CHAIN;
    }
    while (left > 0) {
      CK(cudaGraphLaunch(ctx->graph1, ctx->stream));
      ctx->launches += (unsigned long long)kpi;
      --left;
    }
  } else {
    for (; left > 0; --left) TRY(enqueue_iteration(ctx, P));
  }
  ctx->k_host += n_iters;
  return GCADA_OK;
}

gcada_status gcada_step(gcada_ctx* ctx, int n_iters) {
  if (!ctx) return GCADA_EINVAL;
  return run_iterations(ctx, n_iters, nullptr);
}

gcada_status gcada_step_forced(gcada_ctx* ctx, int n_iters, const unsigned char* mask) {
  if (!ctx) return GCADA_EINVAL;
  if (!mask) return fail(ctx, GCADA_EINVAL, "mask is NULL");
  return run_iterations(ctx, n_iters, mask);
}

gcada_status gcada_step_host_batch(gcada_ctx* ctx, const void* Xb_host, const void* yb_host) {
  if (!ctx) return GCADA_EINVAL;
  if (!Xb_host || !yb_host) return fail(ctx, GCADA_EINVAL, "Xb_host / yb_host is NULL");
  TRY(check_runnable(ctx, false));
  DeviceGuard dg(ctx->device);
  TRY(make_plans(ctx));
  const long long rows = (long long)ctx->G * ctx->B;
  const int d = ctx->dims[0];
  const size_t esz = ctx->compute == GCADA_COMPUTE_BF16 ? 2 : 4;
  if (!ctx->stage_x) {
    ctx->stage_ld = (d + 7) / 8 * 8;
    CK(cudaMalloc(&ctx->stage_x, (size_t)rows * ctx->stage_ld * esz));
    CK(cudaMalloc(&ctx->stage_y, (size_t)rows * 4));
    CK(cudaMemsetAsync(ctx->stage_x, 0, (size_t)rows * ctx->stage_ld * esz, ctx->stream));
  }
  CK(cudaMemcpy2DAsync(ctx->stage_x, (size_t)ctx->stage_ld * esz, Xb_host, (size_t)d * esz, (size_t)d * esz,
                       (size_t)rows, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(ctx->stage_y, yb_host, (size_t)rows * 4, cudaMemcpyHostToDevice, ctx->stream));
  Params P = ctx->P;
  P.X = ctx->stage_x;
  P.y = ctx->stage_y;
  P.ld = ctx->stage_ld;
  P.identity_batch = 1;
  P.n_g = ctx->B;
  TRY(enqueue_iteration(ctx, P));
  ctx->k_host += 1;
  return GCADA_OK;
}

gcada_status gcada_get_theta(gcada_ctx* ctx, float* out, long long p) {
  if (!ctx) return GCADA_EINVAL;
  if (!out || p != ctx->p) return fail(ctx, GCADA_EINVAL, "need a buffer of p = %lld floats", ctx->p);
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  const long long slot = s.k % (ctx->D + 1);
  CK(cudaMemcpy(out, ctx->P.theta_ring + slot * ctx->p_pad, sizeof(float) * p, cudaMemcpyDeviceToHost));
  return GCADA_OK;
}

gcada_status gcada_get_selection_mask(gcada_ctx* ctx, unsigned char* out, long long first_iter, int n_iters) {
  if (!ctx) return GCADA_EINVAL;
  if (!out || n_iters < 0 || first_iter < 0) return fail(ctx, GCADA_EINVAL, "bad arguments");
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  if (first_iter + n_iters > s.k) return fail(ctx, GCADA_EINVAL, "only %lld iterations have run", s.k);
  if (first_iter < s.k - ctx->hist_cap) return fail(ctx, GCADA_EINVAL, "iteration %lld is no longer in the history", first_iter);
  for (long long i = 0; i < n_iters;) {
    const long long slot = (first_iter + i) % ctx->hist_cap;
    long long run = ctx->hist_cap - slot;
    if (run > n_iters - i) run = n_iters - i;
    CK(cudaMemcpy(out + i * ctx->G, ctx->P.hist + slot * ctx->G, (size_t)run * ctx->G, cudaMemcpyDeviceToHost));
    i += run;
  }
  return GCADA_OK;
}

gcada_status gcada_get_comm_count(gcada_ctx* ctx, unsigned long long* uploads, unsigned long long* paper_comm,
                                  unsigned long long* paper_comp) {
  if (!ctx) return GCADA_EINVAL;
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  if (uploads) *uploads = s.uploads;
  if (paper_comm) *paper_comm = s.comm;
  if (paper_comp) *paper_comp = s.comp;
  return GCADA_OK;
}

gcada_status gcada_get_wallclock(gcada_ctx* ctx, double* total, double* last_iter) {
  if (!ctx) return GCADA_EINVAL;
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  if (total) *total = s.wall;
  if (last_iter) *last_iter = s.last_dt;
  return GCADA_OK;
}

gcada_status gcada_get_iteration(gcada_ctx* ctx, long long* k) {
  if (!ctx || !k) return GCADA_EINVAL;
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  *k = s.k;
  return GCADA_OK;
}

gcada_status gcada_get_debug(gcada_ctx* ctx, int what, void* out, long long bytes) {
  if (!ctx) return GCADA_EINVAL;
  if (!out) return fail(ctx, GCADA_EINVAL, "out is NULL");
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  const Params& P = ctx->P;
  const long long G = ctx->G, p = ctx->p, pp = ctx->p_pad;
  const void* src = nullptr;
  long long rows = 1, row_bytes = 0, src_pitch = 0;
  int per_group = -1;
  switch (what) {
    case GCADA_DBG_FRESH: per_group = 0; break;
    case GCADA_DBG_STALE:
      if (!P.stale) return fail(ctx, GCADA_ESTATE, "stale gradients are not kept: set GCADA_OPT_KEEP_STALE");
      src = P.stale; rows = G; row_bytes = p * 4; src_pitch = pp * 4; break;
    case GCADA_DBG_GLAST: per_group = 1; break;
    case GCADA_DBG_LHS: src = P.lhs; row_bytes = G * 8; break;
    case GCADA_DBG_RHS: src = &ctx->st->rhs; row_bytes = 8; break;
    case GCADA_DBG_TAU: src = P.tau; row_bytes = G * 4; break;
    case GCADA_DBG_AGG: src = P.agg_hi; row_bytes = p * 4; break;
    case GCADA_DBG_H: src = P.h; row_bytes = p * 4; break;
    case GCADA_DBG_VHAT: src = P.vhat; row_bytes = p * 4; break;
    case GCADA_DBG_TGROUP: src = P.t_g; row_bytes = G * 8; break;
    case GCADA_DBG_SRING: src = P.s_ring; row_bytes = (long long)ctx->D * 8; break;
    default: return fail(ctx, GCADA_EINVAL, "unknown debug item %d", what);
  }
  if (per_group >= 0) {
    if (bytes != G * p * 4) return fail(ctx, GCADA_EINVAL, "item %d has %lld bytes, buffer has %lld", what, G * p * 4, bytes);
    std::vector<unsigned char> cur((size_t)G), mask((size_t)G);
    CK(cudaMemcpy(cur.data(), P.cur, (size_t)G, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(mask.data(), P.mask_cur, (size_t)G, cudaMemcpyDeviceToHost));
    for (int g = 0; g < (int)G; ++g) {
      const float* row = nullptr;
      TRY(group_row_dev(ctx, per_group, g, cur, mask, &row));
      CK(cudaMemcpy(static_cast<float*>(out) + (long long)g * p, row, (size_t)p * 4, cudaMemcpyDeviceToHost));
    }
    return GCADA_OK;
  }
  if (bytes != rows * row_bytes) return fail(ctx, GCADA_EINVAL, "item %d has %lld bytes, buffer has %lld", what, rows * row_bytes, bytes);
  if (rows == 1)
    CK(cudaMemcpy(out, src, (size_t)row_bytes, cudaMemcpyDeviceToHost));
  else
    CK(cudaMemcpy2D(out, (size_t)row_bytes, src, (size_t)src_pitch, (size_t)row_bytes, (size_t)rows, cudaMemcpyDeviceToHost));
  return GCADA_OK;
}

gcada_status gcada_get_group_gradient(gcada_ctx* ctx, int what, int g, float* out, long long p) {
  if (!ctx) return GCADA_EINVAL;
  if (!out || p != ctx->p) return fail(ctx, GCADA_EINVAL, "need a buffer of p = %lld floats", ctx->p);
  if (g < 0 || g >= ctx->G) return fail(ctx, GCADA_EINVAL, "group %d out of range", g);
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  DeviceGuard dg(ctx->device);
  DevState s;
  TRY(read_state(ctx, &s));
  const float* src = nullptr;
  if (what == GCADA_DBG_STALE) {
    if (!ctx->P.stale) return fail(ctx, GCADA_ESTATE, "stale gradients are not kept: set GCADA_OPT_KEEP_STALE");
    src = ctx->P.stale + (long long)g * ctx->p_pad;
  } else if (what == GCADA_DBG_FRESH || what == GCADA_DBG_GLAST) {
    std::vector<unsigned char> cur((size_t)ctx->G), mask((size_t)ctx->G);
    CK(cudaMemcpy(cur.data(), ctx->P.cur, (size_t)ctx->G, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(mask.data(), ctx->P.mask_cur, (size_t)ctx->G, cudaMemcpyDeviceToHost));
    TRY(group_row_dev(ctx, what == GCADA_DBG_GLAST ? 1 : 0, g, cur, mask, &src));
  } else {
    return fail(ctx, GCADA_EINVAL, "item %d is not a per-group gradient", what);
  }
  CK(cudaMemcpy(out, src, sizeof(float) * (size_t)p, cudaMemcpyDeviceToHost));
  return GCADA_OK;
}

gcada_status gcada_get_launch_count(gcada_ctx* ctx, unsigned long long* launches) {
  if (!ctx || !launches) return GCADA_EINVAL;
  *launches = ctx->launches;
  return GCADA_OK;
}

gcada_status gcada_get_kernel_times(gcada_ctx* ctx, double ms[3], int* n_timed) {
  if (!ctx || !ms || !n_timed) return GCADA_EINVAL;
  DeviceGuard dg(ctx->device);
  CK(cudaStreamSynchronize(ctx->stream));
  const long long n = ctx->timed < TIMING_CAP ? ctx->timed : TIMING_CAP;
  ms[0] = ms[1] = ms[2] = 0.0;
  *n_timed = (int)n;
  if (n == 0) return GCADA_OK;
  for (long long i = 0; i < n; ++i) {
    cudaEvent_t* ev = &ctx->events[(size_t)i * 5];
    // normal order: gradient, selection, gradient (post-selection part), update;
    // skip mode (rule PS on linear models): selection first, then the selected groups' gradients
    const int normal[4] = {0, 1, 0, 2}, skip_first[4] = {1, 0, 2, 2}, agg_after[4] = {0, 1, 2, 2};
    const int* phase_of = ctx->P.skip_unselected ? skip_first : (ctx->P.agg_direct ? agg_after : normal);
    for (int j = 0; j < 4; ++j) {
      float t = 0.f;
      CK(cudaEventElapsedTime(&t, ev[j], ev[j + 1]));
      ms[phase_of[j]] += t;
    }
  }
  for (int j = 0; j < 3; ++j) ms[j] /= (double)n;
  return GCADA_OK;
}

gcada_status gcada_time_gradient(gcada_ctx* ctx, int reps, double* ms_per_rep) {
  if (!ctx || !ms_per_rep || reps < 1) return GCADA_EINVAL;
  TRY(check_runnable(ctx, true));
  DeviceGuard dg(ctx->device);
  TRY(make_plans(ctx));
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  CK(cudaEventCreate(&e0));
  CK(cudaEventCreate(&e1));
  Params P = ctx->P;
  P.skip_unselected = 0;  // every group, as in the default rule
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaEventRecord(e0, ctx->stream));
  for (int r = 0; r < reps; ++r) {
    if (is_linear(ctx)) {
      CK(launch_grad_linear(P, ctx->lin, ctx->kind == GCADA_MODEL_QUADRATIC, ctx->stream));
      ctx->launches += 1;
    } else {
      int n = 0;
      CK(launch_grad_mlp(P, ctx->mlp, ctx->stream, &n));
      ctx->launches += (unsigned long long)n;
    }
  }
  CK(cudaEventRecord(e1, ctx->stream));
  CK(cudaEventSynchronize(e1));
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, e0, e1));
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  *ms_per_rep = (double)ms / reps;
  return GCADA_OK;
}

gcada_status gcada_time_empty_chain(gcada_ctx* ctx, int n_iters, double* us_per_iter) {
  if (!ctx || !us_per_iter || n_iters < 1) return GCADA_EINVAL;
  TRY(check_runnable(ctx, true));
  DeviceGuard dg(ctx->device);
  TRY(make_plans(ctx));
  if (ctx->stream == nullptr) return fail(ctx, GCADA_ESTATE, "gcada_time_empty_chain needs a stream other than the default one");
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  CK(cudaEventCreate(&e0));
  CK(cudaEventCreate(&e1));
  float ms = 0.f;
  int iters_run = 0;
  if (is_linear(ctx) && ctx->cluster.usable) {
    CK(launch_linear_cluster_empty(ctx->cluster, 16, ctx->stream));  // warm-up
    CK(cudaStreamSynchronize(ctx->stream));
    CK(cudaEventRecord(e0, ctx->stream));
    CK(launch_linear_cluster_empty(ctx->cluster, n_iters, ctx->stream));
    CK(cudaEventRecord(e1, ctx->stream));
    iters_run = n_iters;
  } else {
    // the captured iterations with every kernel node's function replaced by an empty kernel: same nodes,
    // same edges, same grids, blocks, shared-memory sizes and cluster shapes, no work
    cudaGraph_t graph = nullptr;
    TRY(capture_graph(ctx, GRAPH_CHAIN, &graph));
    size_t n_nodes = 0;
    CK(cudaGraphGetNodes(graph, nullptr, &n_nodes));
    std::vector<cudaGraphNode_t> nodes(n_nodes);
    CK(cudaGraphGetNodes(graph, nodes.data(), &n_nodes));
    CK(cudaFuncSetAttribute(empty_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->smem_optin));
    CK(cudaFuncSetAttribute(empty_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    for (cudaGraphNode_t nd : nodes) {
      cudaGraphNodeType type;
      CK(cudaGraphNodeGetType(nd, &type));
      if (type != cudaGraphNodeTypeKernel) continue;
      cudaKernelNodeParams kp{};
      CK(cudaGraphKernelNodeGetParams(nd, &kp));
      kp.func = reinterpret_cast<void*>(empty_kernel);
      kp.kernelParams = nullptr;
      kp.extra = nullptr;
      CK(cudaGraphKernelNodeSetParams(nd, &kp));
    }
    cudaGraphExec_t exec = nullptr;
    cudaError_t e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    CK(e);
    const int reps = (n_iters + GRAPH_CHAIN - 1) / GRAPH_CHAIN;
    CK(cudaGraphLaunch(exec, ctx->stream));  // warm-up
    CK(cudaStreamSynchronize(ctx->stream));
    CK(cudaEventRecord(e0, ctx->stream));
    for (int r = 0; r < reps; ++r) CK(cudaGraphLaunch(exec, ctx->stream));
    CK(cudaEventRecord(e1, ctx->stream));
    CK(cudaEventSynchronize(e1));
    cudaGraphExecDestroy(exec);
    iters_run = reps * GRAPH_CHAIN;
  }
  CK(cudaEventSynchronize(e1));
  CK(cudaEventElapsedTime(&ms, e0, e1));
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  *us_per_iter = (double)ms * 1e3 / iters_run;
  return GCADA_OK;
}

gcada_status gcada_eval_loss(gcada_ctx* ctx, long long first_row, long long n_rows, double* mean_loss) {
  if (!ctx) return GCADA_EINVAL;
  if (!mean_loss) return fail(ctx, GCADA_EINVAL, "mean_loss is NULL");
  TRY(check_runnable(ctx, true));
  if (first_row < 0 || n_rows < 1 || first_row + n_rows > ctx->N)
    return fail(ctx, GCADA_EINVAL, "rows [%lld, %lld) are outside the training set of %lld rows", first_row,
                first_row + n_rows, ctx->N);
  DeviceGuard dg(ctx->device);
  TRY(make_plans(ctx));
  if (!ctx->eval_scratch) TRY(dev_alloc(ctx, &ctx->eval_scratch, (size_t)eval_loss_scratch_doubles()));
  DevState s;
  TRY(read_state(ctx, &s));
  if (!is_linear(ctx)) {
    if (!ctx->mlp_eval.part) {  // slab buffers, on first use
      int widest = 0;
      for (int v : ctx->dims) widest = v > widest ? v : widest;
      TRY(dev_alloc(ctx, &ctx->mlp_eval.buf[0], (size_t)MLP_EVAL_SLAB * widest));
      TRY(dev_alloc(ctx, &ctx->mlp_eval.buf[1], (size_t)MLP_EVAL_SLAB * widest));
      TRY(dev_alloc(ctx, &ctx->mlp_eval.ones, (size_t)MLP_EVAL_SLAB / 64));
      CK(cudaMemsetAsync(ctx->mlp_eval.ones, 1, (size_t)MLP_EVAL_SLAB / 64, ctx->stream));
      TRY(dev_alloc(ctx, &ctx->mlp_eval.part, (size_t)1024));
    }
    CK(mlp_eval_loss(ctx->P, ctx->mlp, first_row, n_rows, ctx->mlp_eval, ctx->eval_scratch, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    CK(cudaMemcpy(mean_loss, ctx->eval_scratch, sizeof(double), cudaMemcpyDeviceToHost));
    return GCADA_OK;
  }
  const float* theta = ctx->P.theta_ring + (s.k % (ctx->D + 1)) * ctx->p_pad;
  CK(launch_eval_loss_linear(ctx->P, theta, ctx->kind == GCADA_MODEL_QUADRATIC, first_row, n_rows, ctx->eval_scratch,
                             ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaMemcpy(mean_loss, ctx->eval_scratch, sizeof(double), cudaMemcpyDeviceToHost));
  return GCADA_OK;
}

namespace {
struct CkptHeader {
  char magic[8];
  long long kind, compute, n_dims, dims[MLP_MAX_LAYERS + 1], M, M_G, D, B, p, hist_cap, keep_stale, n_seg, total;
};
constexpr char CKPT_MAGIC[8] = {'G', 'C', 'A', 'D', 'A', 'C', 'K', '1'};

gcada_status checkpoint_layout(gcada_ctx* ctx, CkptHeader* h, std::vector<std::pair<void*, size_t>>* segs) {
  TRY(check_runnable(ctx, false));
  TRY(make_plans(ctx));
  *segs = ctx->state;
  if (!is_linear(ctx)) segs->insert(segs->end(), ctx->mlp.state.begin(), ctx->mlp.state.end());
  memset(h, 0, sizeof *h);
  memcpy(h->magic, CKPT_MAGIC, 8);
  h->kind = ctx->kind;
  h->compute = ctx->compute;
  h->n_dims = (long long)ctx->dims.size();
  for (size_t i = 0; i < ctx->dims.size(); ++i) h->dims[i] = ctx->dims[i];
  h->M = ctx->M;
  h->M_G = ctx->M_G;
  h->D = ctx->D;
  h->B = ctx->B;
  h->p = ctx->p;
  h->hist_cap = ctx->hist_cap;
  h->keep_stale = ctx->keep_stale;
  h->n_seg = (long long)segs->size();
  size_t total = sizeof(CkptHeader) + sizeof(unsigned long long) * segs->size();
  for (auto& s : *segs) total += s.second;
  h->total = (long long)total;
  return GCADA_OK;
}
}  // namespace

gcada_status gcada_checkpoint_size(gcada_ctx* ctx, unsigned long long* bytes) {
  if (!ctx || !bytes) return GCADA_EINVAL;
  DeviceGuard dg(ctx->device);
  CkptHeader h;
  std::vector<std::pair<void*, size_t>> segs;
  TRY(checkpoint_layout(ctx, &h, &segs));
  *bytes = (unsigned long long)h.total;
  return GCADA_OK;
}

gcada_status gcada_checkpoint_save(gcada_ctx* ctx, void* host_buf, unsigned long long bytes) {
  if (!ctx) return GCADA_EINVAL;
  if (!host_buf) return fail(ctx, GCADA_EINVAL, "host_buf is NULL");
  DeviceGuard dg(ctx->device);
  CkptHeader h;
  std::vector<std::pair<void*, size_t>> segs;
  TRY(checkpoint_layout(ctx, &h, &segs));
  if (bytes != (unsigned long long)h.total)
    return fail(ctx, GCADA_EINVAL, "a checkpoint of this context has %lld bytes, the buffer has %llu", h.total, bytes);
  DevState s;
  TRY(read_state(ctx, &s));  // synchronises the stream and refuses to save after a device-side error
  unsigned char* out = static_cast<unsigned char*>(host_buf);
  memcpy(out, &h, sizeof h);
  out += sizeof h;
  for (auto& sg : segs) {
    const unsigned long long n = sg.second;
    memcpy(out, &n, sizeof n);
    out += sizeof n;
  }
  for (auto& sg : segs) {
    CK(cudaMemcpy(out, sg.first, sg.second, cudaMemcpyDeviceToHost));
    out += sg.second;
  }
  return GCADA_OK;
}

gcada_status gcada_checkpoint_load(gcada_ctx* ctx, const void* host_buf, unsigned long long bytes) {
  if (!ctx) return GCADA_EINVAL;
  if (!host_buf) return fail(ctx, GCADA_EINVAL, "host_buf is NULL");
  DeviceGuard dg(ctx->device);
  CkptHeader h;
  std::vector<std::pair<void*, size_t>> segs;
  TRY(checkpoint_layout(ctx, &h, &segs));
  if (bytes < sizeof(CkptHeader)) return fail(ctx, GCADA_EINVAL, "buffer too small for a checkpoint");
  CkptHeader in;
  memcpy(&in, host_buf, sizeof in);
  if (memcmp(in.magic, CKPT_MAGIC, 8) != 0) return fail(ctx, GCADA_EINVAL, "not a checkpoint of this library");
  if (memcmp(&in, &h, sizeof h) != 0 || bytes != (unsigned long long)h.total)
    return fail(ctx, GCADA_EINVAL,
                "the checkpoint was saved by a context with another model, grouping, D, batch size or options");
  const unsigned char* src = static_cast<const unsigned char*>(host_buf) + sizeof h;
  for (auto& sg : segs) {
    unsigned long long n;
    memcpy(&n, src, sizeof n);
    src += sizeof n;
    if (n != sg.second) return fail(ctx, GCADA_EINVAL, "checkpoint segment sizes do not match this context");
  }
  CK(cudaStreamSynchronize(ctx->stream));
  for (auto& sg : segs) {
    CK(cudaMemcpy(sg.first, src, sg.second, cudaMemcpyHostToDevice));
    src += sg.second;
  }
  DevState s;
  TRY(read_state(ctx, &s));
  ctx->k_host = s.k;
  return GCADA_OK;
}

int gcada_is_debug_build(void) {
#ifdef GCADA_DEBUG
  return 1;
#else
  return 0;
#endif
}

gcada_status gcada_debug_set_error(gcada_ctx* ctx, int dev_err) {
  if (!ctx) return GCADA_EINVAL;
#ifdef GCADA_DEBUG
  if (!ctx->have_theta) return fail(ctx, GCADA_ESTATE, "gcada_set_theta has not been called");
  if (dev_err < 0 || dev_err > DEV_ERR_CHAIN) return fail(ctx, GCADA_EINVAL, "unknown device error word %d", dev_err);
  DeviceGuard dg(ctx->device);
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaMemcpy(&ctx->st->err, &dev_err, sizeof(int), cudaMemcpyHostToDevice));
  return GCADA_OK;
#else
  (void)dev_err;
  return fail(ctx, GCADA_ESTATE, "gcada_debug_set_error exists in the debug library (libgcada_dbg.so) only");
#endif
}

const char* gcada_last_error(const gcada_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

void gcada_destroy(gcada_ctx* ctx) {
  if (!ctx) return;
  {
    DeviceGuard dg(ctx->device);
    if (ctx->st) cudaStreamSynchronize(ctx->stream);
    free_all(ctx);
  }
  delete ctx;
}

}  // extern "C"
