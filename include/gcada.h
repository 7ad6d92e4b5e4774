/*
 * gcada.h - C ABI of the G-CADA step library (CUDA, sm_100a).
 *
 * G-CADA = grouping-based communication-adaptive distributed Adam (Zhu, Zhang,
 * Simeone, Wang, "Adaptive Worker Grouping for Communication-Efficient and
 * Straggler-Tolerant Distributed SGD").  One context simulates the parameter
 * server and all M workers (G = M / M_G groups) on one GPU.  One call of
 * gcada_step runs iterations of Algorithm 1:
 *
 *   1. every group g draws a minibatch xi_g^k from its shard (Section II-A);
 *   2. its gradient is evaluated at theta^k and at the group's stale iterate
 *      theta^{k - tau_g} on the same samples; LHS_g = ||difference||^2, the
 *      quantity the left side of Eq. (9) estimates (rule INNOV), or the
 *      printed left side L_g^2 ||theta^k - theta^{k-tau_g}||^2 (rule PS);
 *   3. group g is selected if tau_g >= D or LHS_g > c * sum_{d=1..D}
 *      ||theta^{k+1-d} - theta^{k-d}||^2 (Eq. 9 and the age rule, Section IV);
 *   4. the lazily aggregated gradient (Eq. 3) swaps in the fresh gradients of
 *      the selected groups; theta, h, v-hat follow Eq. (8a)-(8c);
 *   5. the simulated wall-clock advances by the slowest selected group, a
 *      group being as fast as its fastest worker (Section II-B, Section V-A);
 *      communication and computation loads follow Eqs. (5), (6), (19), (22).
 *
 * Conventions
 *   - Every function returns a gcada_status; nothing throws or aborts.  After a
 *     non-OK status gcada_last_error(ctx) describes it.
 *   - "device" pointers are CUDA device pointers of the current device,
 *     "host" pointers are ordinary host memory.  Borrowed buffers must outlive
 *     their use by the context; the library never frees caller memory.
 *     Output buffers are caller-allocated with the size passed.
 *   - gcada_step only enqueues work on the context's stream (its first call
 *     on a context also builds launch plans and captures its CUDA graphs,
 *     which allocates); getters synchronise that stream.  The harness
 *     variants gcada_step_forced and gcada_step_host_batch are not free of
 *     host work: the first synchronises the stream, copies the mask with a
 *     blocking copy and grows its device buffer when needed, the second
 *     allocates a staging area on first use.
 *   - Contexts are independent and share no state.  The only process-wide
 *     state of the library is the fixed scratch array of
 *     gcada_innovation_norms_noalloc (see there).  A context is bound to the
 *     device that was current in gcada_create.
 *   - There is no CPU fallback: without a usable CUDA device gcada_create
 *     fails with GCADA_ECUDA.
 */
#ifndef GCADA_H
#define GCADA_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gcada_ctx gcada_ctx; /* opaque; owns all internal device state */

typedef enum {
  GCADA_OK = 0,
  GCADA_EINVAL = 1,   /* bad argument; nothing was changed */
  GCADA_ENOMEM = 2,   /* host or device allocation failed */
  GCADA_ECUDA = 3,    /* a CUDA call failed; text in gcada_last_error */
  GCADA_ESTATE = 4,   /* call not allowed in the context's current state */
  GCADA_ETIMEOUT = 5  /* a bounded device-side wait gave up */
} gcada_status;

/* Model kinds (per-sample loss l(theta; z) of Eq. 1). */
#define GCADA_MODEL_LOGISTIC 0  /* -y ln s - (1-y) ln(1-s), s = sigmoid(x.theta), y in {0,1} */
#define GCADA_MODEL_MLP 1       /* ReLU hidden layers, softmax cross-entropy, integer class y */
#define GCADA_MODEL_QUADRATIC 2 /* (x.theta - y)^2 / 2, the loss of Section VI */

/* Arithmetic. */
#define GCADA_COMPUTE_FP32 0 /* fp32 data, fp32 arithmetic */
#define GCADA_COMPUTE_BF16 1 /* bf16 features and weight copies, fp32 accumulation and state (MLP only) */

typedef struct {
  int kind;        /* GCADA_MODEL_* */
  int n_dims;      /* logistic / quadratic: 1; MLP: number of layers + 1 */
  const int *dims; /* host; {d} or {n_0, n_1, ..., n_L}; copied */
  int compute;     /* GCADA_COMPUTE_* */
} gcada_model;

/* Options for gcada_set_option (set before the first step). */
#define GCADA_OPT_RULE 0       /* 0 = INNOV (default), 1 = PS (printed Eq. 9; needs gcada_set_smoothness) */
#define GCADA_OPT_REDUCTION 1  /* 0 = mean over the minibatch (default), 1 = sum (Section II-A as printed) */
#define GCADA_OPT_HISTORY 2    /* iterations of selection masks kept for gcada_get_selection_mask (default 65536) */
#define GCADA_OPT_KEEP_STALE 3 /* 1 = also keep each group's stale-point gradient for gcada_get_debug (default 0) */
#define GCADA_OPT_GRAPH 4      /* 1 = replay iterations from a captured CUDA graph (default 1) */
#define GCADA_OPT_TIMING 5     /* 1 = bracket each kernel phase with CUDA events (plain launches; see
                                  gcada_get_kernel_times); may be switched at any time (default 0) */

/* (key 6 is not used) */
#define GCADA_OPT_PERSISTENT 7     /* 1 (default) = logistic / quadratic models with d <= 256, at most 64 groups and
                                      1024 workers run free-running steps of the default rule as ONE launch of a
                                      single thread-block cluster per gcada_step call, whatever n_iters is (the
                                      whole iteration stays on chip; one cluster barrier per iteration);
                                      0 = always the chain of kernels.  Both give the same results up to summation
                                      order; forced, host-fed, timed and rule-PS steps always use the chain */

/* Items for gcada_get_debug.  Sizes are in elements of the stated type. */
#define GCADA_DBG_FRESH 0   /* float [G][p]: gradient of each group at theta^k, last iteration run */
#define GCADA_DBG_STALE 1   /* float [G][p]: gradient at the stale iterate (needs GCADA_OPT_KEEP_STALE) */
#define GCADA_DBG_LHS 2     /* double [G]: left side of the test, last iteration */
#define GCADA_DBG_RHS 3     /* double [1]: right side of the test, last iteration */
#define GCADA_DBG_TAU 4     /* int [G]: age of information entering the NEXT iteration */
#define GCADA_DBG_AGG 5     /* float [p]: lazily aggregated gradient (Eq. 3) after the last iteration */
#define GCADA_DBG_H 6       /* float [p]: h (Eq. 8a) */
#define GCADA_DBG_VHAT 7    /* float [p]: v-hat (Eq. 8b and the max below it) */
#define GCADA_DBG_TGROUP 8  /* double [G]: fastest-worker time of each group, last iteration */
#define GCADA_DBG_GLAST 9   /* float [G][p]: last uploaded gradient of each group */
#define GCADA_DBG_SRING 10  /* double [D]: ||theta^{j+1}-theta^j||^2 for the last D steps, slot j mod D */

/*
 * Create a context.  Arguments are Algorithm 1's inputs and the constants of
 * Eq. (8) and (9): M workers in groups of M_G (Section IV), maximum delay D,
 * threshold constant c, step size alpha, momentum weights beta1, beta2,
 * epsilon.  GCADA_EINVAL unless M > 0, M_G > 0, M % M_G == 0, D >= 1, c >= 0,
 * alpha > 0, 0 < beta1, beta2 < 1, eps > 0 and the model is supported:
 * logistic / quadratic need 1 <= d <= 4096; MLP needs n_dims >= 2.
 * Initial state: h = v-hat = 0, aggregate 0, every tau_g = D (so the first
 * iteration selects every group), k = 0, seed 0, delay model shift 1 rate 1.
 * *out receives the context (owned by the caller until gcada_destroy).
 */
gcada_status gcada_create(const gcada_model *model, int M, int M_G, int D, double c, double alpha,
                          double beta1, double beta2, double eps, gcada_ctx **out);

/* CUDA stream (cudaStream_t passed as void*) all work is enqueued on;
 * borrowed; NULL = the legacy default stream (the initial setting). */
gcada_status gcada_set_stream(gcada_ctx *ctx, void *cuda_stream);

/*
 * Training set (Section II-A): X_dev is a row-major device matrix of N rows
 * with row stride ld_x elements (>= d): float for GCADA_COMPUTE_FP32, bfloat16
 * for GCADA_COMPUTE_BF16.  y_dev holds N labels: float (0/1 or real) for
 * logistic / quadratic, int32 class ids for the MLP.  Both are BORROWED.
 * Shard of group g = rows g*floor(N/G) .. (g+1)*floor(N/G)-1 (Section IV:
 * equal-sized disjoint shards; trailing rows unused).  `batch` = minibatch
 * size per group.  For logistic / quadratic models with d > 256, X_dev must
 * be 16-byte aligned and ld_x a multiple of 4.  GCADA_EINVAL otherwise, or if
 * floor(N/G) == 0, batch <= 0.
 */
gcada_status gcada_set_data(gcada_ctx *ctx, const void *X_dev, const void *y_dev, long long N,
                            long long ld_x, int batch);

/* theta^0: p floats, copied (from the device if on_device != 0, else from the
 * host).  Resets the run to k = 0 with the initial state listed above.
 * MLP layout: for each layer W_l (n_l rows of n_{l-1}) then b_l (n_l). */
gcada_status gcada_set_theta(gcada_ctx *ctx, const float *theta0, long long p, int on_device);

/* Seed of the counter-based generator (Philox4x32-10) that draws minibatches
 * and worker computing times.  Minibatch draw j of group g at iteration k is
 * 32-bit word j%4 of counter (j/4, g, k, 0), mapped to floor(w*n_g/2^32);
 * worker m's uniform at iteration k is word m%4 of counter (m/4, 0, k, 1),
 * u = (w + 0.5) / 2^32.  Key = (seed low 32 bits, seed high 32 bits). */
gcada_status gcada_set_seed(gcada_ctx *ctx, unsigned long long seed);

/* Computing time of worker m at iteration k (Section II-B):
 * T = shift - ln(1 - u) / rate.  The paper's exponential of mean eta is
 * shift 0, rate 1/eta.  GCADA_EINVAL unless shift >= 0 and rate > 0. */
gcada_status gcada_set_delay_model(gcada_ctx *ctx, double shift, double rate);

/* Law of the computing times.  Section II-B takes them exponential; the analysis of Section V only uses
 * that they are i.i.d., so two more laws are offered, with the (shift, rate) of gcada_set_delay_model:
 * GCADA_DELAY_EXP      T = shift - ln(1-u)/rate           (default)
 * GCADA_DELAY_PARETO   T = shift * (1-u)^(-1/rate)        heavy tail, P(T > t) = (shift/t)^rate, shift > 0
 * GCADA_DELAY_UNIFORM  T = shift + u/rate                 bounded */
#define GCADA_DELAY_EXP 0
#define GCADA_DELAY_PARETO 1
#define GCADA_DELAY_UNIFORM 2
gcada_status gcada_set_delay_law(gcada_ctx *ctx, int law);

/* Per-lag constants {c_d} (host, D doubles >= 0; copied) of Algorithm 1's input list: the right side of
 * the test becomes sum_{d=1..D} c_d ||theta^{k+1-d} - theta^{k-d}||^2.  NULL restores c_d = c, which is
 * Eq. (9) as printed.  Set before the first step (GCADA_ESTATE afterwards). */
gcada_status gcada_set_lag_weights(gcada_ctx *ctx, const double *c_d, int D);

/* Step size alpha^k of Eq. (2) / Eq. (8c), alpha being gcada_create's:
 * GCADA_SCHEDULE_CONST  alpha^k = alpha                          (default; a, b ignored)
 * GCADA_SCHEDULE_POLY   alpha^k = alpha / (1 + k/a)^b            a > 0, b >= 0
 * GCADA_SCHEDULE_STEP   alpha^k = alpha * b^floor(k/a)           integer a >= 1, b > 0
 * k counts from 0.  May be changed between steps. */
#define GCADA_SCHEDULE_CONST 0
#define GCADA_SCHEDULE_POLY 1
#define GCADA_SCHEDULE_STEP 2
gcada_status gcada_set_step_schedule(gcada_ctx *ctx, int kind, double a, double b);

gcada_status gcada_set_option(gcada_ctx *ctx, int key, double value);

/* Smoothness constants L_g >= 0 (host, G doubles; copied) for rule PS, the left side of Eq. (9) as
 * printed: L_g^2 ||theta^k - theta^{k-tau_g}||^2, evaluated from the ring of the last D+1 iterates.  Set
 * them before the first step; stepping with GCADA_OPT_RULE = 1 and no constants gives GCADA_ESTATE.  The
 * printed test needs no gradient, so for logistic / quadratic models (up to 1024 groups) an iteration runs in
 * Algorithm 1's order: test, selection, then gradients at theta^k for the selected groups only (the cost of
 * an iteration scales with the number of uploads; GCADA_DBG_FRESH / _STALE / _LHS-by-innovation of
 * unselected groups are then not produced).  The MLPs run in the same order (forward and backward pass
 * of the selected groups at theta^k only; no stale-point pass, no innovation norms) unless
 * GCADA_OPT_KEEP_STALE is set, in which case both gradients of every group are still evaluated. */
gcada_status gcada_set_smoothness(gcada_ctx *ctx, const double *L, int G);

/* Run n_iters iterations of Algorithm 1 on the stream (asynchronous).
 * GCADA_ESTATE before gcada_set_data and gcada_set_theta. */
gcada_status gcada_step(gcada_ctx *ctx, int n_iters);

/* As gcada_step, but the selected set of iteration i is mask[i*G + g] != 0
 * (host, n_iters*G bytes, copied before return) instead of the test's
 * outcome.  LHS, RHS and every other quantity are still computed.  The
 * method's own rule never lets an age exceed D; if a forced mask does, the
 * group's stale iterate is theta^{k-D}, the oldest one kept. */
gcada_status gcada_step_forced(gcada_ctx *ctx, int n_iters, const unsigned char *mask);

/*
 * One iteration whose minibatches come from the HOST: Xb_host holds G*batch
 * rows of d elements (row stride d; group g's minibatch = rows g*batch ..),
 * yb_host the matching labels.  They are copied to a device staging area
 * (asynchronously if the host memory is pinned) and the step uses them in
 * place of draws from the resident training set, which may be absent.
 * Needs gcada_set_batch or gcada_set_data first.
 */
gcada_status gcada_step_host_batch(gcada_ctx *ctx, const void *Xb_host, const void *yb_host);

/* Minibatch size when no resident training set is given (host-fed steps). */
gcada_status gcada_set_batch(gcada_ctx *ctx, int batch);

/* Getters: synchronise the stream, copy to HOST memory. */
gcada_status gcada_get_theta(gcada_ctx *ctx, float *out, long long p);
/* mask[i*G + g] for iterations first_iter .. first_iter + n_iters - 1
 * (0-based); GCADA_EINVAL if not run yet or no longer in the history. */
gcada_status gcada_get_selection_mask(gcada_ctx *ctx, unsigned char *out, long long first_iter,
                                      int n_iters);
/* uploads = sum of all selection masks (|M_U| summed over iterations);
 * paper_comm = sum of |M_D| + |M_U| = (M_G + 1) * uploads (Eqs. 5, 19);
 * paper_comp = sum of |M_D| = M_G * uploads, in minibatch gradients (Eqs. 6,
 * 22; multiply by the batch size for samples).  Any pointer may be NULL. */
gcada_status gcada_get_comm_count(gcada_ctx *ctx, unsigned long long *uploads,
                                  unsigned long long *paper_comm, unsigned long long *paper_comp);
/* Simulated wall-clock (Eq. 4 summed over iterations) and its last increment. */
gcada_status gcada_get_wallclock(gcada_ctx *ctx, double *total, double *last_iter);
/* Number of iterations run since gcada_set_theta. */
gcada_status gcada_get_iteration(gcada_ctx *ctx, long long *k);
/* Internal quantities (GCADA_DBG_*); `bytes` must equal the item's size. */
gcada_status gcada_get_debug(gcada_ctx *ctx, int what, void *out, long long bytes);
/* One group's row of GCADA_DBG_FRESH / GCADA_DBG_STALE / GCADA_DBG_GLAST (p floats to the host), for models
 * whose [G][p] arrays are too large to copy whole.  With the bf16 MLP and GCADA_OPT_KEEP_STALE off no
 * per-group gradient vector exists on the device: each upload is kept as the two bf16 factors of every
 * layer's weight gradient, GCADA_DBG_GLAST rebuilds the group's last uploaded gradient from them on demand,
 * and GCADA_DBG_FRESH returns the same (a fresh gradient survives only as an upload). */
gcada_status gcada_get_group_gradient(gcada_ctx *ctx, int what, int g, float *out, long long p);
/* Number of kernel launches enqueued by this context so far (graph replays
 * count the kernels they contain). */
gcada_status gcada_get_launch_count(gcada_ctx *ctx, unsigned long long *launches);

/* With GCADA_OPT_TIMING on: mean device time in milliseconds of the three
 * phases of an iteration, ms[0] gradient kernels (including any that run
 * after the selection), ms[1] selection kernel,
 * ms[2] update kernel, over the (at most 512) most recent timed iterations,
 * whose number goes to *n_timed.  Synchronises the stream. */
gcada_status gcada_get_kernel_times(gcada_ctx *ctx, double ms[3], int *n_timed);

/*
 * Innovation norms without any allocation.  (The paper has no counterpart of
 * this call; it exists for the sake of callers, not of the method.)
 *
 * Some users of this library run where device memory may not be allocated:
 * inside a region whose memory plan is frozen (a serving process that
 * pre-allocated its pool, a real-time loop, code running between the capture
 * and replay of someone else's graph) or under an allocator they do not
 * control.  gcada_create and gcada_set_theta allocate, so such callers cannot
 * use a context.  This call gives them the test quantity of the selection
 * rule on gradients they already hold:
 *     lhs_dev[g] = || fresh_dev[g*ld .. g*ld+p) - stale_dev[g*ld .. g*ld+p) ||^2
 * for g < G: each difference is taken in float, squared and accumulated in
 * double in a fixed order (the order differs from a context's own reduction,
 * and for logistic / quadratic models a context squares innovation partial
 * sums that its gradient kernel formed directly, so the two agree to
 * rounding, not bit for bit).  All three pointers are device
 * memory of the CURRENT device, owned by the caller; lhs_dev receives G
 * doubles.  The work is enqueued on cuda_stream (cudaStream_t as void*, NULL =
 * legacy default stream) and is asynchronous.
 *
 * Scratch space is a fixed 512 KiB array inside the library image: every GPU
 * that loads the library carries it until the process exits.  Limit:
 * G <= GCADA_NOALLOC_MAX_GROUPS, otherwise GCADA_EINVAL and nothing runs (p
 * is not limited).  All calls on one device share that array, so two calls
 * whose kernels may overlap on the GPU (different streams without ordering
 * between them) race and give wrong sums; order them.  The array keeps the
 * previous call's contents; the one word that must start at zero is cleared
 * on the stream by every call.  The first call on each device looks up the
 * array's device address (cudaGetSymbolAddress, with that device current)
 * and keeps it for the life of the process: make that first call outside any
 * stream capture, and do not use this entry point again on a device after
 * cudaDeviceReset or from a second CUDA context on the same device (the kept
 * address belongs to the context that first loaded the library).  No call here uses
 * cudaMalloc, cudaFree or any other allocating routine.
 * On failure a message is written to errbuf (if non-NULL, errbuf_len bytes).
 */
#define GCADA_NOALLOC_MAX_GROUPS 1024
gcada_status gcada_innovation_norms_noalloc(const float *fresh_dev, const float *stale_dev, int G,
                                            long long p, long long ld, double *lhs_dev,
                                            void *cuda_stream, char *errbuf, size_t errbuf_len);

/* Measurement aid: enqueue the gradient kernel(s) of the current iteration `reps` times back to back on the
 * stream, bracketed by ONE pair of CUDA events, and return the mean device time per repetition in
 * milliseconds (per-launch event brackets, as GCADA_OPT_TIMING uses, add the launch gaps of each bracket to
 * a kernel that lasts tens of microseconds).  The repetitions recompute the same gradients and change no
 * state that an iteration reads.  Synchronises the stream before and after. */
gcada_status gcada_time_gradient(gcada_ctx *ctx, int reps, double *ms_per_rep);

/* Measurement aid: the latency floor of this context's iteration structure.  Enqueues what gcada_step(n_iters)
 * would launch with all work removed - for the kernel chain a copy of the captured iteration graph (same
 * nodes and dependencies, same grid, block, shared-memory and cluster shapes) whose kernels are empty, run in
 * multiples of 16 iterations; for narrow linear models that run whole steps in one thread-block cluster, that
 * cluster with nothing but its one cluster-wide barrier per iteration - and returns the device time per
 * iteration in microseconds.  Touches no state of the run.  Needs a stream other than the default one
 * (GCADA_ESTATE otherwise).  Synchronises the stream. */
gcada_status gcada_time_empty_chain(gcada_ctx *ctx, int n_iters, double *us_per_iter);

/* Reporting aid (not a step of Algorithm 1): the mean per-sample loss of the current iterate over rows
 * first_row .. first_row + n_rows - 1 of the resident training set, i.e. the objective of Eq. (1) restricted
 * to those rows, to *mean_loss (host).  Logistic / quadratic models: double precision.  MLPs: the softmax
 * cross-entropy of the fp32 master parameters in fp32 arithmetic (whatever the model's compute type; the
 * per-row terms and their sum in double), rows pushed through the tile kernels in slabs; scratch buffers are
 * allocated on the first call.  Synchronises the stream. */
gcada_status gcada_eval_loss(gcada_ctx *ctx, long long first_row, long long n_rows, double *mean_loss);

/*
 * Checkpoints (the paper has no counterpart).  A checkpoint is everything an iteration inherits from
 * earlier ones: iteration counter, counters and wall-clock, the last D+1 iterates, h, v-hat, the
 * aggregate, every group's last uploaded gradient (or its factors), ages, the ring of squared step norms
 * and the mask history.  It does NOT hold the constructor arguments, seed, delay model, options or the
 * training set: load into a context created and configured like the one that saved (gcada_create, options,
 * gcada_set_data or gcada_set_batch, gcada_set_theta with any theta), otherwise GCADA_EINVAL and nothing is
 * changed.  After a load the run continues bit-for-bit as the saved one would have.
 * gcada_checkpoint_size gives the byte count for this context; save / load need a host buffer of exactly
 * that size.  All three synchronise the stream.
 */
gcada_status gcada_checkpoint_size(gcada_ctx *ctx, unsigned long long *bytes);
gcada_status gcada_checkpoint_save(gcada_ctx *ctx, void *host_buf, unsigned long long bytes);
gcada_status gcada_checkpoint_load(gcada_ctx *ctx, const void *host_buf, unsigned long long bytes);

/*
 * The debug library.  libgcada_dbg.so is this same source compiled with -DGCADA_DEBUG: every store whose
 * position a kernel computes at run time (partial-sum slots, innovation-norm partial sums, the mask history,
 * the list of selected groups, gradient rows, the entries of the bf16 factor arrays) is checked against the
 * size of its buffer first.  A failed check does not trap: the store is skipped, the run's device error word
 * is raised, and from then on every getter returns GCADA_ECUDA with the buffer named in gcada_last_error
 * (a bounded device-side wait that gave up is reported as GCADA_ETIMEOUT the same way, in both libraries).
 * gcada_is_debug_build tells the two libraries apart (1 / 0).  gcada_debug_set_error writes the device error
 * word from the host (dev_err: 0 none, 1 a wait gave up, 2 an index check failed, 3 a kernel that started early
 * inside a replayed chain of iterations found the iteration counter elsewhere than the chain's bookkeeping:
 * reported as GCADA_ECUDA) so that the reporting path
 * can be exercised without any device-side failure; in the ordinary library it returns GCADA_ESTATE.
 */
int gcada_is_debug_build(void);
gcada_status gcada_debug_set_error(gcada_ctx *ctx, int dev_err);

/* Text of the last error of this context ("" if none); valid until the next
 * call on the context.  ctx == NULL returns the text of the last failed
 * gcada_create of the calling thread. */
const char *gcada_last_error(const gcada_ctx *ctx);

void gcada_destroy(gcada_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* GCADA_H */
