// bf16 tensor-core path of the dual-point MLP gradients (Algorithm 1's
// gradient step for every group at theta^k and at theta^{k-tau_g}).
//
// Operands are bf16 (features as stored; weights rounded from the fp32 master
// iterate once per iteration), accumulation is fp32 in tensor memory.  Per-group
// weight gradients are never materialised on the production path: the squared
// innovation norms come from two Gram products per group and layer over the
// differences of the two points (bf16_gram_kernel), and the server's aggregate (Eq. 3,
// the sum over groups of each group's last uploaded gradient) is one product per
// layer over the factors (dz_l, a_{l-1}) of every group's last
// upload, with K running over all groups' rows.  The factors at theta^k are
// written into one of two buffers per group; the other one holds the group's last
// upload, and selecting the group flips the two (Params::cur), so an upload moves
// no data.  One kernel serves every product  C[M x N] = sum_k A[m][k] B[n][k]:
//     forward   z_l   = a_{l-1} W_l^T        A = a_{l-1} [rows][n_{l-1}],  B = W_l   [n_l][n_{l-1}]   (both K-major)
//     backward  da    = dz_l W_l             A = dz_l    [rows][n_l],      B = W_l^T [n_{l-1}][n_l]   (both K-major)
//     aggregate sum_g dz_l(g)^T a_{l-1}(g)   A = dz_l [rows][n_l], B = a_{l-1} [rows][n_{l-1}] of the groups' last
//                                            uploads, K = rows: both operands are read as they lie (MN-major:
//                                            the M / N index is the contiguous one), so no transposed copy of
//                                            an activation or error matrix is ever written
// (only the weights are kept in both orientations, by the conversion kernel).
//
// Kernels: persistent CTAs, one per SM; warp 0 = TMA producer
// (cp.async.bulk.tensor, 128-byte swizzle, mbarrier ring), warp 1 = MMA issuer
// (tcgen05.mma, cta_group::1, bf16 -> fp32 in TMEM, two accumulator slots),
// warps 2-9 = epilogue (tcgen05.ld, fused bias / ReLU / ReLU-mask, stores).  A group's
// minibatch is padded to a multiple of 128 rows, so an M tile never mixes
// groups and the stale-point weights of a tile are one slot of the bf16
// weight ring.  Every wait is bounded; a timeout raises the device error word.
#include "mlp_bf16.h"

#include <cuda.h>
#include <cuda_bf16.h>

namespace gcada {

namespace {

constexpr int BM = 128, BK = 64;  // M tile; K block (BK * 2 bytes = one 128-byte swizzle row)
constexpr int MAX_STAGES = 8;

enum { EPI_HIDDEN = 0, EPI_SCORES = 1, EPI_DA = 2, EPI_AGG = 3 };
enum { ZB_BATCH = 0, ZB_GROUP = 1, ZB_RING = 2 };

struct Bf16Impl {
  int Bp = 0;                   // rows per group padded to a multiple of 128
  long long slot_elems = 0;     // bf16 elements per weight-ring slot
  long long w_pos[MLP_MAX_LAYERS + 1] = {0};   // W_l   [n_l][ldk_l] inside a slot
  long long wt_pos[MLP_MAX_LAYERS + 1] = {0};  // W_l^T [n_{l-1}][ldn_l]
  long long bias_pos[MLP_MAX_LAYERS + 1] = {0};  // floats (bf16-rounded biases) inside the bias ring slot
  long long bias_slot = 0;
  int ld[MLP_MAX_LAYERS + 1] = {0};            // row stride (elements) of activation-like buffers of width n_l
  __nv_bfloat16* wb = nullptr;   // (D+1) slots
  float* bias = nullptr;         // (D+1) slots of rounded biases
  int* yb = nullptr;             // [G*Bp], -1 on padding rows
  float* scores = nullptr;       // [2][G*Bp][n_L]
  // Activations and back-propagated errors, row-major [entry][Bp][ld_l]: they are the operands of the next
  // product AND the factors of the weight gradients, dW_l(g) = dz[l](g)^T act[l-1](g).  Entries [0, 2G) are
  // two upload buffers per group (entry b*G + g): buffer cur[g] holds the factors of the group's last
  // upload, the other one receives the factors at theta^k; the selection flips cur[g] and thereby keeps the
  // upload.  Entries [2G, 3G) hold the stale point's matrices of this iteration (never kept).
  __nv_bfloat16* xb = nullptr;                          // [2][G][Bp][ld_0] (the features serve both points)
  __nv_bfloat16* act[MLP_MAX_LAYERS + 1] = {nullptr};   // [3][G][Bp][ld_l]
  __nv_bfloat16* dz[MLP_MAX_LAYERS + 1] = {nullptr};    // [3][G][Bp][ld_l]
  int nbias = 0;                                         // bias entries of all layers
  int bias_loc[MLP_MAX_LAYERS + 2] = {0};                // first entry of layer l in the compact bias arrays
  float* db = nullptr;           // [2][G][nbias] bias gradients, the same two buffers per group
  // column sums of dz_l over row blocks, written by the kernels that produce dz_l (the backward-data epilogue:
  // blocks of 128 rows; the loss-gradient kernel: blocks of 32 rows): [2][G][blocks][n_l]
  float* dbp[MLP_MAX_LAYERS + 1] = {nullptr};
  int dbp_blocks[MLP_MAX_LAYERS + 1] = {0};
  uint32_t* relu_bits[MLP_MAX_LAYERS + 1] = {nullptr};  // [2G][(n_l + 31) / 32][Bp]: a_l > 0, l = 1..L-1
  // differences between the two points, row-major [G*Bp][ld_l] (see bf16_gram_kernel)
  __nv_bfloat16* dE[MLP_MAX_LAYERS + 1] = {nullptr};  // dz_l(theta^k) - dz_l(stale), l = 1..L
  __nv_bfloat16* dF[MLP_MAX_LAYERS + 1] = {nullptr};  // a_l(theta^k) - a_l(stale),  l = 1..L-1
  int gram_part_base[MLP_MAX_LAYERS + 1] = {0};
  CUtensorMap tm_dE[MLP_MAX_LAYERS + 1], tm_dF[MLP_MAX_LAYERS + 1];
  int dw_part_base[MLP_MAX_LAYERS + 1] = {0}, bias_part_base[MLP_MAX_LAYERS + 1] = {0};
  int n_parts = 0;               // innovation-norm partial sums per group
  CUtensorMap tm_fwd_a[MLP_MAX_LAYERS + 1], tm_fwd_b[MLP_MAX_LAYERS + 1];
  CUtensorMap tm_da_a[MLP_MAX_LAYERS + 1], tm_da_b[MLP_MAX_LAYERS + 1];
  CUtensorMap tm_dw_a[MLP_MAX_LAYERS + 1], tm_dw_b[MLP_MAX_LAYERS + 1];  // dz[l] / act[l-1] in boxes of 64 rows x 64 columns (MN-major operands)
};

struct GemmB {
  int M, N, K;
  int a_shared;      // 1: operand A is the same for both points (the gathered features)
  int zb_mode;       // ZB_*
  int epi;           // EPI_*
  int stages;
  int k_batched;     // 1: one output [M][N]; K runs over the batch entries of both operands (kpg K blocks each)
  int kpg, n_batch;
                     // k_batched products maintain the aggregate of Eq. (3) from the groups' upload buffers
                     // (run after the selection has flipped cur[] of the selected groups).  When fewer than half
                     // of the groups are selected, K runs over the SELECTED groups twice - their replaced
                     // uploads (buffer 1 - cur[g]) with the A operand negated, then their new ones (buffer
                     // cur[g]) - and the result is added to the output.  Otherwise, and every AGG_REFRESH-th
                     // iteration (so that rounding cannot pile up), K runs over every group's buffer cur[g] and
                     // the sum is written anew.
  // epilogue operands
  __nv_bfloat16* out;    // row-major bf16 [entry][M][ldo], entry = factor_entry(point, group)
  float* out_f32;        // EPI_SCORES: [z][M][N]
  uint32_t* relu_bits;        // one bit per hidden unit: the (bf16-rounded) activation is positive.  Layout
                              // [z][N / 32 rounded up][M] words (rows of a word position are contiguous).
                              // EPI_HIDDEN writes them, EPI_DA of the same layer reads them as the ReLU derivative
  int nw;                     // words per row: (N + 31) / 32
  int n_entries;              // entries of `out` (checked by the debug library)
  int point;                  // forward / backward-data products: the point this launch computes (0: theta^k,
                              // 1: the stale iterates).  One launch per point: all tiles of the first share one
                              // slot of the weight ring, which then stays in L2; the second walks the groups by
                              // age, one stale slot after the other; interleaving the two kept two slots (64 MB
                              // at 4096 x 4096) live at a time and every wave of CTAs fetched both from HBM again
  float* colsum;              // EPI_DA: [z][tiles_m][N] column sums of the (bf16-rounded) output tile, or null
  __nv_bfloat16* diff;        // EPI_HIDDEN / EPI_DA, or null: row-major [G][M][ldo]; the stale-point tile also
                              // writes (fresh output - its own output) here, rounded to bf16: the small
                              // factors of the innovation's rank-one terms (see bf16_gram_kernel)
  const float* bias_ring;     // EPI_HIDDEN / EPI_SCORES: rounded biases, ring slots of bias_slot floats
  long long bias_slot, bias_pos;
  long long ldo;
  long long z_stride_out;
  long long c_off, ldc;       // EPI_AGG: offset inside out_f32 (a p-vector), row stride
};

// ----------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait of the single-thread producer / MMA loops: the hardware parks the thread for at most about a
// microsecond per try (suspend-time hint) and wakes it when the phase flips, so a waiting thread issues next
// to nothing (busy polling with test_wait reacted no faster in practice and cost the step ~0.5 % under the
// power cap).  2^20 tries: about a second before the wait is given up.
__device__ __forceinline__ bool mbar_spin_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < (1u << 20); ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(1000u)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  // no back-off for the first polls: a sleeping producer or MMA thread adds its wake-up time to every
  // pipeline step, which dominates when a tile has only a few steps
  for (uint32_t it = 0; it < (1u << 24); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > (1u << 16)) __nanosleep(128);
  }
  return false;
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_c, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      :
      : "r"(tmem_c), "l"(da), "l"(db), "r"(idesc), "r"(accum), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// Issues the load only; the registers are valid after tc_ld_wait().
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes
// (64 bf16) under the 128-byte swizzle: 8-row atoms of 1024 bytes, start
// address in 16-byte units, leading offset 1, stride offset 1024 bytes,
// descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// The same for an MN-major tile (the M / N index contiguous): 64 x 64 blocks as the copies deliver them, i.e.
// 64 K-rows of 128 bytes (64 M / N values) under the 128-byte swizzle.  Atoms are 8 K-rows x 128 bytes; the
// stride offset is the distance between K-groups of 8 rows (1024 bytes), the leading offset the distance
// between blocks of 64 M / N values (one whole block: 8192 bytes).  One MMA (K = 16) spans two K-groups.
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(8192 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
constexpr int MN_BLK = 64 * BK * 2;  // bytes of one 64 x 64 block
// Instruction descriptor: fp32 accumulator, bf16 A and B, N >> 3 at bit 17, M >> 4 at bit 24; bits 15 / 16
// set = A / B is MN-major (clear = K-major).

__device__ __forceinline__ int ring_slot(const Params& P, int g, int q, long long k) {
  long long j = q == 0 ? k : k - P.tau[g];
  if (j < k - P.D) j = k - P.D;  // ages beyond D only arise under forced masks: oldest kept iterate
  if (j < 0) j = 0;
  return (int)(j % (P.D + 1));
}

// Upload buffer that receives group g's factors at theta^k.  Normally the gradients come before the
// selection: the buffer that does not hold the last upload.  When the selection came first (printed rule,
// only the selected groups compute) cur[g] has already been flipped and names the buffer to fill.
__device__ __forceinline__ int fresh_buf(const Params& P, int g) { return P.skip_unselected ? P.cur[g] : 1 - P.cur[g]; }
// Batch entry of (point q, group g) in the factor arrays.
__device__ __forceinline__ int factor_entry(const Params& P, int g, int q) {
  return q == 0 ? fresh_buf(P, g) * P.G + g : 2 * P.G + g;
}

// ----------------------------------------------------------------- GEMM (forward and backward-data products)
// Persistent: one CTA per SM walks 128 x 256 output tiles (N fastest, so that
// the CTAs running together share operand tiles in L2); tensor memory holds
// two 256-column accumulators, so the eight epilogue warps drain tile i while
// the producer and the MMA warp work on tile i+1.  A forward / backward-data
// product is two launches, theta^k for all groups and then the stale iterates
// with the groups taken in order of age (GemmB::point).
constexpr int AGG_REFRESH = 16;  // the aggregate is recomputed in full at least every so many iterations (a replaced
                                 // pair of uploads moves it by ~1e-7 of its norm from the recomputed value)
constexpr int GN = 256;                                  // N tile of this kernel (the epilogue assumes 2 x 4 chunks of 32)
constexpr int G_STAGE_BYTES = (BM + GN) * BK * 2;        // 48 KiB
constexpr int G_STAGES = 4;
constexpr int G_EPI_WARPS = 8;
constexpr int G_THREADS = 64 + 32 * G_EPI_WARPS;
constexpr int TRP = 20;  // words per row of a transposition tile: rows 16-byte aligned, and the eight lanes of a
                        // 128-bit access phase (row stride 20 words) fall on 32 different banks
constexpr int G_TR_BYTES = G_EPI_WARPS * 32 * TRP * 4;  // per-warp transposition tiles of the epilogue
constexpr int G_CS_BYTES = 2 * 4 * GN * 4;             // column sums of a tile per 32-row quadrant, two tiles in flight
constexpr int G_BIAS_BYTES = G_EPI_WARPS * (GN / 2) * 4;  // each epilogue warp's 128 bias values of the current tile
constexpr int G_SMEM_BYTES = G_STAGES * G_STAGE_BYTES + 1024 + G_TR_BYTES + G_CS_BYTES + G_BIAS_BYTES;
constexpr uint32_t IDESC_G = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
constexpr uint32_t IDESC_MN = IDESC_G | (1u << 15) | (1u << 16);

// Difference of two packed bf16 pairs: each half is the exact difference rounded once to nearest-even bf16.
__device__ __forceinline__ uint32_t bf16x2_sub(uint32_t x, uint32_t y) {
  uint32_t r;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
  return r;
}
// (lo, hi) -> packed bf16 pair, round to nearest even; the second form also replaces negative values by zero.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t pack_relu_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(G_THREADS, 1) bf16_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                 const __grid_constant__ CUtensorMap tmB,
                                                                 const Params P, const GemmB a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ uint64_t full_bar[G_STAGES], empty_bar[G_STAGES], tfull_bar[2], tempty_bar[2];
  __shared__ uint32_t tmem_base_sm;
  unsigned char* tiles = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // aggregate passes: which batch entries, with which sign, written or added (the same in every thread of the grid)
  int n_batch = a.n_batch;
  int n_sel = 0;
  bool listed = false;
  if (a.k_batched) {
    n_sel = P.sel_count[0];
    const bool refresh = 2 * n_sel >= P.G || (P.st->k % AGG_REFRESH) == 0;
    if (!refresh) {
      if (n_sel == 0) return;  // no upload: the aggregate stands
      listed = true;
      n_batch = 2 * n_sel;     // the replaced uploads (negated), then the new ones
    }
  }
  const bool accumulate = listed;
  const int nkb = a.k_batched ? a.kpg * n_batch : (a.K + BK - 1) / BK;
  const int tiles_n = (a.N + GN - 1) / GN, tiles_m = (a.M + BM - 1) / BM;
  // batch entries: (point, group) for every group, or - when only the selected groups compute (rule PS:
  // Algorithm 1's own order, the selection is already known) - the selected groups at theta^k only
  const int n_grp = P.skip_unselected ? P.sel_count[0] : P.G;
  // A CTA walks units (column tile, row tile, group) of the launch's point.
  const int total_units = tiles_n * tiles_m * (a.k_batched ? 1 : n_grp);
  const int n_local = (int)blockIdx.x < total_units ? (total_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const long long k_it = P.st->k;

  if (threadIdx.x == 0) {
    for (int s = 0; s < G_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], G_EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sm)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sm;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int i = 0; i < n_local && ok; ++i) {
        const int u = blockIdx.x + i * gridDim.x, q = a.k_batched ? 0 : a.point;
        const int nt = u % tiles_n, mt = (u / tiles_n) % tiles_m, gi = u / (tiles_n * tiles_m);
        const int g = a.k_batched ? 0 : (P.skip_unselected ? P.sel_list[gi] : P.age_order[gi]);
        const int z = q * P.G + g;
        int zA = 0, zB = 0, ent = 0;
        // entry e of a k_batched product: every group's last upload, or (listed) the selected groups' replaced
        // uploads followed by their new ones
        auto agg_entry = [&](int e) {
          if (!listed) return (int)P.cur[e] * P.G + e;
          const int gs = P.sel_list[e < n_sel ? e : e - n_sel];
          return (e < n_sel ? 1 - (int)P.cur[gs] : (int)P.cur[gs]) * P.G + gs;
        };
        if (a.k_batched) {
          zA = zB = agg_entry(0);
        } else {
          zA = factor_entry(P, g, a.a_shared ? 0 : q);
          zB = a.zb_mode == ZB_RING ? ring_slot(P, g, q, k_it) : (a.zb_mode == ZB_GROUP ? g : z);
        }
        int kin = 0;  // K block inside the current batch entry (k_batched)
        for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
          const int s = it % G_STAGES;
          ok = mbar_spin_bounded(&empty_bar[s], (uint32_t)(((it / G_STAGES) & 1) ^ 1));
          if (!ok) break;
          unsigned char* sa = tiles + (size_t)s * G_STAGE_BYTES;
          mbar_expect_tx(&full_bar[s], G_STAGE_BYTES);
          const int kc = (a.k_batched ? kin : kb) * BK;
          if (a.k_batched) {  // MN-major: 64-row x 64-column blocks of the row-major factors, two for A, four for B
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_3d(sa + j * MN_BLK, &tmA, mt * BM + j * 64, kc, zA, &full_bar[s]);
#pragma unroll
            for (int j = 0; j < GN / 64; ++j)
              tma_load_3d(sa + BM * BK * 2 + j * MN_BLK, &tmB, nt * GN + j * 64, kc, zB, &full_bar[s]);
          } else {
            tma_load_3d(sa, &tmA, kc, mt * BM, zA, &full_bar[s]);
            tma_load_3d(sa + BM * BK * 2, &tmB, kc, nt * GN, zB, &full_bar[s]);
          }
          if (a.k_batched && ++kin == a.kpg) {
            kin = 0;
            ++ent;
            if (ent < n_batch) zA = zB = agg_entry(ent);
          }
        }
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int i = 0; i < n_local && ok; ++i) {
        const int slot = i & 1;
        ok = mbar_spin_bounded(&tempty_bar[slot], (uint32_t)(((i >> 1) & 1) ^ 1));
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
          const int s = it % G_STAGES;
          ok = mbar_spin_bounded(&full_bar[s], (uint32_t)((it / G_STAGES) & 1));
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(tiles + (size_t)s * G_STAGE_BYTES);
          const bool negate = listed && kb < a.kpg * n_sel;  // the replaced uploads leave the sum (A negated, bit 13)
          if (a.k_batched) {
            const uint64_t da = make_desc_mn(sa), db = make_desc_mn(sa + BM * BK * 2);
            const uint32_t idesc = negate ? (IDESC_MN | (1u << 13)) : IDESC_MN;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)  // 16 K-rows = two K-groups of 1024 bytes = 128 descriptor units
              tc_mma_bf16(tmem_base + (uint32_t)(slot * GN), da + (uint64_t)(kk * 128), db + (uint64_t)(kk * 128), idesc,
                          (kb | kk) != 0 ? 1u : 0u);
          } else {
            const uint64_t da = make_desc(sa), db = make_desc(sa + BM * BK * 2);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)  // 16 bf16 = 32 bytes = 2 descriptor units per MMA
              tc_mma_bf16(tmem_base + (uint32_t)(slot * GN), da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), IDESC_G,
                          (kb | kk) != 0 ? 1u : 0u);
          }
          tc_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(&tfull_bar[slot]);
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else {
    // epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31; the two warps of a quadrant split the columns
    const int ew = warp - 2;
    const int quad = warp & 3;
    const int half = ew >> 2;
    uint32_t* tr = reinterpret_cast<uint32_t*>(tiles + (size_t)G_STAGES * G_STAGE_BYTES) + ew * (32 * TRP);
    float* cs_all = reinterpret_cast<float*>(tiles + (size_t)G_STAGES * G_STAGE_BYTES + G_TR_BYTES);  // [2][4][GN]
    float* bias_w = reinterpret_cast<float*>(tiles + (size_t)G_STAGES * G_STAGE_BYTES + G_TR_BYTES + G_CS_BYTES) + ew * (GN / 2);
    bool ok = true;
    for (int i = 0; i < n_local; ++i) {
      const int slot = i & 1;
      const int u = blockIdx.x + i * gridDim.x, q = a.k_batched ? 0 : a.point;
      const int nt = u % tiles_n, mt = (u / tiles_n) % tiles_m, gi = u / (tiles_n * tiles_m);
      const int g = a.k_batched ? 0 : (P.skip_unselected ? P.sel_list[gi] : P.age_order[gi]);
      const int z = q * P.G + g;
      const bool write_diff = q == 1 && a.diff != nullptr;
      const int zT = a.k_batched ? 0 : factor_entry(P, g, q);  // entry of the output in its factor array
      const int zF = a.k_batched ? 0 : factor_entry(P, g, 0);  // entry of the fresh point's output
      // (debug library) the entry of the factor array this tile stores to
      const bool entry_ok = a.k_batched || a.epi == EPI_SCORES || GCADA_INDEX_OK(P.st, zT, a.n_entries, CHK_FACTOR);
      const int m = mt * BM + quad * 32 + lane;
      const int n0 = nt * GN;
      // EPI_DA: the ReLU derivative of this thread's row does not depend on the accumulator: its four words
      // (one bit per column of the four chunks) are fetched while the MMAs of the tile are still running
      uint32_t mbits[4] = {0u, 0u, 0u, 0u};
      if (a.epi == EPI_DA && m < a.M) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const int nc = n0 + half * (GN / 2) + ch * 32;
          if (nc < a.N) mbits[ch] = a.relu_bits[((long long)z * a.nw + (nc >> 5)) * a.M + m];
        }
      }
      if (ok) {
        ok = mbar_wait_bounded(&tfull_bar[slot], (uint32_t)((i >> 1) & 1));
        ok = __all_sync(0xffffffffu, ok);
      }
      if (!ok) {  // (the barrier below is still taken: the other epilogue warps may be waiting at it)
        if (a.colsum) asm volatile("bar.sync 1, %0;" ::"n"(32 * G_EPI_WARPS) : "memory");
        continue;
      }
      tc_fence_after();
      if (a.epi == EPI_HIDDEN || a.epi == EPI_SCORES) {
        // the 128 biases of this warp's columns, once per tile, into the warp's own shared-memory strip (read
        // back as broadcasts); zeros beyond the matrix
        const float* bias = a.bias_ring + (long long)ring_slot(P, g, q, k_it) * a.bias_slot + a.bias_pos;
        const int col = n0 + half * (GN / 2) + lane * 4;
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col + 3 < a.N) {
          b4 = *reinterpret_cast<const float4*>(bias + col);
        } else {
          if (col < a.N) b4.x = bias[col];
          if (col + 1 < a.N) b4.y = bias[col + 1];
          if (col + 2 < a.N) b4.z = bias[col + 2];
        }
        __syncwarp();
        *reinterpret_cast<float4*>(bias_w + lane * 4) = b4;
        __syncwarp();
      }
      const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * GN);
      // one 32-column chunk of this thread's row
      auto chunk = [&](const uint32_t (&v)[32], int c) {
        const int nc = n0 + c;
        if (nc >= a.N || !entry_ok) return;  // uniform across the warp
        const bool row_ok = m < a.M;
        const bool full = nc + 32 <= a.N;
        const float* bw = bias_w + (c - half * (GN / 2));  // this chunk's biases (EPI_HIDDEN / EPI_SCORES)
        // The stale point's tile also writes fresh - stale: the fresh point's values (written by the launch
        // before this one) at the places this thread will store to are fetched now, so that their latency
        // is covered by the conversion work
        const long long off0 = (long long)(mt * BM + quad * 32) * a.ldo + nc;
        const bool fast = full && a.M - (mt * BM + quad * 32) >= 32;
        uint4 frv[4] = {};
        if (write_diff && fast) {
#pragma unroll
          for (int it = 0; it < 4; ++it)
            frv[it] = *reinterpret_cast<const uint4*>(a.out + (long long)zF * a.z_stride_out + off0 +
                                                      (long long)(it * 8 + (lane >> 2)) * a.ldo + (lane & 3) * 8);
        }
        if (a.epi == EPI_AGG) {  // a block of the aggregated weight gradient, straight into the p-vector
          float* dst = a.out_f32 + a.c_off + (long long)m * a.ldc + nc;
          if (row_ok) {
            if (full && ((a.c_off | a.ldc) & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                float4 o4 = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                                        __uint_as_float(v[j + 3]));
                if (accumulate) {
                  const float4 c4 = *reinterpret_cast<const float4*>(dst + j);
                  o4 = make_float4(c4.x + o4.x, c4.y + o4.y, c4.z + o4.z, c4.w + o4.w);
                }
                *reinterpret_cast<float4*>(dst + j) = o4;
              }
            } else {
              for (int j = 0; j < 32 && nc + j < a.N; ++j) dst[j] = (accumulate ? dst[j] : 0.f) + __uint_as_float(v[j]);
            }
          }
        } else if (a.epi == EPI_SCORES) {
          float* dst = a.out_f32 + ((long long)z * a.M + m) * a.N + nc;
          if (row_ok) {
            if (full && (a.N & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(dst + j) =
                    make_float4(__uint_as_float(v[j]) + bw[j], __uint_as_float(v[j + 1]) + bw[j + 1],
                                __uint_as_float(v[j + 2]) + bw[j + 2], __uint_as_float(v[j + 3]) + bw[j + 3]);
            } else {
              for (int j = 0; j < 32 && nc + j < a.N; ++j) dst[j] = __uint_as_float(v[j]) + bw[j];
            }
          }
        } else {
          // bf16 pairs of this thread's row
          float f[32];
          uint32_t h[16];
          if (a.epi == EPI_HIDDEN) {  // bias, ReLU and rounding (the conversion clamps at zero)
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 b4 = *reinterpret_cast<const float4*>(bw + j);
              f[j] = __uint_as_float(v[j]) + b4.x;
              f[j + 1] = __uint_as_float(v[j + 1]) + b4.y;
              f[j + 2] = __uint_as_float(v[j + 2]) + b4.z;
              f[j + 3] = __uint_as_float(v[j + 3]) + b4.w;
              h[j >> 1] = pack_relu_bf16x2(f[j], f[j + 1]);
              h[(j >> 1) + 1] = pack_relu_bf16x2(f[j + 2], f[j + 3]);
            }
          } else {  // EPI_DA: ReLU derivative of the layer below (bits of rows / columns outside the matrix are 0)
            const uint32_t bits = mbits[(c - half * (GN / 2)) >> 5];
#pragma unroll
            for (int j = 0; j < 32; ++j) f[j] = ((bits >> j) & 1u) ? __uint_as_float(v[j]) : 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) h[j >> 1] = pack_bf16x2(f[j], f[j + 1]);
          }
          if (a.epi == EPI_HIDDEN && row_ok) {
            // After the clamp a value is positive iff its 16 bits are non-zero (a NaN counts as positive, as
            // before), i.e. iff adding 0x7FFF sets bit 15 (no half exceeds 0x7FFF, so nothing carries over).  The
            // four flag bytes of two words are gathered into one word and a multiplication moves their top bits
            // next to each other: (a 2^7 + b 2^15 + c 2^23 + d 2^31) * (2^21 + 2^14 + 2^7 + 1) has a, b, c, d at
            // bits 28..31 and every other product below bit 24 or beyond bit 31.
            uint32_t bits = 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint32_t s0 = h[2 * k] + 0x7FFF7FFFu, s1 = h[2 * k + 1] + 0x7FFF7FFFu;
              const uint32_t x = __byte_perm(s0, s1, 0x7531) & 0x80808080u;
              bits |= ((x * 0x00204081u) >> 28) << (4 * k);
            }
            a.relu_bits[((long long)z * a.nw + (nc >> 5)) * a.M + m] = bits;
          }
          // The warp's 32 x 32 block goes through shared memory (rows of 17 words), so that every store
          // instruction writes whole 32-byte sectors: a lane that stored 16 bytes of its own row touched half
          // a sector, and the L2 counted twice the sectors the data needs.
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<uint4*>(tr + lane * TRP + j) = make_uint4(h[j], h[j + 1], h[j + 2], h[j + 3]);
          __syncwarp();
          if (a.colsum) {
            // column `lane` of the warp's 32 x 32 block summed over its rows in row order (the rounded values:
            // what the bias gradient is the column sum of); rows and columns outside the matrix hold zeros
            float csum = 0.f;
#pragma unroll
            for (int r = 0; r < 32; ++r) {
              const uint32_t wd = tr[r * TRP + (lane >> 1)];
              csum += __uint_as_float((lane & 1) ? (wd & 0xFFFF0000u) : (wd << 16));
            }
            cs_all[((i & 1) * 4 + quad) * GN + c + lane] = csum;
          }
          if (fast) {
            // row-major copy: lanes 4r..4r+3 write the 64 bytes of row r, eight rows per instruction
            __nv_bfloat16* dst0 = a.out + (long long)zT * a.z_stride_out + off0;
#pragma unroll
            for (int it = 0; it < 4; ++it) {
              const int r = it * 8 + (lane >> 2), qd = lane & 3;
              const uint4 mine = *reinterpret_cast<const uint4*>(tr + r * TRP + qd * 4);
              *reinterpret_cast<uint4*>(dst0 + (long long)r * a.ldo + qd * 8) = mine;
              if (write_diff) {
                const uint4 fr = frv[it];
                *reinterpret_cast<uint4*>(a.diff + (long long)g * a.z_stride_out + off0 + (long long)r * a.ldo + qd * 8) =
                    make_uint4(bf16x2_sub(fr.x, mine.x), bf16x2_sub(fr.y, mine.y), bf16x2_sub(fr.z, mine.z),
                               bf16x2_sub(fr.w, mine.w));
              }
            }
            return;
          }
          if (row_ok) {
            __nv_bfloat16* dst = a.out + (long long)zT * a.z_stride_out + (long long)m * a.ldo + nc;
            const unsigned short* hv = reinterpret_cast<const unsigned short*>(h);  // the row's 32 rounded values
            unsigned short* dst16 = reinterpret_cast<unsigned short*>(dst);
            for (int j = 0; j < 32 && nc + j < a.N; ++j) dst16[j] = hv[j];
            if (write_diff) {
              const unsigned short* fr =
                  reinterpret_cast<const unsigned short*>(a.out + (long long)zF * a.z_stride_out + (long long)m * a.ldo + nc);
              unsigned short* df =
                  reinterpret_cast<unsigned short*>(a.diff + (long long)g * a.z_stride_out + (long long)m * a.ldo + nc);
              for (int j = 0; j < 32 && nc + j < a.N; ++j)
                df[j] = (unsigned short)(bf16x2_sub((uint32_t)fr[j], (uint32_t)hv[j]) & 0xFFFFu);
            }
          }
        }
      };
      // The four chunks of this warp, software-pipelined: the tensor-memory load of the next chunk is in
      // flight while the current one is converted and stored (a load takes far longer than its issue).
      {
        const int cb = half * (GN / 2);
        uint32_t va[32], vb[32];
        tc_ld32_issue(tbase + (uint32_t)cb, va);
        tc_ld_wait();
        tc_ld32_issue(tbase + (uint32_t)(cb + 32), vb);
        chunk(va, cb);
        tc_ld_wait();
        tc_ld32_issue(tbase + (uint32_t)(cb + 64), va);
        chunk(vb, cb + 32);
        tc_ld_wait();
        tc_ld32_issue(tbase + (uint32_t)(cb + 96), vb);
        chunk(va, cb + 64);
        tc_ld_wait();
        chunk(vb, cb + 96);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[slot]);
      if (a.colsum) {
        // the tile's column sums: the four 32-row quadrants added in order, one column per epilogue thread.
        // The buffer alternates between tiles, so a warp that runs ahead writes the other half; it cannot
        // reach this half again before every warp has passed the next tile's barrier.
        asm volatile("bar.sync 1, %0;" ::"n"(32 * G_EPI_WARPS) : "memory");
        const int col = ew * 32 + lane;  // 0..255
        if (n0 + col < a.N) {
          const float* cs = cs_all + (size_t)(i & 1) * 4 * GN + col;
          a.colsum[((long long)z * tiles_m + mt) * a.N + n0 + col] = ((cs[0] + cs[GN]) + cs[2 * GN]) + cs[3 * GN];
        }
      }
    }
    if (!ok && lane == 0) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ----------------------------------------------------------------- innovation norm of the weight gradients
// ||dW_l(theta^k) - dW_l(stale)||_F^2 of one group without forming either gradient.  With r over the group's
// minibatch rows, dz / a the back-propagated errors / input activations of layer l at theta^k and a tilde for
// the stale point,
//     dW - dW~ = sum_r dz_r (x) a_r - dz~_r (x) a~_r = sum_r (dz_r - dz~_r) (x) a_r + dz~_r (x) (a_r - a~_r),
// a sum of 2B rank-one terms u_k (x) v_k in which one factor of every term is a small difference:
//     U = [E; dz~],  V = [a; F],  E = dz - dz~,  F = a - a~   (E, F formed exactly from the bf16 values and
//                                                              rounded to bf16 by the kernels that produce dz, a).
// Then ||sum_k u_k (x) v_k||_F^2 = sum_{k,k'} (u_k . u_k') (v_k . v_k') = <U U^T, V V^T>: two Gram matrices of
// 2B x 2B entries (K = n_l and n_{l-1}) and their elementwise product summed.  Every term is of the size of
// the innovation itself, so nothing cancels (Grams of [dz; -dz~] and [a; a~] would sum terms of the size of
// the gradients to a result of the size of the innovation).  Compared with forming dW - dW~ tile by tile the
// tensor cores do 2 (2B)^2 (n_l + n_{l-1}) instead of 4 B n_l n_{l-1} flops and, decisive here, only 2 (2B)^2
// accumulators per group and layer are read from tensor memory instead of n_l n_{l-1}: the direct pass was
// bound by draining its accumulators.  Layer 1 has a = a~ (the features), so U = E, V = x.
//
// Unit = (group, 128-row block mi, column block nj of up to 256) of the two Grams: accumulator columns
// [0, BN) receive U_mi U_nj^T, columns [BN, 2 BN) V_mi V_nj^T; the epilogue multiplies them elementwise and
// adds up; one partial sum per unit goes to lhs_part.  Operand blocks of 128 rows come from up to two arrays
// per matrix (part 0 / part 1) through their own tensor maps.
struct GramArgs {
  int parts;         // 1: U = E_l, V = a_{l-1} (layer 1); 2: U = [E_l; dz~_l], V = [a_{l-1}; F_{l-1}]
  int nb;            // 128-row blocks per part (padded minibatch rows / 128)
  int BN;            // column block of the Grams: min(parts * nb * 128, 256)
  int Ku, Kv;        // n_l, n_{l-1}
  int part_base, n_parts;
};

__global__ void __launch_bounds__(G_THREADS, 1) bf16_gram_kernel(const __grid_constant__ CUtensorMap tmU0,
                                                                 const __grid_constant__ CUtensorMap tmU1,
                                                                 const __grid_constant__ CUtensorMap tmV0,
                                                                 const __grid_constant__ CUtensorMap tmV1,
                                                                 const Params P, const GramArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], tfull_bar, tempty_bar;
  __shared__ uint32_t tmem_base_sm;
  __shared__ double norm_sm[G_EPI_WARPS];
  unsigned char* tiles = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int RB = a.parts * a.nb;             // 128-row blocks of U and V
  const int bpn = a.BN / BM;                 // row blocks per column block
  const int tiles_nj = RB / bpn;
  const int units_per_group = RB * tiles_nj;
  const int total_units = units_per_group * P.G;
  const int nku = (a.Ku + BK - 1) / BK, nkv = (a.Kv + BK - 1) / BK;
  // The 128 rows of the A operand are rows of the same matrix as the B operand's: when they lie inside the B
  // tile (always, if one column block covers the whole Gram) they are not fetched a second time and the
  // stages shrink to the B tile, which makes the ring deeper.
  const bool always_inside = tiles_nj == 1;
  const int stage_bytes = (always_inside ? a.BN : BM + a.BN) * BK * 2;
  const int stages = (G_STAGES * G_STAGE_BYTES) / stage_bytes < MAX_STAGES ? (G_STAGES * G_STAGE_BYTES) / stage_bytes : MAX_STAGES;
  const int b_off = always_inside ? 0 : BM * BK * 2;  // where the B tile starts inside a stage
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&tfull_bar, 1);
    mbar_init(&tempty_bar, G_EPI_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sm)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sm;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const int g = u / units_per_group, r = u - g * units_per_group;
        const int mi = r / tiles_nj, nj = r - mi * tiles_nj;
        const bool inside = mi / bpn == nj;  // the A rows are among the B rows of this unit
        for (int ph = 0; ph < 2 && ok; ++ph) {  // the U Gram, then the V Gram
          const int nk = ph == 0 ? nku : nkv;
          for (int kb = 0; kb < nk && ok; ++kb, ++it) {
            const int s = it % stages;
            ok = mbar_spin_bounded(&empty_bar[s], (uint32_t)(((it / stages) & 1) ^ 1));
            if (!ok) break;
            unsigned char* sa = tiles + (size_t)s * stage_bytes;
            mbar_expect_tx(&full_bar[s], (uint32_t)((inside ? a.BN : BM + a.BN) * BK * 2));
            // block b of the matrix: part b / nb, rows (b % nb) * 128 of the group's entry in that part's array
            auto load_block = [&](unsigned char* dst, int b) {
              const int part = b / a.nb, row = (b - part * a.nb) * BM;
              const CUtensorMap* tm = ph == 0 ? (part == 0 ? &tmU0 : &tmU1) : (part == 0 ? &tmV0 : &tmV1);
              // U: part 0 = E_l (entry g), part 1 = dz_l at the stale point; V: part 0 = a_{l-1} at theta^k (in
              // the group's upload buffer being filled), part 1 = F_{l-1} (entry g)
              const int z = ph == 0 ? (part == 1 ? factor_entry(P, g, 1) : g) : (part == 0 ? factor_entry(P, g, 0) : g);
              tma_load_3d(dst, tm, kb * BK, row, z, &full_bar[s]);
            };
            if (!inside) load_block(sa, mi);
            for (int j = 0; j < bpn; ++j) load_block(sa + b_off + (size_t)(j * BM) * BK * 2, nj * bpn + j);
          }
        }
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      int it = 0, i = 0;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++i) {
        const int r = u % units_per_group, mi = r / tiles_nj, nj = r - mi * tiles_nj;
        const bool inside = mi / bpn == nj;
        ok = mbar_spin_bounded(&tempty_bar, (uint32_t)((i & 1) ^ 1));  // the epilogue has drained the accumulators
        if (!ok) break;
        tc_fence_after();
        for (int ph = 0; ph < 2 && ok; ++ph) {
          const int nk = ph == 0 ? nku : nkv;
          for (int kb = 0; kb < nk && ok; ++kb, ++it) {
            const int s = it % stages;
            ok = mbar_spin_bounded(&full_bar[s], (uint32_t)((it / stages) & 1));
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = smem_u32(tiles + (size_t)s * stage_bytes);
            const uint64_t db = make_desc(sa + b_off);
            const uint64_t da = make_desc(inside ? sa + b_off + (uint32_t)((mi % bpn) * BM * BK * 2) : sa);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma_bf16(tmem_base + (uint32_t)(ph * a.BN), da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc,
                          (kb | kk) != 0 ? 1u : 0u);
            tc_commit(&empty_bar[s]);
          }
        }
        if (ok) tc_commit(&tfull_bar);
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else {
    const int ew = warp - 2, quad = warp & 3, half = ew >> 2;
    bool ok = true;
    int i = 0;
    for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++i) {
      const int g = u / units_per_group, r = u - g * units_per_group;
      double local = 0.0;
      if (ok) {
        ok = mbar_wait_bounded(&tfull_bar, (uint32_t)(i & 1));
        ok = __all_sync(0xffffffffu, ok);
      }
      if (ok) {
        tc_fence_after();
        const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int c0 = half * (a.BN / 2), c1 = c0 + a.BN / 2;  // this warp's columns of both accumulators
        for (int c = c0; c < c1; c += 32) {
          uint32_t gu[32], gv[32];
          tc_ld32_issue(tbase + (uint32_t)c, gu);
          tc_ld32_issue(tbase + (uint32_t)(a.BN + c), gv);
          tc_ld_wait();
          float part = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) part = fmaf(__uint_as_float(gu[j]), __uint_as_float(gv[j]), part);
          local += (double)part;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar);
      }
      // one partial sum per unit, the eight warps added in warp order (two barriers: the slots are reused)
      local = warp_sum(local);
      if (lane == 0) norm_sm[ew] = local;
      asm volatile("bar.sync 1, %0;" ::"n"(32 * G_EPI_WARPS) : "memory");
      if (ew == 0 && lane == 0) {
        double tsum = 0.0;
#pragma unroll
        for (int w = 0; w < G_EPI_WARPS; ++w) tsum += norm_sm[w];
        if (GCADA_INDEX_OK(P.st, (long long)g * a.n_parts + a.part_base + r, P.lim.lhs_parts, CHK_LHS_PART))
          P.lhs_part[(long long)g * a.n_parts + a.part_base + r] = tsum;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(32 * G_EPI_WARPS) : "memory");
    }
    if (!ok && lane == 0) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ----------------------------------------------------------------- weight gradients, both points in one CTA
// dW_l of one group at theta^k (accumulator 0) and at the stale iterate
// (accumulator 1), 128 x 256 tiles, written out: the inspection mode (every
// group's two gradients are kept; the epilogue also forms the squared norm of
// their difference, the tile's share of the left side of Eq. (9)) and the
// getters' rebuild of one group's last upload from its kept factors.  The
// production path never forms a group's weight gradient (bf16_gram_kernel).
//
// Persistent: one CTA per SM walks work units u = blockIdx.x, + gridDim.x,
// ...; a unit is one (group, 128-row block of W_l) and its tiles are all the
// column blocks.  The unit's A operand (128 columns of dz_l at both points, 2 x K x 128
// bf16, read MN-major as it lies) stays in shared memory for the whole unit and only B is streamed: with
// K = 128 the product is bound by operand traffic from L2, and this halves it.
// Tensor memory holds two accumulator pairs (2 x 256 columns) so that the
// eight epilogue warps drain tile i while the producer and the MMA warp work
// on tile i+1.  Rows reach global memory as full 128-byte lines through a
// per-warp staging tile.
struct DwArgs {
  int M, N, K;            // n_l, n_{l-1}, padded rows per group
  int b_shared;           // 1: operand B is the same for both points (the gathered features)
  int nkb;                // K blocks per point
  int stages;
  int tiles_m, tiles_n, total_tiles;
  long long c_off, ldc;   // position of W_l inside the gradient vector, row stride
  int part_base, n_parts; // this layer's first slot in lhs_part and slots per group
  int mode;               // DW_BOTH: both points in two accumulators, norm, gradients written for every group
                          //          (inspection mode; the production path takes the norm in bf16_gram_kernel);
                          // DW_ONE: one group's last uploaded gradient rebuilt from its kept factors and
                          //          written to out_row; used by getters
  int g_only;             // DW_ONE: the group
  float* out_row;         // DW_ONE: a p-vector
};
enum { DW_BOTH = 0, DW_ONE = 2 };

constexpr int DW_BN = 256;     // N tile: the MMA issue rate, not the tensor pipe, limits 128-wide instructions
constexpr int DW_PITCH = 36;   // floats per staged row (16-byte aligned, conflict-free 16-byte stores)
constexpr int DW_EPI_WARPS = 8;
constexpr int DW_THREADS = 64 + 32 * DW_EPI_WARPS;
constexpr int DW_STAGE_FLOATS = DW_EPI_WARPS * 32 * DW_PITCH;

__global__ void __launch_bounds__(DW_THREADS, 1) bf16_dw_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                const __grid_constant__ CUtensorMap tmB,
                                                                const Params P, const DwArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], tfull_bar[4], tempty_bar[4], afull_bar, aempty_bar;
  __shared__ uint32_t tmem_base_sm;
  __shared__ double norm_sm[4][DW_EPI_WARPS];
  // accumulator slots in the 512 columns of tensor memory: one pair, or two single accumulators
  const int n_slots = a.mode == DW_BOTH ? 1 : 2;
  const int slot_cols = a.mode == DW_BOTH ? 2 * DW_BN : DW_BN;
  constexpr int BLK = BM * BK * 2;      // one 128 x 64 bf16 block of A, 16 KiB
  constexpr int BBLK = DW_BN * BK * 2;  // one 256 x 64 bf16 block of B, 32 KiB
  unsigned char* a_res = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* tiles = a_res + (size_t)2 * a.nkb * BLK;  // ring of B blocks
  float* stage_all = reinterpret_cast<float*>(tiles + (size_t)a.stages * BBLK);
  const int n_units = a.mode == DW_ONE ? a.tiles_m : a.tiles_m * P.G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stages = a.stages;
  const int kb_per_tile = a.mode == DW_ONE ? a.nkb : 2 * a.nkb;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 4; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], DW_EPI_WARPS);
    }
    mbar_init(&afull_bar, 1);
    mbar_init(&aempty_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // all 512 columns: two slots of two fp32 accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sm)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sm;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int it = 0, ui = 0;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const int mt = u % a.tiles_m, g = a.mode == DW_ONE ? a.g_only : u / a.tiles_m;
        const int zone = (int)P.cur[g] * P.G + g;  // DW_ONE: the group's last upload
        // the unit's A blocks, once the MMAs of the previous unit have finished reading them
        ok = mbar_spin_bounded(&aempty_bar, (uint32_t)((ui & 1) ^ 1));
        if (!ok) break;
        mbar_expect_tx(&afull_bar, (uint32_t)(kb_per_tile * BLK));
        for (int j = 0; j < kb_per_tile; ++j) {
          const int q = j / a.nkb, kb = j - q * a.nkb;
          const int zA = a.mode == DW_ONE ? zone : factor_entry(P, g, q);
#pragma unroll
          for (int h = 0; h < BM / 64; ++h)  // MN-major: 64 batch rows x 64 columns of dz_l per block
            tma_load_3d(a_res + (size_t)j * BLK + h * MN_BLK, &tmA, mt * BM + h * 64, kb * BK, zA, &afull_bar);
        }
        ++ui;
        for (int nt = 0; nt < a.tiles_n && ok; ++nt) {
          for (int j = 0; j < kb_per_tile && ok; ++j, ++it) {
            const int q = j / a.nkb, kb = j - q * a.nkb;
            const int s = it % stages;
            ok = mbar_spin_bounded(&empty_bar[s], (uint32_t)(((it / stages) & 1) ^ 1));
            if (!ok) break;
            mbar_expect_tx(&full_bar[s], BBLK);
            const int zB = a.mode == DW_ONE ? zone : factor_entry(P, g, a.b_shared ? 0 : q);
#pragma unroll
            for (int h = 0; h < DW_BN / 64; ++h)
              tma_load_3d(tiles + (size_t)s * BBLK + h * MN_BLK, &tmB, nt * DW_BN + h * 64, kb * BK, zB, &full_bar[s]);
          }
        }
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      int it = 0, i = 0, ui = 0;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        ok = mbar_spin_bounded(&afull_bar, (uint32_t)(ui & 1));
        if (!ok) break;
        ++ui;
        for (int nt = 0; nt < a.tiles_n && ok; ++nt, ++i) {
          const int slot = i % n_slots;
          ok = mbar_spin_bounded(&tempty_bar[slot], (uint32_t)(((i / n_slots) & 1) ^ 1));  // epilogue has drained the slot
          if (!ok) break;
          tc_fence_after();
          for (int j = 0; j < kb_per_tile && ok; ++j, ++it) {
            const int q = j / a.nkb, kb = j - q * a.nkb;
            const int s = it % stages;
            ok = mbar_spin_bounded(&full_bar[s], (uint32_t)((it / stages) & 1));
            if (!ok) break;
            tc_fence_after();
            const uint64_t da = make_desc_mn(smem_u32(a_res + (size_t)j * BLK));
            const uint64_t db = make_desc_mn(smem_u32(tiles + (size_t)s * BBLK));
            const uint32_t idesc = IDESC_MN;
            const uint32_t acc_col = (uint32_t)(slot * slot_cols + (a.mode == DW_BOTH ? q * DW_BN : 0));
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma_bf16(tmem_base + acc_col, da + (uint64_t)(kk * 128), db + (uint64_t)(kk * 128), idesc,
                          (kb | kk) != 0 ? 1u : 0u);
            tc_commit(&empty_bar[s]);
          }
          if (ok) tc_commit(&tfull_bar[slot]);
        }
        if (ok) tc_commit(&aempty_bar);  // the A blocks may be overwritten once these MMAs are done
      }
      if (!ok) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
    }
  } else {
    const int ew = warp - 2;           // 0..7
    const int quad = warp & 3;         // TMEM lanes this warp may read
    const int half = ew >> 2;          // which 128 columns of the tile
    float* stg = stage_all + (size_t)ew * 32 * DW_PITCH;
    const bool vec_ok = ((a.c_off | a.ldc) & 3) == 0 && (P.p_pad & 3) == 0 &&
                        (reinterpret_cast<uintptr_t>(a.mode == DW_ONE ? a.out_row : P.gbuf) & 15) == 0;
    bool ok = true;
    int i = 0, ui = 0;
    for (int u = blockIdx.x; u < n_units; u += gridDim.x, ++ui) {
      const int mt = u % a.tiles_m, g = a.mode == DW_ONE ? a.g_only : u / a.tiles_m;
      double local = 0.0;  // this warp's share of the unit's squared innovation norm (all its column tiles)
      for (int nt = 0; nt < a.tiles_n; ++nt) {
      const int slot = i % n_slots;
      const int phase = (i / n_slots) & 1;
      ++i;
      if (ok) {
        ok = mbar_wait_bounded(&tfull_bar[slot], (uint32_t)phase);
        ok = __all_sync(0xffffffffu, ok);
      }
      if (ok) {
        tc_fence_after();
        // kept for inspection: the fresh gradient goes to the row that is not the last uploaded one
        float* fresh = (a.mode == DW_ONE ? a.out_row : fresh_row(P, g)) + a.c_off;
        float* stale = (a.mode == DW_BOTH && P.stale) ? P.stale + (long long)g * P.p_pad + a.c_off : nullptr;
        const int n_pass = stale ? 2 : 1;
        const int mrow = mt * BM + quad * 32;
        const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * slot_cols);
#pragma unroll 1
        for (int c = half * (DW_BN / 2); c < (half + 1) * (DW_BN / 2); c += 32) {
          const int nc = nt * DW_BN + c;
          if (nc >= a.N) break;
          uint32_t v0[32], v1[32];
          tc_ld32_issue(tbase + (uint32_t)c, v0);
          if (a.mode == DW_BOTH) tc_ld32_issue(tbase + (uint32_t)(DW_BN + c), v1);
          tc_ld_wait();  // one wait for both accumulators
          if (a.mode != DW_ONE) {
            const bool row_ok = mrow + lane < a.M;
            const bool interior = nc + 32 <= a.N;
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float d = __uint_as_float(v0[j]) - __uint_as_float(v1[j]);
              if (interior || nc + j < a.N) part += d * d;
            }
            if (row_ok) local += (double)part;
          }
          for (int pass = 0; pass < n_pass; ++pass) {
            const uint32_t* v = pass == 0 ? v0 : v1;
            float* out = pass == 0 ? fresh : stale;
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(stg + lane * DW_PITCH + j) =
                  make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                              __uint_as_float(v[j + 3]));
            __syncwarp();
            const int rr = lane >> 3, c4 = (lane & 7) * 4;  // lanes 8r..8r+7 write the 128 bytes of one row
#pragma unroll
            for (int r0 = 0; r0 < 32; r0 += 4) {
              const int r = r0 + rr;
              const int m = mrow + r;
              if (m >= a.M) continue;
              const float4 tv = *reinterpret_cast<const float4*>(stg + r * DW_PITCH + c4);
              float* dst = out + (long long)m * a.ldc + nc + c4;
              if (vec_ok && nc + c4 + 3 < a.N) {
                *reinterpret_cast<float4*>(dst) = tv;
              } else {
                const float tt[4] = {tv.x, tv.y, tv.z, tv.w};
                for (int e = 0; e < 4 && nc + c4 + e < a.N; ++e) dst[e] = tt[e];
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[slot]);  // this warp is done with the slot's tensor memory
      }
      }
      // one partial sum per unit (the eight warps in warp order); the buffer alternates between units, so a
      // warp that runs ahead cannot overwrite values that thread 0 of the first warp is still adding
      local = warp_sum(local);
      if (lane == 0) norm_sm[ui & 1][ew] = local;
      asm volatile("bar.sync 1, %0;" ::"n"(32 * DW_EPI_WARPS) : "memory");
      if (ew == 0 && lane == 0 && a.mode != DW_ONE) {
        double tsum = 0.0;
#pragma unroll
        for (int w = 0; w < DW_EPI_WARPS; ++w) tsum += norm_sm[ui & 1][w];
        if (GCADA_INDEX_OK(P.st, (long long)g * a.n_parts + a.part_base + mt, P.lim.lhs_parts, CHK_LHS_PART))
          P.lhs_part[(long long)g * a.n_parts + a.part_base + mt] = tsum;
      }
    }
    if (!ok && lane == 0) atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ----------------------------------------------------------------- weights -> bf16 (both orientations)
// grid (col tiles, row tiles, layer-1); 64 x 64 tiles through shared memory, two elements per thread so that a warp
// reads 256 bytes of a row and writes 128 bytes of a row in either orientation.
struct ConvArgs {
  int n_out[MLP_MAX_LAYERS + 1], n_in[MLP_MAX_LAYERS + 1];
  long long w_off[MLP_MAX_LAYERS + 1], b_off[MLP_MAX_LAYERS + 1];
  long long w_pos[MLP_MAX_LAYERS + 1], wt_pos[MLP_MAX_LAYERS + 1], bias_pos[MLP_MAX_LAYERS + 1];
  int ldk[MLP_MAX_LAYERS + 1], ldn[MLP_MAX_LAYERS + 1];
  long long slot_elems, bias_slot;
};

__global__ void __launch_bounds__(256) bf16_convert_kernel(const Params P, const ConvArgs a, __nv_bfloat16* wb,
                                                           float* bias) {
  __shared__ float tile[64][65];
  const int l = blockIdx.z + 1;
  const int no = a.n_out[l], ni = a.n_in[l];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  if (r0 >= no || c0 >= ni) return;
  const long long k = P.st->k;
  const int slot = (int)(k % (P.D + 1));
  const float* th = P.theta_ring + (long long)slot * P.p_pad;
  __nv_bfloat16* W = wb + (long long)slot * a.slot_elems + a.w_pos[l];
  __nv_bfloat16* WT = wb + (long long)slot * a.slot_elems + a.wt_pos[l];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const bool pair_ok = ((a.w_off[l] | (long long)ni) & 1) == 0;  // 8-byte loads of the fp32 master weights
  for (int i = ty; i < 64; i += 8) {
    const int r = r0 + i, c = c0 + 2 * tx;
    float v0 = 0.f, v1 = 0.f;
    if (r < no) {
      const float* src = th + a.w_off[l] + (long long)r * ni + c;
      if (pair_ok && c + 1 < ni) {
        const float2 t = *reinterpret_cast<const float2*>(src);
        v0 = t.x;
        v1 = t.y;
      } else {
        if (c < ni) v0 = src[0];
        if (c + 1 < ni) v1 = src[1];
      }
      __nv_bfloat16* dst = W + (long long)r * a.ldk[l] + c;  // (even leading dimension, even c: 4-byte aligned)
      if (c + 1 < ni)
        *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(v0, v1);
      else if (c < ni)
        dst[0] = __float2bfloat16_rn(v0);
    }
    tile[i][2 * tx] = v0;
    tile[i][2 * tx + 1] = v1;
  }
  __syncthreads();
  for (int i = ty; i < 64; i += 8) {
    const int c = c0 + i, r = r0 + 2 * tx;
    if (c < ni) {
      __nv_bfloat16* dst = WT + (long long)c * a.ldn[l] + r;
      if (r + 1 < no)
        *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(tile[2 * tx][i], tile[2 * tx + 1][i]);
      else if (r < no)
        dst[0] = __float2bfloat16_rn(tile[2 * tx][i]);
    }
  }
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    float* bo = bias + (long long)slot * a.bias_slot + a.bias_pos[l];
    for (int n = threadIdx.x; n < no; n += 256) bo[n] = __bfloat162float(__float2bfloat16_rn(th[a.b_off[l] + n]));
  }
  // One warp of one block also lists the groups by age (stable; ages beyond D, which only forced masks
  // produce, count as D + 1): groups of equal age read the same slot of the weight ring at the stale point,
  // and the products schedule their tiles in this order so that the CTAs running together touch few slots.
  // The order has no influence on any result.
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x < 32) {
    const int lane = threadIdx.x, G = P.G, chunks = (G + 31) / 32;
    if ((long long)(P.D + 1) * chunks <= 8192) {
      int base = 0;
      for (int age = 1; age <= P.D + 1; ++age) {
        for (int c = 0; c < chunks; ++c) {
          const int g = c * 32 + lane;
          int t = g < G ? P.tau[g] : 0;
          if (t > P.D + 1) t = P.D + 1;
          if (t < 1 && g < G) t = 1;
          const unsigned int m = __ballot_sync(0xffffffffu, t == age);
          if (t == age) P.age_order[base + __popc(m & ((1u << lane) - 1u))] = g;
          base += __popc(m);
        }
      }
    } else {
      for (int g = lane; g < G; g += 32) P.age_order[g] = g;
    }
  }
}

// ----------------------------------------------------------------- gather
// Block = 32 consecutive minibatch rows of one group, copied with 16-byte loads and stores into the group's
// upload buffer that receives this iteration's factors.
// Inside a chain of captured iterations (P.pdl) the kernel runs beside the previous iteration's update kernel:
// the draw does not depend on the iterate (Section II-A), the iteration number comes from the chain's start,
// and neither cur[] nor the buffer written here is touched by the update.  It waits for the update at its end,
// so that its completion implies the update's.
__global__ void __launch_bounds__(256) bf16_gather_kernel(const Params P, __nv_bfloat16* xb, int* yb, int d, int ld0,
                                                          int Bp) {
  __shared__ long long rows_sm[32];
  const int g = blockIdx.y, rb = blockIdx.x * 32;
  const int tid = threadIdx.x;
  const bool early = P.pdl != 0 && !P.skip_unselected;
  pdl_launch_dependents();
  if (!early) pdl_wait();
  const uint32_t k32 = (uint32_t)(early ? P.st->k_chain + P.k_off : P.st->k);
  if (P.skip_unselected && !P.mask_cur[g]) return;
  const int fb = fresh_buf(P, g);
  if (tid < 32) {
    const int j = rb + tid;
    long long row = -1;
    if (j < P.B) row = batch_row(P, k32, g, j);
    rows_sm[tid] = row;
    yb[(long long)g * Bp + j] = row >= 0 ? reinterpret_cast<const int*>(P.y)[row] : -1;
  }
  __syncthreads();
  const __nv_bfloat16* X = reinterpret_cast<const __nv_bfloat16*>(P.X);
  __nv_bfloat16* out = xb + (((long long)fb * P.G + g) * Bp + rb) * ld0;
  const bool vec = (P.ld & 7) == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0 && (d & 7) == 0;
  if (vec) {
    const int per_row = d / 8;
    for (int e = tid; e < 32 * per_row; e += 256) {
      const int r = e / per_row, c = (e - r * per_row) * 8;
      const long long row = rows_sm[r];
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (row >= 0) v = *reinterpret_cast<const uint4*>(X + row * P.ld + c);
      *reinterpret_cast<uint4*>(out + (long long)r * ld0 + c) = v;
    }
  } else {
    for (int e = tid; e < 32 * d; e += 256) {
      const int r = e / d, c = e - r * d;
      const long long row = rows_sm[r];
      out[(long long)r * ld0 + c] = row >= 0 ? X[row * P.ld + c] : __float2bfloat16_rn(0.f);
    }
  }
  if (early) {
    pdl_wait();
    if (blockIdx.x == 0 && g == 0 && tid == 0 && (uint32_t)P.st->k != k32)
      atomicCAS(&P.st->err, (int)DEV_OK, (int)DEV_ERR_CHAIN);
  }
}

// ----------------------------------------------------------------- loss gradient
// dz = (softmax(scores) - onehot(y)) * scale in both orientations; padding rows (y < 0) get zeros.
// Block = 32 consecutive rows of one group; each of the 8 warps takes 4 rows; the bf16 results also go to a
// shared tile from which the column sums (the block's share of the last layer's bias gradient) are taken.
// With `both` the block handles the rows at theta^k and then at the stale point, and also writes the
// difference of the two (fresh - stale, rounded to bf16) to `diff`; otherwise grid.y selects the point.
__global__ void __launch_bounds__(256) bf16_softmax_grad_kernel(const Params P, const float* scores, const int* yb,
                                                                __nv_bfloat16* dz, int n_cls, int ldz, int Bp,
                                                                int pitch, float* colsum, __nv_bfloat16* diff,
                                                                int both) {
  extern __shared__ __nv_bfloat16 sm_tile[];  // [32][pitch]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long rows = (long long)P.G * Bp;
  const long long r0 = (long long)blockIdx.x * 32;  // first row of the block inside a point
  const int g = (int)(r0 / Bp), m0 = (int)(r0 - (long long)g * Bp);
  if (P.skip_unselected && (blockIdx.y != 0 || !P.mask_cur[g])) return;
  const int q_first = both ? 0 : blockIdx.y, q_last = both ? 1 : blockIdx.y;
  for (int q = q_first; q <= q_last; ++q) {
    const long long w0 = (long long)q * rows + r0;
    const bool write_diff = both && q == 1;
    for (int i = 0; i < 4; ++i) {
      const int lr = warp * 4 + i;
      const long long w = w0 + lr;
      const float* s = scores + w * n_cls;
      __nv_bfloat16* o = dz + (((long long)factor_entry(P, g, q) * Bp) + m0 + lr) * ldz;
      const __nv_bfloat16* o0 = dz + (((long long)factor_entry(P, g, 0) * Bp) + m0 + lr) * ldz;  // the same row at theta^k (written by this thread)
      __nv_bfloat16* df = diff + (r0 + lr) * ldz;
      __nv_bfloat16* t = sm_tile + lr * pitch;
      const int y = yb[r0 + lr];
      if (y < 0) {
        for (int c = lane; c < n_cls; c += 32) {
          o[c] = __float2bfloat16_rn(0.f);
          t[c] = __float2bfloat16_rn(0.f);
          if (write_diff) df[c] = __float2bfloat16_rn(0.f);
        }
        continue;
      }
      float mx = -3.0e38f;
      for (int c = lane; c < n_cls; c += 32) mx = fmaxf(mx, s[c]);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      // p_y - 1 = -(sum of the other classes' exponentials) / sum, free of cancellation
      float others = 0.f;
      for (int c = lane; c < n_cls; c += 32)
        if (c != y) others += expf(s[c] - mx);
      others = warp_sum(others);
      const float inv = 1.0f / (others + expf(s[y] - mx));
      for (int c = lane; c < n_cls; c += 32) {
        const float v = (c == y ? -others * inv : expf(s[c] - mx) * inv) * P.scale;
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        o[c] = b;
        t[c] = b;
        if (write_diff) df[c] = __float2bfloat16_rn(__bfloat162float(o0[c]) - __bfloat162float(b));
      }
    }
    __syncthreads();
    // column sums of the block's 32 rows in row order: this block's share of the bias gradient of the last layer
    float* cs = colsum + (((long long)(q * P.G + g)) * (Bp / 32) + m0 / 32) * n_cls;
    for (int c = threadIdx.x; c < n_cls; c += 256) {
      float v = 0.f;
#pragma unroll 8
      for (int r = 0; r < 32; ++r) v += __bfloat162float(sm_tile[r * pitch + c]);
      cs[c] = v;
    }
    __syncthreads();  // the tile is reused for the second point
  }
}

// The same for an even number of classes up to 64 * NP: a lane keeps its NP class pairs of a row in registers,
// so the scores are read once (8-byte loads), every exponential is taken once, and the results leave as bf16
// pairs.
template <int NP>
__global__ void __launch_bounds__(256) bf16_softmax_grad_pairs_kernel(const Params P, const float* scores, const int* yb,
                                                                      __nv_bfloat16* dz, int n_cls, int ldz, int Bp,
                                                                      int pitch, float* colsum, __nv_bfloat16* diff,
                                                                      int both) {
  extern __shared__ __nv_bfloat16 sm_tile[];  // [32][pitch]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long rows = (long long)P.G * Bp;
  const long long r0 = (long long)blockIdx.x * 32;  // first row of the block inside a point
  const int g = (int)(r0 / Bp), m0 = (int)(r0 - (long long)g * Bp);
  if (P.skip_unselected && (blockIdx.y != 0 || !P.mask_cur[g])) return;
  const int q_first = both ? 0 : blockIdx.y, q_last = both ? 1 : blockIdx.y;
  for (int q = q_first; q <= q_last; ++q) {
    const long long w0 = (long long)q * rows + r0;
    const bool write_diff = both && q == 1;
    const long long zq = (long long)factor_entry(P, g, q) * Bp + m0;
    for (int i = 0; i < 4; i += 2) {  // two rows at a time: the loads of both are in flight together
      float2 v[2][NP];
      int y[2];
      float mx[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int lr = warp * 4 + i + u;
        const float* s = scores + (w0 + lr) * n_cls;
        y[u] = yb[r0 + lr];
        mx[u] = -3.0e38f;
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          const int c = 2 * lane + 64 * j;
          v[u][j] = (y[u] >= 0 && c < n_cls) ? *reinterpret_cast<const float2*>(s + c) : make_float2(-3.0e38f, -3.0e38f);
        }
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
#pragma unroll
        for (int j = 0; j < NP; ++j) mx[u] = fmaxf(mx[u], fmaxf(v[u][j].x, v[u][j].y));
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], off));
        mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], off));
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int lr = warp * 4 + i + u;
        __nv_bfloat16* o = dz + (zq + lr) * ldz;
        __nv_bfloat16* df = diff + (r0 + lr) * ldz;
        __nv_bfloat16* t = sm_tile + lr * pitch;
        // p_y - 1 = -(sum of the other classes' exponentials) / sum, free of cancellation
        float others = 0.f, ey = 0.f;
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          const int c = 2 * lane + 64 * j;
          v[u][j].x = expf(v[u][j].x - mx[u]);  // classes beyond n_cls: exp of a huge negative number, zero
          v[u][j].y = expf(v[u][j].y - mx[u]);
          if (c == y[u]) ey = v[u][j].x; else others += v[u][j].x;
          if (c + 1 == y[u]) ey = v[u][j].y; else others += v[u][j].y;
        }
        others = warp_sum(others);
        ey = warp_sum(ey);
        const float inv = y[u] >= 0 ? 1.0f / (others + ey) : 0.f;
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          const int c = 2 * lane + 64 * j;
          if (c < n_cls) {
            const float a = y[u] < 0 ? 0.f : (c == y[u] ? -others * inv : v[u][j].x * inv) * P.scale;
            const float b = y[u] < 0 ? 0.f : (c + 1 == y[u] ? -others * inv : v[u][j].y * inv) * P.scale;
            const __nv_bfloat162 pr = __floats2bfloat162_rn(a, b);
            *reinterpret_cast<__nv_bfloat162*>(o + c) = pr;
            if (write_diff) {  // the tile still holds this row at theta^k (this thread put it there)
              const uint32_t fr = *reinterpret_cast<const uint32_t*>(t + c);
              *reinterpret_cast<uint32_t*>(df + c) = bf16x2_sub(fr, *reinterpret_cast<const uint32_t*>(&pr));
            }
            *reinterpret_cast<__nv_bfloat162*>(t + c) = pr;
          }
        }
      }
    }
    __syncthreads();
    float* cs = colsum + (((long long)(q * P.G + g)) * (Bp / 32) + m0 / 32) * n_cls;
    for (int c = threadIdx.x; c < n_cls; c += 256) {
      float v2 = 0.f;
#pragma unroll 8
      for (int r = 0; r < 32; ++r) v2 += __bfloat162float(sm_tile[r * pitch + c]);
      cs[c] = v2;
    }
    __syncthreads();  // the tile is reused for the second point
  }
}

// ----------------------------------------------------------------- bias gradients
// db_l at both points = column sums of dz_l over the group's rows.  The kernels that produce dz_l leave the
// sums of their row blocks (BiasArgsB::part); here the blocks are added in order, the fresh one is kept, and
// the squared difference of the two points is summed into the layer's lhs_part slot of the group.  One block
// per (group, layer): the selection kernel's single scheduling block adds up every group's partial sums, so
// there should be few of them.
struct BiasArgsB {
  const float* part[MLP_MAX_LAYERS + 1];  // [2][G][blocks[l]][n[l]]
  int blocks[MLP_MAX_LAYERS + 1];
  int n[MLP_MAX_LAYERS + 1];
  long long b_off[MLP_MAX_LAYERS + 1];
  int part_base[MLP_MAX_LAYERS + 1];
  int n_parts;
  float* db;                          // [2][G][nbias], buffer fresh_buf(g) receives this iteration's
  int bias_loc[MLP_MAX_LAYERS + 1];   // first entry of layer l in a db row
  int nbias;
};
__global__ void __launch_bounds__(256) bf16_bias_grad_kernel(const Params P, const BiasArgsB a) {
  __shared__ double scratch[40];
  const int l = blockIdx.y + 1;
  const int n_l = a.n[l];
  const int g = blockIdx.x;
  if (P.skip_unselected && !P.mask_cur[g]) return;
  double d2 = 0.0;
  for (int c = threadIdx.x; c < n_l; c += 256) {
    const int nb = a.blocks[l];
    const float* p0 = a.part[l] + ((long long)g * nb) * n_l + c;
    const float* p1 = p0 + (long long)P.G * nb * n_l;
    float f = 0.f, sv = 0.f;
    for (int b = 0; b < nb; ++b) f += p0[(long long)b * n_l];
    if (!P.skip_unselected)                      // (no stale point when only the selected groups compute)
      for (int b = 0; b < nb; ++b) sv += p1[(long long)b * n_l];
    a.db[((long long)fresh_buf(P, g) * P.G + g) * a.nbias + a.bias_loc[l] + c] = f;
    if (P.gbuf) (fresh_row(P, g) + a.b_off[l])[c] = f;  // kept for inspection
    if (P.stale) (P.stale + (long long)g * P.p_pad + a.b_off[l])[c] = sv;
    d2 += (double)(f - sv) * (double)(f - sv);
  }
  d2 = block_sum(d2, scratch);
  if (threadIdx.x == 0 && GCADA_INDEX_OK(P.st, (long long)g * a.n_parts + a.part_base[l], P.lim.lhs_parts, CHK_LHS_PART))
    P.lhs_part[(long long)g * a.n_parts + a.part_base[l]] = d2;
}

// ----------------------------------------------------------------- bias part of the aggregate
// Bias part of the aggregate: sum over groups (ascending) of the last uploaded bias gradients.
struct BiasAggArgs {
  const float* db;   // [2][G][nbias]; buffer cur[g] holds group g's last upload
  int nbias, n_layers;
  int bias_loc[MLP_MAX_LAYERS + 2];
  long long b_off[MLP_MAX_LAYERS + 1];
};
__global__ void __launch_bounds__(256) bf16_bias_agg_kernel(const Params P, const BiasAggArgs a, float* agg) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= a.nbias) return;
  float s = 0.f;
  for (int g = 0; g < P.G; ++g) s += a.db[((long long)P.cur[g] * P.G + g) * a.nbias + i];
  int l = 1;
  while (l < a.n_layers && i >= a.bias_loc[l + 1]) ++l;
  agg[a.b_off[l] + (i - a.bias_loc[l])] = s;
}

// One group's bias gradient of its last upload into a p-vector (getters).
__global__ void __launch_bounds__(256) bf16_bias_row_kernel(const Params P, const BiasAggArgs a, int g, float* row) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= a.nbias) return;
  int l = 1;
  while (l < a.n_layers && i >= a.bias_loc[l + 1]) ++l;
  row[a.b_off[l] + (i - a.bias_loc[l])] = a.db[((long long)P.cur[g] * P.G + g) * a.nbias + i];
}

// ----------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [batch][rows][k] (k contiguous, row stride ld elements, batch stride bs elements);
// box = 64 (k) x box_rows x 1, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap* tm, const void* base, long long k_extent, long long rows, long long batch, long long ld,
              long long bs, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)k_extent, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)bs * 2};
  cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

long long up(long long x, long long m) { return (x + m - 1) / m * m; }

cudaError_t launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const Params& P, GemmB a, int sm_count,
                        cudaStream_t st) {
  a.stages = G_STAGES;
  const long long units = (long long)((a.N + GN - 1) / GN) * ((a.M + BM - 1) / BM) * (a.k_batched ? 1 : P.G);
  const int ctas = (int)(units < sm_count ? units : sm_count);
  bf16_gemm_kernel<<<ctas, G_THREADS, (size_t)G_SMEM_BYTES, st>>>(ta, tb, P, a);
  return cudaGetLastError();
}

cudaError_t launch_dw(const Params& P, const MlpPlan& pl, const Bf16Impl* im, int l, int mode, cudaStream_t st,
                      int g_only = 0, float* out_row = nullptr) {
  DwArgs w{};
  w.g_only = g_only;
  w.out_row = out_row;
  w.M = pl.dims[l];
  w.N = pl.dims[l - 1];
  w.K = im->Bp;
  w.b_shared = l == 1 ? 1 : 0;
  w.nkb = im->Bp / BK;
  // 32 KiB B blocks in whatever shared memory is left beside the resident A blocks (and the staging tile of
  // the modes that write gradients): the B stream is bound by bytes in flight, so every stage counts
  const long long stage_bytes = (long long)DW_STAGE_FLOATS * 4;
  const long long room = 232448 - 1024 - 1024 - (long long)2 * w.nkb * (BM * BK * 2) - stage_bytes;
  w.stages = (int)(room / (DW_BN * BK * 2));
  if (w.stages > MAX_STAGES) w.stages = MAX_STAGES;
  if (w.stages < 1) w.stages = 1;
  w.tiles_m = (w.M + BM - 1) / BM;
  w.tiles_n = (w.N + DW_BN - 1) / DW_BN;
  w.total_tiles = w.tiles_m * w.tiles_n * P.G;
  w.c_off = pl.w_off[l];
  w.ldc = pl.dims[l - 1];
  w.part_base = im->dw_part_base[l];
  w.n_parts = im->n_parts;
  w.mode = mode;
  const int units = mode == DW_ONE ? w.tiles_m : w.tiles_m * P.G;
  const int ctas = units < pl.sm_count ? units : pl.sm_count;
  const size_t smem = (size_t)(2 * w.nkb + 2 * w.stages) * (BM * BK * 2) + 1024 + (size_t)stage_bytes;
  bf16_dw_kernel<<<ctas, DW_THREADS, smem, st>>>(im->tm_dw_a[l], im->tm_dw_b[l], P, w);
  return cudaGetLastError();
}

}  // namespace

const char* mlp_bf16_supported(const std::vector<int>& dims) {
  (void)dims;
  return nullptr;
}

cudaError_t mlp_bf16_plan_create(MlpPlan* plan, cudaStream_t st, std::vector<void*>* owned, const char** why) {
  const int L = plan->n_layers, G = plan->G, B = plan->B, D = plan->D;
  if (plan->B > 256) {
    *why = "the bf16 MLP path supports minibatches of at most 256 rows per group";
    return cudaSuccess;
  }
  if (plan->dims[L] > 3500) {
    *why = "the bf16 MLP path supports at most 3500 classes";
    return cudaSuccess;
  }
  Bf16Impl* im = new Bf16Impl();
  plan->bf16_impl = im;  // lives as long as the process (a few hundred bytes per plan)
  im->Bp = (int)up(B, 128);
  const long long rows = (long long)G * im->Bp;
  long long pos = 0, bpos = 0;
  // row strides of whole 128-byte lines: a K-major row that starts inside a line costs the copies two lines per box row
  for (int l = 0; l <= L; ++l) im->ld[l] = (int)up(plan->dims[l], 64);
  for (int l = 1; l <= L; ++l) {
    im->w_pos[l] = pos;
    pos += up((long long)plan->dims[l] * im->ld[l - 1], 64);
    im->wt_pos[l] = pos;
    pos += up((long long)plan->dims[l - 1] * im->ld[l], 64);
    im->bias_pos[l] = bpos;
    bpos += up(plan->dims[l], 4);
  }
  im->slot_elems = pos;
  im->bias_slot = bpos;
  // partial sums of the innovation norm per group: one per layer for the biases, and for the weights either one
  // per unit of the Gram products or (inspection mode) one per 128-row block of W_l
  int parts = 0;
  for (int l = 1; l <= L; ++l) im->bias_part_base[l] = parts++;
  for (int l = 1; l <= L; ++l) {
    im->dw_part_base[l] = im->gram_part_base[l] = parts;
    const int rb = (l == 1 ? 1 : 2) * (im->Bp / BM), bn = rb * BM < GN ? rb * BM : GN;
    parts += plan->inspect ? (plan->dims[l] + BM - 1) / BM : rb * (rb * BM / bn);
  }
  im->n_parts = parts;
  plan->norm_parts = parts;
  for (int l = 1; l <= L; ++l) im->bias_loc[l + 1] = im->bias_loc[l] + plan->dims[l];
  im->nbias = im->bias_loc[L + 1];
  auto alloc = [&](void** q, size_t bytes) -> cudaError_t {
    cudaError_t e = cudaMalloc(q, bytes);
    if (e != cudaSuccess) return e;
    owned->push_back(*q);
    return cudaMemsetAsync(*q, 0, bytes, st);
  };
#define A_(ptr, count, type)                                                                     \
  do {                                                                                           \
    cudaError_t e_ = alloc(reinterpret_cast<void**>(&(ptr)), sizeof(type) * (size_t)(count));    \
    if (e_ != cudaSuccess) return e_;                                                            \
  } while (0)
  A_(im->wb, (long long)(D + 1) * im->slot_elems, __nv_bfloat16);
  A_(im->bias, (long long)(D + 1) * im->bias_slot, float);
  A_(im->xb, 2 * rows * im->ld[0], __nv_bfloat16);
  A_(im->yb, rows, int);
  for (int l = 1; l <= L; ++l) {
    if (l < L) {
      A_(im->act[l], 3 * rows * im->ld[l], __nv_bfloat16);
    }
    A_(im->dz[l], 3 * rows * im->ld[l], __nv_bfloat16);
  }
  A_(im->scores, 2 * rows * plan->dims[L], float);
  A_(im->db, 2LL * G * im->nbias, float);
  for (int l = 1; l <= L; ++l) {
    A_(im->dE[l], rows * im->ld[l], __nv_bfloat16);
    if (l < L) A_(im->dF[l], rows * im->ld[l], __nv_bfloat16);
    if (l < L) A_(im->relu_bits[l], 2 * rows * ((plan->dims[l] + 31) / 32), uint32_t);
  }
  for (int l = 1; l <= L; ++l) {
    im->dbp_blocks[l] = l < L ? im->Bp / BM : im->Bp / 32;
    A_(im->dbp[l], 2LL * G * im->dbp_blocks[l] * plan->dims[l], float);
  }
#undef A_
  // what an iteration reads from earlier ones: the bf16 copies of the last D+1 iterates and every group's last upload
  plan->state.clear();
  plan->state.emplace_back(im->wb, sizeof(__nv_bfloat16) * (size_t)(D + 1) * im->slot_elems);
  plan->state.emplace_back(im->bias, sizeof(float) * (size_t)(D + 1) * im->bias_slot);
  // (both upload buffers of every group: which of the two holds the last upload is in Params::cur)
  plan->state.emplace_back(im->xb, sizeof(__nv_bfloat16) * (size_t)2 * rows * im->ld[0]);
  for (int l = 1; l <= L; ++l) {
    plan->state.emplace_back(im->dz[l], sizeof(__nv_bfloat16) * (size_t)2 * rows * im->ld[l]);
    if (l < L) plan->state.emplace_back(im->act[l], sizeof(__nv_bfloat16) * (size_t)2 * rows * im->ld[l]);
  }
  plan->state.emplace_back(im->db, sizeof(float) * (size_t)2 * G * im->nbias);
  if (!encode_fn()) {
    *why = "cuTensorMapEncodeTiled is not available from this driver";
    return cudaSuccess;
  }
  bool ok = true;
  const long long Bp = im->Bp;
  for (int l = 1; l <= L; ++l) {
    const int ni = plan->dims[l - 1], no = plan->dims[l];
    // forward: A = a_{l-1} rows, B = W_l (ring)
    if (l == 1)
      ok &= make_map(&im->tm_fwd_a[l], im->xb, ni, Bp, 2LL * G, im->ld[0], Bp * im->ld[0], BM);
    else
      ok &= make_map(&im->tm_fwd_a[l], im->act[l - 1], ni, Bp, 3LL * G, im->ld[l - 1], Bp * im->ld[l - 1], BM);
    ok &= make_map(&im->tm_fwd_b[l], im->wb + im->w_pos[l], ni, no, D + 1, im->ld[l - 1], im->slot_elems, GN);
    // backward data: A = dz_l rows, B = W_l^T (ring)
    ok &= make_map(&im->tm_da_a[l], im->dz[l], no, Bp, 3LL * G, im->ld[l], Bp * im->ld[l], BM);
    ok &= make_map(&im->tm_da_b[l], im->wb + im->wt_pos[l], no, ni, D + 1, im->ld[l], im->slot_elems, GN);
    // weight gradient: A = dz_l^T, B = a_{l-1}^T
    // differences of the two points (row-major, one entry per group): operands of the Gram products
    ok &= make_map(&im->tm_dE[l], im->dE[l], no, Bp, G, im->ld[l], Bp * im->ld[l], BM);
    if (l < L) ok &= make_map(&im->tm_dF[l], im->dF[l], no, Bp, G, im->ld[l], Bp * im->ld[l], BM);
    // weight gradient and aggregate: the same arrays read MN-major, in blocks of 64 batch rows x 64 columns
    static_assert(DW_BN == GN, "the weight-gradient and aggregate products share their B tensor map");
    ok &= make_map(&im->tm_dw_a[l], im->dz[l], no, Bp, 3LL * G, im->ld[l], Bp * im->ld[l], 64);
    if (l == 1)
      ok &= make_map(&im->tm_dw_b[l], im->xb, ni, Bp, 2LL * G, im->ld[0], Bp * im->ld[0], 64);
    else
      ok &= make_map(&im->tm_dw_b[l], im->act[l - 1], ni, Bp, 3LL * G, im->ld[l - 1], Bp * im->ld[l - 1], 64);
  }
  if (!ok) {
    *why = "tensor map creation failed for this MLP shape";
    return cudaSuccess;
  }
  cudaError_t e = cudaFuncSetAttribute(bf16_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       G_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_softmax_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           32 * (plan->dims[L] + 4) * 2);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_softmax_grad_pairs_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32 * (256 + 4) * 2);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_softmax_grad_pairs_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32 * (512 + 4) * 2);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_softmax_grad_pairs_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32 * (1024 + 4) * 2);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_dw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024);  // the kernel's static arrays take under 1 KiB
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bf16_gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, G_STAGES * G_STAGE_BYTES + 1024);
  if (e != cudaSuccess) return e;
  plan->launches_per_iter = 3 + 2 * L + 1 + L + 2 * (L - 1);
  plan->post_launches = L + 1;
  plan->skip_launches = 2 + L + 1 + (L - 1) + 1;
  return cudaSuccess;
}

cudaError_t mlp_bf16_launch(const Params& P, const MlpPlan& pl, cudaStream_t st, int* n_launches) {
  const Bf16Impl* im = static_cast<const Bf16Impl*>(pl.bf16_impl);
  const int L = pl.n_layers, G = P.G, Bp = im->Bp;
  const long long rows = (long long)G * Bp;
  int n = 0;
  cudaError_t e;
  // the minibatch rows first: inside a captured chain this launch is programmatically dependent on the previous
  // iteration's update kernel and runs beside it
  if ((e = launch_k(bf16_gather_kernel, dim3(Bp / 32, G), dim3(256), 0, st, P.pdl != 0 && P.k_off > 0, P, im->xb,
                    im->yb, pl.dims[0], im->ld[0], Bp)) != cudaSuccess)
    return e;
  ++n;
  // weights of theta^k -> bf16 ring slot k (both orientations) and rounded biases
  {
    ConvArgs c{};
    int max_no = 0, max_ni = 0;
    for (int l = 1; l <= L; ++l) {
      c.n_out[l] = pl.dims[l];
      c.n_in[l] = pl.dims[l - 1];
      c.w_off[l] = pl.w_off[l];
      c.b_off[l] = pl.b_off[l];
      c.w_pos[l] = im->w_pos[l];
      c.wt_pos[l] = im->wt_pos[l];
      c.bias_pos[l] = im->bias_pos[l];
      c.ldk[l] = im->ld[l - 1];
      c.ldn[l] = im->ld[l];
      if (pl.dims[l] > max_no) max_no = pl.dims[l];
      if (pl.dims[l - 1] > max_ni) max_ni = pl.dims[l - 1];
    }
    c.slot_elems = im->slot_elems;
    c.bias_slot = im->bias_slot;
    bf16_convert_kernel<<<dim3((max_ni + 63) / 64, (max_no + 63) / 64, L), 256, 0, st>>>(P, c, im->wb, im->bias);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    ++n;
  }
  // production: no group's weight gradient is formed; the stale point's epilogues write differences for the
  // Gram form of the innovation norm.  Inspection mode keeps both gradients of every group instead.
  const bool production = !P.stale && !P.skip_unselected;
  for (int l = 1; l <= L; ++l) {
    GemmB a{};
    a.M = Bp;
    a.N = pl.dims[l];
    a.K = pl.dims[l - 1];
    a.a_shared = l == 1;
    a.zb_mode = ZB_RING;
    a.bias_ring = im->bias;
    a.bias_slot = im->bias_slot;
    a.bias_pos = im->bias_pos[l];
    if (l < L) {
      a.epi = EPI_HIDDEN;
      a.out = im->act[l];
      a.ldo = im->ld[l];
      a.z_stride_out = (long long)Bp * im->ld[l];
      a.diff = production ? im->dF[l] : nullptr;
      a.n_entries = 3 * G;
      a.relu_bits = im->relu_bits[l];
      a.nw = (pl.dims[l] + 31) / 32;
    } else {
      a.epi = EPI_SCORES;
      a.out_f32 = im->scores;
    }
    for (int q = 0; q < (P.skip_unselected ? 1 : 2); ++q) {  // theta^k, then the stale iterates
      a.point = q;
      if ((e = launch_gemm(im->tm_fwd_a[l], im->tm_fwd_b[l], P, a, pl.sm_count, st)) != cudaSuccess) return e;
      ++n;
    }
  }
  {
    const int pitch = pl.dims[L] + 2 + (pl.dims[L] & 1);  // even, and an odd number of 32-bit words when possible
    const int nc = pl.dims[L];
    // production: a block takes both points of its rows and writes their difference; inspection mode (both
    // gradients kept) and the printed rule (one point only): grid.y selects the point
    const int both = (!P.stale && !P.skip_unselected) ? 1 : 0;
    const dim3 blocks((unsigned)(rows / 32), both || P.skip_unselected ? 1 : 2);
    const size_t sm = (size_t)32 * pitch * 2;
    if ((nc & 1) == 0 && nc <= 1024) {  // class pairs in registers
      if (nc <= 256)
        bf16_softmax_grad_pairs_kernel<4><<<blocks, 256, sm, st>>>(P, im->scores, im->yb, im->dz[L], nc, im->ld[L], Bp, pitch, im->dbp[L], im->dE[L], both);
      else if (nc <= 512)
        bf16_softmax_grad_pairs_kernel<8><<<blocks, 256, sm, st>>>(P, im->scores, im->yb, im->dz[L], nc, im->ld[L], Bp, pitch, im->dbp[L], im->dE[L], both);
      else
        bf16_softmax_grad_pairs_kernel<16><<<blocks, 256, sm, st>>>(P, im->scores, im->yb, im->dz[L], nc, im->ld[L], Bp, pitch, im->dbp[L], im->dE[L], both);
    } else {
      bf16_softmax_grad_kernel<<<blocks, 256, sm, st>>>(P, im->scores, im->yb, im->dz[L], nc, im->ld[L], Bp, pitch, im->dbp[L], im->dE[L], both);
    }
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  ++n;
  for (int l = L; l >= 1; --l) {
    if (production) {  // the innovation norm of layer l's weight gradient from the two Gram products
      GramArgs ga{};
      ga.parts = l == 1 ? 1 : 2;
      ga.nb = Bp / BM;
      ga.BN = ga.parts * Bp < GN ? ga.parts * Bp : GN;
      ga.Ku = pl.dims[l];
      ga.Kv = pl.dims[l - 1];
      ga.part_base = im->gram_part_base[l];
      ga.n_parts = im->n_parts;
      const int units = G * ga.parts * ga.nb * (ga.parts * Bp / ga.BN);
      const int ctas = units < pl.sm_count ? units : pl.sm_count;
      // U = [E_l; dz_l at the stale point], V = [a_{l-1} at theta^k; F_{l-1}]
      bf16_gram_kernel<<<ctas, G_THREADS, (size_t)G_STAGES * G_STAGE_BYTES + 1024, st>>>(
          im->tm_dE[l], im->tm_da_a[l], im->tm_fwd_a[l], l == 1 ? im->tm_fwd_a[l] : im->tm_dF[l - 1], P, ga);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      ++n;
    } else if (!P.skip_unselected) {  // inspection mode: both gradients of every group, norm from their difference
      if ((e = launch_dw(P, pl, im, l, DW_BOTH, st)) != cudaSuccess) return e;
      ++n;
    }
    if (l > 1) {
      GemmB d{};
      d.M = Bp;
      d.N = pl.dims[l - 1];
      d.K = pl.dims[l];
      d.a_shared = 0;
      d.zb_mode = ZB_RING;
      d.epi = EPI_DA;
      d.out = im->dz[l - 1];
      d.relu_bits = im->relu_bits[l - 1];
      d.nw = (pl.dims[l - 1] + 31) / 32;
      d.colsum = im->dbp[l - 1];
      d.diff = production ? im->dE[l - 1] : nullptr;
      d.n_entries = 3 * G;
      d.ldo = im->ld[l - 1];
      d.z_stride_out = (long long)Bp * im->ld[l - 1];
      for (int q = 0; q < (P.skip_unselected ? 1 : 2); ++q) {
        d.point = q;
        if ((e = launch_gemm(im->tm_da_a[l], im->tm_da_b[l], P, d, pl.sm_count, st)) != cudaSuccess) return e;
        ++n;
      }
    }
  }
  BiasArgsB ba{};
  int maxn = 0;
  for (int l = 1; l <= L; ++l) {
    ba.part[l] = im->dbp[l];
    ba.blocks[l] = im->dbp_blocks[l];
    ba.n[l] = pl.dims[l];
    ba.b_off[l] = pl.b_off[l];
    ba.part_base[l] = im->bias_part_base[l];
    ba.bias_loc[l] = im->bias_loc[l];
    if (pl.dims[l] > maxn) maxn = pl.dims[l];
  }
  ba.n_parts = im->n_parts;
  ba.db = im->db;
  ba.nbias = im->nbias;
  bf16_bias_grad_kernel<<<dim3(G, L), 256, 0, st>>>(P, ba);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  ++n;
  *n_launches = n;
  return cudaSuccess;
}

}  // namespace gcada

namespace gcada {
namespace {
BiasAggArgs bias_agg_args(const MlpPlan& pl, const Bf16Impl* im) {
  BiasAggArgs b{};
  b.db = im->db;
  b.nbias = im->nbias;
  b.n_layers = pl.n_layers;
  for (int l = 1; l <= pl.n_layers + 1; ++l) b.bias_loc[l] = im->bias_loc[l];
  for (int l = 1; l <= pl.n_layers; ++l) b.b_off[l] = pl.b_off[l];
  return b;
}
}  // namespace

// After the selection (which has flipped cur[] of the selected groups, so that their uploads are kept), the
// server's side of Eq. (3): the aggregate is the sum over ALL groups of the last uploaded gradients.  Each
// layer's share is one product whose K dimension runs over groups' rows: over the selected groups only - their
// replaced uploads with a minus sign, then their new ones - when fewer than half of the groups upload, over
// every group (the sum formed anew) otherwise and at least every AGG_REFRESH iterations, which keeps the
// rounding of the running sum from piling up.
cudaError_t mlp_bf16_launch_post(const Params& P, const MlpPlan& pl, cudaStream_t st, int* n_launches) {
  *n_launches = 0;
  const Bf16Impl* im = static_cast<const Bf16Impl*>(pl.bf16_impl);
  const int L = pl.n_layers, G = P.G, Bp = im->Bp;
  cudaError_t e;
  for (int l = L; l >= 1; --l) {
    GemmB a{};
    a.M = pl.dims[l];
    a.N = pl.dims[l - 1];
    a.K = G * Bp;
    a.k_batched = 1;
    a.kpg = Bp / BK;
    a.n_batch = G;
    a.epi = EPI_AGG;
    a.out_f32 = P.agg_hi;
    a.c_off = pl.w_off[l];
    a.ldc = pl.dims[l - 1];
    if ((e = launch_gemm(im->tm_dw_a[l], im->tm_dw_b[l], P, a, pl.sm_count, st)) != cudaSuccess) return e;
    ++*n_launches;
  }
  bf16_bias_agg_kernel<<<(im->nbias + 255) / 256, 256, 0, st>>>(P, bias_agg_args(pl, im), P.agg_hi);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  ++*n_launches;
  return cudaSuccess;
}

// Group g's last uploaded gradient, rebuilt from its stored factors into `row` (a p-vector on the device).
cudaError_t mlp_bf16_group_gradient(const Params& P, const MlpPlan& pl, int g, float* row, cudaStream_t st) {
  const Bf16Impl* im = static_cast<const Bf16Impl*>(pl.bf16_impl);
  for (int l = pl.n_layers; l >= 1; --l) {
    cudaError_t e = launch_dw(P, pl, im, l, DW_ONE, st, g, row);
    if (e != cudaSuccess) return e;
  }
  bf16_bias_row_kernel<<<(im->nbias + 255) / 256, 256, 0, st>>>(P, bias_agg_args(pl, im), g, row);
  return cudaGetLastError();
}
}  // namespace gcada
