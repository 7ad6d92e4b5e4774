// Dual-point minibatch gradients of the multilayer perceptron (ReLU hidden
// layers, softmax cross-entropy) for all groups: the gradient step of
// Algorithm 1 evaluated at theta^k (point 0) and at each group's stale
// iterate theta^{k - tau_g} (point 1) on the same gathered samples.
//
// fp32 path (this file): plain FFMA tiles, because single-pass tensor-core
// arithmetic (tf32 / bf16 operands) cannot hold a 1e-5 relative tolerance.
// The bf16 path lives in mlp_bf16.cu.
//
// theta layout: for l = 1..L, W_l (n_l rows of n_{l-1}) then b_l (n_l).
// Batch index z = q * G + g (q = point, g = group).
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "mlp.h"

#include "mlp_bf16.h"

namespace gcada {

namespace cg = cooperative_groups;

namespace {

__device__ __forceinline__ const float* ring_ptr(const Params& P, int g, int q, long long k) {
  long long j = q == 0 ? k : k - P.tau[g];
  if (j < k - P.D) j = k - P.D;  // ages beyond D only arise under forced masks: oldest kept iterate
  if (j < 0) j = 0;
  return P.theta_ring + (j % (P.D + 1)) * P.p_pad;
}

// ------------------------------------------------------------------ gather
// Warp per sampled row: xb[r] = X[row(r)], yb[r] = y[row(r)].
// Inside a chain of captured iterations (P.pdl) the kernel runs while the previous iteration's update kernel
// does: the draw does not depend on the iterate (Section II-A), the iteration number comes from the chain's
// start, and the buffers it writes were last read before that update began.  It waits for the update at its
// end, so that its completion implies the update's.
__global__ void __launch_bounds__(256) mlp_gather_kernel(const Params P, float* xb, int* yb, int d) {
  const int warp = (int)((blockIdx.x * 256 + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  const long long rows = (long long)P.G * P.B;
  const bool early = P.pdl != 0 && !P.skip_unselected;
  pdl_launch_dependents();
  if (!early) pdl_wait();
  const uint32_t k32 = (uint32_t)(early ? P.st->k_chain + P.k_off : P.st->k);
  if (warp >= rows) {
    if (early) pdl_wait();
    return;
  }
  const int g = warp / P.B, j = warp - g * P.B;
  if (P.skip_unselected && !P.mask_cur[g]) return;  // rule PS: only the selected groups compute
  const long long row = batch_row(P, k32, g, j);
  const float* src = reinterpret_cast<const float*>(P.X) + row * P.ld;
  float* dst = xb + (long long)warp * d;
  if (((d | P.ld) & 3) == 0 && ((reinterpret_cast<uintptr_t>(P.X) | reinterpret_cast<uintptr_t>(xb)) & 15) == 0) {
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(dst);
    const int n4 = d >> 2;
    for (int c0 = 0; c0 < n4; c0 += 256) {  // eight 16-byte loads in flight per lane
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (c0 + lane + 32 * u < n4) v[u] = s4[c0 + lane + 32 * u];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (c0 + lane + 32 * u < n4) d4[c0 + lane + 32 * u] = v[u];
    }
  } else {
    for (int c = lane; c < d; c += 32) dst[c] = src[c];
  }
  if (lane == 0) yb[warp] = reinterpret_cast<const int*>(P.y)[row];
  if (early) {
    pdl_wait();
    if (warp == 0 && lane == 0 && (uint32_t)P.st->k != k32) atomicCAS(&P.st->err, (int)DEV_OK, (int)DEV_ERR_CHAIN);
  }
}

// ------------------------------------------------------------------ GEMM
struct Operand {
  const float* base;  // plain buffer, or unused when ring != 0
  long long off;      // ring != 0: offset inside theta
  long long zg, zq;   // batch strides (group, point)
  long long rs, cs;   // strides of the first / second matrix index
  int ring;           // 1: the operand lives in the iterate ring (theta^k for q = 0, theta^{k-tau_g} for q = 1)
};

struct GemmArgs {
  int M, N, K;
  Operand A;   // A(m, k)
  Operand Bm;  // B(k, n)
  float* C;    // plain output (c_grad == 0): C + g*c_zg + q*c_zq + m*c_rs + n
  long long c_zg, c_zq, c_rs;
  int c_grad;  // 1: output goes to the gradient vectors, (q == 0 ? fresh : stale) + g*p_pad + c_off
  long long c_off;
  int bias;    // add b[n] from the iterate ring at bias_off
  long long bias_off;
  int relu;
  const float* mask;  // multiply by (mask(m, n) > 0); same indexing as C
  int split;          // CTAs (one thread-block cluster along x) that share an output tile, each summing over
  int kchunk;         // kchunk values of k (a multiple of TK); 1: no split
};

constexpr int TM = 64, TN = 64, TK = 32;
constexpr int EPT = TM * TK / 256;  // elements of each operand tile a thread moves per K step

// 64 x 64 output tile per CTA, 4 x 4 per thread, K in steps of 32 through two shared-memory buffers: the next
// step's operands are fetched into registers before the current step is multiplied and stored into the other
// buffer after it, one block barrier per step.  A product with few tiles and a long K (the first layer of a
// small network) is split over the CTAs of one thread-block cluster: CTA r sums k in [r kchunk, (r+1) kchunk),
// the partial tiles meet in CTA 0 through distributed shared memory in rank order (fixed, so results are
// reproducible).
__global__ void __launch_bounds__(256) mlp_sgemm_kernel(const Params P, const GemmArgs a) {
  __shared__ __align__(16) float sm[2][2][TK][TM + 4];  // [buffer][A, B][k][m or n]
  float4* red = reinterpret_cast<float4*>(&sm[0][0][0][0]);  // [4][256]: this CTA's partial tile (split products), after the loop
  static_assert(sizeof(sm) >= 4 * 256 * sizeof(float4), "the partial tile reuses the operand buffers");
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int z = blockIdx.z, q = z / P.G, g = z - q * P.G;
  // rule PS (the selection is already known): selected groups at theta^k only
  if (P.skip_unselected && (q != 0 || !P.mask_cur[g])) return;  // (the same for every CTA of a cluster)
  const int rank = a.split > 1 ? (int)(blockIdx.x % a.split) : 0;
  const int m0 = blockIdx.y * TM, n0 = (a.split > 1 ? (int)(blockIdx.x / a.split) : (int)blockIdx.x) * TN;
  const int k_lo = rank * a.kchunk, k_hi = a.split > 1 ? (k_lo + a.kchunk < a.K ? k_lo + a.kchunk : a.K) : a.K;
  const long long k_it = P.st->k;
  const float* Ab = a.A.ring ? ring_ptr(P, g, q, k_it) + a.A.off : a.A.base + g * a.A.zg + q * a.A.zq;
  const float* Bb = a.Bm.ring ? ring_ptr(P, g, q, k_it) + a.Bm.off : a.Bm.base + g * a.Bm.zg + q * a.Bm.zq;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  // The eight A and eight B elements this thread moves per K step.  An operand that runs along m (or n) is
  // read and stored 32 consecutive m per warp.  One that runs along k is stored transposed: a warp takes
  // 8 consecutive k of 4 rows, which are 32 different banks under the row pitch of 68 floats.
  static_assert(TM == 64 && TN == 64 && TK == 32, "index arithmetic below");
  int a_mm[EPT], a_kk[EPT], b_nn[EPT], b_kk[EPT];
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int e = tid + 256 * i;
    const int t_k = (e & 7) | (((e >> 5) & 3) << 3), t_m = ((e >> 3) & 3) | ((e >> 7) << 2);
    if (a.A.cs == 1) {
      a_kk[i] = t_k;
      a_mm[i] = t_m;
    } else {
      a_mm[i] = e & (TM - 1);
      a_kk[i] = e >> 6;
    }
    if (a.Bm.cs == 1) {
      b_nn[i] = e & (TN - 1);
      b_kk[i] = e >> 6;
    } else {
      b_kk[i] = t_k;
      b_nn[i] = t_m;
    }
  }
  float ra[EPT], rb[EPT];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      const int m = m0 + a_mm[i], kx = k0 + a_kk[i];
      ra[i] = (m < a.M && kx < k_hi) ? Ab[m * a.A.rs + kx * a.A.cs] : 0.f;
      const int n = n0 + b_nn[i], ky = k0 + b_kk[i];
      rb[i] = (n < a.N && ky < k_hi) ? Bb[ky * a.Bm.rs + n * a.Bm.cs] : 0.f;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      sm[buf][0][a_kk[i]][a_mm[i]] = ra[i];
      sm[buf][1][b_kk[i]][b_nn[i]] = rb[i];
    }
  };
  if (k_lo < k_hi) {
    fetch(k_lo);
    stash(0);
  }
  __syncthreads();
  int buf = 0;
  for (int k0 = k_lo; k0 < k_hi; k0 += TK, buf ^= 1) {
    const bool more = k0 + TK < k_hi;
    if (more) fetch(k0 + TK);
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&sm[buf][0][kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&sm[buf][1][kk][tx * 4]);
      const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += av[i] * bv[j];
    }
    if (more) stash(buf ^ 1);  // (last read before the barrier that ended the previous step)
    __syncthreads();
  }

  if (a.split > 1) {
    cg::cluster_group cluster = cg::this_cluster();
#pragma unroll
    for (int i = 0; i < 4; ++i) red[i * 256 + tid] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    cluster.sync();
    if (rank == 0) {
      for (int r = 1; r < a.split; ++r) {
        const float4* rr = cluster.map_shared_rank(red, r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 v = rr[i * 256 + tid];
          acc[i][0] += v.x;
          acc[i][1] += v.y;
          acc[i][2] += v.z;
          acc[i][3] += v.w;
        }
      }
    }
    cluster.sync();  // no CTA leaves while CTA 0 may still read its tile
    if (rank != 0) return;
  }

  float* Cb;
  if (a.c_grad)  // (after the selection the flip of cur[g] has made the target row the last uploaded one)
    Cb = (q == 0 ? (P.skip_unselected ? last_row(P, g) : fresh_row(P, g)) : P.stale + (long long)g * P.p_pad) + a.c_off;
  else
    Cb = a.C + g * a.c_zg + q * a.c_zq;
  const float* Mb = a.mask ? a.mask + g * a.c_zg + q * a.c_zq : nullptr;
  const float* bias = a.bias ? ring_ptr(P, g, q, k_it) + a.bias_off : nullptr;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= a.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= a.N) continue;
      float v = acc[i][j];
      if (bias) v += bias[n];
      if (a.relu) v = fmaxf(v, 0.f);
      if (Mb) v = Mb[m * a.c_rs + n] > 0.f ? v : 0.f;
      Cb[m * a.c_rs + n] = v;
    }
  }
}

// Products with at most 16 output columns whose operands both run along k (the class scores of a small
// network): the CTA stages the N x K weights of its (point, group) in shared memory, then a warp per output
// row: lanes stride over k, one shuffle reduction per column.  Grid (ceil(M / 8), 2 G).
constexpr int ROWDOT_MAX_N = 16;
__global__ void __launch_bounds__(256) mlp_rowdot_kernel(const Params P, const GemmArgs a) {
  extern __shared__ float wsm[];  // [N][K]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int z = blockIdx.y, q = z / P.G, g = z - q * P.G;
  if (P.skip_unselected && (q != 0 || !P.mask_cur[g])) return;
  const long long k_it = P.st->k;
  const float* Bb = a.Bm.ring ? ring_ptr(P, g, q, k_it) + a.Bm.off : a.Bm.base + g * a.Bm.zg + q * a.Bm.zq;
  for (int e = threadIdx.x; e < a.N * a.K; e += 256) {
    const int n = e / a.K, k = e - n * a.K;
    wsm[e] = Bb[k + n * a.Bm.cs];
  }
  const int m = blockIdx.x * 8 + warp;
  // the row's share of this lane, up to 8 values at a time, all loads in flight before the weights are needed
  const float* Ab = (a.A.ring ? ring_ptr(P, g, q, k_it) + a.A.off : a.A.base + g * a.A.zg + q * a.A.zq) + (m < a.M ? m : 0) * a.A.rs;
  float part[ROWDOT_MAX_N];
#pragma unroll
  for (int n = 0; n < ROWDOT_MAX_N; ++n) part[n] = 0.f;
  float av[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) av[u] = lane + 32 * u < a.K ? Ab[lane + 32 * u] : 0.f;
  __syncthreads();
  for (int k0 = 0; k0 < a.K; k0 += 256) {
    float nx[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) nx[u] = k0 + 256 + lane + 32 * u < a.K ? Ab[k0 + 256 + lane + 32 * u] : 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int k = k0 + lane + 32 * u;
      if (k < a.K) {
#pragma unroll
        for (int n = 0; n < ROWDOT_MAX_N; ++n)
          if (n < a.N) part[n] += av[u] * wsm[n * a.K + k];
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) av[u] = nx[u];
  }
  float mine = 0.f;
#pragma unroll
  for (int n = 0; n < ROWDOT_MAX_N; ++n) {
    if (n < a.N) {  // (uniform)
      float v = part[n];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == n) mine = v;
    }
  }
  if (m < a.M && lane < a.N) {
    float v = mine;
    if (a.bias) v += (ring_ptr(P, g, q, k_it) + a.bias_off)[lane];
    if (a.relu) v = fmaxf(v, 0.f);
    const long long o = g * a.c_zg + q * a.c_zq + m * a.c_rs + lane;
    if (a.mask) v = a.mask[o] > 0.f ? v : 0.f;
    a.C[o] = v;
  }
}

// ------------------------------------------------------------------ loss
// Warp per (point, row): dz = (softmax(scores) - onehot(y)) * scale.  Class ids outside [0, n_cls) are
// the caller's error (undefined result).
__global__ void __launch_bounds__(256) mlp_softmax_grad_kernel(const Params P, const float* scores, const int* yb,
                                                               float* dz, int n_cls) {
  const long long rows = (long long)P.G * P.B;
  const long long w = ((long long)blockIdx.x * 256 + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= 2 * rows) return;
  const long long r = w % rows;
  if (P.skip_unselected && (w >= rows || !P.mask_cur[r / P.B])) return;
  const float* s = scores + w * n_cls;
  float* o = dz + w * n_cls;
  float mx = -3.0e38f;
  for (int c = lane; c < n_cls; c += 32) mx = fmaxf(mx, s[c]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  // p_y - 1 = -(sum of the other classes' exponentials) / sum: formed without
  // the cancellation that p_y - 1 suffers once a sample is classified well
  const int y = yb[r];
  float others = 0.f;
  for (int c = lane; c < n_cls; c += 32)
    if (c != y) others += expf(s[c] - mx);
  others = warp_sum(others);
  const float ey = expf(s[y] - mx);
  const float inv = 1.0f / (others + ey);
  for (int c = lane; c < n_cls; c += 32)
    o[c] = (c == y ? -others * inv : expf(s[c] - mx) * inv) * P.scale;
}

// ------------------------------------------------------------------ bias gradients
// db_l[n] = sum over the group's rows of dz_l[row][n]; grid (n blocks, 2G, L).
struct BiasArgs {
  const float* dz[MLP_MAX_LAYERS + 1];
  int n[MLP_MAX_LAYERS + 1];
  long long b_off[MLP_MAX_LAYERS + 1];
};

__global__ void __launch_bounds__(256) mlp_bias_grad_kernel(const Params P, const BiasArgs a) {
  const int l = blockIdx.z + 1;
  const int n = blockIdx.x * 256 + threadIdx.x;
  if (n >= a.n[l]) return;
  const int z = blockIdx.y, q = z / P.G, g = z - q * P.G;
  if (P.skip_unselected && (q != 0 || !P.mask_cur[g])) return;
  const float* src = a.dz[l] + ((long long)z * P.B) * a.n[l] + n;
  float s = 0.f;
  int r = 0;
  for (; r + 8 <= P.B; r += 8) {  // eight loads in flight, added in row order
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = src[(long long)(r + u) * a.n[l]];
#pragma unroll
    for (int u = 0; u < 8; ++u) s += v[u];
  }
  for (; r < P.B; ++r) s += src[(long long)r * a.n[l]];
  ((q == 0 ? (P.skip_unselected ? last_row(P, g) : fresh_row(P, g)) : P.stale + (long long)g * P.p_pad) + a.b_off[l])[n] = s;
}

// ------------------------------------------------------------------ small output layer, fused
// Networks whose last layer is small (at most 16 classes on at most 256 hidden units: the 784-200-10 workload)
// spend their time in launch and dependency latency, not in arithmetic.  Everything on the back-propagation
// chain above the last hidden layer is local to a minibatch row, so one launch does it, a warp per row:
// class scores z_L = a_{L-1} W_L^T + b_L, the loss gradient dz_L, and the back-propagated error
// dz_{L-1} = (dz_L W_L) masked by a_{L-1} > 0.  It replaces three dependent launches (scores, loss gradient,
// backward-data).  Grid (ceil(B / 8), 2 G); the CTA stages W_L of its (point, group) in shared memory.
constexpr int HEAD_MAX_N = 16;   // classes
constexpr int HEAD_CH = 8;       // hidden units per lane: up to 256 hidden units
struct HeadArgs {
  int n1, nL;                    // hidden units n_{L-1}, classes n_L
  long long w_off, b_off;        // W_L and b_L inside theta
  const float* a1;               // [2][G*B][n1]  activations of the last hidden layer
  const int* yb;                 // [G*B]
  float* dzL;                    // [2][G*B][nL]
  float* dz1;                    // [2][G*B][n1]
};

__global__ void __launch_bounds__(256) mlp_head_kernel(const Params P, const HeadArgs a) {
  extern __shared__ float hsm[];  // W_L [nL][n1]
  const int n1 = a.n1, nL = a.nL;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int z = blockIdx.y, q = z / P.G, g = z - q * P.G;
  if (P.skip_unselected && (q != 0 || !P.mask_cur[g])) return;
  const long long k_it = P.st->k;
  const float* theta = ring_ptr(P, g, q, k_it);
  const int r = blockIdx.x * 8 + warp;
  const long long row = (long long)q * P.G * P.B + (long long)g * P.B + (r < P.B ? r : 0);
  // the row's activations and label are on their way while the weights are staged
  const float* ar = a.a1 + row * n1;
  float av[HEAD_CH];
#pragma unroll
  for (int u = 0; u < HEAD_CH; ++u) av[u] = lane + 32 * u < n1 ? ar[lane + 32 * u] : 0.f;
  const int y = a.yb[(long long)g * P.B + (r < P.B ? r : 0)];
  const float bl = lane < nL ? theta[a.b_off + lane] : 0.f;
  for (int e = threadIdx.x; e < nL * n1; e += 256) hsm[e] = theta[a.w_off + e];
  __syncthreads();
  if (r >= P.B) return;
  // class scores: lane c ends up with z_L[c]
  float mine = 0.f;
#pragma unroll
  for (int c = 0; c < HEAD_MAX_N; ++c) {
    if (c < nL) {  // (uniform)
      float v = 0.f;
#pragma unroll
      for (int u = 0; u < HEAD_CH; ++u)
        if (lane + 32 * u < n1) v += av[u] * hsm[c * n1 + lane + 32 * u];
      v = warp_sum(v);
      if (lane == c) mine = v + bl;
    }
  }
  // loss gradient across the lanes; p_y - 1 = -(sum of the other classes' exponentials) / sum, free of cancellation
  float mx = lane < nL ? mine : -3.0e38f;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  const float ex = lane < nL ? expf(mine - mx) : 0.f;
  const float others = warp_sum(lane == y ? 0.f : ex);
  const float ey = __shfl_sync(0xffffffffu, ex, y & 31);
  const float inv = 1.0f / (others + ey);
  const float dzc = lane < nL ? (lane == y ? -others * inv : ex * inv) * P.scale : 0.f;
  if (lane < nL) a.dzL[row * nL + lane] = dzc;
  // back-propagated error of the last hidden layer
  float acc[HEAD_CH];
#pragma unroll
  for (int u = 0; u < HEAD_CH; ++u) acc[u] = 0.f;
#pragma unroll
  for (int c = 0; c < HEAD_MAX_N; ++c) {
    if (c < nL) {
      const float d = __shfl_sync(0xffffffffu, dzc, c);
#pragma unroll
      for (int u = 0; u < HEAD_CH; ++u)
        if (lane + 32 * u < n1) acc[u] += d * hsm[c * n1 + lane + 32 * u];
    }
  }
  float* d1 = a.dz1 + row * n1;
#pragma unroll
  for (int u = 0; u < HEAD_CH; ++u)
    if (lane + 32 * u < n1) d1[lane + 32 * u] = av[u] > 0.f ? acc[u] : 0.f;
}

size_t head_smem_bytes(const MlpPlan& pl) {
  const int L = pl.n_layers;
  return (size_t)pl.dims[L] * pl.dims[L - 1] * sizeof(float);
}
bool head_fits(const MlpPlan& pl) {
  const int L = pl.n_layers;
  return pl.compute == 0 && L >= 2 && pl.dims[L] <= HEAD_MAX_N && pl.dims[L - 1] <= 32 * HEAD_CH &&
         head_smem_bytes(pl) <= 96 * 1024;
}

cudaError_t launch_gemm(const Params& P, GemmArgs a, int sm_count, cudaStream_t st) {
  if (a.N <= ROWDOT_MAX_N && a.A.cs == 1 && a.Bm.rs == 1 && !a.c_grad && (size_t)a.N * a.K * sizeof(float) <= 48 * 1024) {
    mlp_rowdot_kernel<<<dim3((a.M + 7) / 8, 2 * P.G), 256, (size_t)a.N * a.K * sizeof(float), st>>>(P, a);
    return cudaGetLastError();
  }
  const int gx = (a.N + TN - 1) / TN, gy = (a.M + TM - 1) / TM;
  const long long tiles = (long long)gx * gy * 2 * P.G;
  // few tiles and a long K: split K over a cluster so that about one CTA per SM is busy (measured on the
  // 784-200-10 network: 3 and 5 shares of K equally good, 2, 4 and 7 slower)
  a.split = 1;
  a.kchunk = a.K;
  if (a.K >= 8 * TK && tiles < sm_count) {
    long long s = sm_count / tiles;
    if (s > 8) s = 8;
    if (s > a.K / (2 * TK)) s = a.K / (2 * TK);
    if (s > 1) {
      a.kchunk = (int)(((a.K + s - 1) / s + TK - 1) / TK * TK);
      a.split = (a.K + a.kchunk - 1) / a.kchunk;
    }
  }
  if (a.split == 1) {
    mlp_sgemm_kernel<<<dim3(gx, gy, 2 * P.G), 256, 0, st>>>(P, a);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(gx * a.split, gy, 2 * P.G);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = a.split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, mlp_sgemm_kernel, P, a);
}

}  // namespace

const char* mlp_supported(const std::vector<int>& dims, int compute) {
  if ((int)dims.size() - 1 > MLP_MAX_LAYERS) return "too many layers (at most 15)";
  if (compute == 1) return mlp_bf16_supported(dims);
  return nullptr;
}

cudaError_t mlp_plan_create(const std::vector<int>& dims, int compute, int G, int B, int D, long long p_pad,
                            int sm_count, cudaStream_t st, MlpPlan* plan, std::vector<void*>* owned,
                            const char** why) {
  *why = "";
  const int L = (int)dims.size() - 1;
  plan->n_layers = L;
  plan->compute = compute;
  plan->G = G;
  plan->B = B;
  plan->D = D;
  plan->p_pad = p_pad;
  plan->sm_count = sm_count;
  long long off = 0;
  for (int l = 0; l <= L; ++l) plan->dims[l] = dims[l];
  for (int l = 1; l <= L; ++l) {
    plan->w_off[l] = off;
    off += (long long)dims[l] * dims[l - 1];
    plan->b_off[l] = off;
    off += dims[l];
  }
  if (compute == 1) return mlp_bf16_plan_create(plan, st, owned, why);
  const long long rows = (long long)G * B;
  auto alloc = [&](void** q, size_t bytes) -> cudaError_t {
    cudaError_t e = cudaMalloc(q, bytes);
    if (e != cudaSuccess) return e;
    owned->push_back(*q);
    return cudaMemsetAsync(*q, 0, bytes, st);
  };
  cudaError_t e;
  if ((e = alloc(reinterpret_cast<void**>(&plan->xb), sizeof(float) * rows * dims[0])) != cudaSuccess) return e;
  if ((e = alloc(reinterpret_cast<void**>(&plan->yb), sizeof(int) * rows)) != cudaSuccess) return e;
  for (int l = 1; l <= L; ++l) {
    if ((e = alloc(reinterpret_cast<void**>(&plan->act[l]), sizeof(float) * 2 * rows * dims[l])) != cudaSuccess) return e;
    if ((e = alloc(reinterpret_cast<void**>(&plan->dz[l]), sizeof(float) * 2 * rows * dims[l])) != cudaSuccess) return e;
  }
  plan->launches_per_iter = 3 * L + 2;
  if (head_fits(*plan)) {  // scores, loss gradient and the first backward-data product in one launch
    plan->launches_per_iter = 3 * L;
    if ((e = cudaFuncSetAttribute(mlp_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)head_smem_bytes(*plan))) != cudaSuccess)
      return e;
  }
  plan->skip_launches = plan->launches_per_iter;  // the same kernels; blocks of unselected groups and of the stale point exit at once
  if (L >= 2) {
    if ((e = cudaStreamCreateWithFlags(&plan->side, cudaStreamNonBlocking)) != cudaSuccess) return e;
    for (int l = 1; l <= L; ++l)
      if ((e = cudaEventCreateWithFlags(&plan->ev_dz[l], cudaEventDisableTiming)) != cudaSuccess) return e;
    if ((e = cudaEventCreateWithFlags(&plan->ev_join, cudaEventDisableTiming)) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

void mlp_plan_release(MlpPlan* plan) {
  if (plan->side) {
    cudaStreamSynchronize(plan->side);
    cudaStreamDestroy(plan->side);
    plan->side = nullptr;
  }
  for (int l = 0; l <= MLP_MAX_LAYERS; ++l)
    if (plan->ev_dz[l]) {
      cudaEventDestroy(plan->ev_dz[l]);
      plan->ev_dz[l] = nullptr;
    }
  if (plan->ev_join) {
    cudaEventDestroy(plan->ev_join);
    plan->ev_join = nullptr;
  }
}

cudaError_t launch_grad_mlp_post(const Params& P, const MlpPlan& pl, cudaStream_t st, int* n_launches) {
  *n_launches = 0;
  if (pl.compute == 1) return mlp_bf16_launch_post(P, pl, st, n_launches);
  return cudaSuccess;
}

cudaError_t mlp_group_gradient(const Params& P, const MlpPlan& pl, int g, float* row, cudaStream_t st) {
  if (pl.compute != 1) return cudaErrorNotSupported;
  return mlp_bf16_group_gradient(P, pl, g, row, st);
}

// ------------------------------------------------------------------ loss of the current iterate (reporting)
namespace {
constexpr int EVAL_CHUNK = 64;  // rows per "group" of the tile kernels
__global__ void __launch_bounds__(256) mlp_eval_convert_kernel(const __nv_bfloat16* X, long long ld, int d, long long rows,
                                                               float* out) {
  const long long n = rows * d;
  for (long long e = (long long)blockIdx.x * 256 + threadIdx.x; e < n; e += (long long)gridDim.x * 256) {
    const long long r = e / d;
    out[e] = __bfloat162float(X[r * ld + (e - r * d)]);
  }
}
// Warp per row: -ln softmax(scores)[y] in double; one partial sum per block.
__global__ void __launch_bounds__(256) mlp_eval_rows_kernel(const float* scores, const int* y, long long rows, int n_cls,
                                                            double* part) {
  __shared__ double scratch[40];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double local = 0.0;
  for (long long r = (long long)blockIdx.x * 8 + warp; r < rows; r += (long long)gridDim.x * 8) {
    const float* s = scores + r * n_cls;
    float mx = -3.0e38f;
    for (int c = lane; c < n_cls; c += 32) mx = fmaxf(mx, s[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    double sum = 0.0;
    for (int c = lane; c < n_cls; c += 32) sum += exp((double)s[c] - (double)mx);
    sum = warp_sum(sum);
    if (lane == 0) local += log(sum) + (double)mx - (double)s[y[r]];
  }
  const double tot = block_sum(local, scratch);
  if (threadIdx.x == 0) part[blockIdx.x] = tot;
}
// out[0] = (add ? out[0] : 0) + sum(part), divided by `div` when div > 0 (the last slab).
__global__ void __launch_bounds__(256) mlp_eval_add_kernel(const double* part, int n_part, int add, double div, double* out) {
  __shared__ double scratch[40];
  double s = 0.0;
  for (int i = threadIdx.x; i < n_part; i += 256) s += part[i];
  s = block_sum(s, scratch);
  if (threadIdx.x == 0) {
    double v = (add ? out[0] : 0.0) + s;
    if (div > 0.0) v /= div;
    out[0] = v;
  }
}
}  // namespace

cudaError_t mlp_eval_loss(const Params& P, const MlpPlan& pl, long long first, long long n, const MlpEvalScratch& sc,
                          double* out, cudaStream_t st) {
  const int L = pl.n_layers;
  cudaError_t e;
  for (long long s0 = 0; s0 < n; s0 += MLP_EVAL_SLAB) {
    const long long m = n - s0 < MLP_EVAL_SLAB ? n - s0 : MLP_EVAL_SLAB;
    const float* in = nullptr;
    long long in_ld = 0;
    int cur = 0;
    if (pl.compute == 1) {  // bf16 features: a dense fp32 copy of the slab
      mlp_eval_convert_kernel<<<592, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(P.X) + (first + s0) * P.ld, P.ld,
                                                   pl.dims[0], m, sc.buf[0]);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      in = sc.buf[0];
      in_ld = pl.dims[0];
      cur = 1;
    } else {
      in = reinterpret_cast<const float*>(P.X) + (first + s0) * P.ld;
      in_ld = P.ld;
    }
    for (int l = 1; l <= L; ++l) {
      const int ni = pl.dims[l - 1], no = pl.dims[l];
      float* outp = sc.buf[cur];
      // whole chunks of 64 rows as "groups" of the tile kernels at the current iterate, then the remaining rows
      for (int part = 0; part < 2; ++part) {
        const long long chunks = m / EVAL_CHUNK, done = chunks * EVAL_CHUNK;
        const long long rows_here = part == 0 ? EVAL_CHUNK : m - done;
        const long long groups = part == 0 ? chunks : 1;
        if (groups == 0 || rows_here == 0) continue;
        Params Q = P;
        Q.G = (int)groups;
        Q.B = (int)rows_here;
        Q.skip_unselected = 1;   // point 0 only ...
        Q.mask_cur = sc.ones;    // ... of every "group"
        GemmArgs a{};
        a.M = (int)rows_here;
        a.N = no;
        a.K = ni;
        a.A = Operand{in + (part == 0 ? 0 : done * in_ld), 0, (long long)EVAL_CHUNK * in_ld, 0, in_ld, 1, 0};
        a.Bm = Operand{nullptr, pl.w_off[l], 0, 0, 1, ni, 1};
        a.C = outp + (part == 0 ? 0 : done * no);
        a.c_zg = (long long)EVAL_CHUNK * no;
        a.c_zq = 0;
        a.c_rs = no;
        a.bias = 1;
        a.bias_off = pl.b_off[l];
        a.relu = l < L;
        if ((e = launch_gemm(Q, a, pl.sm_count, st)) != cudaSuccess) return e;
      }
      in = outp;
      in_ld = no;
      cur ^= 1;
    }
    mlp_eval_rows_kernel<<<512, 256, 0, st>>>(in, reinterpret_cast<const int*>(P.y) + first + s0, m, pl.dims[L], sc.part);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    mlp_eval_add_kernel<<<1, 256, 0, st>>>(sc.part, 512, s0 > 0 ? 1 : 0, s0 + m >= n ? (double)n : 0.0, out);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_grad_mlp(const Params& P, const MlpPlan& pl, cudaStream_t st, int* n_launches) {
  if (pl.compute == 1) return mlp_bf16_launch(P, pl, st, n_launches);
  const int L = pl.n_layers, G = P.G, B = P.B;
  const long long rows = (long long)G * B;
  int n = 0;
  cudaError_t e;
  // inside a captured chain (P.pdl) the gather is launched programmatically dependent on the previous
  // iteration's update kernel and runs beside it (784-200-10 network: 67.1 -> 64.9 us per iteration).  Launching
  // the forward product and the loss-gradient kernel in the same way, their blocks resident and waiting, was
  // slower (73.3 us): where nothing overlaps, a programmatic edge with an early release costs about a
  // microsecond more than an ordinary edge of the graph.
  if ((e = launch_k(mlp_gather_kernel, dim3((unsigned)((rows * 32 + 255) / 256)), dim3(256), 0, st,
                    P.pdl != 0 && P.k_off > 0, P, pl.xb, pl.yb, pl.dims[0])) != cudaSuccess)
    return e;
  ++n;
  // a small output layer: everything above the last hidden layer in one launch (see mlp_head_kernel)
  const size_t head_smem = head_smem_bytes(pl);
  const bool head = head_fits(pl);
  const int L_top = head ? L - 1 : L;   // layers handled by the tile kernels
  // forward
  for (int l = 1; l <= L_top; ++l) {
    const int ni = pl.dims[l - 1], no = pl.dims[l];
    GemmArgs a{};
    a.M = B;
    a.N = no;
    a.K = ni;
    if (l == 1)
      a.A = Operand{pl.xb, 0, (long long)B * ni, 0, ni, 1, 0};
    else
      a.A = Operand{pl.act[l - 1], 0, (long long)B * ni, rows * ni, ni, 1, 0};
    a.Bm = Operand{nullptr, pl.w_off[l], 0, 0, 1, ni, 1};  // B(k, n) = W_l[n][k]
    a.C = pl.act[l];
    a.c_zg = (long long)B * no;
    a.c_zq = rows * no;
    a.c_rs = no;
    a.bias = 1;
    a.bias_off = pl.b_off[l];
    a.relu = l < L;
    if ((e = launch_gemm(P, a, pl.sm_count, st)) != cudaSuccess) return e;
    ++n;
  }
  if (head) {
    HeadArgs h{};
    h.n1 = pl.dims[L - 1];
    h.nL = pl.dims[L];
    h.w_off = pl.w_off[L];
    h.b_off = pl.b_off[L];
    h.a1 = pl.act[L - 1];
    h.yb = pl.yb;
    h.dzL = pl.dz[L];
    h.dz1 = pl.dz[L - 1];
    mlp_head_kernel<<<dim3((B + 7) / 8, 2 * G), 256, head_smem, st>>>(P, h);
  } else {
    mlp_softmax_grad_kernel<<<(unsigned)((2 * rows * 32 + 255) / 256), 256, 0, st>>>(P, pl.act[L], pl.yb, pl.dz[L],
                                                                                    pl.dims[L]);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  ++n;
  // backward.  Main stream: the back-propagation chain dz_L -> ... -> dz_1, then dW_1.  Second stream (when
  // there is more than one layer): dW_l for l >= 2 as soon as dz_l is there, then all bias gradients.
  // (with the fused output layer dz_L and dz_{L-1} are both there already)
  const bool side = pl.side != nullptr;
  cudaStream_t s2 = side ? pl.side : st;
  if (side) {
    if ((e = cudaEventRecord(pl.ev_dz[L], st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(pl.side, pl.ev_dz[L], 0)) != cudaSuccess) return e;
  }
  for (int l = L; l >= 1; --l) {
    const int ni = pl.dims[l - 1], no = pl.dims[l];
    GemmArgs w{};  // dW_l = dz_l^T a_{l-1}
    w.M = no;
    w.N = ni;
    w.K = B;
    w.A = Operand{pl.dz[l], 0, (long long)B * no, rows * no, 1, no, 0};  // A(m, k) = dz_l[k][m]
    if (l == 1)
      w.Bm = Operand{pl.xb, 0, (long long)B * ni, 0, ni, 1, 0};
    else
      w.Bm = Operand{pl.act[l - 1], 0, (long long)B * ni, rows * ni, ni, 1, 0};
    w.c_grad = 1;
    w.c_off = pl.w_off[l];
    w.c_rs = ni;
    if ((e = launch_gemm(P, w, pl.sm_count, l == 1 ? st : s2)) != cudaSuccess) return e;
    ++n;
    if (l > 1 && !(head && l == L)) {
      GemmArgs d{};  // dz_{l-1} = (dz_l W_l) masked by a_{l-1} > 0
      d.M = B;
      d.N = ni;
      d.K = no;
      d.A = Operand{pl.dz[l], 0, (long long)B * no, rows * no, no, 1, 0};
      d.Bm = Operand{nullptr, pl.w_off[l], 0, 0, ni, 1, 1};  // B(k, n) = W_l[k][n]
      d.C = pl.dz[l - 1];
      d.c_zg = (long long)B * ni;
      d.c_zq = rows * ni;
      d.c_rs = ni;
      d.mask = pl.act[l - 1];
      if ((e = launch_gemm(P, d, pl.sm_count, st)) != cudaSuccess) return e;
      ++n;
      if (side) {
        if ((e = cudaEventRecord(pl.ev_dz[l - 1], st)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(pl.side, pl.ev_dz[l - 1], 0)) != cudaSuccess) return e;
      }
    }
  }
  const int L_bias = L;
  {
    BiasArgs ba{};
    int maxn = 0;
    for (int l = 1; l <= L_bias; ++l) {
      ba.dz[l] = pl.dz[l];
      ba.n[l] = pl.dims[l];
      ba.b_off[l] = pl.b_off[l];
      if (pl.dims[l] > maxn) maxn = pl.dims[l];
    }
    mlp_bias_grad_kernel<<<dim3((maxn + 255) / 256, 2 * G, L_bias), 256, 0, s2>>>(P, ba);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    ++n;
  }
  if (side) {
    if ((e = cudaEventRecord(pl.ev_join, pl.side)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(st, pl.ev_join, 0)) != cudaSuccess) return e;
  }
  *n_launches = n;
  return cudaSuccess;
}

}  // namespace gcada
