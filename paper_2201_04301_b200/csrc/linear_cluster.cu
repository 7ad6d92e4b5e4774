// Whole iterations of Algorithm 1 for narrow linear models inside ONE
// thread-block cluster.
//
// Workloads such as logistic regression on a few dozen features move about a
// megabyte per iteration: a chain of kernels (gradients, selection, update)
// spends its time in launch and dependency latency, not in memory traffic.
// Here a single cluster of up to 16 CTAs runs any number of iterations in one
// launch:
//   * the G*B minibatch rows of an iteration are dealt to all warps of the
//     cluster in batches of RR rows (warp per row, lane l owns columns
//     l + 32*i); each warp keeps the gradient at theta^k and its change since
//     the group's stale iterate in registers (the same cancellation-free
//     form as the multi-kernel path);
//   * warps are combined inside a CTA through shared memory, CTAs through
//     distributed shared memory after ONE hardware cluster barrier per
//     iteration (the exchange buffer is double-buffered, so no second barrier
//     is needed), always in a fixed order; a CTA works on a contiguous range
//     of batches, so a group's sum is read only from the CTAs that hold a
//     share of it;
//   * every CTA then holds every group's gradient and innovation norm and
//     redundantly evaluates Eq. (9), the age rule, the computing times and
//     wall-clock (Section II-B), the aggregate (Eq. 3) and Eq. (8a)-(8c) on
//     its own copy of the state in shared memory: identical inputs and
//     identical code give identical bits, so the copies never diverge.
// The iterate ring, h, v-hat, the aggregate and every group's last uploaded
// gradient live in shared memory for the whole launch; CTA 0 writes the mask
// history as it goes and the state back to global memory at the end.
#include <cooperative_groups.h>

#include "common.cuh"
#include "launch.h"

namespace gcada {

namespace cg = cooperative_groups;

namespace {

constexpr int LC_THREADS = 512, LC_WARPS = LC_THREADS / 32;

// a = f(z) - y (residual at theta^k); e = f(z) - f(z - dz) (its change), without cancellation.
template <bool QUAD>
__device__ __forceinline__ void residuals(float z, float dz, float y, float& a, float& e) {
  if (QUAD) {
    a = z - y;
    e = dz;
  } else {
    const float sz = 1.0f / (1.0f + expf(-z));
    const float snt = 1.0f / (1.0f + expf(z - dz));  // sigmoid(-(z - dz))
    a = sz - y;
    e = -expm1f(-dz) * sz * snt;
  }
}

// (hi, lo) += f - l with both rounding errors kept (TwoSum), as in the update kernel.
__device__ __forceinline__ void fold2(float& hi, float& lo, float f, float l) {
  const float dff = f - l;
  const float bb = dff - f;
  const float e1 = (f - (dff - bb)) + (-l - bb);
  const float s = hi + dff;
  const float b2 = s - hi;
  const float e2 = (hi - (s - b2)) + (dff - b2);
  hi = s;
  lo += e1 + e2;
}

// Sums V values over the 32 lanes with V-1 + log2(32/V) shuffles instead of 5 V: at each of the first
// log2(V) steps a lane keeps half of its values and hands the other half to its partner.  On return
// v[0] of lane l is the total of value number (l * V) / 32 (so 32 / V consecutive lanes hold the same one).
template <int V>
__device__ __forceinline__ void reduce_spread(float (&v)[V], int lane) {
  static_assert(V == 8 || V == 4, "8 or 4 values");
  const unsigned int full = 0xffffffffu;
  if (V == 8) {
    const bool up = lane & 16;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = up ? v[i] : v[i + 4], keep = up ? v[i + 4] : v[i];
      v[i] = keep + __shfl_xor_sync(full, send, 16);
    }
  }
  constexpr int W1 = V == 8 ? 8 : 16;  // lane bit of the step that halves four values to two
  {
    const bool up = lane & W1;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = up ? v[i] : v[i + 2], keep = up ? v[i + 2] : v[i];
      v[i] = keep + __shfl_xor_sync(full, send, W1);
    }
  }
  {
    const bool up = lane & (W1 >> 1);
    const float send = up ? v[0] : v[1], keep = up ? v[1] : v[0];
    v[0] = keep + __shfl_xor_sync(full, send, W1 >> 1);
  }
#pragma unroll
  for (int w = W1 >> 2; w >= 1; w >>= 1) v[0] += __shfl_xor_sync(full, v[0], w);
}

struct Carve {
  float *ring, *h, *vhat, *agg_hi, *agg_lo, *glast, *fresh, *innov, *part, *accw;
  double *s_ring, *lhs, *tg, *tw, *red, *lhsp;
  int* tau;
  unsigned char* mask;
};

__host__ __device__ inline size_t carve(unsigned char* base, int G, int M, int D, int pp, Carve* c) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    off = (off + 15) & ~(size_t)15;
    const size_t o = off;
    off += bytes;
    return o;
  };
  const size_t gp = (size_t)G * pp;
  const size_t o_ring = take(sizeof(float) * (size_t)(D + 1) * pp), o_h = take(4 * (size_t)pp), o_v = take(4 * (size_t)pp),
               o_ah = take(4 * (size_t)pp), o_al = take(4 * (size_t)pp), o_gl = take(4 * gp), o_fr = take(4 * gp),
               o_in = take(4 * gp), o_pa = take(4 * 2 * 2 * gp), o_aw = take(4 * (size_t)LC_WARPS * 2 * gp),
               o_sr = take(8 * (size_t)D), o_lhs = take(8 * (size_t)G), o_tg = take(8 * (size_t)G), o_tw = take(8 * (size_t)M),
               o_red = take(8 * 40), o_lhsp = take(8 * (size_t)G * 8), o_tau = take(4 * (size_t)G),
               o_mask = take((size_t)G);
  if (c) {
    c->ring = reinterpret_cast<float*>(base + o_ring);
    c->h = reinterpret_cast<float*>(base + o_h);
    c->vhat = reinterpret_cast<float*>(base + o_v);
    c->agg_hi = reinterpret_cast<float*>(base + o_ah);
    c->agg_lo = reinterpret_cast<float*>(base + o_al);
    c->glast = reinterpret_cast<float*>(base + o_gl);
    c->fresh = reinterpret_cast<float*>(base + o_fr);
    c->innov = reinterpret_cast<float*>(base + o_in);
    c->part = reinterpret_cast<float*>(base + o_pa);
    c->accw = reinterpret_cast<float*>(base + o_aw);
    c->s_ring = reinterpret_cast<double*>(base + o_sr);
    c->lhs = reinterpret_cast<double*>(base + o_lhs);
    c->tg = reinterpret_cast<double*>(base + o_tg);
    c->tw = reinterpret_cast<double*>(base + o_tw);
    c->red = reinterpret_cast<double*>(base + o_red);
    c->lhsp = reinterpret_cast<double*>(base + o_lhsp);
    c->tau = reinterpret_cast<int*>(base + o_tau);
    c->mask = base + o_mask;
  }
  return off;
}

template <int CPL, int RR, bool QUAD>
__global__ void __launch_bounds__(LC_THREADS, 1) linear_cluster_kernel(const Params P, int n_iters) {
  extern __shared__ __align__(16) unsigned char smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), cta = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = P.G, D = P.D, d = P.d, B = P.B, ring = P.D + 1;
  const int pp = (int)P.p_pad;
  const int gp2 = G * 2 * pp;  // floats of one (group, point, column) array
  Carve S;
  carve(smem, G, P.M, D, pp, &S);
  const float* Xf = reinterpret_cast<const float*>(P.X);
  const float* yf = reinterpret_cast<const float*>(P.y);

  // ---- state: global -> this CTA's shared memory
  DevState st = *P.st;  // every thread keeps the scalars it needs in registers; thread 0 of CTA 0 writes them back
  for (int e = tid; e < ring * pp; e += LC_THREADS) S.ring[e] = P.theta_ring[e];
  for (int e = tid; e < pp; e += LC_THREADS) {
    S.h[e] = P.h[e];
    S.vhat[e] = P.vhat[e];
    S.agg_hi[e] = P.agg_hi[e];
    S.agg_lo[e] = P.agg_lo[e];
  }
  for (int e = tid; e < G * pp; e += LC_THREADS) {
    const int g = e / pp, c = e - g * pp;
    S.glast[e] = P.gbuf[((long long)P.cur[g] * G + g) * pp + c];
    S.fresh[e] = 0.f;
  }
  for (int e = tid; e < D; e += LC_THREADS) S.s_ring[e] = P.s_ring[e];
  for (int e = tid; e < G; e += LC_THREADS) {
    S.tau[e] = P.tau[e];
    S.mask[e] = P.mask_cur[e];
  }
  __syncthreads();

  const int nb_g = (B + RR - 1) / RR;          // batches of RR rows per group
  const int n_batches = G * nb_g;
  // every CTA takes a contiguous range of batches, hence of groups: only the CTAs that worked on a group
  // hold a partial sum of it, and the exchange below reads only those.  Inside the CTA batches are dealt
  // warp-major, so that the last warp has the fewest (it also forms the right side of Eq. (9) while the
  // others fetch their first rows)
  const int bpc = (n_batches + C - 1) / C;
  const int b_lo = cta * bpc < n_batches ? cta * bpc : n_batches, b_hi = b_lo + bpc < n_batches ? b_lo + bpc : n_batches;
  const int wg = b_lo + warp, nw_tot = LC_WARPS;
  // (group, point, column) elements of this CTA's groups: [e_lo, e_hi)
  const int e_lo = b_lo < b_hi ? (b_lo / nb_g) * 2 * pp : 0, e_hi = b_lo < b_hi ? ((b_hi - 1) / nb_g + 1) * 2 * pp : 0;
  // ring positions are kept as small counters (no 64-bit division inside the loop)
  int kslot = (int)(st.k % ring), dslot = (int)(st.k % D), hslot = (int)(st.k % P.hist_cap);
  // computing times of the first iteration (those of iteration k+1 are drawn while iteration k updates)
  for (int m = LC_THREADS - 1 - tid; m < P.M; m += LC_THREADS) S.tw[m] = worker_time(P, (uint32_t)st.k, m);
  __syncthreads();

  for (int it = 0; it < n_iters; ++it) {
    const long long k = st.k;
    const uint32_t k32 = (uint32_t)k;
    const int kfill = k < D ? (int)k : D;       // how many earlier iterates exist, up to D
    const float* theta_k = S.ring + kslot * pp;
    float* accw_w = S.accw + (size_t)warp * gp2;
    for (int e = e_lo + lane; e < e_hi; e += 32) accw_w[e] = 0.f;  // groups this warp does not visit contribute zero
    __syncwarp();

    // the last warp forms the right side of Eq. (9) (it depends on earlier iterations only)
    if (warp == LC_WARPS - 1 && lane == 0) {
      double rhs = 0.0;
      for (int dd = 1; dd <= kfill; ++dd) {  // ||theta^{k+1-dd} - theta^{k-dd}||^2 sits in slot (k-dd) mod D
        int sl = dslot - dd;
        if (sl < 0) sl += D;
        rhs += (P.c_d ? P.c_d[dd - 1] : P.c) * S.s_ring[sl];
      }
      S.red[39] = rhs;
    }

    // ---- gradients: this warp's batches (ascending, so its groups come in one run each); the rows of
    // the next batch are fetched before the current one is worked on
    float th[CPL], ths[CPL], acc0[CPL], acc1[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) th[i] = lane + 32 * i < pp ? theta_k[lane + 32 * i] : 0.f;  // (the pad of a p-vector is zero)
    int cur_g = -1;
    constexpr int SPREAD = 32 / RR;  // lanes that end up holding the same row's dot products
    auto fetch = [&](int b, float& yy, float (&x)[RR][CPL]) {
      const int g = b / nb_g, rb = (b - g * nb_g) * RR;
      long long myrow = 0;
      yy = 0.f;
      if (lane < RR && rb + lane < B) {
        myrow = batch_row(P, k32, g, rb + lane);
        yy = yf[myrow];
      }
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        const long long row = __shfl_sync(0xffffffffu, myrow, r);
        const bool valid = rb + r < B;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          const int c = lane + 32 * i;
          x[r][i] = (valid && c < d) ? Xf[row * P.ld + c] : 0.f;
        }
      }
    };
    float xc[RR][CPL], yc = 0.f;
    int b = wg;
    if (b < b_hi) fetch(b, yc, xc);
    while (b < b_hi) {
      const int bn = b + nw_tot;
      float xn[RR][CPL], yn = 0.f;
      constexpr bool PREFETCH = RR * CPL <= 16;  // wider rows would not fit two batches in registers
      if (PREFETCH && bn < b_hi) fetch(bn, yn, xn);
      const int g = b / nb_g, rb = (b - g * nb_g) * RR;
      if (g != cur_g) {
        if (cur_g >= 0) {
#pragma unroll
          for (int i = 0; i < CPL; ++i)
            if (lane + 32 * i < pp) {
              accw_w[(cur_g * 2 + 0) * pp + lane + 32 * i] = acc0[i];
              accw_w[(cur_g * 2 + 1) * pp + lane + 32 * i] = acc1[i];
            }
        }
        cur_g = g;
        // stale iterate theta^{k - min(tau, D)} (theta^0 before the run began)
        int age = S.tau[g] < kfill ? S.tau[g] : kfill;
        int sslot = kslot - age;
        if (sslot < 0) sslot += ring;
        const float* theta_s = S.ring + sslot * pp;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          ths[i] = lane + 32 * i < pp ? th[i] - theta_s[lane + 32 * i] : 0.f;
          acc0[i] = 0.f;
          acc1[i] = 0.f;
        }
      }
      float z[RR], zs[RR];
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        z[r] = 0.f;
        zs[r] = 0.f;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          z[r] += xc[r][i] * th[i];
          zs[r] += xc[r][i] * ths[i];
        }
      }
      reduce_spread<RR>(z, lane);
      reduce_spread<RR>(zs, lane);
      // lane l now holds both dot products of row l / SPREAD and turns them into that row's two coefficients
      // (every lane used to repeat this for all RR rows)
      const int my_r = lane / SPREAD;
      const float my_y = __shfl_sync(0xffffffffu, yc, my_r);
      float my_a = 0.f, my_e = 0.f;
      if (rb + my_r < B) residuals<QUAD>(z[0], zs[0], my_y, my_a, my_e);
      my_a *= P.scale;
      my_e *= P.scale;
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        const float a = __shfl_sync(0xffffffffu, my_a, r * SPREAD), e = __shfl_sync(0xffffffffu, my_e, r * SPREAD);
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          acc0[i] += a * xc[r][i];
          acc1[i] += e * xc[r][i];
        }
      }
      if (!PREFETCH && bn < b_hi) fetch(bn, yn, xn);
      b = bn;
      yc = yn;
#pragma unroll
      for (int r = 0; r < RR; ++r)
#pragma unroll
        for (int i = 0; i < CPL; ++i) xc[r][i] = xn[r][i];
    }
    if (cur_g >= 0) {
#pragma unroll
      for (int i = 0; i < CPL; ++i)
        if (lane + 32 * i < pp) {
          accw_w[(cur_g * 2 + 0) * pp + lane + 32 * i] = acc0[i];
          accw_w[(cur_g * 2 + 1) * pp + lane + 32 * i] = acc1[i];
        }
    }
    __syncthreads();

    // ---- warps -> CTA partial (fixed order), published in this iteration's exchange buffer
    float* part = S.part + (size_t)(it & 1) * gp2;
    for (int e = e_lo + tid; e < e_hi; e += LC_THREADS) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < LC_WARPS; ++w) s += S.accw[(size_t)w * gp2 + e];
      part[e] = s;
    }
    cluster.sync();  // the one cluster-wide barrier of the iteration

    // ---- CTA partials -> every group's gradient and innovation, in every CTA (CTA order).  One element per
    // thread; the 32 elements of a warp lie in one (group, point) row, so the warp also forms its share of
    // the squared innovation norm
    for (int e = tid; e < gp2; e += LC_THREADS) {
      const int gq = e / pp, c = e - gq * pp, g = gq >> 1;
      const int r_lo = (g * nb_g) / bpc, r_hi = ((g + 1) * nb_g - 1) / bpc;  // the CTAs that worked on group g
      float v[16];  // all remote loads in flight before the first add
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] = r_lo + j <= r_hi ? cluster.map_shared_rank(part, r_lo + j)[e] : 0.f;
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) s += v[j];
      if (gq & 1) {
        S.innov[g * pp + c] = s;
        const double nrm = warp_sum((double)s * (double)s);
        if (lane == 0) S.lhsp[g * 8 + (c >> 5)] = nrm;
      } else {
        S.fresh[g * pp + c] = s;
      }
    }
    __syncthreads();

    // ---- the server's decision (Eq. 9, the age rule), ages, clock and counters
    if (tid < G) {
      const int g = tid, tau = S.tau[g];
      const double rhs = S.red[39];
      double lhs = 0.0;
      for (int ch = 0; ch < (pp >> 5); ++ch) lhs += S.lhsp[g * 8 + ch];  // LHS_g = ||innovation_g||^2
      S.lhs[g] = lhs;
      double t = 1.0e300;
      for (int m = g * P.M_G; m < (g + 1) * P.M_G; ++m) t = fmin(t, S.tw[m]);
      const bool sel = (tau >= D) || (lhs > rhs);
      S.tg[g] = t;
      S.mask[g] = sel ? 1 : 0;
      S.tau[g] = sel ? 1 : tau + 1;
      if (cta == 0 && GCADA_INDEX_OK(P.st, (long long)hslot * G + g, P.lim.hist_bytes, CHK_HIST))
        P.hist[(long long)hslot * G + g] = sel ? 1 : 0;
    }
    __syncthreads();
    int nsel = 0;
    double tmax = 0.0;
    for (int g = 0; g < G; ++g)
      if (S.mask[g]) {
        ++nsel;
        tmax = fmax(tmax, S.tg[g]);
      }
    st.uploads += (unsigned long long)nsel;
    st.comm += (unsigned long long)nsel * (unsigned long long)(P.M_G + 1);
    st.comp += (unsigned long long)nsel * (unsigned long long)P.M_G;
    st.wall += tmax;
    st.last_dt = tmax;
    st.rhs = S.red[39];

    // ---- aggregate (Eq. 3) and Eq. (8a)-(8c): one thread per coordinate; the threads at the other end of the
    // block meanwhile draw the computing times of the next iteration
    const float alpha_k = step_size(P, k);
    int nslot = kslot + 1;
    if (nslot == ring) nslot = 0;
    float* theta_n = S.ring + nslot * pp;
    double sq = 0.0;
    for (int c = tid; c < pp; c += LC_THREADS) {
      float hi = S.agg_hi[c], lo = S.agg_lo[c];
      for (int g = 0; g < G; ++g)
        if (S.mask[g]) {
          fold2(hi, lo, S.fresh[g * pp + c], S.glast[g * pp + c]);
          S.glast[g * pp + c] = S.fresh[g * pp + c];
        }
      const float t = hi + lo;
      lo = lo - (t - hi);
      hi = t;
      S.agg_hi[c] = hi;
      S.agg_lo[c] = lo;
      const float hh = P.beta1 * S.h[c] + P.omb1 * hi;
      const float v = P.beta2 * S.vhat[c] + P.omb2 * (hi * hi);
      const float vh = fmaxf(S.vhat[c], v);
      const float up = alpha_k * hh / sqrtf(P.eps + vh);
      S.h[c] = hh;
      S.vhat[c] = vh;
      theta_n[c] = theta_k[c] - up;
      sq += (double)up * (double)up;
    }
    if (warp < (pp + 31) / 32 || warp < 8) {  // the warps that hold coordinates (p_pad <= 256: at most 8)
      sq = warp_sum(sq);
      if (lane == 0 && warp < 8) S.red[warp] = sq;
    }
    for (int m = LC_THREADS - 1 - tid; m < P.M; m += LC_THREADS) S.tw[m] = worker_time(P, k32 + 1u, m);
    __syncthreads();
    if (tid == 0) {
      double s = 0.0;
      for (int w = 0; w < 8; ++w) s += S.red[w];  // warps without coordinates contributed zero
      S.s_ring[dslot] = s;
    }
    st.k = k + 1;
    kslot = nslot;
    if (++dslot == D) dslot = 0;
    if (++hslot == P.hist_cap) hslot = 0;
    __syncthreads();
  }

  // ---- state back to global memory (CTA 0; every CTA holds the same bits)
  if (cta == 0) {
    for (int e = tid; e < ring * pp; e += LC_THREADS) P.theta_ring[e] = S.ring[e];
    for (int e = tid; e < pp; e += LC_THREADS) {
      P.h[e] = S.h[e];
      P.vhat[e] = S.vhat[e];
      P.agg_hi[e] = S.agg_hi[e];
      P.agg_lo[e] = S.agg_lo[e];
    }
    for (int e = tid; e < G * pp; e += LC_THREADS) {
      const int g = e / pp, c = e - g * pp;
      const int cur = P.cur[g];
      P.gbuf[((long long)cur * G + g) * pp + c] = S.glast[e];
      // an unselected group's fresh gradient of the last iteration sits in its other row
      if (n_iters > 0 && !S.mask[g]) P.gbuf[((long long)(1 - cur) * G + g) * pp + c] = S.fresh[e];
    }
    for (int e = tid; e < D; e += LC_THREADS) P.s_ring[e] = S.s_ring[e];
    for (int e = tid; e < G; e += LC_THREADS) {
      P.tau[e] = S.tau[e];
      P.mask_cur[e] = S.mask[e];
      P.lhs[e] = S.lhs[e];
      P.t_g[e] = S.tg[e];
    }
    if (tid == 0) {
      st.err = P.st->err;
      st.k_chain = st.k;
      *P.st = st;
    }
  }
  cluster.sync();  // no CTA leaves while another may still read its exchange buffer
}

template <int CPL, int RR>
cudaError_t launch_cpl(const Params& P, const ClusterPlan& plan, bool quad, int n_iters, cudaStream_t st) {
  void (*kern)(const Params, int) = quad ? linear_cluster_kernel<CPL, RR, true> : linear_cluster_kernel<CPL, RR, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (e != cudaSuccess) return e;
  if (plan.n_cta > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(plan.n_cta);
  cfg.blockDim = dim3(LC_THREADS);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = plan.n_cta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, P, n_iters);
}

// The cluster kernel's launch shape with nothing in it but its one cluster-wide barrier per iteration:
// the floor an iteration of this design cannot go below (measurement aid).
__global__ void __launch_bounds__(LC_THREADS, 1) linear_cluster_empty_kernel(int n_iters) {
  cg::cluster_group cluster = cg::this_cluster();
  for (int i = 0; i < n_iters; ++i) cluster.sync();
}

}  // namespace

cudaError_t launch_linear_cluster_empty(const ClusterPlan& plan, int n_iters, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(linear_cluster_empty_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)plan.smem_bytes);
  if (e != cudaSuccess) return e;
  if (plan.n_cta > 8) {
    e = cudaFuncSetAttribute(linear_cluster_empty_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(plan.n_cta);
  cfg.blockDim = dim3(LC_THREADS);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = plan.n_cta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, linear_cluster_empty_kernel, n_iters);
}

bool plan_linear_cluster(int d, int G, int M, int D, int B, long long p_pad, size_t smem_optin, ClusterPlan* plan) {
  plan->usable = false;
  if (d > 256 || G > 64 || M > 1024 || G * p_pad > 2048 || (long long)(D + 1) * p_pad > 8192) return false;
  plan->cpl = d <= 32 ? 1 : (d <= 64 ? 2 : (d <= 128 ? 4 : 8));
  plan->rr = plan->cpl <= 2 ? 8 : 4;
  plan->smem_bytes = carve(nullptr, G, M, D, (int)p_pad, nullptr) + 16;
  if (plan->smem_bytes > smem_optin) return false;
  const long long batches = (long long)G * ((B + plan->rr - 1) / plan->rr);
  long long c = (batches + 2 * LC_WARPS - 1) / (2 * LC_WARPS);  // about two batches per warp
  plan->n_cta = (int)(c < 1 ? 1 : (c > 16 ? 16 : c));
  plan->usable = true;
  return true;
}

cudaError_t launch_linear_cluster(const Params& P, const ClusterPlan& plan, bool quad, int n_iters, cudaStream_t st) {
  switch (plan.cpl) {
    case 1: return launch_cpl<1, 8>(P, plan, quad, n_iters, st);
    case 2: return launch_cpl<2, 8>(P, plan, quad, n_iters, st);
    case 4: return launch_cpl<4, 4>(P, plan, quad, n_iters, st);
    default: return launch_cpl<8, 4>(P, plan, quad, n_iters, st);
  }
}

}  // namespace gcada
