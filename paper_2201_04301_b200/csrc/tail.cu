// Server-side kernels of one G-CADA iteration.
//
// select_kernel: adds the gradient partial sums of every group in a fixed
//   order, forms LHS_g = ||fresh_g - stale_g||^2 (the gradient innovation the
//   left side of Eq. (9) estimates; the linear-model kernels hand over the
//   innovation itself, the MLP kernels both gradients), and its last block
//   evaluates the right side c * sum_d ||theta^{k+1-d} - theta^{k-d}||^2, the age rule tau_g >= D
//   (Section IV), the selection mask, the ages for the next iteration
//   (Algorithm 1, last step), the workers' computing times with the
//   fastest-in-group / slowest-selected-group wall-clock (Section II-B,
//   Section V-A) and the load counters (Eqs. 5, 6, 19, 22).
// update_kernel: swaps the selected groups' fresh gradients into the lazily
//   aggregated gradient (Eq. 3), applies Eq. (8a)-(8c), stores theta^{k+1} in
//   the iterate ring and ||theta^{k+1} - theta^k||^2 in the ring of squared
//   step norms that feeds the next D right sides.
#include "common.cuh"
#include "launch.h"

namespace gcada {

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

// what: SEL_ALL = reduce the partial sums, then schedule (last block); SEL_SCHEDULE = schedule only (one
// block; the left sides come from lhs_part as it stands, or from rule PS); SEL_REDUCE = reduce only (skip
// mode: the gradient kernels ran after the scheduling, on the selected groups, and only their partial sums
// have to become gradients).
enum { SEL_ALL = 0, SEL_SCHEDULE = 1, SEL_REDUCE = 2 };

template <int U>
__global__ void __launch_bounds__(256) select_kernel(const Params P, int blocks_x, int what) {
  __shared__ double scratch[40];
  __shared__ int sh_nsel[8];
  __shared__ int sh_cnt[8];
  __shared__ double sh_tmax[8];
  __shared__ double tw_sm[1024];
  __shared__ double lhs_sm[256];
  __shared__ bool is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = blockIdx.y;
  const long long cols4 = P.p_pad >> 2;
  pdl_wait();  // (no pdl_launch_dependents here: see enqueue_iteration)
  const long long k = P.st->k;

  // ---- phase 1: partial sums -> fresh_g (and stale_g), innovation norm
  // (skipped when the gradient kernels have already delivered the norm partial sums)
  const bool tg_early = P.pm.n_cta >= 0 && what == SEL_ALL;  // the groups' computing times are taken in phase 1
  if (P.pm.n_cta >= 0 && what != SEL_SCHEDULE) {
    // The group's computing time (fastest of its workers, Section II-B) needs nothing from the gradients: the
    // first warp of the group's first block takes it here, off the single block's chain of phase 2.
    if (tg_early && blockIdx.x == 0 && warp == 0) {
      double t = 1.0e300;
      for (int j = lane; j < P.M_G; j += 32) t = fmin(t, worker_time(P, (uint32_t)k, g * P.M_G + j));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) t = fmin(t, __shfl_xor_sync(0xffffffffu, t, o));
      if (lane == 0) P.t_g[g] = t;  // (thread 0: published by the fence before this block's ticket)
    }
    // skip mode: the group's rank among the selected ones locates its partial sums, and its fresh gradient
    // goes to the row that the flip of cur[g] has already made the last uploaded one
    int gi = g, n_groups = P.G;
    if (what == SEL_REDUCE) {
      if (!P.mask_cur[g]) return;
      int before = 0, total = 0;
      for (int j = tid; j < P.G; j += 256) {
        const int m = P.mask_cur[j] != 0;
        total += m;
        before += (j < g) ? m : 0;
      }
      gi = (int)(block_sum((double)before, scratch) + 0.5);
      n_groups = (int)(block_sum((double)total, scratch) + 0.5);
    }
    if (!GCADA_INDEX_OK(P.st, P.cur[g], 2, CHK_GRAD_ROW) ||
        !GCADA_INDEX_OK(P.st, (long long)P.G + g, P.lim.grad_rows, CHK_GRAD_ROW))
      return;  // (debug library: the group's two gradient rows are rows g and G + g of gbuf)
    float* fresh_g = what == SEL_REDUCE ? last_row(P, g) : fresh_row(P, g);
    int c_lo = 0, c_hi = -1;
    const long long Rtot = (long long)n_groups * P.pm.rows_per_group;
    // CTA c of the gradient kernel owns rows [c*Rtot/n, (c+1)*Rtot/n), n = the CTAs that got rows (all of them
    // unless only a few selected groups compute); 32-bit arithmetic where the products fit
    const int n = (P.pm.n_cta > 0 && Rtot < (long long)P.pm.n_cta) ? (int)Rtot : P.pm.n_cta;
    const bool small = (Rtot + 1) * (long long)(n + 1) < 0x7fffffffLL;
    if (n > 0) {
      const long long x0 = (long long)gi * P.pm.rows_per_group;
      const long long x1 = x0 + P.pm.rows_per_group - 1;
      if (small) {
        c_lo = (int)(((unsigned)(x0 + 1) * (unsigned)n - 1u) / (unsigned)Rtot);
        c_hi = (int)(((unsigned)(x1 + 1) * (unsigned)n - 1u) / (unsigned)Rtot);
      } else {
        c_lo = (int)(((x0 + 1) * n - 1) / Rtot);
        c_hi = (int)(((x1 + 1) * n - 1) / Rtot);
      }
    }
    double local = 0.0;
  #pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i4 = ((long long)blockIdx.x * U + u) * 256 + tid;
      if (i4 >= cols4) continue;
      float4 f, s;
      if (n > 0) {
        f = make_float4(0.f, 0.f, 0.f, 0.f);
        s = f;
        for (int c0 = c_lo; c0 <= c_hi; c0 += 4) {  // four partial sums per round: loads first, adds in CTA order
          float4 a[4], b[4];
  #pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int c = c0 + u;
            if (c <= c_hi) {
              const int gf = small ? (int)(((unsigned)c * (unsigned)Rtot / (unsigned)n) / (unsigned)P.pm.rows_per_group)
                                   : (int)(((long long)c * Rtot / n) / P.pm.rows_per_group);
              const float* src = P.partial + ((long long)(c * P.pm.maxseg + (gi - gf)) * 2) * P.p_pad + i4 * 4;
              a[u] = ld4(src);
              b[u] = ld4(src + P.p_pad);
            }
          }
  #pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (c0 + u <= c_hi) {
              f.x += a[u].x; f.y += a[u].y; f.z += a[u].z; f.w += a[u].w;
              s.x += b[u].x; s.y += b[u].y; s.z += b[u].z; s.w += b[u].w;
            }
          }
        }
        // second slot half = innovation; the stale-point gradient is fresh - innovation
        st4(fresh_g + i4 * 4, f);
        if (P.stale)
          st4(P.stale + (long long)g * P.p_pad + i4 * 4, make_float4(f.x - s.x, f.y - s.y, f.z - s.z, f.w - s.w));
      } else {
        f = ld4(fresh_g + i4 * 4);
        s = ld4(P.stale + (long long)g * P.p_pad + i4 * 4);
        s = make_float4(f.x - s.x, f.y - s.y, f.z - s.z, f.w - s.w);
      }
      const float dx = s.x, dy = s.y, dz = s.z, dw = s.w;  // the innovation
      local += (double)dx * dx + (double)dy * dy + (double)dz * dz + (double)dw * dw;
    }
    if (what == SEL_REDUCE) return;
    const double tot = block_sum(local, scratch);
    if (tid == 0) {
      if (GCADA_INDEX_OK(P.st, (long long)g * blocks_x + blockIdx.x, P.lim.lhs_parts, CHK_LHS_PART))
        P.lhs_part[(long long)g * blocks_x + blockIdx.x] = tot;
      __threadfence();
      const unsigned int total = (unsigned int)blocks_x * (unsigned int)P.G;
      is_last = atomicAdd(&P.st->ticket_select, 1u) == total - 1u;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
  }

  // ---- phase 2 (last block only): the server's scheduling decision.
  // One thread per group, 256 groups at a time; everything a group needs is
  // fetched in one round of independent loads.
  // Everything below is one dependency chain in one block, so all loads are issued before the arithmetic
  // that does not need them (the computing times) and consumed after it.
  // Right side of Eq. (9).  With one constant c it is c times the sum of the ring of squared step norms
  // (slots of steps that have not happened yet hold zero), which needs no slot arithmetic.
  constexpr int RING_REGS = 16;
  const bool ring_in_regs = !P.c_d && P.D <= RING_REGS;
  double sv[RING_REGS];
#pragma unroll
  for (int i = 0; i < RING_REGS; ++i) sv[i] = (ring_in_regs && i < P.D) ? P.s_ring[i] : 0.0;
  double rhs = 0.0;
  const uint32_t k32 = (uint32_t)k;
  const volatile double* parts = P.lhs_part;
  // (the counters that thread 0 advances at the end are fetched now, with everything else)
  unsigned long long up0 = 0ull, comm0 = 0ull, comp0 = 0ull;
  double wall0 = 0.0;
  if (tid == 0) {
    up0 = P.st->uploads;
    comm0 = P.st->comm;
    comp0 = P.st->comp;
    wall0 = P.st->wall;
  }
  int nsel = 0;
  int listed = 0;  // selected groups of earlier chunks (the same in every thread)
  double tmax = 0.0;
  for (int gc = 0; gc < P.G; gc += 256) {
    const int gg = gc + tid;
    const bool have = gg < P.G;
    const int ng = P.G - gc < 256 ? P.G - gc : 256;
    // loads first: age, forced bit, partial sums of the innovation norm
    const int tau = have ? P.tau[gg] : 0;
    bool sel_forced = false;
    if (have && P.forced) sel_forced = P.forced[(k - P.forced_base) * P.G + gg] != 0;
    double lhs = 0.0;
    constexpr int PART_REGS = 8;
    double pv[PART_REGS];
    if (blocks_x <= PART_REGS) {  // issued now, added (in block order) after the computing times
#pragma unroll
      for (int b = 0; b < PART_REGS; ++b) pv[b] = (have && b < blocks_x) ? parts[(long long)gg * blocks_x + b] : 0.0;
    } else if (blocks_x <= 64) {
      if (have)
        for (int b = 0; b < blocks_x; ++b) lhs += parts[(long long)gg * blocks_x + b];
    } else {
      for (int lg = warp; lg < ng; lg += 8) {
        double v = 0.0;
        for (int b = lane; b < blocks_x; b += 32) v += parts[(long long)(gc + lg) * blocks_x + b];
        v = warp_sum(v);
        if (lane == 0) lhs_sm[lg] = v;
      }
      __syncthreads();
      if (have) lhs = lhs_sm[tid];
    }
    // computing times: one thread per worker into shared memory (tiles of 1024
    // workers), then each group's thread takes the minimum over its workers
    double t = 1.0e300;
    if (tg_early && have) t = reinterpret_cast<const volatile double*>(P.t_g)[gg];
    const long long w_lo = (long long)gc * P.M_G, w_hi = tg_early ? w_lo : (long long)(gc + ng) * P.M_G;
    for (long long m0 = w_lo; m0 < w_hi; m0 += 1024) {
      const int cnt = (int)(w_hi - m0 < 1024 ? w_hi - m0 : 1024);
      __syncthreads();
      for (int i = tid; i < cnt; i += 256) tw_sm[i] = worker_time(P, k32, (int)(m0 + i));
      __syncthreads();
      if (have) {
        const long long lo = (long long)gg * P.M_G > m0 ? (long long)gg * P.M_G : m0;
        const long long hi = (long long)(gg + 1) * P.M_G < m0 + cnt ? (long long)(gg + 1) * P.M_G : m0 + cnt;
        for (long long m = lo; m < hi; ++m) t = fmin(t, tw_sm[m - m0]);
      }
    }
    bool sel = false;
    if (blocks_x <= PART_REGS) {
#pragma unroll
      for (int b = 0; b < PART_REGS; ++b) lhs += pv[b];
    }
    if (gc == 0) {
      if (ring_in_regs) {
#pragma unroll
        for (int i = 0; i < RING_REGS; ++i) rhs += sv[i];
        rhs *= P.c;
      } else {
        int slot = (int)(k % P.D);  // ||theta^{k+1-d} - theta^{k-d}||^2 sits in slot (k-d) mod D
        const int terms = k < P.D ? (int)k : P.D;
        for (int d = 1; d <= terms; ++d) {
          if (--slot < 0) slot = P.D - 1;
          rhs += (P.c_d ? P.c_d[d - 1] : P.c) * P.s_ring[slot];
        }
      }
    }
    if (have) {
      if (P.ps_L2) lhs = P.ps_lhs[gg];  // rule PS: the test uses the printed left side, not the measured innovation
      sel = P.forced ? sel_forced : ((tau >= P.D) || (lhs > rhs));
      P.lhs[gg] = lhs;
      P.t_g[gg] = t;
      P.mask_cur[gg] = sel ? 1 : 0;
      if (GCADA_INDEX_OK(P.st, (k % P.hist_cap) * P.G + gg, P.lim.hist_bytes, CHK_HIST))
        P.hist[(k % P.hist_cap) * P.G + gg] = sel ? 1 : 0;
      P.tau[gg] = sel ? 1 : tau + 1;
      if (sel) P.cur[gg] ^= 1;  // the fresh gradient's row becomes the last uploaded one
      if (sel) {
        ++nsel;
        tmax = fmax(tmax, t);
      }
    }
    // ascending list of the selected groups (for kernels that work on the selected groups only)
    {
      const unsigned int b = __ballot_sync(0xffffffffu, sel);
      __syncthreads();
      if (lane == 0) sh_cnt[warp] = __popc(b);
      __syncthreads();
      int base = listed, all = 0;
      for (int w = 0; w < 8; ++w) {
        if (w < warp) base += sh_cnt[w];
        all += sh_cnt[w];
      }
      if (sel && GCADA_INDEX_OK(P.st, base + __popc(b & ((1u << lane) - 1u)), P.G, CHK_SEL_LIST))
        P.sel_list[base + __popc(b & ((1u << lane) - 1u))] = gg;
      listed += all;
    }
  }
  if (tid == 0) P.sel_count[0] = listed;
  // block-wide count and maximum
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    nsel += __shfl_xor_sync(0xffffffffu, nsel, o);
    tmax = fmax(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  }
  if (lane == 0) {
    sh_nsel[warp] = nsel;
    sh_tmax[warp] = tmax;
  }
  __syncthreads();
  if (tid == 0) {
    int ns = 0;
    double tm = 0.0;
    for (int w = 0; w < 8; ++w) {
      ns += sh_nsel[w];
      tm = fmax(tm, sh_tmax[w]);
    }
    DevState* st = P.st;
    st->uploads = up0 + (unsigned long long)ns;
    st->comm = comm0 + (unsigned long long)ns * (unsigned long long)(P.M_G + 1);
    st->comp = comp0 + (unsigned long long)ns * (unsigned long long)P.M_G;
    st->wall = wall0 + tm;
    st->last_dt = tm;
    st->rhs = rhs;
    st->ticket_select = 0u;
  }
}

// Error-free difference and compensated accumulation: (hi, lo) += f - l with
// the rounding errors of both operations kept in lo (Knuth's TwoSum), so that
// the aggregate stays equal to the sum of the last uploaded gradients however
// many swaps have been folded in.
__device__ __forceinline__ void fold(float& hi, float& lo, float f, float l) {
  const float dff = f - l;
  const float bb = dff - f;
  const float e1 = (f - (dff - bb)) + (-l - bb);
  const float s = hi + dff;
  const float b2 = s - hi;
  const float e2 = (hi - (s - b2)) + (dff - b2);
  hi = s;
  lo += e1 + e2;
}
__device__ __forceinline__ void renorm(float& hi, float& lo) {
  const float t = hi + lo;
  lo = lo - (t - hi);
  hi = t;
}

// Block = 32 float4 columns (lanes) x 8 warps.  Warp w folds the selected
// groups number w, w+8, ... of the (ascending) list into its own compensated
// partial sum; the eight partial sums are then added to the aggregate in warp
// order, so the result does not depend on timing.
__global__ void __launch_bounds__(256) update_kernel(const Params P) {
  extern __shared__ int sel_list[];  // selected groups, ascending; bit 30 set = the group's cur[] is 1
  __shared__ int n_sel_sh;
  __shared__ float4 wsum_hi[8][32], wsum_lo[8][32];
  __shared__ bool is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long cols4 = P.p_pad >> 2;
  pdl_launch_dependents();
  pdl_wait();
  const long long k = P.st->k;
  const int ring = P.D + 1;
  const float alpha_k = step_size(P, k);

  if (warp == 0) {
    int cnt = 0;
    for (int g0 = 0; g0 < P.G; g0 += 32) {
      const int gg = g0 + lane;
      const bool s = gg < P.G && P.mask_cur[gg] != 0;
      const int cur = gg < P.G ? P.cur[gg] : 0;  // read with the mask, so that the fold need not wait for it
      const unsigned int b = __ballot_sync(0xffffffffu, s);
      if (s) sel_list[cnt + __popc(b & ((1u << lane) - 1u))] = gg | (cur << 30);
      cnt += __popc(b);
    }
    if (lane == 0) n_sel_sh = cnt;
  }
  const long long i4 = (long long)blockIdx.x * 32 + lane;
  const bool active = i4 < cols4;
  const long long o = i4 * 4;
  // the vectors Eq. (8) needs do not depend on the selection: fetched now, used after the fold
  float4 ahi = make_float4(0.f, 0.f, 0.f, 0.f), alo = ahi, h = ahi, vh = ahi, th = ahi;
  if (warp == 0 && active) {
    ahi = ld4(P.agg_hi + o);
    alo = ld4(P.agg_lo + o);
    h = ld4(P.h + o);
    vh = ld4(P.vhat + o);
    th = ld4(P.theta_ring + (k % ring) * P.p_pad + o);
  }
  __syncthreads();
  const int n_sel = n_sel_sh;

  float4 hi = make_float4(0.f, 0.f, 0.f, 0.f), lo = hi;
  if (active) {
    for (int j0 = warp; j0 < n_sel; j0 += 32) {  // four groups of this warp per round, loads first
      float4 f[4], l[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j = j0 + 8 * u;
        if (j < n_sel) {
          const int e = sel_list[j], g = e & 0x3fffffff, cur = e >> 30;
          f[u] = ld4(P.gbuf + ((long long)cur * P.G + g) * P.p_pad + o);        // selected: cur[g] already points at the fresh gradient
          l[u] = ld4(P.gbuf + ((long long)(1 - cur) * P.G + g) * P.p_pad + o);  // the gradient it replaces
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (j0 + 8 * u < n_sel) {
          fold(hi.x, lo.x, f[u].x, l[u].x);
          fold(hi.y, lo.y, f[u].y, l[u].y);
          fold(hi.z, lo.z, f[u].z, l[u].z);
          fold(hi.w, lo.w, f[u].w, l[u].w);
        }
      }
    }
  }
  wsum_hi[warp][lane] = hi;
  wsum_lo[warp][lane] = lo;
  __syncthreads();
  if (warp == 0) {
    double local = 0.0;
    if (active) {
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const float4 h2 = wsum_hi[w][lane], l2 = wsum_lo[w][lane];
        fold(ahi.x, alo.x, h2.x, 0.f);
        fold(ahi.y, alo.y, h2.y, 0.f);
        fold(ahi.z, alo.z, h2.z, 0.f);
        fold(ahi.w, alo.w, h2.w, 0.f);
        alo.x += l2.x;
        alo.y += l2.y;
        alo.z += l2.z;
        alo.w += l2.w;
      }
      renorm(ahi.x, alo.x);
      renorm(ahi.y, alo.y);
      renorm(ahi.z, alo.z);
      renorm(ahi.w, alo.w);
      st4(P.agg_hi + o, ahi);
      st4(P.agg_lo + o, alo);
      // Eq. (8a)-(8c)
      float4 tn;
#define GCADA_AMSGRAD(c)                                   \
  {                                                        \
    const float gr = ahi.c;                                \
    h.c = P.beta1 * h.c + P.omb1 * gr;                     \
    const float v = P.beta2 * vh.c + P.omb2 * (gr * gr);   \
    vh.c = fmaxf(vh.c, v);                                 \
    const float up = alpha_k * h.c / sqrtf(P.eps + vh.c);   \
    tn.c = th.c - up;                                      \
    local += (double)up * (double)up;                      \
  }
      GCADA_AMSGRAD(x)
      GCADA_AMSGRAD(y)
      GCADA_AMSGRAD(z)
      GCADA_AMSGRAD(w)
#undef GCADA_AMSGRAD
      st4(P.h + o, h);
      st4(P.vhat + o, vh);
      st4(P.theta_ring + ((k + 1) % ring) * P.p_pad + o, tn);
    }
    local = warp_sum(local);
    if (lane == 0) {
      P.upd_part[blockIdx.x] = local;
      __threadfence();
      is_last = atomicAdd(&P.st->ticket_update, 1u) == gridDim.x - 1u;
    }
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const volatile double* parts = P.upd_part;
  double s = 0.0;
  for (unsigned int b = tid; b < gridDim.x; b += 256) s += parts[b];
  s = block_sum(s, reinterpret_cast<double*>(&wsum_hi[0][0]));
  if (tid == 0) {
    P.s_ring[k % P.D] = s;
    P.st->k = k + 1;
    if (P.chain_last) P.st->k_chain = k + 1;
    P.st->ticket_update = 0u;
  }
}

// The same step for long parameter vectors (tens of thousands of 16-byte columns and more): one column per
// thread, which folds every selected group itself in ascending order (loads of four groups in flight), so a
// block is 256 columns wide and needs no exchange between its warps.
__global__ void __launch_bounds__(256) update_wide_kernel(const Params P) {
  extern __shared__ int sel_list[];  // selected groups, ascending; bit 30 set = the group's cur[] is 1
  __shared__ int n_sel_sh;
  __shared__ double scratch[40];
  __shared__ bool is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long cols4 = P.p_pad >> 2;
  pdl_launch_dependents();
  pdl_wait();
  const long long k = P.st->k;
  const int ring = P.D + 1;
  const float alpha_k = step_size(P, k);
  const long long i4 = (long long)blockIdx.x * 256 + tid;
  const bool active = i4 < cols4;
  const long long o = i4 * 4;
  float4 ahi = make_float4(0.f, 0.f, 0.f, 0.f), alo = ahi, h = ahi, vh = ahi, th = ahi;
  if (active) {  // independent of the selection: fetched first
    ahi = ld4(P.agg_hi + o);
    alo = ld4(P.agg_lo + o);
    h = ld4(P.h + o);
    vh = ld4(P.vhat + o);
    th = ld4(P.theta_ring + (k % ring) * P.p_pad + o);
  }
  if (warp == 0) {
    int cnt = 0;
    for (int g0 = 0; g0 < P.G; g0 += 32) {
      const int gg = g0 + lane;
      const bool s = gg < P.G && P.mask_cur[gg] != 0;
      const int cur = gg < P.G ? P.cur[gg] : 0;
      const unsigned int b = __ballot_sync(0xffffffffu, s);
      if (s) sel_list[cnt + __popc(b & ((1u << lane) - 1u))] = gg | (cur << 30);
      cnt += __popc(b);
    }
    if (lane == 0) n_sel_sh = cnt;
  }
  __syncthreads();
  const int n_sel = n_sel_sh;
  double local = 0.0;
  if (active) {
    for (int j0 = 0; j0 < n_sel; j0 += 4) {
      float4 f[4], l[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (j0 + u < n_sel) {
          const int e = sel_list[j0 + u], g = e & 0x3fffffff, cur = e >> 30;
          f[u] = ld4(P.gbuf + ((long long)cur * P.G + g) * P.p_pad + o);        // the fresh gradient (cur[g] already flipped)
          l[u] = ld4(P.gbuf + ((long long)(1 - cur) * P.G + g) * P.p_pad + o);  // the gradient it replaces
        }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (j0 + u < n_sel) {
          fold(ahi.x, alo.x, f[u].x, l[u].x);
          fold(ahi.y, alo.y, f[u].y, l[u].y);
          fold(ahi.z, alo.z, f[u].z, l[u].z);
          fold(ahi.w, alo.w, f[u].w, l[u].w);
        }
    }
    renorm(ahi.x, alo.x);
    renorm(ahi.y, alo.y);
    renorm(ahi.z, alo.z);
    renorm(ahi.w, alo.w);
    st4(P.agg_hi + o, ahi);
    st4(P.agg_lo + o, alo);
    float4 tn;
#define GCADA_AMSGRAD(c)                                   \
  {                                                        \
    const float gr = ahi.c;                                \
    h.c = P.beta1 * h.c + P.omb1 * gr;                     \
    const float v = P.beta2 * vh.c + P.omb2 * (gr * gr);   \
    vh.c = fmaxf(vh.c, v);                                 \
    const float up = alpha_k * h.c / sqrtf(P.eps + vh.c);   \
    tn.c = th.c - up;                                      \
    local += (double)up * (double)up;                      \
  }
    GCADA_AMSGRAD(x)
    GCADA_AMSGRAD(y)
    GCADA_AMSGRAD(z)
    GCADA_AMSGRAD(w)
#undef GCADA_AMSGRAD
    st4(P.h + o, h);
    st4(P.vhat + o, vh);
    st4(P.theta_ring + ((k + 1) % ring) * P.p_pad + o, tn);
  }
  const double tot = block_sum(local, scratch);
  if (tid == 0) {
    P.upd_part[blockIdx.x] = tot;
    __threadfence();
    is_last = atomicAdd(&P.st->ticket_update, 1u) == gridDim.x - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const volatile double* parts = P.upd_part;
  double s = 0.0;
  for (unsigned int b = tid; b < gridDim.x; b += 256) s += parts[b];
  s = block_sum(s, scratch);
  if (tid == 0) {
    P.s_ring[k % P.D] = s;
    P.st->k = k + 1;
    if (P.chain_last) P.st->k_chain = k + 1;
    P.st->ticket_update = 0u;
  }
}

// Eq. (8a)-(8c) when the aggregate has already been formed in agg_hi (P.agg_direct): one float4 per thread.
__global__ void __launch_bounds__(256) update_direct_kernel(const Params P) {
  __shared__ double scratch[40];
  __shared__ bool is_last;
  const int tid = threadIdx.x;
  const long long cols4 = P.p_pad >> 2;
  pdl_launch_dependents();
  pdl_wait();
  const long long k = P.st->k;
  const int ring = P.D + 1;
  const float alpha_k = step_size(P, k);
  // a block walks the columns with the grid's stride, two columns of a thread in flight together (a few
  // blocks per SM: one partial sum and one ticket per block, not per 256 columns)
  const long long stride = (long long)gridDim.x * 256;
  const float* th_k = P.theta_ring + (k % ring) * P.p_pad;
  float* th_n = P.theta_ring + ((k + 1) % ring) * P.p_pad;
  double local = 0.0;
  for (long long i4 = (long long)blockIdx.x * 256 + tid; i4 < cols4; i4 += 2 * stride) {
    const long long o[2] = {i4 * 4, (i4 + stride) * 4};
    const bool have[2] = {true, i4 + stride < cols4};
    float4 ahi[2], h[2], vh[2], th[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (have[u]) {
        ahi[u] = ld4(P.agg_hi + o[u]);
        h[u] = ld4(P.h + o[u]);
        vh[u] = ld4(P.vhat + o[u]);
        th[u] = ld4(th_k + o[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (!have[u]) continue;
      float4 tn;
#define GCADA_AMSGRAD(c)                                        \
  {                                                             \
    const float gr = ahi[u].c;                                  \
    h[u].c = P.beta1 * h[u].c + P.omb1 * gr;                    \
    const float v = P.beta2 * vh[u].c + P.omb2 * (gr * gr);     \
    vh[u].c = fmaxf(vh[u].c, v);                                \
    const float up = alpha_k * h[u].c / sqrtf(P.eps + vh[u].c); \
    tn.c = th[u].c - up;                                        \
    local += (double)up * (double)up;                           \
  }
      GCADA_AMSGRAD(x)
      GCADA_AMSGRAD(y)
      GCADA_AMSGRAD(z)
      GCADA_AMSGRAD(w)
#undef GCADA_AMSGRAD
      st4(P.h + o[u], h[u]);
      st4(P.vhat + o[u], vh[u]);
      st4(th_n + o[u], tn);
    }
  }
  const double tot = block_sum(local, scratch);
  if (tid == 0) {
    P.upd_part[blockIdx.x] = tot;
    __threadfence();
    is_last = atomicAdd(&P.st->ticket_update, 1u) == gridDim.x - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const volatile double* parts = P.upd_part;
  double s = 0.0;
  for (unsigned int b = tid; b < gridDim.x; b += 256) s += parts[b];
  s = block_sum(s, scratch);
  if (tid == 0) {
    P.s_ring[k % P.D] = s;
    P.st->k = k + 1;
    if (P.chain_last) P.st->k_chain = k + 1;
    P.st->ticket_update = 0u;
  }
}

// Rule PS: left side of Eq. (9) exactly as printed, L_g^2 ||theta^k - theta^{k-tau_g}||^2, from the
// iterate ring.  Grid (column blocks, D): block (b, d-1) sums its slice of ||theta^k - theta^{k-d}||^2
// (theta^j = theta^0 for j < 0); the last block adds the slices in a fixed order and scales by L_g^2.
__global__ void __launch_bounds__(256) ps_lhs_kernel(const Params P) {
  __shared__ double scratch[40];
  __shared__ bool is_last;
  const int tid = threadIdx.x;
  const int d = blockIdx.y + 1;
  const long long cols4 = P.p_pad >> 2;
  pdl_wait();
  const long long k = P.st->k;
  const int ring = P.D + 1;
  long long j = k - d;
  if (j < 0) j = 0;
  const float* a = P.theta_ring + (k % ring) * P.p_pad;
  const float* b = P.theta_ring + (j % ring) * P.p_pad;
  double local = 0.0;
  for (long long i4 = (long long)blockIdx.x * 256 + tid; i4 < cols4; i4 += (long long)gridDim.x * 256) {
    const float4 x = ld4(a + i4 * 4), y = ld4(b + i4 * 4);
    const float dx = x.x - y.x, dy = x.y - y.y, dz = x.z - y.z, dw = x.w - y.w;
    local += (double)dx * dx + (double)dy * dy + (double)dz * dz + (double)dw * dw;
  }
  const double tot = block_sum(local, scratch);
  if (tid == 0) {
    P.ps_part[(long long)(d - 1) * gridDim.x + blockIdx.x] = tot;
    __threadfence();
    is_last = atomicAdd(&P.st->ticket_aux, 1u) == gridDim.x * gridDim.y - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const volatile double* parts = P.ps_part;
  for (int g = tid; g < P.G; g += 256) {
    const int tau = P.tau[g];
    const int dd = tau < 1 ? 1 : (tau > P.D ? P.D : tau);
    double s = 0.0;
    for (unsigned int bb = 0; bb < gridDim.x; ++bb) s += parts[(long long)(dd - 1) * gridDim.x + bb];
    P.ps_lhs[g] = P.ps_L2[g] * s;
  }
  if (tid == 0) P.st->ticket_aux = 0u;
}

cudaError_t launch_ps_lhs(const Params& P, const TailPlan& plan, cudaStream_t st, bool pdl) {
  return launch_k(ps_lhs_kernel, dim3(plan.ps_blocks, P.D), dim3(256), 0, st, pdl, P);
}

void plan_tail(long long p_pad, int G, int sm_count, TailPlan* plan) {
  const long long cols4 = p_pad / 4;
  // four columns per thread once one per thread would give more than four blocks per SM
  const int U = (cols4 > 256 * 1024 || cols4 * G > 256LL * 4 * sm_count) ? 4 : 1;
  plan->select_cols4_per_block = 256 * U;
  plan->select_blocks_x = (int)((cols4 + 256 * U - 1) / (256 * U));
  plan->update_blocks = (int)((cols4 + 31) / 32);
  const long long db = (cols4 + 255) / 256;
  plan->direct_blocks = (int)(db < 8LL * sm_count ? db : 8LL * sm_count);
  long long pb = (cols4 + 256 * 8 - 1) / (256 * 8);  // about eight float4 per thread
  plan->ps_blocks = (int)(pb < 1 ? 1 : (pb > 1024 ? 1024 : pb));
}

cudaError_t launch_select(const Params& P, const TailPlan& plan, cudaStream_t st, int what, bool pdl) {
  if (what == SEL_SCHEDULE || P.pm.n_cta < 0) {
    // nothing to reduce: with n_cta < 0 the norm partial sums are already in lhs_part (maxseg per group);
    // in skip mode (rule PS) the left sides come from ps_lhs and lhs_part is not read (0 slots)
    return launch_k(select_kernel<1>, dim3(1, 1), dim3(256), 0, st, pdl, P, P.pm.n_cta < 0 ? P.pm.maxseg : 0,
                    (int)SEL_SCHEDULE);
  }
  dim3 grid(plan.select_blocks_x, P.G);
  if (plan.select_cols4_per_block == 256)
    return launch_k(select_kernel<1>, grid, dim3(256), 0, st, pdl, P, plan.select_blocks_x, what);
  return launch_k(select_kernel<4>, grid, dim3(256), 0, st, pdl, P, plan.select_blocks_x, what);
}

cudaError_t launch_update(const Params& P, const TailPlan& plan, cudaStream_t st, bool pdl) {
  if (P.agg_direct)
    return launch_k(update_direct_kernel, dim3(plan.direct_blocks), dim3(256), 0, st, pdl, P);
  if (P.p_pad >= 4 * 256 * 128)  // enough 16-byte columns to fill the machine with one per thread
    return launch_k(update_wide_kernel, dim3((plan.update_blocks + 7) / 8), dim3(256), (size_t)P.G * sizeof(int), st,
                    pdl, P);
  return launch_k(update_kernel, dim3(plan.update_blocks), dim3(256), (size_t)P.G * sizeof(int), st, pdl, P);
}

}  // namespace gcada
