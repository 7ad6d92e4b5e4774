// Dual-point minibatch gradients of the linear models (logistic regression,
// quadratic loss) for all groups in one launch.
//
// For every group g the kernel evaluates, on the same B sampled rows,
//     fresh_g = scale * sum_i r_i x_i,         r_i = f(z_i) - y_i,  z_i = x_i . theta^k
//     innov_g = scale * sum_i (r_i - r~_i) x_i, r~_i = f(z~_i) - y_i, z~_i = x_i . theta^{k-tau_g}
// with f the logistic sigmoid (or the identity for the quadratic loss):
// the gradient at the current iterate and its change since the group's stale
// iterate, whose squared norm is what Eq. (9)'s left side estimates
// (Section IV; Algorithm 1's gradient step).  The stale-point gradient is
// fresh_g - innov_g.  The change is accumulated directly, from
// z_i - z~_i = x_i . (theta^k - theta^{k-tau_g}) and
// f(z) - f(z~) = -expm1(-(z - z~)) * sigmoid(z) * sigmoid(-z~), so that it
// keeps full relative accuracy when the two gradients nearly cancel.  Each
// sampled row is read from HBM once and serves both points and both passes
// (x . theta, then r x).
//
// Work split: the G*B minibatch rows form one list; CTA c owns the
// contiguous range [c*R/n, (c+1)*R/n) and writes one partial sum per group
// it touches (PartialMap).  A later kernel adds the partials in a fixed
// order, so results are bitwise reproducible.
#include "common.cuh"
#include "launch.h"

namespace gcada {

// ------------------------------------------------------------------ helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
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
// Bounded wait: false if the phase did not complete within the limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < (1u << 22); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}
// One contiguous global -> shared copy of `bytes` (multiple of 16, both
// addresses 16-byte aligned), completion signalled on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// a = f(z) - y (residual at theta^k); e = f(z) - f(z - dz) (its change).
template <bool QUAD>
__device__ __forceinline__ void coefficients(float z, float dz, float y, float& a, float& e) {
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

// ---------------------------------------------------------------------------
// Large-d kernel (256 < d <= THREADS*CPT*4).  Thread t owns the 16-byte
// column chunks t + THREADS*i, i < CPT, of every row: theta, the stale iterate
// (as theta^k minus it) and both accumulators stay in registers; rows arrive
// in a shared-memory ring through bulk asynchronous copies (one per 4*d-byte
// row) issued ahead by thread 0, so each row crosses HBM -> SM exactly once.
// FULL = the row is exactly THREADS*CPT chunks (no column predicates).
// ---------------------------------------------------------------------------
constexpr int LG_CHUNK_ROWS = 256;  // rows whose indices / labels are staged at once

template <int THREADS, int CPT, int R, int MINB, bool QUAD, bool FULL>
__global__ void __launch_bounds__(THREADS, MINB) grad_linear_large_kernel(const Params P, int nslot) {
  constexpr int V = 2 * R;
  constexpr int NW = THREADS / 32;
  // the copies are issued by lane 0 of the last warp: the first R warps are on the critical path of every
  // batch (they turn the dot products into coefficients), the last one is not
  constexpr int ISSUER = THREADS - 32;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = P.d;
  const int nchunks = FULL ? THREADS * CPT : (d + 3) >> 2;
  const uint32_t rowbytes = (uint32_t)nchunks * 16u;

  // shared memory carve-up
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);                       // nslot (<= 32)
  long long* row_sm = reinterpret_cast<long long*>(smem_raw + 8 * 32);          // LG_CHUNK_ROWS
  float* y_sm = reinterpret_cast<float*>(row_sm + LG_CHUNK_ROWS);               // LG_CHUNK_ROWS
  float* part = y_sm + LG_CHUNK_ROWS;                                           // V * THREADS
  float* res = part + V * THREADS;                                              // V (padded to 32)
  unsigned char* slots = reinterpret_cast<unsigned char*>(res + 32);
  slots = reinterpret_cast<unsigned char*>(((uintptr_t)slots + 127) & ~(uintptr_t)127);

  const float* Xf = reinterpret_cast<const float*>(P.X);
  const float* yf = reinterpret_cast<const float*>(P.y);
  const int B = P.B;
  const bool skip = P.skip_unselected != 0;
  // Inside a chain of captured iterations the kernel may start while the previous iteration's selection and
  // update kernels are still running.  Which rows it reads follows from the draw alone (Section II-A: the
  // minibatch does not depend on the iterate), so the first copies are started before the wait below; the
  // iteration number for the draw then comes from the chain's start, which no running kernel writes.
  const bool early = P.pdl != 0 && !skip;
  pdl_launch_dependents();
  if (!early) pdl_wait();
  const long long k_pre = early ? P.st->k_chain + P.k_off : P.st->k;  // the iteration (confirmed after the wait)
  const uint32_t k32 = (uint32_t)k_pre;
  const int ring = P.D + 1;

  // group numbers below are positions in the list of groups worked on (all groups, or the selected ones)
  __shared__ int sel_sm[SKIP_MAX_GROUPS];
  __shared__ int n_groups_sm;
  const int n_groups = build_group_list(P, sel_sm, &n_groups_sm);
  const long long Rtot = (long long)n_groups * B;
  // (when only the selected groups compute there may be fewer rows than CTAs: the first Rtot CTAs take one each,
  // so that no CTA with an empty range sits between two that hold a group's partial sums)
  const long long n_eff = Rtot < (long long)gridDim.x ? Rtot : (long long)gridDim.x;
  if ((long long)blockIdx.x >= n_eff) return;
  const long long r0 = (long long)blockIdx.x * Rtot / n_eff;
  const long long r1 = (long long)(blockIdx.x + 1) * Rtot / n_eff;
  if (r0 >= r1) return;
  const int rows_cta = (int)(r1 - r0);
  const int g_first = (int)(r0 / B);
  const int in_g0 = (int)(r0 - (long long)g_first * B);  // position of the CTA's first row in its group

  if (tid == 0) {
    for (int s = 0; s < nslot; ++s) mbar_init(&bars[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // Index and label of the rows of a chunk, then the first copies (as many as the ring has slots).
  // Returns how many copies were issued (meaningful in the issuing thread).
  int cslot = 0;          // ring slot of the next row to consume
  auto stage_chunk = [&](int cs, int nrows) -> int {
    __syncthreads();  // previous chunk fully consumed; barriers initialised (first pass)
    for (int i = tid; i < nrows; i += THREADS) {
      const int pos = in_g0 + cs + i;
      const int gi = pos / B;
      const long long row = batch_row(P, k32, skip ? sel_sm[g_first + gi] : g_first + gi, pos - gi * B);
      row_sm[i] = row * P.ld;
      y_sm[i] = yf[row];
    }
    __syncthreads();
    int issued = 0;
    if (tid == ISSUER) {
      const int n0 = nrows < nslot ? nrows : nslot;
      for (; issued < n0; ++issued) {
        int s = cslot + issued;
        if (s >= nslot) s -= nslot;
        mbar_expect_tx(&bars[s], rowbytes);
        bulk_load(slots + (size_t)s * rowbytes, Xf + row_sm[issued], rowbytes, &bars[s]);
      }
    }
    return issued;
  };
  // column ownership
  bool own[CPT];
  float4 th[CPT], ths[CPT], acc0[CPT], acc1[CPT];
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const bool ragged = !FULL && (d & 3) != 0;
#pragma unroll
  for (int i = 0; i < CPT; ++i) ths[i] = zero4;
  int issued_early = 0;
  // The stale iterate of the CTA's first group can be fetched early as well: the ages were written by the
  // previous selection kernel, which had finished before the update kernel started, and theta^{k - tau} with
  // tau >= 1 sits in a slot of the ring that the running update does not write.
  bool ths_raw = false;  // ths[] holds the first group's stale iterate itself, not yet theta^k minus it
  if (early) {
    issued_early = stage_chunk(0, rows_cta < LG_CHUNK_ROWS ? rows_cta : LG_CHUNK_ROWS);
    if (FULL) {
      long long js = k_pre - P.tau[g_first];
      if (js < k_pre - P.D) js = k_pre - P.D;
      if (js < 0) js = 0;
      const float* theta_s = P.theta_ring + (js % ring) * P.p_pad;
#pragma unroll
      for (int i = 0; i < CPT; ++i) ths[i] = *reinterpret_cast<const float4*>(theta_s + (tid + THREADS * i) * 4);
      ths_raw = true;
    }
    pdl_wait();
  }
  // theta^k: its slot follows from the iteration number already at hand, so these loads and the one that
  // confirms the number leave together
  const long long k = early ? *reinterpret_cast<volatile const long long*>(&P.st->k) : k_pre;
  const float* theta_k = P.theta_ring + (k_pre % ring) * P.p_pad;
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const int q = tid + THREADS * i;
    own[i] = FULL || q < nchunks;
    th[i] = zero4;
    if (own[i]) {
      const int c0 = q * 4;
      if (FULL) {
        th[i] = *reinterpret_cast<const float4*>(theta_k + c0);
      } else {
        th[i].x = theta_k[c0];
        th[i].y = c0 + 1 < d ? theta_k[c0 + 1] : 0.f;
        th[i].z = c0 + 2 < d ? theta_k[c0 + 2] : 0.f;
        th[i].w = c0 + 3 < d ? theta_k[c0 + 3] : 0.f;
      }
    }
    acc0[i] = zero4;
    acc1[i] = zero4;
  }
  int failed = 0;
  if (k != k_pre) {  // the chain's bookkeeping and the iteration counter disagree: nothing is computed
    if (tid == 0) atomicCAS(&P.st->err, (int)DEV_OK, (int)DEV_ERR_CHAIN);
    if (tid == ISSUER)  // the copies already started get a bounded chance to land before the CTA leaves
      for (int j = 0; j < issued_early; ++j) mbar_wait_bounded(&bars[j], 0u);
    return;
  }

  int cur_g = -1;
  int g_end = 0;          // CTA-local row at which the current group ends
  uint32_t cphase = 0;    // barrier parity of that slot's current fill

  auto flush = [&](int g) {
    const long long slot = (long long)blockIdx.x * P.pm.maxseg + (g - g_first);
    if (!GCADA_INDEX_OK(P.st, g - g_first, P.pm.maxseg, CHK_PARTIAL) ||
        !GCADA_INDEX_OK(P.st, slot, P.lim.partial_slots, CHK_PARTIAL))
      return;
    float* dst = P.partial + (slot * 2) * P.p_pad;
#pragma unroll
    for (int i = 0; i < CPT; ++i) {
      if (!own[i]) continue;
      const int c0 = (tid + THREADS * i) * 4;
      if (!ragged || c0 + 3 < d) {
        *reinterpret_cast<float4*>(dst + c0) = acc0[i];
        *reinterpret_cast<float4*>(dst + P.p_pad + c0) = acc1[i];
      } else {
        const float a0[4] = {acc0[i].x, acc0[i].y, acc0[i].z, acc0[i].w};
        const float a1[4] = {acc1[i].x, acc1[i].y, acc1[i].z, acc1[i].w};
        for (int e = 0; e < 4 && c0 + e < d; ++e) {
          dst[c0 + e] = a0[e];
          dst[P.p_pad + c0 + e] = a1[e];
        }
      }
    }
  };

  for (int cs = 0; cs < rows_cta && !failed; cs += LG_CHUNK_ROWS) {
    const int nrows = rows_cta - cs < LG_CHUNK_ROWS ? rows_cta - cs : LG_CHUNK_ROWS;
    int issued = (early && cs == 0) ? issued_early : stage_chunk(cs, nrows);
    int consumed = 0;
    while (consumed < nrows) {
      const int lr = cs + consumed;
      if (lr == g_end) {  // first row of a group (g_end starts at 0)
        if (cur_g >= 0) flush(cur_g);
        cur_g = cur_g < 0 ? g_first : cur_g + 1;
        g_end = (cur_g + 1 - g_first) * B - in_g0;
        long long js = k - (ths_raw ? 0 : P.tau[skip ? sel_sm[cur_g] : cur_g]);
        if (js < k - P.D) js = k - P.D;  // ages beyond D only arise under forced masks: oldest kept iterate
        if (js < 0) js = 0;
        const float* theta_s = P.theta_ring + (js % ring) * P.p_pad;
#pragma unroll
        for (int i = 0; i < CPT; ++i) {
          acc0[i] = zero4;
          acc1[i] = zero4;
          if (own[i]) {
            const int c0 = (tid + THREADS * i) * 4;
            if (FULL) {
              const float4 t = ths_raw ? ths[i] : *reinterpret_cast<const float4*>(theta_s + c0);
              ths[i] = make_float4(th[i].x - t.x, th[i].y - t.y, th[i].z - t.z, th[i].w - t.w);
            } else {
              ths[i].x = th[i].x - theta_s[c0];
              ths[i].y = c0 + 1 < d ? th[i].y - theta_s[c0 + 1] : 0.f;
              ths[i].z = c0 + 2 < d ? th[i].z - theta_s[c0 + 2] : 0.f;
              ths[i].w = c0 + 3 < d ? th[i].w - theta_s[c0 + 3] : 0.f;
            }
          }
        }
        ths_raw = false;
      }
      int lim = (g_end < cs + nrows ? g_end : cs + nrows) - lr;
      const int nb = lim < R ? lim : R;

      // pass 1: rows -> registers, partial dot products z = x.theta and dz = x.(theta - theta_stale)
      float4 x[R][CPT];
      float pz[V];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        pz[r] = 0.f;
        pz[R + r] = 0.f;
        if (r < nb) {
          int s = cslot + r;
          uint32_t ph = cphase;
          if (s >= nslot) {
            s -= nslot;
            ph ^= 1u;
          }
          if (!mbar_wait_bounded(&bars[s], ph)) failed = 1;
          const float4* src = reinterpret_cast<const float4*>(slots + (size_t)s * rowbytes);
#pragma unroll
          for (int i = 0; i < CPT; ++i) {
            if (FULL) {
              x[r][i] = src[tid + THREADS * i];
            } else {
              x[r][i] = own[i] ? src[tid + THREADS * i] : zero4;
              if (ragged && own[i]) {
                const int c0 = (tid + THREADS * i) * 4;
                if (c0 + 1 >= d) x[r][i].y = 0.f;
                if (c0 + 2 >= d) x[r][i].z = 0.f;
                if (c0 + 3 >= d) x[r][i].w = 0.f;
              }
            }
            // (one fused multiply-add per term: written as a sum of products the compiler must keep the
            // grouping and spends a multiplication and an addition more per four columns)
            pz[r] = fmaf(x[r][i].w, th[i].w, fmaf(x[r][i].z, th[i].z, fmaf(x[r][i].y, th[i].y, fmaf(x[r][i].x, th[i].x, pz[r]))));
            pz[R + r] = fmaf(x[r][i].w, ths[i].w,
                             fmaf(x[r][i].z, ths[i].z, fmaf(x[r][i].y, ths[i].y, fmaf(x[r][i].x, ths[i].x, pz[R + r]))));
          }
        } else {
#pragma unroll
          for (int i = 0; i < CPT; ++i) x[r][i] = zero4;
        }
      }
#pragma unroll
      for (int v = 0; v < V; ++v) part[v * THREADS + tid] = pz[v];
      failed = __syncthreads_or(failed);  // (A) rows are in registers: their slots are free
      if (failed) break;
      if (tid == ISSUER) {
        for (int r = 0; r < nb && issued < nrows; ++r, ++issued) {
          int s = cslot + r;  // slot of a row consumed just now
          if (s >= nslot) s -= nslot;
          mbar_expect_tx(&bars[s], rowbytes);
          bulk_load(slots + (size_t)s * rowbytes, Xf + row_sm[issued], rowbytes, &bars[s]);
        }
      }
      // stage 2: warp r finishes both dot products of row r and turns them
      // into the two rank-one coefficients
      for (int r = warp; r < R; r += NW) {
        float s = 0.f, t = 0.f;
#pragma unroll
        for (int i = 0; i < NW; ++i) {
          s += part[r * THREADS + lane + 32 * i];
          t += part[(R + r) * THREADS + lane + 32 * i];
        }
        s = warp_sum(s);
        t = warp_sum(t);
        if (lane == 0) {
          float a = 0.f, e = 0.f;
          if (r < nb) coefficients<QUAD>(s, t, y_sm[consumed + r], a, e);
          res[r] = a * P.scale;
          res[R + r] = e * P.scale;
        }
      }
      __syncthreads();  // (B)
      // pass 2: rank-one accumulation
      float cf[V];
      if (V % 4 == 0) {
#pragma unroll
        for (int v = 0; v < V; v += 4) {
          const float4 t = *reinterpret_cast<const float4*>(res + v);
          cf[v] = t.x;
          cf[v + 1] = t.y;
          cf[v + 2] = t.z;
          cf[v + 3] = t.w;
        }
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) cf[v] = res[v];
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float a = cf[r], b = cf[R + r];
#pragma unroll
        for (int i = 0; i < CPT; ++i) {
          acc0[i].x += a * x[r][i].x;
          acc0[i].y += a * x[r][i].y;
          acc0[i].z += a * x[r][i].z;
          acc0[i].w += a * x[r][i].w;
          acc1[i].x += b * x[r][i].x;
          acc1[i].y += b * x[r][i].y;
          acc1[i].z += b * x[r][i].z;
          acc1[i].w += b * x[r][i].w;
        }
      }
      consumed += nb;
      cslot += nb;
      if (cslot >= nslot) {
        cslot -= nslot;
        cphase ^= 1u;
      }
    }
    if (failed) {
      // give copies already in flight a bounded chance to land before leaving
      if (tid == ISSUER) {
        atomicExch(&P.st->err, DEV_ERR_COPY_TIMEOUT);
        for (int j = consumed; j < issued; ++j) {
          int s = cslot + (j - consumed);
          uint32_t ph = cphase;
          if (s >= nslot) {
            s -= nslot;
            ph ^= 1u;
          }
          mbar_wait_bounded(&bars[s], ph);
        }
      }
      return;
    }
  }
  if (cur_g >= 0) flush(cur_g);
}

// ---------------------------------------------------------------------------
// Small-d kernel (d <= 32*CPL <= 256): one warp per row, lane l owns columns
// l + 32*i.  Rows are short (<= 1 KB), loads are coalesced per row; four rows
// are in flight per warp.  Warps of a CTA combine their accumulators through
// shared memory when the CTA leaves a group.
// ---------------------------------------------------------------------------
template <int CPL, bool QUAD>
__global__ void __launch_bounds__(256) grad_linear_small_kernel(const Params P) {
  constexpr int NW = 8, RR = 4;
  __shared__ float accw[NW][2][32 * CPL];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = P.d;
  pdl_launch_dependents();
  pdl_wait();
  const long long k = P.st->k;
  const uint32_t k32 = (uint32_t)k;
  const int ring = P.D + 1;
  const float* theta_k = P.theta_ring + (k % ring) * P.p_pad;
  const float* Xf = reinterpret_cast<const float*>(P.X);
  const float* yf = reinterpret_cast<const float*>(P.y);
  __shared__ int sel_sm[SKIP_MAX_GROUPS];
  __shared__ int n_groups_sm;
  const int n_groups = build_group_list(P, sel_sm, &n_groups_sm);  // positions in this list are called g below
  const bool skip = P.skip_unselected != 0;
  const long long Rtot = (long long)n_groups * P.B;
  const long long n_eff = Rtot < (long long)gridDim.x ? Rtot : (long long)gridDim.x;  // see the wide kernel
  if ((long long)blockIdx.x >= n_eff) return;
  const long long r0 = (long long)blockIdx.x * Rtot / n_eff;
  const long long r1 = (long long)(blockIdx.x + 1) * Rtot / n_eff;
  if (r0 >= r1) return;
  const int g_first = (int)(r0 / P.B);

  float th[CPL], ths[CPL], acc0[CPL], acc1[CPL];
#pragma unroll
  for (int i = 0; i < CPL; ++i) {
    const int c = lane + 32 * i;
    th[i] = c < d ? theta_k[c] : 0.f;
  }
  long long seg0 = r0;
  while (seg0 < r1) {
    const int g = (int)(seg0 / P.B);
    const long long seg1 = (long long)(g + 1) * P.B < r1 ? (long long)(g + 1) * P.B : r1;
    const int g_real = skip ? sel_sm[g] : g;
    long long js = k - P.tau[g_real];
    if (js < k - P.D) js = k - P.D;  // ages beyond D only arise under forced masks: oldest kept iterate
    if (js < 0) js = 0;
    const float* theta_s = P.theta_ring + (js % ring) * P.p_pad;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = lane + 32 * i;
      ths[i] = c < d ? th[i] - theta_s[c] : 0.f;
      acc0[i] = 0.f;
      acc1[i] = 0.f;
    }
    // warp w takes rows seg0 + RR*(w + NW*t) ..
    for (long long rb = seg0 + (long long)RR * warp; rb < seg1; rb += (long long)RR * NW) {
      // lanes 0..RR-1 fetch the row number and label of one row each
      long long myrow = 0;
      float myy = 0.f;
      if (lane < RR && rb + lane < seg1) {
        myrow = batch_row(P, k32, g_real, (int)(rb + lane - (long long)g * P.B));
        myy = yf[myrow];
      }
      float x[RR][CPL], z[RR], zs[RR];
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        const long long row = __shfl_sync(0xffffffffu, myrow, r);
        const bool valid = rb + r < seg1;
        z[r] = 0.f;
        zs[r] = 0.f;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          const int c = lane + 32 * i;
          x[r][i] = (valid && c < d) ? Xf[row * P.ld + c] : 0.f;
          z[r] += x[r][i] * th[i];
          zs[r] += x[r][i] * ths[i];
        }
      }
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        z[r] = warp_sum(z[r]);
        zs[r] = warp_sum(zs[r]);
      }
#pragma unroll
      for (int r = 0; r < RR; ++r) {
        const float yy = __shfl_sync(0xffffffffu, myy, r);
        const bool valid = rb + r < seg1;
        float a = 0.f, b = 0.f;
        if (valid) coefficients<QUAD>(z[r], zs[r], yy, a, b);
        a *= P.scale;
        b *= P.scale;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
          acc0[i] += a * x[r][i];
          acc1[i] += b * x[r][i];
        }
      }
    }
    // combine the warps in a fixed order and write the CTA's partial sum
    __syncthreads();
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      accw[warp][0][lane + 32 * i] = acc0[i];
      accw[warp][1][lane + 32 * i] = acc1[i];
    }
    __syncthreads();
    const long long slot = (long long)blockIdx.x * P.pm.maxseg + (g - g_first);
    const bool slot_ok = GCADA_INDEX_OK(P.st, g - g_first, P.pm.maxseg, CHK_PARTIAL) &&
                         GCADA_INDEX_OK(P.st, slot, P.lim.partial_slots, CHK_PARTIAL);
    float* dst = P.partial + (slot * 2) * P.p_pad;
    for (int e = tid; slot_ok && e < 2 * 32 * CPL; e += 256) {
      const int pt = e / (32 * CPL), c = e - pt * 32 * CPL;
      if (c < d) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) s += accw[w][pt][c];
        dst[(long long)pt * P.p_pad + c] = s;
      }
    }
    seg0 = seg1;
  }
}

// ------------------------------------------------------------------ launch
static size_t large_smem_fixed(int threads, int R) {
  return 8 * 32 + LG_CHUNK_ROWS * (sizeof(long long) + sizeof(float)) + (size_t)2 * R * threads * 4 + 32 * 4 + 128;
}

template <int CPT, int R, int MINB>
static cudaError_t launch_large(const Params& P, const LinearPlan& plan, bool quad, cudaStream_t st,
                                bool attr_only, bool pdl) {
  void (*kern)(const Params, int);
  if (plan.full)
    kern = quad ? grad_linear_large_kernel<256, CPT, R, MINB, true, true>
                : grad_linear_large_kernel<256, CPT, R, MINB, false, true>;
  else
    kern = quad ? grad_linear_large_kernel<256, CPT, R, MINB, true, false>
                : grad_linear_large_kernel<256, CPT, R, MINB, false, false>;
  if (attr_only)
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  return launch_k(kern, dim3(plan.n_cta), dim3(256), plan.smem_bytes, st, pdl, P, plan.nslot);
}

template <int CPL>
static cudaError_t launch_small(const Params& P, const LinearPlan& plan, bool quad, cudaStream_t st, bool pdl) {
  if (quad) return launch_k(grad_linear_small_kernel<CPL, true>, dim3(plan.n_cta), dim3(256), 0, st, pdl, P);
  return launch_k(grad_linear_small_kernel<CPL, false>, dim3(plan.n_cta), dim3(256), 0, st, pdl, P);
}

bool plan_linear(int d, long long ld, const void* X, int G, int B, int sm_count, size_t smem_optin,
                 LinearPlan* plan, const char** why) {
  const long long Rtot = (long long)G * B;
  plan->small = d <= 256;
  if (plan->small) {
    plan->cpl = d <= 32 ? 1 : (d <= 64 ? 2 : (d <= 128 ? 4 : 8));
    long long n = (Rtot + 31) / 32;
    const long long cap = (long long)sm_count * 8;
    plan->n_cta = (int)(n < 1 ? 1 : (n > cap ? cap : n));
    plan->smem_bytes = 0;
    plan->nslot = 0;
  } else {
    if (d > 4096) {
      *why = "logistic / quadratic models support d <= 4096";
      return false;
    }
    if ((ld & 3) != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0) {
      *why = "for d > 256 X must be 16-byte aligned with a row stride that is a multiple of 4";
      return false;
    }
    const int nchunks = (d + 3) / 4;
    plan->cpt = nchunks <= 256 ? 1 : (nchunks <= 512 ? 2 : 4);
    plan->threads = 256;
    plan->full = (d & 3) == 0 && nchunks == 256 * plan->cpt;
    // two CTAs per SM with 2-row batches: each hides the other's barriers (one CTA per SM with 4-row
    // batches measured 15 % slower on the d = 4096 workload)
    plan->ctas_per_sm = 2;
    plan->R = 2;
    const size_t rowbytes = (size_t)nchunks * 16;
    const size_t fixed = large_smem_fixed(plan->threads, plan->R);
    // per CTA: the opt-in limit (or half an SM's shared memory) less the kernel's static arrays
    const long long budget = ((long long)smem_optin + 1024) / 2 - 1024 - 4608;
    long long nslot = (budget - (long long)fixed) / (long long)rowbytes;
    if (nslot > 32) nslot = 32;
    if (nslot < 2 * plan->R) {
      *why = "not enough shared memory for the row ring";
      return false;
    }
    // no more than 64 KiB of copies in flight per CTA (two batches of 2 rows at d = 4096): a copy-only kernel of
    // this shape over the same rows moves 6.3 TB/s with 96 KiB in flight per CTA and 6.7 TB/s with 48 KiB, and
    // the d = 4096 workload runs 0.8 % faster with four slots than with six
    if (nslot * (long long)rowbytes > 65536) nslot = 65536 / (long long)rowbytes;
    if (nslot < 2 * plan->R) nslot = 2 * plan->R;
    plan->nslot = (int)nslot;
    plan->smem_bytes = fixed + (size_t)nslot * rowbytes;
    const long long want = (long long)sm_count * plan->ctas_per_sm;
    plan->n_cta = (int)(Rtot < want ? Rtot : want);
  }
  const long long per = (Rtot + plan->n_cta - 1) / plan->n_cta;
  plan->maxseg = (int)((per + B - 2) / B + 1);
  return true;
}

static cudaError_t dispatch_large(const Params& P, const LinearPlan& plan, bool quad, cudaStream_t st,
                                  bool attr_only, bool pdl) {
  switch (plan.cpt) {
    case 1: return launch_large<1, 2, 2>(P, plan, quad, st, attr_only, pdl);
    case 2: return launch_large<2, 2, 2>(P, plan, quad, st, attr_only, pdl);
    default: return launch_large<4, 2, 2>(P, plan, quad, st, attr_only, pdl);
  }
}

cudaError_t prepare_grad_linear(const LinearPlan& plan, bool quad) {
  if (plan.small) return cudaSuccess;
  return dispatch_large(Params{}, plan, quad, nullptr, true, false);
}

cudaError_t launch_grad_linear(const Params& P, const LinearPlan& plan, bool quad, cudaStream_t st, bool pdl) {
  if (plan.small) {
    switch (plan.cpl) {
      case 1: return launch_small<1>(P, plan, quad, st, pdl);
      case 2: return launch_small<2>(P, plan, quad, st, pdl);
      case 4: return launch_small<4>(P, plan, quad, st, pdl);
      default: return launch_small<8>(P, plan, quad, st, pdl);
    }
  }
  return dispatch_large(P, plan, quad, st, false, pdl);
}

}  // namespace gcada
