// gcada_innovation_norms_noalloc: the innovation-norm reduction of the
// selection kernel for callers that are not allowed to allocate device
// memory.  Its scratch (per-block partial sums and the "last block" ticket)
// lives in a fixed array that is part of the loaded library image.
#include <cuda_runtime.h>
#include <stdio.h>

#include <mutex>

#include "../../include/gcada.h"
#include "common.cuh"

namespace {

constexpr int NA_MAX_GROUPS = GCADA_NOALLOC_MAX_GROUPS;
constexpr int NA_BLOCKS_PER_GROUP = 64;
constexpr int NA_MAX_DEVICES = 64;

struct NoAllocScratch {
  double part[NA_MAX_GROUPS * NA_BLOCKS_PER_GROUP];  // per-block partial sums
  unsigned int ticket;                               // blocks finished so far; must be 0 at launch
};

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

// Host side: the symbol above is only a stand-in here; its device address is
// looked up once per device and cached.
std::mutex g_mu;
NoAllocScratch* g_scratch_addr[NA_MAX_DEVICES] = {nullptr};

__global__ void __launch_bounds__(256) innovation_norms_static_kernel(const float* __restrict__ fresh,
                                                                      const float* __restrict__ stale, int G,
                                                                      long long p, long long ld, double* lhs,
                                                                      NoAllocScratch* sc) {
  __shared__ double scratch[40];
  __shared__ bool is_last;
  const int g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* f = fresh + (long long)g * ld;
  const float* s = stale + (long long)g * ld;
  double local = 0.0;
  for (long long i = (long long)blockIdx.x * 256 + tid; i < p; i += (long long)NA_BLOCKS_PER_GROUP * 256) {
    const float dlt = f[i] - s[i];
    local += (double)dlt * (double)dlt;
  }
  const double tot = gcada::block_sum(local, scratch);
  if (tid == 0) {
    sc->part[g * NA_BLOCKS_PER_GROUP + blockIdx.x] = tot;
    __threadfence();
    is_last = atomicAdd(&sc->ticket, 1u) == (unsigned int)(G * NA_BLOCKS_PER_GROUP) - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const volatile double* parts = sc->part;
  for (int gg = warp; gg < G; gg += 8) {
    double v = 0.0;
    for (int b = lane; b < NA_BLOCKS_PER_GROUP; b += 32) v += parts[gg * NA_BLOCKS_PER_GROUP + b];
    v = gcada::warp_sum(v);
    if (lane == 0) lhs[gg] = v;
  }
  if (tid == 0) sc->ticket = 0u;
}

gcada_status na_fail(char* errbuf, size_t len, gcada_status st, const char* msg, const char* detail = "") {
  if (errbuf && len) snprintf(errbuf, len, "%s%s", msg, detail);
  return st;
}

}  // namespace

extern "C" gcada_status gcada_innovation_norms_noalloc(const float* fresh_dev, const float* stale_dev, int G,
                                                       long long p, long long ld, double* lhs_dev,
                                                       void* cuda_stream, char* errbuf, size_t errbuf_len) {
  if (errbuf && errbuf_len) errbuf[0] = 0;
  if (!fresh_dev || !stale_dev || !lhs_dev) return na_fail(errbuf, errbuf_len, GCADA_EINVAL, "a pointer is NULL");
  if (G < 1 || p < 1 || ld < p) return na_fail(errbuf, errbuf_len, GCADA_EINVAL, "need G >= 1, p >= 1 and ld >= p");
  if (G > NA_MAX_GROUPS) {
    char d[96];
    snprintf(d, sizeof d, ": G = %d, the fixed scratch area holds at most %d groups", G, NA_MAX_GROUPS);
    return na_fail(errbuf, errbuf_len, GCADA_EINVAL, "too many groups for the no-allocation entry point", d);
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return na_fail(errbuf, errbuf_len, GCADA_ECUDA, "cudaGetDevice: ", cudaGetErrorString(e));
  if (dev < 0 || dev >= NA_MAX_DEVICES) return na_fail(errbuf, errbuf_len, GCADA_EINVAL, "device index out of range");
  NoAllocScratch* sc = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
      // first call on this device (which is current): resolve the device address of the array
      void* q = nullptr;
      e = cudaGetSymbolAddress(&q, g_noalloc_scratch);
      if (e != cudaSuccess)
        return na_fail(errbuf, errbuf_len, GCADA_ECUDA, "cudaGetSymbolAddress: ", cudaGetErrorString(e));
      g_scratch_addr[dev] = static_cast<NoAllocScratch*>(q);
    }
    sc = g_scratch_addr[dev];
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // the ticket must start at zero even if an earlier call was cut short
  e = cudaMemsetAsync(&sc->ticket, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return na_fail(errbuf, errbuf_len, GCADA_ECUDA, "cudaMemsetAsync: ", cudaGetErrorString(e));
  dim3 grid(NA_BLOCKS_PER_GROUP, G);
  innovation_norms_static_kernel<<<grid, 256, 0, st>>>(fresh_dev, stale_dev, G, p, ld, lhs_dev, sc);
  e = cudaGetLastError();
  if (e != cudaSuccess) return na_fail(errbuf, errbuf_len, GCADA_ECUDA, "kernel launch: ", cudaGetErrorString(e));
  return GCADA_OK;
}
