// Kernel 1: proxy-query build (Eq. 4) and the row / group planners.
//
// A warp forms the proxy vectors of four (e4m3) or two (bf16) heads of a group: members are de-quantised, summed in member
// order in fp32, scaled by fl32(1/m) and rounded once to the storage type.  For FP8 the proxy
// gets a fresh per-head scale a/448 (a = max(amax, 1e-4)) which is folded into the proxy gate,
// so the shared scan (Eq. 5) runs on plain e4m3 codes.  Every fp32 step uses the explicit
// round-to-nearest intrinsics so the compiler cannot contract a multiply into an add.
#include "kernels.h"
#include "proxy_math.cuh"

namespace pivot {

long long& launch_counter() {
  static long long n = 0;
  return n;
}

template <int DT>
__global__ void __launch_bounds__(256)
proxy_build_kernel(const void* __restrict__ q, const float* __restrict__ qscale,
                   const float* __restrict__ w, void* __restrict__ proxy_q,
                   float* __restrict__ proxy_w, int rows, int g, int first_group, int n_proxy, int pool) {
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  proxy_build_unit<DT>(q, qscale, w, proxy_q, proxy_w, rows, g, first_group, n_proxy, pool, wid, threadIdx.x & 31);
}

void launch_proxy_build(const void* q, const float* qscale, const float* w, void* proxy_q,
                        float* proxy_w, int rows, int g, int first_group, int n_proxy, int dtype,
                        int pool, cudaStream_t st) {
  if (n_proxy <= 0) return;
  const long long warps = (long long)n_proxy * (dtype == DT_FP8 ? kHeads / 4 : kHeads / 2);
  const int blocks = (int)((warps + 7) / 8);
  if (dtype == DT_FP8)
    proxy_build_kernel<DT_FP8><<<blocks, 256, 0, st>>>(q, qscale, w, proxy_q, proxy_w, rows, g, first_group, n_proxy, pool);
  else
    proxy_build_kernel<DT_BF16><<<blocks, 256, 0, st>>>(q, qscale, w, proxy_q, proxy_w, rows, g, first_group, n_proxy, pool);
  ++launch_counter();
}

}  // namespace pivot
