// Kernel 1: proxy-query build (Eq. 4) and the row / group planners.
//
// One warp forms one (group, head) proxy vector: members are de-quantised, summed in member
// order in fp32, scaled by fl32(1/m) and rounded once to the storage type.  For FP8 the proxy
// gets a fresh per-head scale a/448 (a = max(amax, 1e-4)) which is folded into the proxy gate,
// so the shared scan (Eq. 5) runs on plain e4m3 codes.  Every fp32 step uses the explicit
// round-to-nearest intrinsics so the compiler cannot contract a multiply into an add.
#include "kernels.h"

namespace pivot {

long long& launch_counter() {
  static long long n = 0;
  return n;
}

__global__ void __launch_bounds__(256)
proxy_build_kernel(const void* __restrict__ q, const float* __restrict__ qscale,
                   const float* __restrict__ w, void* __restrict__ proxy_q,
                   float* __restrict__ proxy_w, int rows, int g, int first_group, int n_proxy,
                   int dtype, int pool) {
  const int lane = threadIdx.x & 31;
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= (long long)n_proxy * kHeads) return;
  const int r = (int)(wid / kHeads);
  const int h = (int)(wid % kHeads);
  const int t0 = (first_group + r) * g;
  const int m = min(g, rows - t0);
  int lo = 0, hi = m;                       // members pooled
  if (pool == 1) hi = 1;
  if (pool == 2) lo = m - 1;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float wacc = 0.f;
  for (int i = lo; i < hi; ++i) {
    const size_t row = (size_t)(t0 + i) * kHeads + h;
    float x[4];
    if (dtype == DT_FP8) {
      const uint32_t pk = reinterpret_cast<const uint32_t*>(q)[row * (kDim / 4) + lane];
      const float s = qscale[row];
#pragma unroll
      for (int e = 0; e < 4; ++e) x[e] = __fmul_rn(e4m3_to_float((pk >> (8 * e)) & 0xff), s);
    } else {
      const uint2 pk = reinterpret_cast<const uint2*>(q)[row * (kDim / 4) + lane];
      x[0] = bf16_bits_to_float(pk.x & 0xffff);
      x[1] = bf16_bits_to_float(pk.x >> 16);
      x[2] = bf16_bits_to_float(pk.y & 0xffff);
      x[3] = bf16_bits_to_float(pk.y >> 16);
    }
    const float wv = w[row];
    if (i == lo) {
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] = x[e];
      wacc = wv;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], x[e]);
      wacc = __fadd_rn(wacc, wv);
    }
  }
  if (pool == 0) {
    const float inv_m = __fdiv_rn(1.0f, (float)m);
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = __fmul_rn(acc[e], inv_m);
    wacc = __fmul_rn(wacc, inv_m);
  }
  const size_t orow = (size_t)r * kHeads + h;
  if (dtype == DT_FP8) {
    float amax = fmaxf(fmaxf(fabsf(acc[0]), fabsf(acc[1])), fmaxf(fabsf(acc[2]), fabsf(acc[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float a = fmaxf(amax, 1e-4f);
    const float sbar = __fdiv_rn(a, 448.0f);
    const float inv = __fdiv_rn(448.0f, a);
    uint32_t pk = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t code =
          (uint32_t)__nv_cvt_float_to_fp8(__fmul_rn(acc[e], inv), __NV_SATFINITE, __NV_E4M3);
      pk |= (code & 0xffu) << (8 * e);
    }
    reinterpret_cast<uint32_t*>(proxy_q)[orow * (kDim / 4) + lane] = pk;
    if (lane == 0) proxy_w[orow] = __fmul_rn(wacc, sbar);
  } else {
    uint2 pk;
    pk.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[0])) |
           ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[1])) << 16);
    pk.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[2])) |
           ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[3])) << 16);
    reinterpret_cast<uint2*>(proxy_q)[orow * (kDim / 4) + lane] = pk;
    if (lane == 0) proxy_w[orow] = wacc;
  }
}

void launch_proxy_build(const void* q, const float* qscale, const float* w, void* proxy_q,
                        float* proxy_w, int rows, int g, int first_group, int n_proxy, int dtype,
                        int pool, cudaStream_t st) {
  if (n_proxy <= 0) return;
  const long long warps = (long long)n_proxy * kHeads;
  const int blocks = (int)((warps + 7) / 8);
  proxy_build_kernel<<<blocks, 256, 0, st>>>(q, qscale, w, proxy_q, proxy_w, rows, g, first_group,
                                             n_proxy, dtype, pool);
  ++launch_counter();
}

}  // namespace pivot
