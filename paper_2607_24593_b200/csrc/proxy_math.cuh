// Proxy-query arithmetic (Eq. 4) shared by the proxy-build kernel and the decode path's prepare
// kernel: members are de-quantised, summed in member order in fp32, scaled by fl32(1/m) and rounded
// once to the storage type; FP8 proxies get a fresh per-head scale a/448 (a = max(amax, 1e-4))
// which is folded into the proxy gate.  Every fp32 step uses the explicit round-to-nearest
// intrinsics so the compiler cannot contract a multiply into an add.
#pragma once
#include "common.cuh"

namespace pivot {

template <int DT>
constexpr int proxy_units_per_group() { return kHeads / (32 / (kDim / (DT == DT_FP8 ? 16 : 8))); }

// 16 bytes per lane: a warp covers four heads (e4m3: 8 lanes x 16 codes per head) or two
// (bf16: 16 lanes x 8 values), and the members' loads go out four at a time -- with 4-byte
// loads issued one member after the other the kernel had too few bytes in flight to get near
// the HBM rate (it reads every query once: 1.07 GB at the 128K FP8 configuration).
// `wid` numbers the warp-sized units of work: unit wid forms heads (wid % WPG) * HPW .. of proxy wid / WPG.
template <int DT>
__device__ __forceinline__ void proxy_build_unit(const void* __restrict__ q, const float* __restrict__ qscale,
                                                 const float* __restrict__ w, void* __restrict__ proxy_q,
                                                 float* __restrict__ proxy_w, int rows, int g, int first_group, int n_proxy,
                                                 int pool, long long wid, int lane) {
  constexpr bool FP8 = DT == DT_FP8;
  constexpr int E = FP8 ? 16 : 8;            // elements per lane
  constexpr int LPH = kDim / E;              // lanes per head: 8 or 16
  constexpr int HPW = 32 / LPH;              // heads per warp: 4 or 2
  constexpr int WPG = kHeads / HPW;          // warps per group
  if (wid >= (long long)n_proxy * WPG) return;
  const int r = (int)(wid / WPG);
  const int h = (int)(wid % WPG) * HPW + lane / LPH;
  const int sub = lane % LPH;                // which 16 bytes of the head's row
  const int t0 = (first_group + r) * g;
  const int m = min(g, rows - t0);
  int lo = 0, hi = m;                        // members pooled
  if (pool == 1) hi = 1;
  if (pool == 2) lo = m - 1;
  float acc[E];
  float wacc = 0.f;
  const uint4* q4 = reinterpret_cast<const uint4*>(q);
  for (int i0 = lo; i0 < hi; i0 += 4) {
    uint4 pk[4];
    float sc[4], wv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {            // up to four members in flight
      if (i0 + u < hi) {
        const size_t row = (size_t)(t0 + i0 + u) * kHeads + h;
        pk[u] = __ldg(q4 + row * LPH + sub);
        sc[u] = FP8 ? __ldg(qscale + row) : 1.f;
        wv[u] = __ldg(w + row);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u < hi) {
        const uint32_t wd[4] = {pk[u].x, pk[u].y, pk[u].z, pk[u].w};
        float x[E];
        if (FP8) {                           // two codes per conversion (e4m3 -> half is exact, and so is half -> float)
#pragma unroll
          for (int e = 0; e < E; e += 2) {
            const __half2_raw h2 = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)((wd[e >> 2] >> (8 * (e & 3))) & 0xffff), __NV_E4M3);
            const float2 f2 = __half22float2(__half2(h2));
            x[e] = __fmul_rn(f2.x, sc[u]);
            x[e + 1] = __fmul_rn(f2.y, sc[u]);
          }
        } else {
#pragma unroll
          for (int e = 0; e < E; ++e) x[e] = bf16_bits_to_float((wd[e >> 1] >> (16 * (e & 1))) & 0xffff);
        }
        if (i0 + u == lo) {
#pragma unroll
          for (int e = 0; e < E; ++e) acc[e] = x[e];
          wacc = wv[u];
        } else {
#pragma unroll
          for (int e = 0; e < E; ++e) acc[e] = __fadd_rn(acc[e], x[e]);
          wacc = __fadd_rn(wacc, wv[u]);
        }
      }
    }
  }
  if (pool == 0) {
    const float inv_m = __fdiv_rn(1.0f, (float)m);
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = __fmul_rn(acc[e], inv_m);
    wacc = __fmul_rn(wacc, inv_m);
  }
  const size_t orow = (size_t)r * kHeads + h;
  uint4 out;
  uint32_t* ow = reinterpret_cast<uint32_t*>(&out);
  if (FP8) {
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) amax = fmaxf(amax, fabsf(acc[e]));
#pragma unroll
    for (int o = LPH / 2; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));   // over the head's lanes
    const float a = fmaxf(amax, 1e-4f);
    const float sbar = __fdiv_rn(a, 448.0f);
    const float inv = __fdiv_rn(448.0f, a);
#pragma unroll
    for (int j = 0; j < 4; ++j) ow[j] = 0u;
#pragma unroll
    for (int e = 0; e < E; e += 2) {         // two values per conversion, same rounding as one at a time
      const uint32_t code2 = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(acc[e], inv), __fmul_rn(acc[e + 1], inv)),
                                                                __NV_SATFINITE, __NV_E4M3);
      ow[e >> 2] |= (code2 & 0xffffu) << (8 * (e & 3));
    }
    if (sub == 0) proxy_w[orow] = __fmul_rn(wacc, sbar);
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      ow[j] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[2 * j])) |
              ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[2 * j + 1])) << 16);
    if (sub == 0) proxy_w[orow] = wacc;
  }
  reinterpret_cast<uint4*>(proxy_q)[orow * LPH + sub] = out;
}


}  // namespace pivot
