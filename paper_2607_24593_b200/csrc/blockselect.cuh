// Block-wide (1024 threads) exact top-K over packed entries, used by the decode path where one
// CTA serves one sequence or one query.  Same order and entry format as segselect.cuh:
// entry = (score key << 32) | ~position, larger is better, all entries distinct.
#pragma once
#include "segselect.cuh"

namespace pivot {

constexpr int kBlk = 1024;

struct BlkSelSmem {
  uint32_t hist[4096];
  entry_t small[kSelSmall];
  entry_t vmin, vmax, cut;
  uint32_t wsum[32];
  uint32_t bin, need, pop, small_n, out_count, list_n;
};

// Largest bin b (walking from the top) such that bins >= b hold at least `need` entries.
// nbins is a multiple of 1024 (at most 16384).  Results in sm.bin / sm.need (still wanted inside
// bin b) / sm.pop (population of bin b); bin = 0, pop = need = 0 if the total is below `need`.
__device__ __forceinline__ void blk_boundary(BlkSelSmem& sm, const uint32_t* hist, int nbins, uint32_t need) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int per = nbins >> 10;                // 1 .. 16 bins per thread, walked from the top
  __syncthreads();
  // this thread's bins in registers, highest first: all loads are issued before the first is used
  uint32_t h[16];
  const uint32_t* top = hist + nbins - 1 - per * tid;
  if (per == 8 && (reinterpret_cast<uintptr_t>(hist) & 15) == 0) {
    const uint4 a = *reinterpret_cast<const uint4*>(top - 7), c4 = *reinterpret_cast<const uint4*>(top - 3);
    h[0] = c4.w; h[1] = c4.z; h[2] = c4.y; h[3] = c4.x; h[4] = a.w; h[5] = a.z; h[6] = a.y; h[7] = a.x;
#pragma unroll
    for (int i = 8; i < 16; ++i) h[i] = 0u;
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) h[i] = i < per ? top[-i] : 0u;
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += h[i];
  uint32_t incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) sm.wsum[wid] = incl;
  if (tid == 0) { sm.bin = 0; sm.need = 0; sm.pop = 0; }
  __syncthreads();
  // entries in the warps before this one: a warp scan over the 32 warp totals
  uint32_t wincl = sm.wsum[lane];
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, wincl, o);
    if (lane >= o) wincl += v;
  }
  const uint32_t wtot = sm.wsum[wid];
  const uint32_t base = __shfl_sync(0xffffffffu, wincl, wid) - wtot;
  const uint32_t excl = base + incl - s;
  if (excl < need && need <= excl + s) {
    uint32_t cum = excl;
    bool done = false;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (!done && i < per && cum + h[i] >= need) {
        sm.bin = (uint32_t)(nbins - 1 - per * tid - i);
        sm.need = need - cum;
        sm.pop = h[i];
        done = true;
      }
      cum += h[i];
    }
  }
  __syncthreads();
}

// K-th largest of list[0..n) (n > K); list may live in shared or global memory.
__device__ __forceinline__ entry_t blk_find_cut(BlkSelSmem& sm, const entry_t* list, int n, int K) {
  const int tid = threadIdx.x, lane = tid & 31;
  entry_t mn = ~0ull, mx = 0ull;
  for (int i = tid; i < n; i += kBlk) {
    const entry_t x = list[i];
    mn = (x < mn && x != kPadEntry) ? x : mn;
    mx = x > mx ? x : mx;
  }
  if (tid == 0) { sm.vmin = ~0ull; sm.vmax = 0ull; }
  __syncthreads();
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const entry_t a = __shfl_xor_sync(0xffffffffu, mn, o);
    const entry_t b = __shfl_xor_sync(0xffffffffu, mx, o);
    mn = a < mn ? a : mn;
    mx = b > mx ? b : mx;
  }
  if (lane == 0) { atomicMin(&sm.vmin, mn); atomicMax(&sm.vmax, mx); }
  __syncthreads();
  entry_t lo = sm.vmin, hi = sm.vmax;
  uint32_t need = (uint32_t)K;
  for (int iter = 0; iter < 8; ++iter) {
    const entry_t span = hi - lo;
    const int bitsw = span ? 64 - __clzll((long long)span) : 0;
    const int shift = bitsw > 11 ? bitsw - 11 : 0;
    for (int i = tid; i < kSelBins; i += kBlk) sm.hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += kBlk) {
      const entry_t x = list[i];
      if (x >= lo && x <= hi) atomicAdd(&sm.hist[(uint32_t)((x - lo) >> shift)], 1u);
    }
    blk_boundary(sm, sm.hist, kSelBins, need);
    const uint32_t b = sm.bin, pop = sm.pop;
    need = sm.need;
    const entry_t lo2 = lo + ((entry_t)b << shift);
    const entry_t width1 = shift ? (((entry_t)1 << shift) - 1ull) : 0ull;
    const entry_t hi2 = (hi - lo2) < width1 ? hi : lo2 + width1;
    if (pop == need) {
      __syncthreads();
      return lo2;
    }
    if (pop <= (uint32_t)kSelSmall) {
      if (tid == 0) sm.small_n = 0;
      __syncthreads();
      for (int i = tid; i < n; i += kBlk) {
        const entry_t x = list[i];
        if (x >= lo2 && x <= hi2) {
          const uint32_t p = atomicAdd(&sm.small_n, 1u);
          if (p < (uint32_t)kSelSmall) sm.small[p] = x;
        }
      }
      __syncthreads();
      const int P = min((int)sm.small_n, kSelSmall);
      for (int t = tid; t < P; t += kBlk) {
        const entry_t xt = sm.small[t];
        uint32_t rank = 0;
        for (int u = 0; u < P; ++u) rank += sm.small[u] > xt ? 1u : 0u;
        if (rank == need - 1) sm.cut = xt;
      }
      __syncthreads();
      const entry_t c = sm.cut;
      __syncthreads();
      return c;
    }
    lo = lo2;
    hi = hi2;
    __syncthreads();
  }
  return lo;
}

// Writes the K best entries of list[0..n) (positions, optional scores; unordered; padding
// entries skipped) to out / out_score and pads to K with -1 / -inf; `copies` further rows
// `stride` apart receive the same set.
__device__ __forceinline__ void blk_emit_topk(BlkSelSmem& sm, const entry_t* list, int n, int n_valid, int K,
                                              int32_t* out, float* out_score, int copies, int stride) {
  const int tid = threadIdx.x, lane = tid & 31;
  entry_t cut = 0ull;
  if (n_valid > K) cut = blk_find_cut(sm, list, n, K);
  if (tid == 0) sm.out_count = 0;
  __syncthreads();
  for (int i0 = 0; i0 < n; i0 += kBlk) {
    const int i = i0 + tid;
    const entry_t x = i < n ? list[i] : kPadEntry;
    const bool keep = i < n && entry_pos(x) >= 0 && x >= cut;
    const uint32_t m = __ballot_sync(0xffffffffu, keep);
    if (m) {
      uint32_t pos = 0;
      const int leader = __ffs(m) - 1;
      if (lane == leader) pos = atomicAdd(&sm.out_count, (uint32_t)__popc(m));
      pos = __shfl_sync(0xffffffffu, pos, leader);
      if (keep) {
        const uint32_t p = pos + __popc(m & ((1u << lane) - 1u));
        if (p < (uint32_t)K) {
          out[p] = entry_pos(x);
          if (out_score) out_score[p] = key_to_score(entry_key(x));
        }
      }
    }
  }
  __syncthreads();
  const int got = min((int)sm.out_count, K);
  for (int i = got + tid; i < K; i += kBlk) {
    out[i] = -1;
    if (out_score) out_score[i] = -INFINITY;
  }
  __syncthreads();
  for (int r = 1; r < copies; ++r)
    for (int i = tid; i < K; i += kBlk) {
      out[(size_t)r * stride + i] = out[i];
      if (out_score) out_score[(size_t)r * stride + i] = out_score[i];
    }
}

}  // namespace pivot
