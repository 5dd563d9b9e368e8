// Exact top-K over entries held in per-warp segments, for a team of four warps (128 threads).
//
// An entry packs a score and its key position into one 64-bit word,
//     entry = (order-preserving score key << 32) | ~position,
// so that "larger entry" is exactly the total order of the TopK operator used for Eq. 6 / 7 / 9
// (higher score first, then the lower position) and all entries are distinct.
//
// The streaming select of the tensor-core kernels keeps, per row, one candidate segment per
// epilogue warp: warp w appends only to its own segment (cursor in a register, no atomics), and
// entry e of a segment belongs to lane e % 32.  A selection loads every lane's entries into
// registers once and then finds the K-th largest entry of the union by histogramming:
//   1. reduce the range [lo, hi] of the entries;
//   2. 2048 bins, linear over [lo, hi]; count; walk the bins from the top to the one that holds
//      the K-th entry (the boundary bin);
//   3. if the boundary bin is small (<= 256 entries) rank its entries by brute force, else
//      narrow [lo, hi] to that bin and repeat (the width shrinks 2048-fold per round).
// The result is the cut: an entry is among the K best iff entry >= cut.
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace pivot {

#ifdef PIVOT_PROFILE
__device__ unsigned long long g_sel_prof[16];
#define SELP_T(var) const long long var = clock64()
#define SELP_ADD(slot, t0, t1) \
  if (tm.tid == 0 && tm.bar == 1 && blockIdx.x == 0) g_sel_prof[slot] += (unsigned long long)((t1) - (t0))
#else
#define SELP_T(var)
#define SELP_ADD(slot, t0, t1)
#endif

constexpr int kSelBins = 2048;
constexpr int kSelSmall = 256;

typedef unsigned long long entry_t;

__device__ __forceinline__ entry_t make_entry(uint32_t key, int32_t pos) {
  return ((entry_t)key << 32) | (entry_t)(~(uint32_t)pos);
}
__device__ __forceinline__ uint32_t entry_key(entry_t e) { return (uint32_t)(e >> 32); }
__device__ __forceinline__ int32_t entry_pos(entry_t e) { return (int32_t)(~(uint32_t)e); }
// Padding entry: lowest possible, position -1.
constexpr entry_t kPadEntry = 0ull;

struct SegSelSmem {
  uint32_t hist[kSelBins];
  entry_t list[kSelSmall];
  entry_t vmin, vmax;
  entry_t cut;
  uint32_t wsum[4];
  uint32_t bin, need, pop;
  uint32_t list_n;
  uint32_t out_count;
  uint32_t total;
};

// One warp's view of its segment (warp-uniform count).
struct Seg {
  const entry_t* e;
  int cnt;
};

// A lane's entries: cached in registers (EPT entries at most) or re-read on each use.
template <int EPT, bool CACHED>
struct SegRegs {
  entry_t v[CACHED ? EPT : 1];
  const entry_t* base;
  __device__ __forceinline__ void load(const Seg& s, int lane, int nj) {
    base = s.e + lane;
    if constexpr (CACHED) {
#pragma unroll
      for (int j = 0; j < EPT; ++j) v[j] = j < nj ? __ldcg(s.e + j * 32 + lane) : kPadEntry;
    }
  }
  __device__ __forceinline__ entry_t get(int j) const {
    if constexpr (CACHED) return v[j];
    else return __ldcg(base + j * 32);
  }
};

// Finds the K-th largest entry among the team's segments (more than K entries in total).
// All 128 threads call; the cut is returned (and left in sm.cut).
template <int EPT, bool CACHED>
__device__ __forceinline__ entry_t seg_find_cut(const Team& tm, SegSelSmem& sm, const SegRegs<EPT, CACHED>& regs,
                                                int nj, int K) {
  const int lane = tm.tid & 31;
  const int wq = tm.tid >> 5;
  SELP_T(q0);
  entry_t mn = ~0ull, mx = 0ull;
#pragma unroll
  for (int j = 0; j < EPT; ++j)
    if (j < nj) {
      const entry_t x = regs.get(j);
      mn = (x < mn && x != kPadEntry) ? x : mn;     // padding never bounds the range
      mx = x > mx ? x : mx;
    }
  if (tm.tid == 0) { sm.vmin = ~0ull; sm.vmax = 0ull; }
  tm.sync();
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const entry_t a = __shfl_xor_sync(0xffffffffu, mn, o);
    const entry_t b = __shfl_xor_sync(0xffffffffu, mx, o);
    mn = a < mn ? a : mn;
    mx = b > mx ? b : mx;
  }
  if (lane == 0) { atomicMin(&sm.vmin, mn); atomicMax(&sm.vmax, mx); }
  tm.sync();
  entry_t lo = sm.vmin, hi = sm.vmax;
  uint32_t need = (uint32_t)K;
  SELP_T(q1);
  SELP_ADD(0, q0, q1);
  for (int iter = 0; iter < 8; ++iter) {
    SELP_T(r0);
    const entry_t span = hi - lo;
    const int bitsw = span ? 64 - __clzll((long long)span) : 0;
    const int shift = bitsw > 11 ? bitsw - 11 : 0;
    for (int i = tm.tid; i < kSelBins; i += tm.nthr) sm.hist[i] = 0;
    tm.sync();
#pragma unroll
    for (int j = 0; j < EPT; ++j)
      if (j < nj) {
        const entry_t x = regs.get(j);
        if (x >= lo && x <= hi) atomicAdd(&sm.hist[(uint32_t)((x - lo) >> shift)], 1u);
      }
    tm.sync();
    SELP_T(r1);
    SELP_ADD(1, r0, r1);
    // boundary bin, walking from the top: thread t owns bins 2047-16t .. 2032-16t
    uint32_t loc[16];
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) { loc[i] = sm.hist[kSelBins - 1 - 16 * tm.tid - i]; s += loc[i]; }
    uint32_t incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sm.wsum[wq] = incl;
    tm.sync();
    uint32_t base = 0;
    for (int w = 0; w < wq; ++w) base += sm.wsum[w];
    const uint32_t excl = base + incl - s;
    if (excl < need && need <= excl + s) {
      uint32_t cum = excl;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (cum + loc[i] >= need) {
          sm.bin = (uint32_t)(kSelBins - 1 - 16 * tm.tid - i);
          sm.need = need - cum;
          sm.pop = loc[i];
          break;
        }
        cum += loc[i];
      }
    }
    tm.sync();
    const uint32_t b = sm.bin, pop = sm.pop;
    need = sm.need;
    const entry_t lo2 = lo + ((entry_t)b << shift);
    const entry_t width1 = shift ? (((entry_t)1 << shift) - 1ull) : 0ull;
    const entry_t hi2 = (hi - lo2) < width1 ? hi : lo2 + width1;
    SELP_T(r2);
    SELP_ADD(2, r1, r2);
#ifdef PIVOT_PROFILE
    if (tm.tid == 0 && tm.bar == 1 && blockIdx.x == 0) { g_sel_prof[8] += 1; g_sel_prof[9] += pop; }
#endif
    if (pop == need) {          // the whole boundary bin is wanted
      if (tm.tid == 0) sm.cut = lo2;
      tm.sync();
      return lo2;
    }
    if (pop <= (uint32_t)kSelSmall) {   // rank the boundary bin's entries by brute force
      if (tm.tid == 0) sm.list_n = 0;
      tm.sync();
#pragma unroll
      for (int j = 0; j < EPT; ++j)
        if (j < nj) {
          const entry_t x = regs.get(j);
          if (x >= lo2 && x <= hi2) {
            const uint32_t p = atomicAdd(&sm.list_n, 1u);
            if (p < (uint32_t)kSelSmall) sm.list[p] = x;
          }
        }
      tm.sync();
      const int P = min((int)sm.list_n, kSelSmall);
      for (int t = tm.tid; t < P; t += tm.nthr) {
        const entry_t xt = sm.list[t];
        uint32_t rank = 0;
        for (int u = 0; u < P; ++u) rank += sm.list[u] > xt ? 1u : 0u;
        if (rank == need - 1) sm.cut = xt;
      }
      tm.sync();
      SELP_T(r3);
      SELP_ADD(3, r2, r3);
      return sm.cut;
    }
    lo = lo2;
    hi = hi2;
  }
  if (tm.tid == 0) sm.cut = lo;     // not reachable: entries are distinct
  tm.sync();
  return lo;
}

// Compaction: keeps the K best entries; every warp rewrites its survivors into `dst` (its own
// segment of the other ping-pong half) and returns its new count.  *cut_out gets the cut.
template <int EPT, bool CACHED>
__device__ __forceinline__ int seg_compact(const Team& tm, SegSelSmem& sm, const Seg& seg, entry_t* dst, int K,
                                           entry_t* cut_out) {
  const int lane = tm.tid & 31;
  const int nj = seg.cnt > lane ? (seg.cnt - lane + 31) >> 5 : 0;
  SegRegs<EPT, CACHED> regs;
  regs.load(seg, lane, nj);
  SELP_T(c1);
  const entry_t cut = seg_find_cut<EPT, CACHED>(tm, sm, regs, nj, K);
  SELP_T(c2);
  SELP_ADD(5, c1, c2);
  int out = 0;
  const int njw = (seg.cnt + 31) >> 5;          // warp-uniform trip count
#pragma unroll
  for (int j = 0; j < EPT; ++j) {
    if (j < njw) {
      const entry_t x = j < nj ? regs.get(j) : kPadEntry;
      const bool keep = j < nj && x >= cut;
      const uint32_t m = __ballot_sync(0xffffffffu, keep);
      if (keep) dst[out + __popc(m & ((1u << lane) - 1u))] = x;
      out += __popc(m);
    }
  }
  *cut_out = cut;
  SELP_T(c3);
  SELP_ADD(6, c2, c3);
#ifdef PIVOT_PROFILE
  if (tm.tid == 0 && tm.bar == 1 && blockIdx.x == 0) g_sel_prof[10] += 1;
#endif
  return out;
}

// Writes the positions (and optionally scores) of the entries flagged by `pred` through the
// team cursor sm.out_count; entries at position -1 (padding) are skipped.
template <int EPT, bool CACHED, typename Pred>
__device__ __forceinline__ void seg_write_out(const Team& tm, SegSelSmem& sm, const SegRegs<EPT, CACHED>& regs,
                                              int nj, int njw, int32_t* out, float* out_score, int K, Pred pred) {
  const int lane = tm.tid & 31;
#pragma unroll
  for (int j = 0; j < EPT; ++j) {
    if (j < njw) {
      const entry_t x = j < nj ? regs.get(j) : kPadEntry;
      const bool keep = j < nj && entry_pos(x) >= 0 && pred(x);
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
  }
}

// Final selection of a row: writes min(K, n_valid) positions (unordered) to out, returns how
// many.  n_valid = real (non-padding) entries in the team's segments.
template <int EPT, bool CACHED>
__device__ __forceinline__ int seg_emit(const Team& tm, SegSelSmem& sm, const Seg& seg, int n_valid, int32_t* out,
                                        float* out_score, int K) {
  const int lane = tm.tid & 31;
  const int nj = seg.cnt > lane ? (seg.cnt - lane + 31) >> 5 : 0;
  const int njw = (seg.cnt + 31) >> 5;
  SegRegs<EPT, CACHED> regs;
  regs.load(seg, lane, nj);
  if (tm.tid == 0) sm.out_count = 0;
  tm.sync();
  if (n_valid > K) {
    const entry_t cut = seg_find_cut<EPT, CACHED>(tm, sm, regs, nj, K);
    seg_write_out<EPT, CACHED>(tm, sm, regs, nj, njw, out, out_score, K, [cut](entry_t x) { return x >= cut; });
  } else {
    seg_write_out<EPT, CACHED>(tm, sm, regs, nj, njw, out, out_score, K, [](entry_t) { return true; });
  }
  tm.sync();
  return n_valid > K ? K : n_valid;
}

}  // namespace pivot
