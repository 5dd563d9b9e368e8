// Exact top-K over entries held in per-warp segments, for a team of four warps (128 threads).
//
// An entry packs a score and its key position into one 64-bit word,
//     entry = (order-preserving score key << 32) | ~position,
// so that "larger entry" is exactly the total order of the TopK operator used for Eq. 6 / 7 / 9
// (higher score first, then the lower position) and all entries are distinct.
//
// The streaming select of the tensor-core kernels keeps, per row, one candidate segment per
// epilogue warp: warp w appends only to its own segment (cursor in a register, no atomics), and
// entry e of a segment belongs to lane e % 32.  A selection finds the K-th largest entry of the
// union of the four segments by histogramming:
//   1. reduce the range [lo, hi] of the entries;
//   2. 2048 bins, linear over [lo, hi]; count; walk the bins from the top to the one that holds
//      the K-th entry (the boundary bin);
//   3. if the boundary bin is small (<= 256 entries) rank its entries by brute force, else
//      narrow [lo, hi] to that bin and repeat (the width shrinks 2048-fold per round).
// The result is the cut: an entry is among the K best iff entry >= cut.
// Lanes hold their entries in registers when a segment has at most 32 * EPT entries
// (CACHED = true, loops unrolled) and re-read them from memory otherwise (rolled loops).
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace pivot {


constexpr int kSelBins = 2048;
constexpr int kSelSmall = 256;
constexpr int kSelEpt = 64;      // register-cached entries per lane

typedef unsigned long long entry_t;

__device__ __forceinline__ entry_t make_entry(uint32_t key, int32_t pos) {
  return ((entry_t)key << 32) | (entry_t)(~(uint32_t)pos);
}
__device__ __forceinline__ uint32_t entry_key(entry_t e) { return (uint32_t)(e >> 32); }
__device__ __forceinline__ int32_t entry_pos(entry_t e) { return (int32_t)(~(uint32_t)e); }
constexpr entry_t kPadEntry = 0ull;   // lowest possible entry, position -1: never selected

struct SegSelSmem {
  alignas(16) uint32_t hist[kSelBins];   // read as uint4 by warp_hist_boundary
  entry_t list[kSelSmall];
  entry_t vmin, vmax;
  entry_t cut;
  uint32_t wsum[8];
  uint32_t bin, need, pop;
  uint32_t list_n;
  uint32_t out_count;
  uint32_t total;
  uint32_t maxcnt;
  uint32_t kmin, kmax;    // key range of a shared-memory score row
};

// One warp's view of its segment (warp-uniform count).
struct Seg {
  entry_t* e;
  int cnt;
};

// A lane's entries: entry j of the lane is segment element j * 32 + lane.
template <bool CACHED, int EPT = kSelEpt>
struct SegRegs {
  entry_t v[CACHED ? EPT : 1];
  const entry_t* base;
  int nj;      // this lane's entry count
  __device__ __forceinline__ void load(const Seg& s, int lane) {
    base = s.e + lane;
    nj = s.cnt > lane ? (s.cnt - lane + 31) >> 5 : 0;
    if constexpr (CACHED) {
#pragma unroll
      for (int j = 0; j < EPT; ++j) v[j] = j < nj ? __ldcg(base + j * 32) : kPadEntry;
    }
  }
  template <typename F>
  __device__ __forceinline__ void for_each(F f) const {
    if constexpr (CACHED) {
#pragma unroll
      for (int j = 0; j < EPT; ++j)
        if (j < nj) f(v[j]);
    } else {
#pragma unroll 4
      for (int j = 0; j < nj; ++j) f(__ldcg(base + j * 32));
    }
  }
  // Warp-uniform trip count njw = ceil(cnt / 32): f(x, valid) runs for every lane.
  template <typename F>
  __device__ __forceinline__ void for_each_uniform(int njw, F f) const {
    if constexpr (CACHED) {
#pragma unroll
      for (int j = 0; j < EPT; ++j)
        if (j < njw) f(j < nj ? v[j] : kPadEntry, j < nj);
    } else {
      for (int j = 0; j < njw; ++j) f(j < nj ? __ldcg(base + j * 32) : kPadEntry, j < nj);
    }
  }
};

// Boundary bin of a 2048-bin histogram walked from the top: the largest bin b such that the
// bins >= b hold at least `need` entries.  Leaves (bin, need inside that bin, its population)
// in sm.bin / sm.need / sm.pop; if the histogram holds fewer than `need` entries, bin = 0 and
// pop = need = 0.  All threads of the team call (128 or 256 threads).
__device__ __forceinline__ void hist_boundary(const Team& tm, SegSelSmem& sm, const uint32_t* hist, uint32_t need) {
  const int lane = tm.tid & 31;
  const int wq = tm.tid >> 5;
  const int per = kSelBins / tm.nthr;       // bins per thread: 16 or 8
  tm.sync();          // everyone is done with the previous result, and the histogram is complete
  uint32_t s = 0;
  for (int i = 0; i < per; ++i) s += hist[kSelBins - 1 - per * tm.tid - i];
  uint32_t incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) sm.wsum[wq] = incl;
  if (tm.tid == 0) { sm.bin = 0; sm.need = 0; sm.pop = 0; }
  tm.sync();
  uint32_t base = 0;
  for (int w = 0; w < wq; ++w) base += sm.wsum[w];
  const uint32_t excl = base + incl - s;
  if (excl < need && need <= excl + s) {
    uint32_t cum = excl;
    for (int i = 0; i < per; ++i) {
      const uint32_t h = hist[kSelBins - 1 - per * tm.tid - i];
      if (cum + h >= need) {
        sm.bin = (uint32_t)(kSelBins - 1 - per * tm.tid - i);
        sm.need = need - cum;
        sm.pop = h;
        break;
      }
      cum += h;
    }
  }
  tm.sync();
}

// Warp-local boundary bin of a 2048-bin histogram (16-byte aligned, shared memory), walked from
// the top: the largest bin b such that the bins >= b hold at least `need` entries.  Returns
// false if the histogram holds fewer than `need`.  No barrier: other warps may keep adding to
// the histogram meanwhile; counts only grow, so a torn snapshot can only give a lower bin, which
// is still a valid bound.  *need_in and *pop describe the boundary bin (entries still wanted
// from it, and its population as read).
// BATCHED issues all level-1 loads before the reductions (faster, 16 more live registers);
// the serial form is for callers inside a register-bound loop.
template <bool BATCHED = true>
__device__ __forceinline__ bool warp_hist_boundary(const uint32_t* hist, uint32_t need, int lane, uint32_t* bin,
                                                   uint32_t* need_in, uint32_t* pop) {
  const uint4* h4 = reinterpret_cast<const uint4*>(hist);
  uint32_t cum = 0;
  int jsel = -1;
  // level 1: chunks of 128 bins, lane holds four consecutive bins of each chunk.  All loads
  // first, then all reductions, so their latencies overlap.
  constexpr int NCH = kSelBins / 128;
  if constexpr (BATCHED) {
    uint32_t part[NCH];
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const uint4 v = h4[j * 32 + lane];
      part[j] = (v.x + v.y) + (v.z + v.w);
    }
#pragma unroll
    for (int j = 0; j < NCH; ++j) part[j] = __reduce_add_sync(0xffffffffu, part[j]);
#pragma unroll
    for (int j = NCH - 1; j >= 0; --j) {
      if (jsel < 0) {
        if (cum + part[j] >= need) jsel = j;
        else cum += part[j];
      }
    }
  } else {
#pragma unroll
    for (int j = NCH - 1; j >= 0; --j) {
      const uint4 v = h4[j * 32 + lane];
      const uint32_t c = __reduce_add_sync(0xffffffffu, (v.x + v.y) + (v.z + v.w));
      if (jsel < 0) {
        if (cum + c >= need) jsel = j;
        else cum += c;
      }
    }
  }
  if (jsel < 0) { *bin = 0; *need_in = 0; *pop = 0; return false; }
  // level 2: inside the chunk, suffix sums over the lanes
  const uint4 v = h4[jsel * 32 + lane];
  const uint32_t s = (v.x + v.y) + (v.z + v.w);
  uint32_t incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += t;
  }
  const uint32_t above = cum + incl - s;              // entries in bins above this lane's four
  const bool here = above < need && need <= above + s;
  uint32_t b = 0, ni = 0, pp = 0;
  if (here) {
    uint32_t c = above;
    if (c + v.w >= need) { b = 3; ni = need - c; pp = v.w; }
    else if ((c += v.w) + v.z >= need) { b = 2; ni = need - c; pp = v.z; }
    else if ((c += v.z) + v.y >= need) { b = 1; ni = need - c; pp = v.y; }
    else { c += v.y; b = 0; ni = need - c; pp = v.x; }
    b += (uint32_t)(jsel * 128 + lane * 4);
  }
  const uint32_t m = __ballot_sync(0xffffffffu, here);
  const int src = __ffs(m) - 1;                        // exactly one lane
  *bin = __shfl_sync(0xffffffffu, b, src);
  *need_in = __shfl_sync(0xffffffffu, ni, src);
  *pop = __shfl_sync(0xffffffffu, pp, src);
  return true;
}

// Finds the K-th largest entry among the team's segments (more than K real entries in total).
// All 128 threads call; the cut is returned (and left in sm.cut).
template <bool CACHED, int EPT = kSelEpt>
__device__ __forceinline__ entry_t seg_find_cut(const Team& tm, SegSelSmem& sm, const SegRegs<CACHED, EPT>& regs, int K) {
  const int lane = tm.tid & 31;
  entry_t mn = ~0ull, mx = 0ull;
  regs.for_each([&](entry_t x) {
    mn = (x < mn && x != kPadEntry) ? x : mn;     // padding never bounds the range
    mx = x > mx ? x : mx;
  });
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
  for (int iter = 0; iter < 8; ++iter) {
    const entry_t span = hi - lo;
    const int bitsw = span ? 64 - __clzll((long long)span) : 0;
    const int shift = bitsw > 11 ? bitsw - 11 : 0;
    for (int i = tm.tid; i < kSelBins; i += tm.nthr) sm.hist[i] = 0;
    tm.sync();
    regs.for_each([&](entry_t x) {
      if (x >= lo && x <= hi) atomicAdd(&sm.hist[(uint32_t)((x - lo) >> shift)], 1u);
    });
    tm.sync();
    hist_boundary(tm, sm, sm.hist, need);
    const uint32_t b = sm.bin, pop = sm.pop;
    need = sm.need;
    const entry_t lo2 = lo + ((entry_t)b << shift);
    const entry_t width1 = shift ? (((entry_t)1 << shift) - 1ull) : 0ull;
    const entry_t hi2 = (hi - lo2) < width1 ? hi : lo2 + width1;
    if (pop == need) {          // the whole boundary bin is wanted
      if (tm.tid == 0) sm.cut = lo2;
      tm.sync();
      return lo2;
    }
    if (pop <= (uint32_t)kSelSmall) {   // rank the boundary bin's entries by brute force
      if (tm.tid == 0) sm.list_n = 0;
      tm.sync();
      regs.for_each([&](entry_t x) {
        if (x >= lo2 && x <= hi2) {
          const uint32_t p = atomicAdd(&sm.list_n, 1u);
          if (p < (uint32_t)kSelSmall) sm.list[p] = x;
        }
      });
      tm.sync();
      const int P = min((int)sm.list_n, kSelSmall);
      for (int t = tm.tid; t < P; t += tm.nthr) {
        const entry_t xt = sm.list[t];
        uint32_t rank = 0;
        for (int u = 0; u < P; ++u) rank += sm.list[u] > xt ? 1u : 0u;
        if (rank == need - 1) sm.cut = xt;
      }
      tm.sync();
      return sm.cut;
    }
    lo = lo2;
    hi = hi2;
  }
  if (tm.tid == 0) sm.cut = lo;     // not reachable: entries are distinct
  tm.sync();
  return lo;
}

// In-place filter of one warp's segment: keeps the entries for which pred holds, in order,
// and returns the new count.  Safe in place: writes never pass the read position.  Warp-local.
template <typename Pred>
__device__ __forceinline__ int seg_filter_inplace(entry_t* e, int cnt, int lane, Pred pred) {
  int out = 0;
  for (int j0 = 0; j0 < cnt; j0 += 128) {        // four rows of 32 in flight
    entry_t x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = j0 + u * 32 + lane;
      x[u] = i < cnt ? __ldcg(e + i) : kPadEntry;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool keep = (j0 + u * 32 + lane) < cnt && pred(x[u]);
      const uint32_t m = __ballot_sync(0xffffffffu, keep);
      if (keep) e[out + __popc(m & ((1u << lane) - 1u))] = x[u];
      out += __popc(m);
    }
    __syncwarp();
  }
  return out;
}

// Exact compaction in place: keeps the K best entries of the team's segments; returns this
// warp's new count and the cut through *cut_out.  Needs more than K real entries in total.
template <bool CACHED, int EPT = kSelEpt>
__device__ __forceinline__ int seg_compact(const Team& tm, SegSelSmem& sm, const Seg& seg, int K, entry_t* cut_out) {
  const int lane = tm.tid & 31;
  SegRegs<CACHED, EPT> regs;
  regs.load(seg, lane);
  const entry_t cut = seg_find_cut<CACHED, EPT>(tm, sm, regs, K);
  *cut_out = cut;
  if constexpr (CACHED) {
    int out = 0;
    regs.for_each_uniform((seg.cnt + 31) >> 5, [&](entry_t x, bool valid) {
      const bool keep = valid && x >= cut;
      const uint32_t m = __ballot_sync(0xffffffffu, keep);
      if (keep) seg.e[out + __popc(m & ((1u << lane) - 1u))] = x;
      out += __popc(m);
    });
    return out;
  } else {
    return seg_filter_inplace(seg.e, seg.cnt, lane, [cut](entry_t x) { return x >= cut; });
  }
}

// Final selection of a row: writes the K best real entries (fewer if the segments hold fewer;
// unordered) to out and returns how many.  n_valid = an upper bound on the real (non-padding)
// entries in the team's segments, used only to skip the cut search when everything fits.
template <bool CACHED, int EPT = kSelEpt>
__device__ __forceinline__ int seg_emit(const Team& tm, SegSelSmem& sm, const Seg& seg, int n_valid, int32_t* out,
                                        float* out_score, int K) {
  const int lane = tm.tid & 31;
  SegRegs<CACHED, EPT> regs;
  regs.load(seg, lane);
  if (tm.tid == 0) sm.out_count = 0;
  tm.sync();
  entry_t cut = 0ull;
  if (n_valid > K) cut = seg_find_cut<CACHED, EPT>(tm, sm, regs, K);
  regs.for_each_uniform((seg.cnt + 31) >> 5, [&](entry_t x, bool valid) {
    const bool keep = valid && entry_pos(x) >= 0 && x >= cut;
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
  });
  tm.sync();
  // what was really written: n_valid is an upper bound only (masked window slots and slots of a
  // short prefix are padding entries), and the caller pads the row from the returned count on
  const int n_out = (int)sm.out_count;
  return n_out > K ? K : n_out;
}

// ---------------------------------------------------------------------------------------------
// Exact top-K by ONE warp over entries that lie in global memory (written by other warps of the
// CTA, read through L2): the rows of score keys the re-score kernel leaves per member, and the
// candidate segments of the shared scan.  A source sweeps its entries past a functor, U per lane
// in flight (0 = empty slot).  The sweeps are what the select costs: their bodies carry no branch
// per entry (a uniform test per entry, let alone a divergent one, makes every entry a basic block
// of its own and exposes each vote's and each load's latency in turn: measured 320 clocks per
// entry against 40).
//
// The K best entries under the entry order (key, then the lower position) are found by
// narrowing a window [lo, hi]: 2048 linear bins over the window, walk from the top to the bin
// that holds the K-th entry, then either the bin is wanted whole, or it is small enough to rank
// by brute force, or it becomes the next window (its width shrinks 2048-fold per round, so at
// most six rounds for 64-bit entries; one round unless many scores tie).  While a bin is wider
// than 2^32 entries it is a range of keys and a source that has to look positions up need not.
// The last sweep writes every entry above the final bin, lists the bin's own and ranks those.
// Positions are written unordered; the functions return how many: min(K, entries).

// A row of score keys: slot s holds keys[s] (0 = empty) and stands for position cand[s]
// (s < n_cand); nslots is a multiple of 32.
struct KeyRowSrc {
  static constexpr bool kKeysApart = true;       // keys can be swept without their positions
  const uint32_t* keys;
  int nslots;
  const int32_t* __restrict__ cand;
  int n_cand;
  template <int U, typename F>
  __device__ __forceinline__ void sweep_keys(int lane, F f) const {
    for (int s0 = 0; s0 < nslots; s0 += 32 * U) {
      uint32_t k[U];
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int sl = s0 + j * 32 + lane;
        k[j] = sl < nslots ? __ldcg(keys + sl) : 0u;
      }
#pragma unroll
      for (int j = 0; j < U; ++j) f(k[j]);
    }
  }
  template <int U, bool NEED_POS, typename F>
  __device__ __forceinline__ void sweep(int lane, F f) const {
    for (int s0 = 0; s0 < nslots; s0 += 32 * U) {
      uint32_t k[U];
      int ps[U];
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int sl = s0 + j * 32 + lane;
        k[j] = sl < nslots ? __ldcg(keys + sl) : 0u;
        ps[j] = (NEED_POS && sl < n_cand) ? __ldg(cand + sl) : -1;
      }
#pragma unroll
      for (int j = 0; j < U; ++j) f(k[j] ? make_entry(k[j], ps[j]) : 0ull);   // without positions: low word 0
    }
  }
};

// A segment of packed entries (padding entries, position -1, count as empty).
struct SegSrc {
  static constexpr bool kKeysApart = false;
  const entry_t* e;
  int cnt;
  template <int U, bool NEED_POS, typename F>
  __device__ __forceinline__ void sweep(int lane, F f) const {
    for (int i0 = 0; i0 < cnt; i0 += 32 * U) {
      entry_t x[U];
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int i = i0 + j * 32 + lane;
        x[j] = i < cnt ? __ldcg(e + i) : 0ull;
      }
#pragma unroll
      for (int j = 0; j < U; ++j) f(entry_pos(x[j]) >= 0 ? x[j] : 0ull);
    }
  }
};

// Last sweep: entries above bhi go out, those in [elo, bhi] are listed and the need_b best of
// the list follow.  elo > bhi: nothing is listed.
template <typename Src>
__device__ __forceinline__ int warp_emit_above(SegSelSmem& sm, const Src& src, entry_t elo, entry_t bhi, uint32_t need_b,
                                               int32_t* out, float* out_score, int K, int lane) {
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t base = 0, ln = 0;
  src.template sweep<16, true>(lane, [&](entry_t e) {
    const bool em = e > bhi;
    const bool edge = e >= elo && e <= bhi;
    const uint32_t m = __ballot_sync(0xffffffffu, em);
    const uint32_t me = __ballot_sync(0xffffffffu, edge);
    const uint32_t p = base + __popc(m & lt);
    const uint32_t q = ln + __popc(me & lt);
    if (em && p < (uint32_t)K) out[p] = entry_pos(e);
    if (edge && q < (uint32_t)kSelSmall) sm.list[q] = e;
    base += __popc(m);
    ln += __popc(me);
  });
  if (out_score) {                           // the scores, when asked for, take a sweep of their own
    uint32_t b2 = 0;
    src.template sweep<16, true>(lane, [&](entry_t e) {
      const bool em = e > bhi;
      const uint32_t m = __ballot_sync(0xffffffffu, em);
      const uint32_t p = b2 + __popc(m & lt);
      if (em && p < (uint32_t)K) out_score[p] = key_to_score(entry_key(e));
      b2 += __popc(m);
    });
  }
  __syncwarp();
  ln = ln < (uint32_t)kSelSmall ? ln : (uint32_t)kSelSmall;
  for (uint32_t t = lane; t < ln; t += 32) {                      // entries are distinct: ranks are slots
    const entry_t xt = sm.list[t];
    uint32_t rank = 0;
    for (uint32_t u = 0; u < ln; ++u) rank += sm.list[u] > xt ? 1u : 0u;
    if (rank < need_b && base + rank < (uint32_t)K) {
      out[base + rank] = entry_pos(xt);
      if (out_score) out_score[base + rank] = key_to_score(entry_key(xt));
    }
  }
  __syncwarp();
  const uint32_t n_out = base + (ln < need_b ? ln : need_b);
  return (int)(n_out < (uint32_t)K ? n_out : (uint32_t)K);
}

// [lo, hi] holds every entry of the source, n_filled of them.
template <typename Src>
__device__ __noinline__ int warp_topk_entries(SegSelSmem& sm, const Src src, entry_t lo, entry_t hi, uint32_t n_filled,
                                              int32_t* out, float* out_score, int K, int lane) {
  entry_t elo = 1ull, bhi = 0ull;            // n_filled <= K: every entry is "above"
  uint32_t need_b = 0;
  if (n_filled > (uint32_t)K) {
    uint32_t need = (uint32_t)K;
    for (int round = 0; round < 8; ++round) {
      const entry_t span = hi - lo;
      const int bits = 64 - __clzll((long long)(span | 1ull));
      const int shift = bits > 11 ? bits - 11 : 0;
      for (int i = lane; i < kSelBins / 4; i += 32) reinterpret_cast<uint4*>(sm.hist)[i] = make_uint4(0, 0, 0, 0);
      __syncwarp();
      auto count = [&](entry_t e) {
        if (e >= lo && e <= hi && e) atomicAdd(&sm.hist[(uint32_t)((e - lo) >> shift)], 1u);
      };
      bool counted = false;
      if constexpr (Src::kKeysApart) {
        if (shift >= 32) {                   // bins are key ranges (lo has a zero low word then)
          const uint32_t klo = (uint32_t)(lo >> 32), khi = (uint32_t)(hi >> 32);
          const int ksh = shift - 32;
          src.template sweep_keys<32>(lane, [&](uint32_t k) {
            if (k >= klo && k <= khi && k) atomicAdd(&sm.hist[(k - klo) >> ksh], 1u);
          });
          counted = true;
        }
      }
      if (!counted) src.template sweep<16, true>(lane, count);
      __syncwarp();
      uint32_t b, pop;
      warp_hist_boundary(sm.hist, need, lane, &b, &need_b, &pop);
      const entry_t blo = lo + ((entry_t)b << shift);
      bhi = shift ? blo + (((entry_t)1 << shift) - 1ull) : blo;
      bhi = bhi < hi ? bhi : hi;
      elo = blo;
      if (pop == need_b) { bhi = blo - 1ull; elo = ~0ull; break; }   // the bin is wanted whole: it counts as "above"
      if (pop <= (uint32_t)kSelSmall) break;
      lo = blo; hi = bhi; need = need_b;     // crowded bin (ties): it is the next window
    }
  }
  return warp_emit_above(sm, src, elo, bhi, need_b, out, out_score, K, lane);
}

__device__ __forceinline__ int warp_row_topk(SegSelSmem& sm, const uint32_t* keys, int nslots,
                                             const int32_t* __restrict__ cand, int n_cand, int32_t* out,
                                             float* out_score, int K, int lane, uint32_t kmin, uint32_t kmax,
                                             uint32_t n_filled) {
  return warp_topk_entries(sm, KeyRowSrc{keys, nslots, cand, n_cand}, (entry_t)kmin << 32,
                           ((entry_t)kmax << 32) | 0xffffffffull, n_filled, out, out_score, K, lane);
}

// A scan row's segment whose entries were all counted in a histogram with bins bin_of(key):
// bsel = the boundary bin (need_b of its pop entries are wanted), -1 = everything is wanted.
// One sweep, unless the boundary bin is too crowded to rank (ties): then the general way.
template <typename BinFn>
__device__ __noinline__ int warp_seg_topk_binned(SegSelSmem& sm, const entry_t* seg, int cnt, BinFn bin_of, int bsel,
                                                 uint32_t need_b, uint32_t pop, int32_t* out, float* out_score, int K,
                                                 int lane) {
  const SegSrc src{seg, cnt};
  if (bsel >= 0 && pop != need_b && pop > (uint32_t)kSelSmall) {
    entry_t mn = ~0ull, mx = 0ull;
    uint32_t nv = 0;
    src.template sweep<16, true>(lane, [&](entry_t e) {
      mn = (e && e < mn) ? e : mn;
      mx = e > mx ? e : mx;
      nv += e ? 1u : 0u;
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const entry_t a = __shfl_xor_sync(0xffffffffu, mn, o), c = __shfl_xor_sync(0xffffffffu, mx, o);
      mn = a < mn ? a : mn;
      mx = c > mx ? c : mx;
    }
    nv = __reduce_add_sync(0xffffffffu, nv);
    return warp_topk_entries(sm, src, mn, mx, nv, out, out_score, K, lane);
  }
  // the boundary bin as a set of entries: {e : bin_of(key(e)) == bsel}; above it: bin > bsel
  const uint32_t lt = (1u << lane) - 1u;
  const bool whole = bsel >= 0 && pop == need_b;
  const int bcut = whole ? bsel - 1 : bsel;  // a bin wanted whole counts as "above"
  uint32_t base = 0, ln = 0;
  src.template sweep<16, true>(lane, [&](entry_t e) {
    const int bn = e ? (int)bin_of(entry_key(e)) : -2;
    const bool em = bn > bcut;
    const bool edge = bn == bcut && bsel >= 0 && !whole;
    const uint32_t m = __ballot_sync(0xffffffffu, em);
    const uint32_t me = __ballot_sync(0xffffffffu, edge);
    const uint32_t p = base + __popc(m & lt);
    const uint32_t q = ln + __popc(me & lt);
    if (em && p < (uint32_t)K) out[p] = entry_pos(e);
    if (edge && q < (uint32_t)kSelSmall) sm.list[q] = e;
    base += __popc(m);
    ln += __popc(me);
  });
  if (out_score) {
    uint32_t b2 = 0;
    src.template sweep<16, true>(lane, [&](entry_t e) {
      const bool em = (e ? (int)bin_of(entry_key(e)) : -2) > bcut;
      const uint32_t m = __ballot_sync(0xffffffffu, em);
      const uint32_t p = b2 + __popc(m & lt);
      if (em && p < (uint32_t)K) out_score[p] = key_to_score(entry_key(e));
      b2 += __popc(m);
    });
  }
  __syncwarp();
  ln = ln < (uint32_t)kSelSmall ? ln : (uint32_t)kSelSmall;
  for (uint32_t t = lane; t < ln; t += 32) {
    const entry_t xt = sm.list[t];
    uint32_t rank = 0;
    for (uint32_t u = 0; u < ln; ++u) rank += sm.list[u] > xt ? 1u : 0u;
    if (rank < need_b && base + rank < (uint32_t)K) {
      out[base + rank] = entry_pos(xt);
      if (out_score) out_score[base + rank] = key_to_score(entry_key(xt));
    }
  }
  __syncwarp();
  const uint32_t n_out = base + (ln < need_b ? ln : need_b);
  return (int)(n_out < (uint32_t)K ? n_out : (uint32_t)K);
}

}  // namespace pivot
