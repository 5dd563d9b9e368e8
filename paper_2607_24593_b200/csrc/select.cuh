// Exact block-cooperative top-K selection over a buffer of (key, index) entries.
//
// Order: larger key first; among equal keys the smaller index first -- the total order of the
// TopK operator used for Eq. 6 / 7 / 9.  MSB-first radix select, 8 bits per pass, with the
// histogram in shared memory; a second radix select over the indices resolves a tie class that
// straddles the K-th place.  The selected entries are written out unordered.
#pragma once
#include "common.cuh"

namespace pivot {

// A set of threads that work together: `nthr` threads with ranks `tid`, synchronised through
// hardware barrier `bar` (0 with all threads of the block is __syncthreads()).
struct Team {
  int tid, nthr, bar;
  __device__ __forceinline__ void sync() const {
    asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(nthr) : "memory");
  }
};

struct SelectSmem {
  uint32_t hist[256];
  uint32_t prefix;     // bits resolved so far
  uint32_t need;       // how many entries are still wanted inside the current prefix
  uint32_t count_eq;   // population of the bin picked in the last pass
  uint32_t out_count;  // compaction cursor
  uint32_t kmin, kmax; // key range of the current selection (register-resident variant)
};

// Warp 0 of the team: find the bin (scanning from the top if DESC, else from the bottom) in
// which the cumulative count reaches sm.need; update prefix / need / count_eq.
template <bool DESC>
__device__ __forceinline__ void pick_bin(SelectSmem& sm, int lane, int width = 8) {
  uint32_t local[8];
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int bin = DESC ? (255 - 8 * lane - i) : (8 * lane + i);
    local[i] = sm.hist[bin];
    s += local[i];
  }
  uint32_t incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  uint32_t excl = incl - s;
  uint32_t need = sm.need;
  __syncwarp();
  if (excl < need && need <= incl) {
    uint32_t cum = excl;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (cum + local[i] >= need) {
        int bin = DESC ? (255 - 8 * lane - i) : (8 * lane + i);
        sm.prefix = (sm.prefix << width) | (uint32_t)bin;
        sm.need = need - cum;
        sm.count_eq = local[i];
        break;
      }
      cum += local[i];
    }
  }
}

// Selects the K best of n entries (K <= n) from (key, idx) into (okey, oidx) (either may be
// nullptr), unordered.  If out_score != nullptr the scores are written instead of keys.
// All threads of the team must call.  key/idx must not alias the outputs.
__device__ inline void team_select_topk(const Team& tm, SelectSmem& sm, const uint32_t* key,
                                        const int32_t* idx, int n, int K, uint32_t* okey,
                                        int32_t* oidx, float* oscore, uint32_t* tau_out) {
  const int lane = tm.tid & 31;
  if (tm.tid == 0) { sm.prefix = 0; sm.need = (uint32_t)K; sm.count_eq = 0; sm.out_count = 0; }
  // ---- K-th largest key
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tm.tid; i < 256; i += tm.nthr) sm.hist[i] = 0;
    tm.sync();
    const uint32_t prefix = sm.prefix;
    for (int i = tm.tid; i < n; i += tm.nthr) {
      uint32_t kx = key[i];
      bool in = (pass == 0) || ((kx >> (shift + 8)) == prefix);
      if (in) atomicAdd(&sm.hist[(kx >> shift) & 255u], 1u);
    }
    tm.sync();
    if (tm.tid < 32) pick_bin<true>(sm, lane);
    tm.sync();
  }
  const uint32_t tau = sm.prefix;
  const uint32_t need_eq = sm.need;      // entries with key == tau to take (>= 1)
  const uint32_t count_eq = sm.count_eq;
  tm.sync();
  // ---- tie class larger than needed: need_eq-th smallest index among key == tau
  int32_t idx_thr = 0x7fffffff;
  if (count_eq > need_eq) {
    if (tm.tid == 0) { sm.prefix = 0; sm.need = need_eq; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tm.tid; i < 256; i += tm.nthr) sm.hist[i] = 0;
      tm.sync();
      const uint32_t prefix = sm.prefix;
      for (int i = tm.tid; i < n; i += tm.nthr) {
        if (key[i] != tau) continue;
        uint32_t ix = (uint32_t)idx[i];
        bool in = (pass == 0) || ((ix >> (shift + 8)) == prefix);
        if (in) atomicAdd(&sm.hist[(ix >> shift) & 255u], 1u);
      }
      tm.sync();
      if (tm.tid < 32) pick_bin<false>(sm, lane);
      tm.sync();
    }
    idx_thr = (int32_t)sm.prefix;
    tm.sync();
  }
  // ---- write the winners (warp-aggregated cursor)
  for (int base = 0; base < n; base += tm.nthr) {
    int i = base + tm.tid;
    bool keep = false;
    uint32_t kx = 0;
    int32_t ix = 0;
    if (i < n) {
      kx = key[i];
      ix = idx[i];
      keep = (kx > tau) || (kx == tau && ix <= idx_thr);
    }
    uint32_t m = __ballot_sync(0xffffffffu, keep);
    if (m) {
      uint32_t pos = 0;
      if (lane == __ffs(m) - 1) pos = atomicAdd(&sm.out_count, (uint32_t)__popc(m));
      pos = __shfl_sync(0xffffffffu, pos, __ffs(m) - 1);
      if (keep) {
        uint32_t p = pos + __popc(m & ((1u << lane) - 1u));
        if (okey) okey[p] = kx;
        if (oidx) oidx[p] = ix;
        if (oscore) oscore[p] = key_to_score(kx);
      }
    }
  }
  tm.sync();
  if (tau_out && tm.tid == 0) *tau_out = tau;
}

// Register-resident variant for n <= EPT * team size: every thread loads its EPT keys once
// (entry i = j * nthr + tid) and all radix passes run from registers.  The passes start below
// the bits that all keys share, so a narrow score range does not pile every entry into one
// histogram bin.  Same result and contract as team_select_topk.
template <int EPT>
__device__ __forceinline__ void team_select_topk_reg(const Team& tm, SelectSmem& sm, const uint32_t* key,
                                                     const int32_t* idx, int n, int K, uint32_t* okey,
                                                     int32_t* oidx, float* oscore, uint32_t* tau_out) {
  const int lane = tm.tid & 31;
  const int nj = n > tm.tid ? (n - tm.tid + tm.nthr - 1) / tm.nthr : 0;   // my valid entries
  uint32_t kv[EPT];
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int j = 0; j < EPT; ++j) kv[j] = j < nj ? __ldcg(key + (size_t)j * tm.nthr + tm.tid) : 0u;
#pragma unroll
  for (int j = 0; j < EPT; ++j)
    if (j < nj) { kmin = min(kmin, kv[j]); kmax = max(kmax, kv[j]); }
  if (tm.tid == 0) { sm.kmin = 0xffffffffu; sm.kmax = 0u; sm.out_count = 0; sm.count_eq = 0; }
  tm.sync();
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { atomicMin(&sm.kmin, kmin); atomicMax(&sm.kmax, kmax); }
  tm.sync();
  kmin = sm.kmin;
  kmax = sm.kmax;
  const int bits = kmin == kmax ? 0 : 32 - __clz(kmin ^ kmax);    // low bits that differ
  uint32_t tau, need_eq, count_eq;
  if (bits == 0) {
    tau = kmin; need_eq = (uint32_t)K; count_eq = (uint32_t)n;
  } else {
    tm.sync();
    if (tm.tid == 0) { sm.prefix = bits == 32 ? 0u : (kmin >> bits); sm.need = (uint32_t)K; }
    const int passes = (bits + 7) >> 3;
    for (int pass = 0; pass < passes; ++pass) {
      const int top = bits - 8 * pass;             // bits [shift, top) are this pass's digit
      const int shift = top > 8 ? top - 8 : 0;
      const int width = top - shift;
      const uint32_t mask = (1u << width) - 1u;
      for (int i = tm.tid; i < 256; i += tm.nthr) sm.hist[i] = 0;
      tm.sync();
      const uint32_t prefix = sm.prefix;
#pragma unroll
      for (int j = 0; j < EPT; ++j) {
        if (j < nj) {
          const bool in = (pass == 0) || ((kv[j] >> top) == prefix);
          if (in) atomicAdd(&sm.hist[(kv[j] >> shift) & mask], 1u);
        }
      }
      tm.sync();
      if (tm.tid < 32) pick_bin<true>(sm, lane, width);
      tm.sync();
    }
    tau = sm.prefix; need_eq = sm.need; count_eq = sm.count_eq;
  }
  tm.sync();
  int32_t idx_thr = 0x7fffffff;
  if (count_eq > need_eq) {       // a tie class straddles the K-th place: lowest indices win
    if (tm.tid == 0) { sm.prefix = 0; sm.need = need_eq; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tm.tid; i < 256; i += tm.nthr) sm.hist[i] = 0;
      tm.sync();
      const uint32_t prefix = sm.prefix;
#pragma unroll
      for (int j = 0; j < EPT; ++j) {
        if (j < nj && kv[j] == tau) {
          const uint32_t ix = (uint32_t)idx[(size_t)j * tm.nthr + tm.tid];
          const bool in = (pass == 0) || ((ix >> (shift + 8)) == prefix);
          if (in) atomicAdd(&sm.hist[(ix >> shift) & 255u], 1u);
        }
      }
      tm.sync();
      if (tm.tid < 32) pick_bin<false>(sm, lane);
      tm.sync();
    }
    idx_thr = (int32_t)sm.prefix;
    tm.sync();
  }
  // winners: one cursor bump per thread, then its kept entries in a row
  const bool ties = idx_thr != 0x7fffffff;
  int cnt = 0;
#pragma unroll
  for (int j = 0; j < EPT; ++j)
    if (j < nj) {
      bool keep = kv[j] > tau;
      if (kv[j] == tau) keep = !ties || idx[(size_t)j * tm.nthr + tm.tid] <= idx_thr;
      cnt += keep ? 1 : 0;
    }
  uint32_t p = cnt ? atomicAdd(&sm.out_count, (uint32_t)cnt) : 0u;
#pragma unroll
  for (int j = 0; j < EPT; ++j)
    if (j < nj && kv[j] >= tau) {
      const int32_t ix = idx[(size_t)j * tm.nthr + tm.tid];
      if (kv[j] > tau || !ties || ix <= idx_thr) {
        if (okey) okey[p] = kv[j];
        if (oidx) oidx[p] = ix;
        if (oscore) oscore[p] = key_to_score(kv[j]);
        ++p;
      }
    }
  tm.sync();
  if (tau_out && tm.tid == 0) *tau_out = tau;
}

// Picks the register-resident variant when the entries fit (team of 128 threads).
__device__ __forceinline__ void team_select_auto(const Team& tm, SelectSmem& sm, const uint32_t* key,
                                                 const int32_t* idx, int n, int K, uint32_t* okey,
                                                 int32_t* oidx, float* oscore, uint32_t* tau_out) {
  if (n <= 32 * tm.nthr) team_select_topk_reg<32>(tm, sm, key, idx, n, K, okey, oidx, oscore, tau_out);
  else if (n <= 64 * tm.nthr) team_select_topk_reg<64>(tm, sm, key, idx, n, K, okey, oidx, oscore, tau_out);
  else team_select_topk(tm, sm, key, idx, n, K, okey, oidx, oscore, tau_out);
}

}  // namespace pivot
