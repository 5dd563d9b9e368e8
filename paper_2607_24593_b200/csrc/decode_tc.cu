// Decode path (Algorithm 1 with the grouping of Eq. 3), built for HBM bandwidth.
//
// One MTP step scores one proxy per sequence against that sequence's whole key cache, so the
// step is a single pass over every visible key (128 B + 4 B scale): memory bound.  The work is
// therefore split by KEY TILES, not by rows:
//   decode_prepare_kernel one block per sequence clears its histogram, plans it, builds its proxy
//                        and writes its share of the tile prefix, candidate chunks and entry lists.
//   decode_scan_kernel   every SM takes an equal, contiguous share of all (sequence, 128-key
//                        tile) pairs; per tile: TMA -> tcgen05 MMA (128 keys x 64 heads x d) ->
//                        epilogue (ReLU, gate-weighted head sum, key scale) -> one fp32 score per
//                        key to an L2-resident score array (3 % of the bytes read), plus a
//                        8192-bin histogram of the scores' top 13 key bits per sequence.
//   decode_select_kernel a cluster of four 1024-thread CTAs per sequence: the histogram gives the
//                        bin holding the K-th best score; each CTA collects the survivors of its
//                        quarter of the score array in its shared memory; after a cluster barrier
//                        CTA 0 reads the other three lists through distributed shared memory and
//                        takes the exact top-K (Eq. 6 / 7) of the union.  If the boundary bin
//                        leaves too many candidates, one CTA alone refines it 12 bits at a time
//                        with further passes over the scores.
//   decode_window_kernel (only with a local window, Appendix B) the union of the step's per-query
//                        windows as one more candidate chunk per sequence, minus the positions
//                        the pool already holds.
//   entries_topk_kernel  exact top-k (Eq. 9) of each query's re-scored candidates, which the
//                        gather + re-score kernel leaves as packed entries (refine_tc.cu, chunked
//                        over candidates so that all SMs take part).
#include <cuda.h>
#include <string.h>

#include <cooperative_groups.h>

#include "blockselect.cuh"
#include "kernels.h"
#include "plan.cuh"
#include "proxy_math.cuh"
#include "ptx.cuh"

namespace pivot {
namespace {

namespace cg = cooperative_groups;
constexpr int TILE_KEYS = 128;
constexpr int DKS_SLOTS = 14;
constexpr int DHIST_BITS = 13;          // histogram digit: top 13 bits of the score key (16 bins per octave)
constexpr int DHIST = 1 << DHIST_BITS;
constexpr int D_N = kHeads;             // MMA N: one proxy
constexpr int D_THREADS = 64 + 256;     // TMA warp, MMA warp, two sets of four epilogue warps
constexpr int SEL_CAP = 16384;          // candidates collected in shared memory per sequence
constexpr int SEL_SPLIT = 4;            // CTAs sharing the collection pass of one sequence

template <int DT>
struct DCfg {
  static constexpr bool FP8 = DT == DT_FP8;
  static constexpr int KHALVES = FP8 ? 1 : 2;
  static constexpr int HALF_TILE_BYTES = TILE_KEYS * 128;
  static constexpr int STAGE_BYTES = KHALVES * HALF_TILE_BYTES;
  static constexpr int QHALF_BYTES = kHeads * 128;
  static constexpr int QBUF_BYTES = KHALVES * QHALF_BYTES;
  static constexpr int STAGES = FP8 ? 8 : 3;
  static constexpr uint32_t IDESC = ptx::make_idesc(FP8 ? 0u : 1u, TILE_KEYS, D_N);
};

struct DCtrl {
  alignas(128) float ks[DKS_SLOTS][TILE_KEYS];
  alignas(16) float w[2][kHeads];       // per epilogue set: gate of its current sequence
  uint32_t hist[2][DHIST];              // per epilogue set: histogram of its current sequence
  uint64_t full[8], empty[8], q_full[2], q_empty[2], tmem_full[2], tmem_empty[2], ks_full[DKS_SLOTS];
  uint32_t tmem_base;
  int abort;
};

template <int DT>
constexpr size_t dsmem_bytes() {
  return 1024 + 2 * DCfg<DT>::QBUF_BYTES + DCfg<DT>::STAGES * DCfg<DT>::STAGE_BYTES + sizeof(DCtrl);
}

// Walks the global tile index space: sequence b owns tiles [prefix[b], prefix[b+1]).
struct TileWalk {
  const int* prefix;
  int B, b;
  __device__ TileWalk(const int* p, int nb) : prefix(p), B(nb), b(0) {}
  __device__ __forceinline__ int seq_of(int g) {     // g non-decreasing between calls
    while (b + 1 < B && g >= prefix[b + 1]) ++b;
    return b;
  }
};

template <int DT>
__global__ void __launch_bounds__(D_THREADS, 1)
decode_scan_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                   const __grid_constant__ CUtensorMap tm_ks, const RowDesc* __restrict__ prox,
                   const int* __restrict__ tile_prefix, int B, int Lmax, float* __restrict__ scores,
                   uint32_t* __restrict__ ghist, int* status) {
  using C = DCfg<DT>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* qbuf = smem;
  uint8_t* kring = smem + 2 * C::QBUF_BYTES;
  DCtrl& ct = *reinterpret_cast<DCtrl*>(kring + C::STAGES * C::STAGE_BYTES);
  volatile int* abort_flag = &ct.abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { ptx::mbar_init(&ct.full[s], 1); ptx::mbar_init(&ct.empty[s], 1); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ct.q_full[i], 1);
      ptx::mbar_init(&ct.q_empty[i], 1);
      ptx::mbar_init(&ct.tmem_full[i], 1);
      ptx::mbar_init(&ct.tmem_empty[i], 4);   // the four warps of the set that owns buffer i
    }
    for (int i = 0; i < DKS_SLOTS; ++i) ptx::mbar_init(&ct.ks_full[i], 1);
    ct.abort = 0;
    ptx::fence_barrier_init();
  }
  for (int i = threadIdx.x; i < 2 * DHIST; i += D_THREADS) (&ct.hist[0][0])[i] = 0;
  if (warp == 1) { ptx::tmem_alloc(&ct.tmem_base, 2 * D_N); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = ct.tmem_base;
  // everything above touches only this CTA's own shared and tensor memory: it may overlap the
  // prepare kernel; from here on the plan, the proxies and the cleared histograms are read
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  const int total = tile_prefix[B];
  const int g_lo = (int)((long long)blockIdx.x * total / gridDim.x);
  const int g_hi = (int)((long long)(blockIdx.x + 1) * total / gridDim.x);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      ptx::prefetch_tensormap(&tm_k);
      ptx::prefetch_tensormap(&tm_q);
      if (C::FP8) ptx::prefetch_tensormap(&tm_ks);
      TileWalk tw(tile_prefix, B);
      int cur_b = -1;
      uint32_t it = 0, blk = 0;
      PIVOT_PROF_DO(long long pwait = 0;)
      for (int g = g_lo; g < g_hi; ++g, ++it) {
        const int b = tw.seq_of(g);
        const int t = g - tile_prefix[b];
        if (b != cur_b) {             // new sequence: its proxy becomes the MMA's B operand
          const int qb = blk & 1;
          if (!ptx::mbar_wait(&ct.q_empty[qb], ((blk >> 1) & 1) ^ 1, abort_flag, 64)) break;
          ptx::mbar_arrive_expect_tx(&ct.q_full[qb], C::QBUF_BYTES);
          for (int h = 0; h < C::KHALVES; ++h)
            ptx::tma_load_2d(qbuf + qb * C::QBUF_BYTES + h * C::QHALF_BYTES, &tm_q, h * 64, prox[b].q_row * kHeads,
                             &ct.q_full[qb]);
          ++blk;
          cur_b = b;
        }
        // Row of the tile inside the key tensor.  Paged cache: the sequence's block table names
        // the pool page (a page outside the pool reads as zero fill, like any out-of-range box).
        const int32_t* pages = prox[b].pages;
        (void)PIVOT_BOUNDS(t * TILE_KEYS < Lmax, status);              // checked build: the tile lies inside the sequence's rows
        const int krow = pages ? __ldg(pages + t) * TILE_KEYS : prox[b].k_row0 + t * TILE_KEYS;
        const int s = it % C::STAGES;
        PIVOT_PROF_DO(const long long pw0 = clock64();)
        if (!ptx::mbar_wait(&ct.empty[s], ((it / C::STAGES) & 1) ^ 1, abort_flag, 64)) break;
        PIVOT_PROF_DO(pwait += clock64() - pw0;)
        ptx::mbar_arrive_expect_tx(&ct.full[s], C::STAGE_BYTES);
        for (int h = 0; h < C::KHALVES; ++h)
          ptx::tma_load_2d(kring + s * C::STAGE_BYTES + h * C::HALF_TILE_BYTES, &tm_k, h * 64, krow, &ct.full[s]);
        if (C::FP8) {
          const int ksl = it % DKS_SLOTS;       // free by construction (see the prefill scan)
          ptx::mbar_arrive_expect_tx(&ct.ks_full[ksl], TILE_KEYS * 4);
          ptx::tma_load_1d(&ct.ks[ksl][0], &tm_ks, krow, &ct.ks_full[ksl]);
        }
      }
      PIVOT_PROF_DO(prof_add(status, PROF_DSCAN_PRODUCER_WAIT, pwait);)
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
      TileWalk tw(tile_prefix, B);
      int cur_b = -1, qb = 0;
      uint32_t it = 0, blk = 0;
      bool ok = true;
      PIVOT_PROF_DO(long long pw[3] = {0, 0, 0}; const long long pstart = clock64();)
#ifdef PIVOT_PROF
#define PW(i, ...) { const long long t_ = clock64(); __VA_ARGS__; pw[i] += clock64() - t_; }
#else
#define PW(i, ...) __VA_ARGS__;
#endif
      for (int g = g_lo; g < g_hi && ok; ++g, ++it) {
        const int b = tw.seq_of(g);
        if (b != cur_b) {
          if (cur_b >= 0) ptx::tc_commit(&ct.q_empty[qb]);     // previous proxy no longer needed
          qb = blk & 1;
          PW(0, ok = ptx::mbar_wait(&ct.q_full[qb], (blk >> 1) & 1, abort_flag, 32))
          if (!ok) break;
          ++blk;
          cur_b = b;
        }
        const int s = it % C::STAGES;
        const int buf = it & 1;
        PW(1, ok = ptx::mbar_wait(&ct.tmem_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, 32))
        if (!ok) break;
        PW(2, ok = ptx::mbar_wait(&ct.full[s], (it / C::STAGES) & 1, abort_flag, 32))
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t k_addr = ptx::smem_u32(kring + s * C::STAGE_BYTES);
        const uint32_t q_addr = ptx::smem_u32(qbuf + qb * C::QBUF_BYTES);
        const uint32_t d_tmem = tmem_base + buf * D_N;
#pragma unroll
        for (int h = 0; h < C::KHALVES; ++h)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            ptx::tc_mma<C::FP8>(d_tmem, ptx::smem_desc_sw128(k_addr + h * C::HALF_TILE_BYTES + ks * 32),
                                ptx::smem_desc_sw128(q_addr + h * C::QHALF_BYTES + ks * 32), C::IDESC,
                                (h | ks) ? 1u : 0u);
        ptx::tc_commit(&ct.empty[s]);
        ptx::tc_commit(&ct.tmem_full[buf]);
      }
#undef PW
      PIVOT_PROF_DO({
        prof_add(status, PROF_DSCAN_WAIT_ACC, pw[0] + pw[1]);       // (the proxy wait, a few clocks per tile, is counted here)
        prof_add(status, PROF_DSCAN_WAIT_KEYS, pw[2]);
        prof_max(status, PROF_DSCAN_MAX_TOTAL, clock64() - pstart);
        prof_add(status, PROF_DSCAN_TOTAL, clock64() - pstart);
        prof_add(status, PROF_DSCAN_TILES, it);
      })
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // Two sets of four warps take alternate tiles (set s drains accumulator buffer s), so one
    // set's head sum overlaps the other's wait; each set keeps its own gate copy and histogram.
    const int set = (warp - 2) >> 2;
    const int tt = (threadIdx.x - 64) & 127;         // 0..127 inside the set
    const int lq = warp & 3;
    const int key_in_tile = lq * 32 + lane;
    const Team tm{tt, 128, 1 + set};
    TileWalk tw(tile_prefix, B);
    int cur_b = -1, n_vis = 0;
    auto flush_hist = [&](int b) {
      tm.sync();
      for (int i = tt; i < DHIST; i += 128) {
        const uint32_t h = ct.hist[set][i];
        if (h) { atomicAdd(&ghist[(size_t)b * DHIST + i], h); ct.hist[set][i] = 0; }
      }
      tm.sync();
    };
    for (int g = g_lo + set; g < g_hi; g += 2) {
      const uint32_t it = (uint32_t)(g - g_lo);
      const int b = tw.seq_of(g);
      const int t = g - tile_prefix[b];
      if (b != cur_b) {
        if (cur_b >= 0) flush_hist(cur_b);
        cur_b = b;
        n_vis = prox[b].n_vis;
        tm.sync();
        if (tt < kHeads) ct.w[set][tt] = 0.5f * prox[b].w[tt];      // proxy gate, halved (ReLU identity)
        tm.sync();
      }
      const int buf = it & 1;                        // == set
      float ksv = 1.f;
      if (C::FP8) {
        const int ksl = it % DKS_SLOTS;
        (void)ptx::mbar_wait(&ct.ks_full[ksl], (it / DKS_SLOTS) & 1, abort_flag);
        ksv = ct.ks[ksl][key_in_tile];
      }
      (void)ptx::mbar_wait(&ct.tmem_full[buf], (it >> 1) & 1, abort_flag);
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(lq * 32) << 16) + buf * D_N;
      uint32_t v0[32], v1[32];
      ptx::tmem_ld_32x32(taddr, v0);
      ptx::tmem_ld_32x32(taddr + 32, v1);
      ptx::tmem_wait_ld();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&ct.tmem_empty[buf]);
      float ap[4] = {0.f, 0.f, 0.f, 0.f}, an[4] = {0.f, 0.f, 0.f, 0.f};
      const float4* wp = reinterpret_cast<const float4*>(&ct.w[set][0]);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float4 wa = wp[j], wbv = wp[8 + j];
        const float x0 = __uint_as_float(v0[4 * j]), x1 = __uint_as_float(v0[4 * j + 1]);
        const float x2 = __uint_as_float(v0[4 * j + 2]), x3 = __uint_as_float(v0[4 * j + 3]);
        const float y0 = __uint_as_float(v1[4 * j]), y1 = __uint_as_float(v1[4 * j + 1]);
        const float y2 = __uint_as_float(v1[4 * j + 2]), y3 = __uint_as_float(v1[4 * j + 3]);
        ap[0] = fmaf(fabsf(x0), wa.x, ap[0]); an[0] = fmaf(x0, wa.x, an[0]);
        ap[1] = fmaf(fabsf(x1), wa.y, ap[1]); an[1] = fmaf(x1, wa.y, an[1]);
        ap[2] = fmaf(fabsf(x2), wa.z, ap[2]); an[2] = fmaf(x2, wa.z, an[2]);
        ap[3] = fmaf(fabsf(x3), wa.w, ap[3]); an[3] = fmaf(x3, wa.w, an[3]);
        ap[0] = fmaf(fabsf(y0), wbv.x, ap[0]); an[0] = fmaf(y0, wbv.x, an[0]);
        ap[1] = fmaf(fabsf(y1), wbv.y, ap[1]); an[1] = fmaf(y1, wbv.y, an[1]);
        ap[2] = fmaf(fabsf(y2), wbv.z, ap[2]); an[2] = fmaf(y2, wbv.z, an[2]);
        ap[3] = fmaf(fabsf(y3), wbv.w, ap[3]); an[3] = fmaf(y3, wbv.w, an[3]);
      }
      float sv = ((ap[0] + an[0]) + (ap[1] + an[1])) + ((ap[2] + an[2]) + (ap[3] + an[3]));
      if (C::FP8) sv *= ksv;
      const int s_key = t * TILE_KEYS + key_in_tile;
      if (s_key < n_vis && PIVOT_BOUNDS(s_key < Lmax, status)) {
        scores[(size_t)b * Lmax + s_key] = sv;
        atomicAdd(&ct.hist[set][score_to_key(sv) >> (32 - DHIST_BITS)], 1u);
      }
    }
    if (cur_b >= 0) flush_hist(cur_b);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, 2 * D_N);
  if (threadIdx.x == 0 && ct.abort) set_status(status, DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------------------ per-sequence select

struct SelSmem {
  BlkSelSmem blk;
  entry_t list[SEL_CAP];
};

// The SEL_SPLIT CTAs of a sequence are one thread-block cluster (blockIdx.x = rank in it).
__global__ void __cluster_dims__(SEL_SPLIT, 1, 1) __launch_bounds__(kBlk, 1)
decode_select_kernel(const RowDesc* __restrict__ prox, int Ls, const float* __restrict__ scores,
                     const uint32_t* __restrict__ ghist, int* status) {
  extern __shared__ uint8_t sel_raw[];
  SelSmem& sm = *reinterpret_cast<SelSmem*>(((uintptr_t)sel_raw + 15) & ~(uintptr_t)15);
  const int split = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();            // the scan's scores and histograms (before any early return)
  PIVOT_PROF_DO(long long pt[5]; pt[0] = clock64();)
  const RowDesc rd = prox[b];
  const int K = rd.K, n0 = rd.n_vis;
  if (K <= 0) return;
  const float* sc = scores + (size_t)b * Ls;
  // ---- narrow the candidates: entries whose top `pbits` bits are >= prefix
  unsigned long long prefix = 0;
  int pbits = 0;
  bool solo = false;              // this CTA handles the whole sequence by itself
  if (n0 > SEL_CAP) {
    blk_boundary(sm.blk, ghist + (size_t)b * DHIST, DHIST, (uint32_t)K);
    uint32_t need = sm.blk.need, pop = sm.blk.pop;
    prefix = sm.blk.bin;
    pbits = DHIST_BITS;
    // too crowded a boundary bin (every CTA of the sequence sees the same histogram): the
    // refinement passes need the whole score array, CTA 0 takes the sequence alone
    solo = (uint32_t)K - need + pop > (uint32_t)SEL_CAP;
    if (solo && split != 0) return;          // (the whole cluster takes this branch or none: no cluster barrier follows)
    while ((uint32_t)K - need + pop > (uint32_t)SEL_CAP && pbits < 64) {
      const int wbits = 64 - pbits < 12 ? 64 - pbits : 12;
      __syncthreads();
      for (int i = tid; i < 4096; i += kBlk) sm.blk.hist[i] = 0;
      __syncthreads();
      for (int i0 = 0; i0 < n0; i0 += 16 * kBlk) {     // four 16-byte loads in flight per thread
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + (u * kBlk + tid) * 4;
          v[u] = i < n0 ? __ldcg(reinterpret_cast<const float4*>(sc + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
          for (int e4 = 0; e4 < 4; ++e4) {
            const int i = i0 + (u * kBlk + tid) * 4 + e4;
            if (i < n0) {
              const entry_t e = make_entry(score_to_key(vv[e4]), i);
              if ((e >> (64 - pbits)) == prefix)
                atomicAdd(&sm.blk.hist[(uint32_t)((e >> (64 - pbits - wbits)) & ((1u << wbits) - 1u))], 1u);
            }
          }
        }
      }
      blk_boundary(sm.blk, sm.blk.hist, 4096, need);
      need = sm.blk.need;
      pop = sm.blk.pop;
      prefix = (prefix << wbits) | sm.blk.bin;
      pbits += wbits;
    }
  }
  PIVOT_PROF_DO(pt[1] = clock64();)
  // ---- collect them in shared memory: this CTA's share of the scores (multiples of four)
  const int lo = solo ? 0 : (int)(((long long)n0 * split / SEL_SPLIT) & ~3ll);
  const int hi = (solo || split == SEL_SPLIT - 1) ? n0 : (int)(((long long)n0 * (split + 1) / SEL_SPLIT) & ~3ll);
  if (tid == 0) sm.blk.list_n = 0;
  __syncthreads();
  for (int i0 = lo; i0 < hi; i0 += 32 * kBlk) {        // eight 16-byte loads in flight per thread
    float4 v4[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + (u * kBlk + tid) * 4;
      v4[u] = i < hi ? __ldcg(reinterpret_cast<const float4*>(sc + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // One list-cursor bump per warp and pass: each thread counts its keepers among its 32
    // scores, a warp scan turns the counts into offsets (a bump per keeper group would queue
    // hundreds of same-address atomics per pass).  The test runs on the 32-bit score key while
    // the prefix is no longer than that (always, unless a crowded bin was refined further):
    // the pass is bound by its instruction count, not by the loads.
    auto score_of = [&](int u) -> float {
      const float4 q4 = v4[u >> 2];
      return (u & 3) == 0 ? q4.x : (u & 3) == 1 ? q4.y : (u & 3) == 2 ? q4.z : q4.w;
    };
    auto pos_of = [&](int u) -> int { return i0 + ((u >> 2) * kBlk + tid) * 4 + (u & 3); };
    uint32_t keepmask = 0;
    if (pbits <= 32) {
      const uint32_t kthr = pbits ? (uint32_t)prefix << (32 - pbits) : 0u;
#pragma unroll
      for (int u = 0; u < 32; ++u)
        keepmask |= (pos_of(u) < hi && score_to_key(score_of(u)) >= kthr) ? 1u << u : 0u;
    } else {
#pragma unroll
      for (int u = 0; u < 32; ++u) {
        const entry_t e = make_entry(score_to_key(score_of(u)), pos_of(u));
        keepmask |= (pos_of(u) < hi && (e >> (64 - pbits)) >= prefix) ? 1u << u : 0u;
      }
    }
    const uint32_t cnt = (uint32_t)__popc(keepmask);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
    if (tot) {                                           // warp-uniform
      uint32_t base = 0;
      if (lane == 31) base = atomicAdd(&sm.blk.list_n, tot);
      base = __shfl_sync(0xffffffffu, base, 31);
      uint32_t p = base + incl - cnt;
      while (keepmask) {                                 // a few per cent of the scores are kept
        const int u = __ffs(keepmask) - 1;
        keepmask &= keepmask - 1u;
        float vu = 0.f;
#pragma unroll
        for (int q = 0; q < 32; ++q) vu = q == u ? score_of(q) : vu;
        if (p < (uint32_t)SEL_CAP) sm.list[p] = make_entry(score_to_key(vu), pos_of(u));
        ++p;
      }
    }
  }
  __syncthreads();
  PIVOT_PROF_DO(pt[2] = clock64();)
  int n = min((int)sm.blk.list_n, SEL_CAP);
  if (!solo) {
    // ---- hand the shares over: the four CTAs of a sequence form a cluster, and CTA 0 reads the
    //      others' lists out of their shared memory
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();                                      // every list is complete
    if (split == 0) {
      for (int r = 1; r < SEL_SPLIT; ++r) {
        const SelSmem* rs = cluster.map_shared_rank(&sm, r);
        const int nr = min((int)rs->blk.list_n, SEL_CAP);
        for (int i = tid; i < nr; i += kBlk)
          if (n + i < SEL_CAP) sm.list[n + i] = rs->list[i];
        n = min(n + nr, SEL_CAP);
      }
    }
    cluster.sync();                                      // nobody leaves while its list is being read
    if (split != 0) return;
    __syncthreads();
  }
  PIVOT_PROF_DO(pt[3] = clock64();)
  blk_emit_topk(sm.blk, sm.list, n, n, K, rd.out, rd.out_score, rd.out_rows, rd.out_stride);
  PIVOT_PROF_DO(__syncthreads(); if (tid == 0) {
    pt[4] = clock64();
    for (int i = 0; i < 4; ++i) prof_add(status, PROF_DSEL_BOUNDARY + i, pt[i + 1] - pt[i]);
    prof_add(status, PROF_DSEL_SEQS, 1);
  })
  (void)status;
}

// ------------------------------------------------------------------------------ top-k of entry lists

__global__ void __launch_bounds__(kBlk, 1) entries_topk_kernel(const EntryList* __restrict__ lists) {
  __shared__ BlkSelSmem sm;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();            // the re-score's entries
  const EntryList el = lists[blockIdx.x];
  if (el.K <= 0) return;
  blk_emit_topk(sm, (const entry_t*)el.list, el.n, el.n, el.K, el.out, el.out_score, 1, el.K);
}

// Union of candidate lists -> packed entries -> exact top-K, one block.
__global__ void __launch_bounds__(kBlk, 1)
merge_topk_kernel(const float* __restrict__ scores, const int32_t* __restrict__ idx, int n_seg, int seg_len,
                  const int32_t* __restrict__ seg_offset, entry_t* __restrict__ entries, int K, int32_t* out_idx,
                  float* out_scores) {
  __shared__ BlkSelSmem sm;
  const int n = n_seg * seg_len;
  for (int i = threadIdx.x; i < n; i += kBlk) {
    const int ix = idx[i];
    const int off = seg_offset ? seg_offset[i / seg_len] : 0;
    entries[i] = ix < 0 ? kPadEntry : make_entry(score_to_key(scores[i]), ix + off);
  }
  __threadfence_block();
  __syncthreads();
  blk_emit_topk(sm, entries, n, n, K, out_idx, out_scores, 1, K);
}

// ------------------------------------------------------------------------------ setup

// One launch prepares a decode step; block b does everything that concerns sequence b and nobody
// waits for anybody: it clears the sequence's histogram and list counters, plans the sequence (row
// and group descriptors, guard test on the device-resident pos0), builds its proxy (Eq. 4), finds
// its place in the tile order of the key-split scan (the tile counts of the sequences before it,
// recomputed from their pos0 -- a few loads instead of a hand-over between blocks), and writes its
// candidate chunks for the re-score and its entry lists for the final top-k.  1024 threads per block.
__device__ __forceinline__ int decode_live_tiles(const DecodePlan& p, int b) {
  // tiles of sequence b's proxy scan, as plan_decode_sequence decides them: 0 for a guarded
  // sequence and for a pos0 outside the cache
  const int p_in = p.pos0[b / p.kv_share];
  const int step = p.g > p.kv_share ? p.g : p.kv_share;
  if (p_in < 0 || p_in > p.Lmax - step) return 0;
  const int n0 = p_in + b % p.kv_share + 1;
  return n0 < p.guard_len ? 0 : (n0 + TILE_KEYS - 1) / TILE_KEYS;
}

__global__ void __launch_bounds__(1024)
decode_prepare_kernel(DecodePlan p, RowDesc* rows, GroupDesc* plan_groups, uint32_t* ghist, int W, int pool, int chunk,
                      int* tile_prefix, GroupDesc* chunks, EntryList* lists, unsigned long long* entries,
                      const int32_t* wcand) {
  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int B = p.B, g = p.g, c = p.c, k = p.k, mode = p.mode;
  ptx::grid_launch_dependents();          // the scan may set itself up meanwhile (it waits before it reads)
  for (int i = tid; i < DHIST; i += blockDim.x) ghist[(size_t)b * DHIST + i] = 0u;
  __shared__ int seq_ok;
  __shared__ int wsum[32];
  if (tid == 0) seq_ok = plan_decode_sequence(p, b, rows, plan_groups) ? 1 : 0;
  // ---- tiles of the sequences before this one
  int part = 0;
  for (int bb = tid; bb < b; bb += blockDim.x) part += decode_live_tiles(p, bb);
  part = __reduce_add_sync(0xffffffffu, part);
  if (lane == 0) wsum[wid] = part;
  __syncthreads();                                 // also: the descriptors thread 0 wrote are visible to the block
  if (tid == 0) {
    int before = 0;
    for (int i = 0; i < 32; ++i) before += wsum[i];
    tile_prefix[b] = before;
    if (b == B - 1) tile_prefix[B] = before + decode_live_tiles(p, b);
  }
  if (!seq_ok) fill_decode_rows_empty(p, b, tid, blockDim.x);     // pos0 outside the cache: rows of -1
  if (p.raw_q) {
    raw_query_gates(p, b, tid, blockDim.x);
  } else {
    // ---- the sequence's proxy: one warp per unit of four (e4m3) or two (bf16) heads
    if (p.dtype == DT_FP8) {
      for (int u = wid; u < proxy_units_per_group<DT_FP8>(); u += 32)
        proxy_build_unit<DT_FP8>(p.q, p.qscale, p.w, p.proxy_q, p.proxy_w, B * g, g, 0, B, pool,
                                 (long long)b * proxy_units_per_group<DT_FP8>() + u, lane);
    } else {
      for (int u = wid; u < proxy_units_per_group<DT_BF16>(); u += 32)
        proxy_build_unit<DT_BF16>(p.q, p.qscale, p.w, p.proxy_q, p.proxy_w, B * g, g, 0, B, pool,
                                  (long long)b * proxy_units_per_group<DT_BF16>() + u, lane);
    }
  }
  if (mode != 1) return;
  // Refine: split every (sequence, member chunk) into candidate chunks so all SMs re-score,
  // each leaving packed entries; one entry list per query for the final top-k.
  const GroupDesc* groups = plan_groups;
  const int mc = (g + kMembersPerDesc - 1) / kMembersPerDesc;
  const int ncc = (c + chunk - 1) / chunk;
  const int nch = ncc + (W > 0 ? 1 : 0);           // with a window: one more chunk, the window slots
  const int w_g = W > 0 ? W + g - 1 : 0;
  const int stride = c + kDecodeWinMax;            // entries per query
  for (int j = tid; j < mc * nch; j += blockDim.x) {
    const int i = b * mc * nch + j;
    const int gi = i / nch, cc = i % nch;
    GroupDesc gd = groups[gi];
    gd.ent_out = entries + (size_t)gd.q_row * stride;
    gd.ent_stride = stride;
    if (cc < ncc) {
      const int left = gd.n_cand - cc * chunk;
      gd.cand = gd.cand + cc * chunk;
      gd.n_cand = left > 0 ? (left < chunk ? left : chunk) : 0;
      gd.slot0 = cc * chunk;
    } else {                 // window slots follow the pool's valid entries
      gd.slot0 = gd.n_cand;
      gd.cand = wcand + (size_t)(gi / mc) * kDecodeWinMax;
      gd.n_cand = gd.n_cand > 0 ? w_g : 0;
      gd.win_span = W;
    }
    chunks[i] = gd;
  }
  for (int j = tid; j < g; j += blockDim.x) {
    const int i = b * g + j;
    const GroupDesc gd = groups[b * mc];
    EntryList el;
    el.list = entries + (size_t)i * stride;
    el.n = gd.n_cand > 0 ? gd.n_cand + w_g : 0;
    el.K = gd.n_cand > 0 ? k : 0;
    el.out = groups[b * mc].out + (size_t)j * gd.out_stride;
    el.out_score = gd.out_score ? groups[b * mc].out_score + (size_t)j * gd.out_stride : nullptr;
    lists[i] = el;
  }
}

// Decode form of the local window (Appendix B): the queries of the step at pos0 .. pos0 + g - 1
// each add their own window [t - W + 1, t] to the pool.  The union of those windows,
// pos0 - W + 1 .. pos0 + g - 1, becomes one more candidate chunk of the sequence; positions the
// pool already holds (and positions before the start of the sequence) are left out as -1, and
// the re-score kernel masks every slot to the members whose window covers it.
__global__ void decode_window_kernel(const GroupDesc* __restrict__ groups, int mc, int g, int W,
                                     int32_t* __restrict__ wcand) {
  __shared__ int dup[kDecodeWinMax];
  const int b = blockIdx.x, tid = threadIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();            // the select's candidate sets
  const GroupDesc gd = groups[b * mc];
  if (gd.n_cand <= 0) return;                      // guarded sequence: scored densely
  const int pos0 = gd.first_pos, lo = pos0 - W + 1, w_g = W + g - 1;
  for (int j = tid; j < w_g; j += blockDim.x) dup[j] = 0;
  __syncthreads();
  for (int i0 = 0; i0 < gd.n_cand; i0 += 4 * blockDim.x) {      // four independent loads per thread
    int p[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * blockDim.x + tid;
      p[u] = i < gd.n_cand ? __ldcg(gd.cand + i) : -1;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (p[u] >= lo && p[u] <= pos0) dup[p[u] - lo] = 1;
  }
  __syncthreads();
  for (int j = tid; j < w_g; j += blockDim.x) {
    const int s = lo + j;
    wcand[(size_t)b * kDecodeWinMax + j] = (s < 0 || dup[j]) ? -1 : s;
  }
}

template <int DT>
cudaError_t launch_scan(const CUtensorMap& mk, const CUtensorMap& mq, const CUtensorMap& mks, const RowDesc* prox,
                        const int* tile_prefix, int B, int Lmax, float* scores, uint32_t* ghist, int* status,
                        int sms, cudaStream_t st) {
  auto kern = decode_scan_kernel<DT>;
  static bool attr_set[kMaxDevices] = {};
  const size_t smem = dsmem_bytes<DT>();
  if (cudaError_t e = opt_in_dynamic_smem(kern, smem, attr_set); e != cudaSuccess) return e;
  ++launch_counter();
  return launch_kernel(kern, dim3(sms), dim3(D_THREADS), smem, st, true, mk, mq, mks, prox, tile_prefix, B, Lmax, scores,
                       ghist, status);
}

}  // namespace

bool make_operand_map(CUtensorMap* m, const void* base, long long rows, int dtype, int box_rows, int row_stride);
bool make_scale_map(CUtensorMap* m, const float* base, long long n, int box);

size_t decode_fast_bytes(int B, int Lmax, int g, int c) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const int mc = group_chunks(g);
  const int ncc = (c + kDecodeCandChunk - 1) / kDecodeCandChunk;
  const size_t Ls = ((size_t)Lmax + 3) & ~(size_t)3;     // score rows start on 16-byte boundaries
  return up(B * Ls * 4) + up((size_t)B * DHIST * 4) + up((size_t)(B + 1) * 4) +
         up((size_t)B * mc * (ncc + 1) * sizeof(GroupDesc)) + up((size_t)B * g * sizeof(EntryList)) +
         up((size_t)B * kDecodeWinMax * 4) + up((size_t)B * g * (c + kDecodeWinMax) * 8);
}

cudaError_t launch_merge_topk(const float* scores, const int32_t* idx, int n_seg, int seg_len, const int32_t* seg_offset,
                              unsigned long long* entries, int K, int32_t* out_idx, float* out_scores, cudaStream_t st) {
  merge_topk_kernel<<<1, kBlk, 0, st>>>(scores, idx, n_seg, seg_len, seg_offset, entries, K, out_idx, out_scores);
  ++launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_decode_fast(const DecodeFast& d, cudaStream_t st) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  char* p = (char*)d.scratch;
  const int Ls = (d.Lmax + 3) & ~3;
  float* scores = (float*)p;                 p += up((size_t)d.B * Ls * 4);
  uint32_t* ghist = (uint32_t*)p;            p += up((size_t)d.B * DHIST * 4);
  int* tile_prefix = (int*)p;                p += up((size_t)(d.B + 1) * 4);
  const int mc = group_chunks(d.g);
  // Candidates per re-score work item: as few items as keep every SM busy in ONE wave (each item pays
  // for its own query load and pipeline ramp), never below kDecodeCandChunk, whole 128-key tiles.
  int chunk = kDecodeCandChunk;
  {
    const int per_group = d.sms / (d.B * mc) > 0 ? d.sms / (d.B * mc) : 1;
    const int want = ((d.c + per_group - 1) / per_group + TILE_KEYS - 1) / TILE_KEYS * TILE_KEYS;
    if (want > chunk) chunk = want;
  }
  const int ncc = (d.c + chunk - 1) / chunk;
  const int W = d.mode == 1 ? d.W : 0;
  const int nch = ncc + (W > 0 ? 1 : 0);
  GroupDesc* chunks = (GroupDesc*)p;         p += up((size_t)d.B * mc * (ncc + 1) * sizeof(GroupDesc));
  EntryList* lists = (EntryList*)p;          p += up((size_t)d.B * d.g * sizeof(EntryList));
  int32_t* wcand = (int32_t*)p;              p += up((size_t)d.B * kDecodeWinMax * 4);
  unsigned long long* entries = (unsigned long long*)p;

  decode_prepare_kernel<<<d.B, 1024, 0, st>>>(d.plan, d.prox, d.groups, ghist, W, d.pool, chunk, tile_prefix, chunks, lists,
                                              entries, wcand);
  ++launch_counter();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  CUtensorMap mk, mq, mks;
  memset(&mks, 0, sizeof(mks));
  if (d.dtype == DT_FP8 && !make_scale_map(&mks, d.kscale, d.k_rows, TILE_KEYS)) return cudaErrorInvalidValue;
  if (!make_operand_map(&mk, d.kc, d.k_rows, d.dtype, TILE_KEYS, d.k_stride) ||
      !make_operand_map(&mq, d.proxy_q, (long long)d.B * kHeads, d.dtype, kHeads, 0))
    return cudaErrorInvalidValue;
  if (d.skip_scan) {
    if (d.mode != 1) return cudaErrorInvalidValue;
  } else {
  if (d.ev_scan_begin) cudaEventRecord(d.ev_scan_begin, st);
  e = d.dtype == DT_FP8
          ? launch_scan<DT_FP8>(mk, mq, mks, d.prox, tile_prefix, d.B, Ls, scores, ghist, d.status, d.sms, st)
          : launch_scan<DT_BF16>(mk, mq, mks, d.prox, tile_prefix, d.B, Ls, scores, ghist, d.status, d.sms, st);
  if (e != cudaSuccess) return e;
  if (d.ev_scan_end) cudaEventRecord(d.ev_scan_end, st);
  static bool sel_attr[kMaxDevices] = {};
  const size_t sel_smem = sizeof(SelSmem) + 16;
  if ((e = opt_in_dynamic_smem(decode_select_kernel, sel_smem, sel_attr)) != cudaSuccess) return e;
  if ((e = launch_kernel(decode_select_kernel, dim3(SEL_SPLIT, d.B), dim3(kBlk), sel_smem, st, true, (const RowDesc*)d.prox,
                         Ls, (const float*)scores, (const uint32_t*)ghist, d.status)) != cudaSuccess)
    return e;
  ++launch_counter();
  if (d.ev_scan_end && d.ev_select_end) cudaEventRecord(d.ev_select_end, st);
  }
  if (d.mode == 1) {
    if (W > 0) {
      if ((e = launch_kernel(decode_window_kernel, dim3(d.B), dim3(1024), 0, st, true, (const GroupDesc*)d.groups, mc, d.g,
                             W, wcand)) != cudaSuccess)
        return e;
      ++launch_counter();
    }
    ScanScratch sc = d.scratch_tc;
    e = launch_refine_tc(d.q, d.B * d.g, d.dtype, chunks, d.B * mc * nch, sc, d.sms, st, false, true, 0, true);
    if (e != cudaSuccess) return e;
    if ((e = launch_kernel(entries_topk_kernel, dim3(d.B * d.g), dim3(kBlk), 0, st, true, (const EntryList*)lists)) !=
        cudaSuccess)
      return e;
    ++launch_counter();
  }
  return cudaGetLastError();
}

}  // namespace pivot
