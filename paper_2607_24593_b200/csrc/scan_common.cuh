// Parts of the shared-scan kernel (scan_tc.cu): the order in which a CTA takes its row blocks,
// and the streaming select behind the scan (Eq. 6 / Eq. 7) -- survivor queues between the warps
// that produce scores and one append warp per row, the row histogram that keeps the running
// threshold, the row's candidate segment, and the final exact selection, which finisher warps
// take one block behind the scan (a row has two segments, used by alternate blocks).
#pragma once
#include "kernels.h"
#include "ptx.cuh"
#include "segselect.cuh"

namespace pivot {
namespace scan {

constexpr int TILE_KEYS = 128;
constexpr int KS_SLOTS = 8;       // key-scale ring: deeper than (key stages + accumulator buffers)
#ifndef PIVOT_CHK
#define PIVOT_CHK 32
#endif
constexpr int kThresholdRefreshTiles = PIVOT_CHK;
#ifndef PIVOT_COMPACT_EVERY
#define PIVOT_COMPACT_EVERY 0
#endif
constexpr int kCompactEveryTiles = PIVOT_COMPACT_EVERY;   // a multiple of the refresh interval, or 0 = never   // the append warp re-reads its row's threshold off the histogram this often

// Block sequence of one CTA: blocks sorted longest-first are dealt in snake order.
struct BlockIter {
  int n_blocks, G, cta, round;
  __device__ BlockIter(int nb, int g, int c) : n_blocks(nb), G(g), cta(c), round(0) {}
  __device__ int next() {   // block index, or -1
    const int pos = (round & 1) ? (G - 1 - cta) : cta;
    const long long d = (long long)round * G + pos;
    ++round;
    if (d >= n_blocks) return -1;
    return n_blocks - 1 - (int)d;
  }
};

// Key tiles a block of nrows_blk consecutive scan rows needs (its longest live row), and the
// first key-tensor row of the block's sequence.
__device__ __forceinline__ int block_tiles(const RowDesc* rows, int n_rows, int b, int nrows_blk, int* k_row0,
                                           int* nv_max = nullptr) {
  int mx = 0;
  for (int r = 0; r < nrows_blk; ++r) {
    const int ri = b * nrows_blk + r;
    if (ri < n_rows) {
      const int K = rows[ri].K;
      const int nv = rows[ri].n_vis;
      if (K > 0 && nv > mx) mx = nv;
      if (r == 0) *k_row0 = rows[ri].k_row0;
    }
  }
  if (nv_max) *nv_max = mx;
  return (mx + TILE_KEYS - 1) / TILE_KEYS;
}

// Shared-memory state of the streaming select of a block of NROWS rows.
template <int NROWS, int QD>
struct SelectCtrl {
  uint32_t rhist[NROWS][kSelBins];      // per row: histogram of every score appended so far
  uint64_t sc_full[QD], sc_empty[QD];   // survivor queues: score warps -> append warps
  alignas(16) unsigned long long q[QD][NROWS][4][32];   // [tile % QD][row][lane quarter]: packed entries
  alignas(16) uint32_t qn[QD][NROWS][4];                // their counts
  // published append threshold of each row, (block sequence number << 32) | key: only grows
  // within a block; a reader that is already in the next block sees a stale tag and takes 0
  volatile unsigned long long thr[NROWS];
  // End of a block: what the row's finisher needs (the append warp moves on to the next block
  // and the row's other segment at once).  Two slots, used by alternate blocks like the segments.
  struct FinRow {
    int cnt;                            // entries held in the row's segment
    int base;                           // the row histogram's anchor
    int bsel;                           // boundary bin of the exact histogram, -1 = everything is wanted
    uint32_t need_b, pop;               // entries wanted from that bin, and its population
  } fin[NROWS][2];
  uint64_t fin_full[NROWS][2], fin_done[NROWS][2];   // append warp -> finisher -> append warp
  int abort_code;                       // device status to report besides a timed-out wait
  SegSelSmem sel[NROWS];                // the row's append warp (segment overflow) or its finisher
};

// The threshold the score warps of block sequence number `seq` compare row r's scores with.
template <int NROWS, int QD>
__device__ __forceinline__ uint32_t row_threshold(const SelectCtrl<NROWS, QD>& s, int r, uint32_t seq) {
  const unsigned long long t = s.thr[r];
  return (uint32_t)(t >> 32) == seq ? (uint32_t)t : 0u;
}

// Row r's segment for the block with sequence number seq.
template <int NROWS>
__device__ __forceinline__ entry_t* row_segment(const ScanScratch& sc, int r, uint32_t seq) {
  return sc.cand64 + (((size_t)blockIdx.x * NROWS + r) * 2 + (seq & 1u)) * sc.cap;
}

// A score warp leaves the survivors of its 32 keys of row r in the tile's queue: compacted by one
// vote, count beside them.  `take` must already include the causal cut and the threshold test.
template <int NROWS, int QD>
__device__ __forceinline__ void push_survivors(SelectCtrl<NROWS, QD>& s, int qb, int r, int lq, int lane, bool take,
                                               uint32_t key, int s_key) {
  const uint32_t m = __ballot_sync(0xffffffffu, take);
  if (take) s.q[qb][r][lq][__popc(m & ((1u << lane) - 1u))] = make_entry(key, s_key);
  if (lane == 0) s.qn[qb][r][lq] = (uint32_t)__popc(m);
}

// Score key -> histogram bin: 256 bins per octave (8 mantissa bits), 2048 bins anchored two
// octaves above the row's first-tile maximum; keys outside land in the end bins.
__device__ __forceinline__ int select_bin(uint32_t key, int base) {
  const int b = (int)(key >> 15) - base;
  return b < 0 ? 0 : (b > kSelBins - 1 ? kSelBins - 1 : b);
}

// The append warp of row r (one warp, all blocks of this CTA): counts the survivors of every tile
// in the row histogram, moves them to the row's segment in the L2-resident scratch and keeps the
// row's threshold fresh -- alone, without barriers.  At the end of a block it reads the boundary
// bin off the (then exact) histogram, hands the segment to the row's finisher and goes on with
// the next block in the row's other segment.
template <int NROWS, int QD>
__device__ __noinline__ void append_role(SelectCtrl<NROWS, QD>& s, int r, int lane, const Team& tm,
                                            const RowDesc* __restrict__ rows, int n_rows, int n_blocks,
                                            const ScanScratch& sc, volatile int* abort_flag) {
  SegSelSmem& sel = s.sel[r];
  const int CAP = sc.cap;                        // entries of this row's candidate segment
  uint32_t* const rhist = s.rhist[r];
  // Lower bound on the K-th best score seen so far, read off the row histogram: the largest
  // bin edge with at least K scores at or above it.  Returned as a key threshold t such that
  // only keys > t can still belong to the top K.
  auto hist_threshold = [&](int K, int base) -> uint32_t {
    uint32_t b, need_in, pop;
    if (!warp_hist_boundary<2>(rhist, (uint32_t)K, lane, &b, &need_in, &pop)) return 0u;
    return b > 0 ? (((uint32_t)((int)b + base)) << 15) - 1u : 0u;
  };
  // The threshold is refreshed every CHK tiles; a tile adds at most TILE_KEYS entries, so a
  // segment checked then always has room until the next check.
  const int CHK = CAP / (2 * TILE_KEYS) < kThresholdRefreshTiles ? (CAP / (2 * TILE_KEYS) > 0 ? CAP / (2 * TILE_KEYS) : 1) : kThresholdRefreshTiles;
  const int headroom = TILE_KEYS * CHK;
  BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
  uint32_t it = 0, seq = 0;
  for (int b = bi.next(); b >= 0; b = bi.next()) {
    int k_row0 = 0;
    const int ntiles = block_tiles(rows, n_rows, b, NROWS, &k_row0);
    if (ntiles == 0) continue;
    const int ri = b * NROWS + r;
    const bool live = ri < n_rows && rows[ri].K > 0;
    const int K = live ? rows[ri].K : 0;
    int cnt = 0, base = 0;
    uint32_t thr = 0;
    for (int i = lane; i < kSelBins; i += 32) rhist[i] = 0;
    if (lane == 0) s.thr[r] = (unsigned long long)seq << 32;
    // this block's segment was the block's before last: its finisher must be through with it
    const int fb = seq & 1;
    (void)ptx::mbar_wait(&s.fin_done[r][fb], ((seq >> 1) & 1) ^ 1, abort_flag, 64);
    entry_t* const seg = row_segment<NROWS>(sc, r, seq);
    bool sel_mine = seq == 0;                    // the finisher of the previous block may still use `sel`
    __syncwarp();
    for (int t = 0; t < ntiles; ++t, ++it) {
      if (K > 0 && t > 0 && (t % CHK) == 0) {
        const uint32_t th = hist_threshold(K, base);
        thr = th > thr ? th : thr;
        // Housekeeping while this warp has slack: every kCompactEveryTiles tiles the entries that fell
        // below the threshold leave the segment, so that the final selection at the end of the block
        // (which stalls the whole pipeline) reads a segment of about K entries instead of
        // K (1 + ln(n / K)).  They lie below every bin the final boundary can be in, so the histogram
        // stays exact for what the selection looks at.
        const bool tidy = kCompactEveryTiles > 0 && (t % kCompactEveryTiles) == 0 && cnt > K + K / 2;
        if (cnt + headroom > CAP || tidy) {
          // (nearly full: the same filter; if that is not enough -- ties, adversarial order -- compact
          // exactly to the K best)
          const uint32_t tcur = thr;
          cnt = seg_filter_inplace(seg, cnt, lane, [tcur](entry_t x) { return entry_key(x) > tcur; });
          if (cnt + headroom > CAP && cnt > K) {
            if (!sel_mine) {                     // (rare path: waiting here costs nothing that matters)
              (void)ptx::mbar_wait(&s.fin_done[r][fb ^ 1], ((seq - 1) >> 1) & 1, abort_flag, 64);
              sel_mine = true;
            }
            entry_t cut;
            cnt = seg_compact<false>(tm, sel, Seg{seg, cnt}, K, &cut);
            thr = entry_key(cut) > thr ? entry_key(cut) : thr;
          }
        }
        if (lane == 0) s.thr[r] = ((unsigned long long)seq << 32) | thr;
      }
      const int sb = it % QD;
      (void)ptx::mbar_wait(&s.sc_full[sb], (it / QD) & 1, abort_flag);
      const uint4 n4 = *reinterpret_cast<const uint4*>(&s.qn[sb][r][0]);
      const uint32_t nq[4] = {n4.x, n4.y, n4.z, n4.w};
      entry_t e[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) e[j] = (uint32_t)lane < nq[j] ? s.q[sb][r][j][lane] : kPadEntry;
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&s.sc_empty[sb]);
      if (K <= 0) continue;                    // a dead row still takes part in the handshake
      if (t == 0) {          // anchor the histogram range on the first tile's maximum
        uint32_t mx = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) mx = entry_key(e[j]) > mx ? entry_key(e[j]) : mx;
        mx = __reduce_max_sync(0xffffffffu, mx);
        const int top = (int)(mx >> 15) + 512 - (kSelBins - 1);
        base = top > 0 ? top : 0;
      }
      // Every entry that reaches the segment is counted: the ones the score warps dropped were
      // at or below a valid threshold and can never reach a bin edge the threshold could still
      // move to, so the counts that matter stay exact.
      int p = cnt + lane;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if ((uint32_t)lane < nq[j]) {
          atomicAdd(&rhist[select_bin(entry_key(e[j]), base)], 1u);
          if (p < CAP) seg[p] = e[j];
          else s.abort_code = DEV_CAND_OVERFLOW;
        }
        p += (int)nq[j];
      }
      cnt = min(cnt + (int)(nq[0] + nq[1] + nq[2] + nq[3]), CAP);
    }
    // ---- end of the block: the histogram is exact for everything the segment still holds; read
    //      the boundary bin off it and hand the row to its finisher
    uint32_t bb = 0, need_b = 0, pop = 0;
    const bool found = K > 0 && warp_hist_boundary<0>(rhist, (uint32_t)K, lane, &bb, &need_b, &pop);
    if (lane == 0) {
      typename SelectCtrl<NROWS, QD>::FinRow& f = s.fin[r][fb];
      f.cnt = cnt; f.base = base; f.bsel = found ? (int)bb : -1; f.need_b = need_b; f.pop = pop;
    }
    __threadfence_block();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&s.fin_full[r][fb]);
    ++seq;
  }
}

// A finisher warp: the final exact selection of rows r0 .. r0 + nr - 1 of every block of this CTA,
// one block behind the scan.  The append warp has counted every entry the segment holds, so its
// boundary bin is exact and one sweep over the segment suffices (a boundary bin too crowded to
// rank takes the general way).  Pads the row with -1 and copies it to the other members of a
// Reuse group.
template <int NROWS, int QD>
__device__ __noinline__ void finisher_role(SelectCtrl<NROWS, QD>& s, int r0, int nr, int lane,
                                              const RowDesc* __restrict__ rows, int n_rows, int n_blocks,
                                              const ScanScratch& sc, volatile int* abort_flag) {
  BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
  uint32_t seq = 0;
  for (int b = bi.next(); b >= 0; b = bi.next()) {
    int k_row0 = 0;
    if (block_tiles(rows, n_rows, b, NROWS, &k_row0) == 0) continue;
    const int fb = seq & 1;
    for (int r = r0; r < r0 + nr; ++r) {
      if (!ptx::mbar_wait(&s.fin_full[r][fb], (seq >> 1) & 1, abort_flag, 64)) return;
      const int ri = b * NROWS + r;
      const int K = (ri < n_rows) ? rows[ri].K : 0;
      if (K > 0) {
        const RowDesc rd = rows[ri];
        const typename SelectCtrl<NROWS, QD>::FinRow f = s.fin[r][fb];
        const int rbase = f.base;
        auto key_bin = [rbase](uint32_t key) { return select_bin(key, rbase); };
        const int n_valid = warp_seg_topk_binned(s.sel[r], row_segment<NROWS>(sc, r, seq), f.cnt, key_bin, f.bsel,
                                                 f.need_b, f.pop, rd.out, rd.out_score, K, lane);
        for (int i = n_valid + lane; i < K; i += 32) {
          rd.out[i] = -1;
          if (rd.out_score) rd.out_score[i] = -INFINITY;
        }
        __syncwarp();
        for (int rr = 1; rr < rd.out_rows; ++rr)
          for (int i = lane; i < K; i += 32) {
            rd.out[(size_t)rr * rd.out_stride + i] = rd.out[i];
            if (rd.out_score) rd.out_score[(size_t)rr * rd.out_stride + i] = rd.out_score[i];
          }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&s.fin_done[r][fb]);
    }
    ++seq;
  }
}

}  // namespace scan
}  // namespace pivot
