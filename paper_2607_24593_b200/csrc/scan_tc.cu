// Kernels 2+3: shared prefix scan on tcgen05 tensor cores with the streaming top-K select
// fused behind it, so the (rows x keys) score matrix never reaches HBM.
//
// Eq. 5 / Eq. 1 as a dense contraction: a tile is 128 keys (MMA M, one key per TMEM lane) by
// NROWS x 64 heads (MMA N) by d = 128 (MMA K).  Keys stream through a TMA-fed shared-memory
// ring; the query block (NROWS rows = NROWS consecutive proxies or queries) sits in shared
// memory for the whole scan of its prefix.  The accumulator lives in TMEM, double-buffered:
// while the tensor core fills one buffer, the epilogue warps drain the other -- each thread owns
// one key, applies ReLU, the gate-weighted head sum, the key scale (Appendix A) and the causal
// cut, and feeds the score to the row's streaming select (filter by the running K-th-best
// threshold, append to an L2-resident candidate buffer, exact radix compaction when it fills).
//
// One persistent CTA per SM; warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, then the
// SCORE warps (two per TMEM lane quarter, each computing two rows of a tile), then one APPEND
// warp per row.  A score warp compares its 32 scores of a row with the row's published
// threshold and leaves the survivors, compacted, in a small double-buffered shared-memory
// queue; the row's append warp counts them in the row histogram, moves them to the row's
// candidate segment (L2-resident scratch) and keeps the threshold fresh -- alone, without
// barriers.  Splitting the epilogue this way puts more warps on every scheduler within the
// register file (the score warps carry no select state) and takes the histogram atomics, the
// global stores and the threshold refresh off the warps that feed the tensor core.  At the end
// of a block the append warp hands its row's segment to a FINISHER warp (one per two rows), which
// takes the final exact select while the other warps are already scanning the next block (a row
// has two segments, used by alternate blocks).  Row blocks are dealt to CTAs longest-first in
// snake order.
//
// FP8 with four rows per block (the prefill configuration) takes the gate-weighted head sum of
// Eq. 5 on the tensor core as well: it is the contraction ReLU(X) [128 keys x 256] . W^T with a
// block-diagonal gate matrix W [16 x 256].  The eight score warps then split into four ReLU
// warps, which turn the fp32 accumulator into packed bf16 ReLU values in place in tensor memory,
// and four compact warps, which read the row scores the second MMA (A operand in tensor memory,
// W in shared memory) leaves in 16 columns of the same buffer.  The fp32 FMA head sum remains for
// bf16 operands, one-row blocks and on request.
#include <cuda.h>
#include <string.h>

#include "kernels.h"
#include "ptx.cuh"
#include "scan_common.cuh"
#include "segselect.cuh"

namespace pivot {
namespace {

using scan::TILE_KEYS;
using scan::KS_SLOTS;
using scan::BlockIter;
using scan::block_tiles;
constexpr int MAX_STAGES = 8;
constexpr int QDEPTH = 4;         // survivor-queue buffers between the score warps and the append warps

// EPI: 1 = the gate-weighted head sum runs on the tensor core where the configuration allows it
// (FP8, four rows); 0 = fp32 FMA epilogue everywhere.
template <int DT, int NROWS, int EPI = 1>
struct Cfg {
  static constexpr bool FP8 = DT == DT_FP8;
  static constexpr int ESZ = FP8 ? 1 : 2;
  static constexpr int KHALVES = FP8 ? 1 : 2;                 // 128-byte K slices per row
  static constexpr int HALF_TILE_BYTES = TILE_KEYS * 128;     // 16 KB: 128 keys x 128 B
  static constexpr int STAGE_BYTES = KHALVES * HALF_TILE_BYTES;
  static constexpr int QROW_HALF_BYTES = kHeads * 128;        // 8 KB: 64 heads x 128 B
  static constexpr int QHALF_BYTES = NROWS * QROW_HALF_BYTES;
  static constexpr int QBUF_BYTES = KHALVES * QHALF_BYTES;
  static constexpr int N = NROWS * kHeads;
  static constexpr int QBUFS = (!FP8 && NROWS == 4) ? 1 : 2;   // bf16 x 4 rows: 64 KB per query buffer
  static constexpr int STAGES = NROWS == 4 ? (FP8 ? 4 : 2) : (FP8 ? 6 : 4);
  // Eight score warps, two rows per 4-warp team (one team per row with sixteen warps leaves too
  // few registers per thread), and one select warp per row.
  static constexpr int EPI_WARPS = NROWS == 4 ? 8 : 4;
  static constexpr int ROWS_PER_TEAM = NROWS == 4 ? 2 : 1;
  static constexpr int TEAMS = EPI_WARPS / 4;
  static constexpr int SEL_WARPS = NROWS;                     // append warps, one per row
  static constexpr int FIN_WARPS = NROWS == 4 ? 2 : 1;        // finisher warps, one per two rows
  static constexpr int THREADS = 64 + (EPI_WARPS + SEL_WARPS + FIN_WARPS) * 32;
  static constexpr int TMEM_COLS = 2 * N < 32 ? 32 : 2 * N;
  // FP8, four rows: the gate-weighted head sum itself runs on the tensor core (see the kernel
  // header).  Other configurations keep the fp32 FMA epilogue.
  static constexpr bool MMA2 = FP8 && NROWS == 4 && EPI == 1;
  static constexpr int QD = MMA2 ? 2 : QDEPTH;                 // survivor-queue depth
  static constexpr int TMEM_EMPTY_ARRIVALS = MMA2 ? 4 : EPI_WARPS;
  static constexpr int SC_FULL_ARRIVALS = MMA2 ? 4 : EPI_WARPS;
  static constexpr uint32_t IDESC2 = ptx::make_idesc(1u, TILE_KEYS, 16);   // bf16 x bf16, N = 16
  static constexpr int KSTEPS = 4;                            // 32 bytes of K per MMA
  static constexpr uint32_t IDESC = ptx::make_idesc(FP8 ? 0u : 1u, TILE_KEYS, N);
};

template <int NROWS, bool MMA2>
struct Ctrl {
  static constexpr int QD = MMA2 ? 2 : QDEPTH;
  // MMA2: the block's gate matrix W [16 x 256] bf16, K-major with 128-byte swizzle (4 slabs of 64
  // columns, 16 rows x 128 B each): row r < 4 holds the bf16 head of row r's effective gates in
  // columns 64 r .. 64 r + 63, row 4 + r the bf16 remainder (so the gates enter with 16 mantissa
  // bits), everything else is zero.  B operand of the second MMA.
  alignas(1024) uint8_t wmat[MMA2 ? 8192 : 16];
  uint64_t a_ready[2], s_ready[2], w_ready;      // MMA2 handshakes (see the kernel)
  alignas(128) float ks[KS_SLOTS][TILE_KEYS];   // key scales of the tiles in flight (TMA destination)
  alignas(16) float w[4][kHeads];       // effective gates of the block's rows (read as float4)
  uint64_t full[MAX_STAGES], empty[MAX_STAGES];
  uint64_t q_full[2], q_empty[2], tmem_full[2], tmem_empty[2];
  uint64_t ks_full[KS_SLOTS];
  uint32_t tmem_base;
  int abort;
  scan::SelectCtrl<NROWS, QD> s;        // streaming select: queues, row histograms, thresholds
};

template <int DT, int NROWS, int EPI = 1>
constexpr size_t smem_bytes() {
  using C = Cfg<DT, NROWS, EPI>;
  return 1024 + C::QBUFS * C::QBUF_BYTES + C::STAGES * C::STAGE_BYTES + sizeof(Ctrl<NROWS, C::MMA2>);
}
static_assert(smem_bytes<DT_FP8, 4, 1>() <= 232448 && smem_bytes<DT_FP8, 4, 0>() <= 232448 &&
              smem_bytes<DT_BF16, 4>() <= 232448, "shared memory budget");

template <int DT, int NROWS, int EPI>
__global__ void __launch_bounds__(Cfg<DT, NROWS, EPI>::THREADS, 1)
scan_select_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q0,
                      const __grid_constant__ CUtensorMap tm_q1, const __grid_constant__ CUtensorMap tm_ks,
                      const RowDesc* __restrict__ rows, int n_rows, ScanScratch sc) {
  using C = Cfg<DT, NROWS, EPI>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* qbuf = smem;                                   // QBUFS x QBUF_BYTES
  uint8_t* kring = smem + C::QBUFS * C::QBUF_BYTES;       // STAGES x STAGE_BYTES
  using CtrlT = Ctrl<NROWS, C::MMA2>;
  CtrlT& ct = *reinterpret_cast<CtrlT*>(kring + C::STAGES * C::STAGE_BYTES);
  constexpr int QD = C::QD;
  volatile int* abort_flag = &ct.abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_blocks = (n_rows + NROWS - 1) / NROWS;

  // A small launch whose rows are all dead (decode: no guarded sequence in the batch) leaves
  // before any barrier or TMEM is set up.
  if (n_rows <= (int)blockDim.x) {
    const bool live = (int)threadIdx.x < n_rows && rows[threadIdx.x].K > 0 && rows[threadIdx.x].n_vis > 0;
    if (!__syncthreads_or(live)) return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { ptx::mbar_init(&ct.full[s], 1); ptx::mbar_init(&ct.empty[s], 1); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ct.q_full[i], 1);
      ptx::mbar_init(&ct.q_empty[i], 1);
      ptx::mbar_init(&ct.tmem_full[i], 1);
      ptx::mbar_init(&ct.tmem_empty[i], C::TMEM_EMPTY_ARRIVALS);
      ptx::mbar_init(&ct.a_ready[i], 4);
      ptx::mbar_init(&ct.s_ready[i], 1);
    }
    ptx::mbar_init(&ct.w_ready, 1);
    for (int i = 0; i < KS_SLOTS; ++i) ptx::mbar_init(&ct.ks_full[i], 1);
    for (int i = 0; i < QD; ++i) {
      ptx::mbar_init(&ct.s.sc_full[i], C::SC_FULL_ARRIVALS);
      ptx::mbar_init(&ct.s.sc_empty[i], C::SEL_WARPS);
    }
    ct.abort = 0;
    ct.s.abort_code = 0;
    for (int r = 0; r < NROWS; ++r) {
      ct.s.thr[r] = 0ull;
      for (int i = 0; i < 2; ++i) { ptx::mbar_init(&ct.s.fin_full[r][i], 1); ptx::mbar_init(&ct.s.fin_done[r][i], 1); }
    }
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&ct.tmem_base, C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  if constexpr (C::MMA2)        // off-diagonal blocks and rows 4..15 of the gate matrix stay zero
    for (int i = threadIdx.x; i < 8192 / 16; i += blockDim.x) reinterpret_cast<uint4*>(ct.wmat)[i] = make_uint4(0, 0, 0, 0);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = ct.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      ptx::prefetch_tensormap(&tm_k);
      ptx::prefetch_tensormap(&tm_q0);
      ptx::prefetch_tensormap(&tm_q1);
      if (C::FP8) ptx::prefetch_tensormap(&tm_ks);
      BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
      uint32_t it = 0, blk = 0;
      bool ok = true;
      for (int b = bi.next(); b >= 0 && ok; b = bi.next()) {
        int k_row0 = 0;
        const int ntiles = block_tiles(rows, n_rows, b, NROWS, &k_row0);
        if (ntiles == 0) continue;
        const int qb = blk % C::QBUFS;
        ok = ptx::mbar_wait(&ct.q_empty[qb], ((blk / C::QBUFS) & 1) ^ 1, abort_flag, 64);
        if (!ok) break;
        int present = 0;
        for (int r = 0; r < NROWS; ++r) present += (b * NROWS + r < n_rows) ? 1 : 0;
        ptx::mbar_arrive_expect_tx(&ct.q_full[qb], present * C::KHALVES * C::QROW_HALF_BYTES);
        for (int r = 0; r < NROWS; ++r) {
          const int ri = b * NROWS + r;
          if (ri >= n_rows) continue;
          const CUtensorMap* tm = rows[ri].q_map ? &tm_q1 : &tm_q0;
          const int y = rows[ri].q_row * kHeads;
          for (int h = 0; h < C::KHALVES; ++h)
            ptx::tma_load_2d(qbuf + qb * C::QBUF_BYTES + h * C::QHALF_BYTES + r * C::QROW_HALF_BYTES, tm,
                             h * 64, y, &ct.q_full[qb]);
        }
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int s = it % C::STAGES;
          const uint32_t ph = (it / C::STAGES) & 1;
          ok = ptx::mbar_wait(&ct.empty[s], ph ^ 1, abort_flag, 64);
          if (!ok) break;
          ptx::mbar_arrive_expect_tx(&ct.full[s], C::STAGE_BYTES);
          for (int h = 0; h < C::KHALVES; ++h)
            ptx::tma_load_2d(kring + s * C::STAGE_BYTES + h * C::HALF_TILE_BYTES, &tm_k, h * 64,
                             k_row0 + t * TILE_KEYS, &ct.full[s]);
          if (C::FP8) {
            // The tile's key scales ride along into their own ring.  A slot is free again
            // by construction: this thread runs at most STAGES tiles ahead of the MMA and the
            // MMA at most two ahead of the epilogue, fewer than KS_SLOTS in total.
            const int ksl = it % KS_SLOTS;
            ptx::mbar_arrive_expect_tx(&ct.ks_full[ksl], TILE_KEYS * 4);
            ptx::tma_load_1d(&ct.ks[ksl][0], &tm_ks, k_row0 + t * TILE_KEYS, &ct.ks_full[ksl]);
          }
        }
        ++blk;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
      BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
      uint32_t it = 0, blk = 0;
      bool ok = true;
      // MMA2: the gate-weighted head sum of tile it-1, S[128 keys x 16] = ReLU(X)[128 x 256] . W^T,
      // is issued right after the first MMA of tile it (its operand -- the accumulator turned into
      // bf16 ReLU values in place -- is produced while that MMA runs).
      bool pend = false;
      uint32_t pend_it = 0, pend_blk = 0, w_blk = 0xffffffffu;
      // (a -DPIVOT_PROF build times this thread's waits: PW(slot, wait) adds the wait's clocks to pw[slot])
      PIVOT_PROF_DO(long long pw[6] = {0, 0, 0, 0, 0, 0}; const long long pstart = clock64();)
#ifdef PIVOT_PROF
#define PW(i, ...) { const long long t_ = clock64(); __VA_ARGS__; pw[i] += clock64() - t_; }
#else
#define PW(i, ...) __VA_ARGS__;
#endif
      auto issue_mma2 = [&]() -> bool {
        if (pend_blk != w_blk) {                 // first tile of a block: its gate matrix must be in place
          bool okw;
          PW(3, okw = ptx::mbar_wait(&ct.w_ready, pend_blk & 1, abort_flag, 32))
          if (!okw) return false;
          w_blk = pend_blk;
        }
        const int pb = pend_it & 1;
        bool oka;
        PW(4, oka = ptx::mbar_wait(&ct.a_ready[pb], (pend_it >> 1) & 1, abort_flag, 32))
        if (!oka) return false;
        ptx::tc_fence_after();
        const uint32_t w_addr = ptx::smem_u32(ct.wmat);
        const uint32_t a_tmem = tmem_base + pb * C::N;
#pragma unroll
        for (int ks = 0; ks < 16; ++ks)          // 16 bf16 of K per step: 8 TMEM columns, 32 bytes of W
          ptx::tc_mma_a_tmem_bf16(a_tmem + 128, a_tmem + ks * 8,
                                  ptx::smem_desc_sw128(w_addr + (ks >> 2) * 2048 + (ks & 3) * 32), C::IDESC2,
                                  ks ? 1u : 0u);
        ptx::tc_commit(&ct.s_ready[pb]);
        return true;
      };
      for (int b = bi.next(); b >= 0 && ok; b = bi.next()) {
        int k_row0 = 0;
        const int ntiles = block_tiles(rows, n_rows, b, NROWS, &k_row0);
        if (ntiles == 0) continue;
        const int qb = blk % C::QBUFS;
        PW(0, ok = ptx::mbar_wait(&ct.q_full[qb], (blk / C::QBUFS) & 1, abort_flag, 32))
        if (!ok) break;
        const uint32_t q_addr = ptx::smem_u32(qbuf + qb * C::QBUF_BYTES);
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int s = it % C::STAGES;
          const uint32_t ph = (it / C::STAGES) & 1;
          const int buf = it & 1;
          PW(1, ok = ptx::mbar_wait(&ct.tmem_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, 32))
          if (!ok) break;
          PW(2, ok = ptx::mbar_wait(&ct.full[s], ph, abort_flag, 32))
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t k_addr = ptx::smem_u32(kring + s * C::STAGE_BYTES);
          const uint32_t d_tmem = tmem_base + buf * C::N;
#pragma unroll
          for (int h = 0; h < C::KHALVES; ++h)
#pragma unroll
            for (int ks = 0; ks < C::KSTEPS; ++ks) {
              const uint64_t a = ptx::smem_desc_sw128(k_addr + h * C::HALF_TILE_BYTES + ks * 32);
              const uint64_t bq = ptx::smem_desc_sw128(q_addr + h * C::QHALF_BYTES + ks * 32);
              ptx::tc_mma<C::FP8>(d_tmem, a, bq, C::IDESC, (h | ks) ? 1u : 0u);
            }
          ptx::tc_commit(&ct.empty[s]);       // key stage free once these MMAs are done
          ptx::tc_commit(&ct.tmem_full[buf]); // accumulator ready
          if constexpr (C::MMA2) {
            if (pend) { ok = issue_mma2(); if (!ok) break; }
            pend = true; pend_it = it; pend_blk = blk;
          }
        }
        ptx::tc_commit(&ct.q_empty[qb]);
        ++blk;
      }
      if constexpr (C::MMA2) {
        if (pend && ok) (void)issue_mma2();
      }
#undef PW
      PIVOT_PROF_DO(if (C::MMA2) {
        pw[5] = clock64() - pstart;
        for (int i = 0; i < 6; ++i) prof_add(sc.status, PROF_SCAN_WAIT_QUERIES + i, pw[i]);
        prof_add(sc.status, PROF_SCAN_TILES, it);
      })
    }
  } else if (warp < 2 + C::EPI_WARPS) {
    // ------------------------------------------------------------------ score warps
    const int ew = warp - 2;                       // 0 .. EPI_WARPS-1
    const int team = ew >> 2;                      // which pair of rows
    const int wq = ew & 3;
    const int lq = warp & 3;                       // TMEM lane quarter this warp may read
    const int key_in_tile = lq * 32 + lane;
    const int tt = wq * 32 + lane;                 // rank inside the team (0..127)
    const Team tm{tt, 128, 1 + team};
    BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
    uint32_t it = 0, seq = 0xffffffffu;            // seq: this block's sequence number in the CTA
    // A failed wait never changes this role's control flow (the team barriers below must stay
    // matched); once the abort flag is up every later wait returns at once.
    for (int b = bi.next(); b >= 0; b = bi.next()) {
      int k_row0 = 0;
      const int ntiles = block_tiles(rows, n_rows, b, NROWS, &k_row0);
      if (ntiles == 0) continue;
      ++seq;
      // ---- effective gates of this team's rows
      tm.sync();
      if constexpr (C::MMA2) {
        // team 1 (the compact warps) writes the four diagonal blocks of the gate matrix; the last
        // second MMA of the previous block is through (its scores have been read)
        if (team == 1) {
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int i = tt + u * 128, r = i >> 6, j = i & 63;
            const int ri = b * NROWS + r;
            float wv = 0.f;
            if (ri < n_rows && rows[ri].K > 0) {
              wv = rows[ri].w[j];
              if (rows[ri].qscale) wv = __fmul_rn(wv, rows[ri].qscale[j]);
            }
            // gate = hi + lo in bf16: matrix rows r and 4 + r (both inside slab r, the row's 64 columns)
            const __nv_bfloat16 hi = __float2bfloat16_rn(wv);
            const __nv_bfloat16 lo = __float2bfloat16_rn(wv - __bfloat162float(hi));
            const uint32_t in_row = (j & 7) * 2;
            *reinterpret_cast<__nv_bfloat16*>(ct.wmat + r * 2048 + r * 128 + (((j >> 3) ^ (r & 7)) << 4) + in_row) = hi;
            *reinterpret_cast<__nv_bfloat16*>(ct.wmat + r * 2048 + (4 + r) * 128 + (((j >> 3) ^ ((4 + r) & 7)) << 4) + in_row) = lo;
          }
          ptx::fence_proxy_async_smem();         // generic-proxy writes -> tensor-core reads
          tm.sync();
          if (tt == 0) ptx::mbar_arrive(&ct.w_ready);
        }
      } else {
        const int rl = tt >> 6, j = tt & 63;
        if (rl < C::ROWS_PER_TEAM) {
          const int r = team * C::ROWS_PER_TEAM + rl;
          const int ri = b * NROWS + r;
          float wv = 0.f;
          if (ri < n_rows && rows[ri].K > 0) {
            wv = rows[ri].w[j];
            if (rows[ri].qscale) wv = __fmul_rn(wv, rows[ri].qscale[j]);
          }
          ct.w[r][j] = 0.5f * wv;       // halved: see the ReLU identity below
        }
      }
      int n_vis[C::ROWS_PER_TEAM];
#pragma unroll
      for (int rl = 0; rl < C::ROWS_PER_TEAM; ++rl) {
        const int ri = b * NROWS + team * C::ROWS_PER_TEAM + rl;
        const bool live = ri < n_rows && rows[ri].K > 0;
        n_vis[rl] = live ? rows[ri].n_vis : 0;
      }
      tm.sync();
      if constexpr (C::MMA2) {
        if (team == 0) {
          // ---- ReLU warps: turn the fp32 accumulator into bf16 ReLU values in place.  Thread =
          // key (TMEM lane); 32 columns at a time come in, 16 packed columns go back to the start
          // of the buffer (writes trail the reads: column 16 c + 16 <= 32 c + 32).
          // Rows missing from a partial block have no queries in shared memory: whatever the first
          // MMA made of the stale bytes there (possibly NaN) must not reach the second one, whose
          // sums run over all 256 columns -- those columns are written as zeros.
          const int present = n_rows - b * NROWS;
          for (int t = 0; t < ntiles; ++t, ++it) {
            const int buf = it & 1;
            (void)ptx::mbar_wait(&ct.tmem_full[buf], (it >> 1) & 1, abort_flag);
            ptx::tc_fence_after();
            const uint32_t xb = tmem_base + ((uint32_t)(lq * 32) << 16) + buf * C::N;
            uint32_t va[32], vb[32];
            ptx::tmem_ld_32x32_async(xb, va);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              if (c & 1) ptx::tmem_wait_ld_regs(vb);
              else ptx::tmem_wait_ld_regs(va);
              if (c + 1 < 8) {
                if (c & 1) ptx::tmem_ld_32x32_async(xb + (c + 1) * 32, va);
                else ptx::tmem_ld_32x32_async(xb + (c + 1) * 32, vb);
              }
              uint32_t pk[16];
#pragma unroll
              for (int i = 0; i < 16; ++i)
                pk[i] = (c & 1) ? ptx::relu_pack_bf16x2(__uint_as_float(vb[2 * i]), __uint_as_float(vb[2 * i + 1]))
                                : ptx::relu_pack_bf16x2(__uint_as_float(va[2 * i]), __uint_as_float(va[2 * i + 1]));
              if ((c >> 1) >= present) {                       // chunk c holds heads of row c / 2 (warp-uniform)
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = 0u;
              }
              ptx::tmem_st_32x16(xb + c * 16, pk);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ct.a_ready[buf]);
          }
        } else {
          // ---- compact warps: read the four row scores of this thread's key, free the
          // accumulator buffer, leave the survivors in the row queues
          int nv4[NROWS];
#pragma unroll
          for (int r = 0; r < NROWS; ++r) {
            const int ri = b * NROWS + r;
            nv4[r] = (ri < n_rows && rows[ri].K > 0) ? rows[ri].n_vis : 0;
          }
          for (int t = 0; t < ntiles; ++t, ++it) {
            const int buf = it & 1;
            const int ksl = it % KS_SLOTS;
            (void)ptx::mbar_wait(&ct.ks_full[ksl], (it / KS_SLOTS) & 1, abort_flag);
            const float ksv = ct.ks[ksl][key_in_tile];
            (void)ptx::mbar_wait(&ct.s_ready[buf], (it >> 1) & 1, abort_flag);
            ptx::tc_fence_after();
            uint32_t sv[8];          // columns r: sum with the gates' bf16 heads, 4 + r: with their remainders
            ptx::tmem_ld_32x8(tmem_base + ((uint32_t)(lq * 32) << 16) + buf * C::N + 128, sv);
            ptx::tmem_wait_ld();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ct.tmem_empty[buf]);
            const int qb = it % QD;
            (void)ptx::mbar_wait(&ct.s.sc_empty[qb], ((it / QD) & 1) ^ 1, abort_flag);
            const int s_key = t * TILE_KEYS + key_in_tile;
#pragma unroll
            for (int r = 0; r < NROWS; ++r) {
              const uint32_t key = score_to_key((__uint_as_float(sv[r]) + __uint_as_float(sv[4 + r])) * ksv);
              scan::push_survivors(ct.s, qb, r, lq, lane, s_key < nv4[r] && key > scan::row_threshold(ct.s, r, seq), key, s_key);
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ct.s.sc_full[qb]);
          }
        }
      } else
      for (int t = 0; t < ntiles; ++t, ++it) {
        const int buf = it & 1;
        // Key scales come through shared memory (TMA): a global load issued by this warp would
        // sit in the same memory queue as its TMEM loads and stall them for an L2 round trip.
        float ksv = 1.f;
        if (C::FP8) {
          const int ksl = it % KS_SLOTS;
          (void)ptx::mbar_wait(&ct.ks_full[ksl], (it / KS_SLOTS) & 1, abort_flag);
          ksv = ct.ks[ksl][key_in_tile];
        }
        (void)ptx::mbar_wait(&ct.tmem_full[buf], (it >> 1) & 1, abort_flag);
        ptx::tc_fence_after();
        // The accumulator comes over in 32-column chunks, two register sets in turn: while one
        // chunk goes through the FMAs the next is already on its way from TMEM.
        // w ReLU(x) = (w/2) x + (w/2) |x|: two full-rate FMAs per element (|x| is a free operand
        // modifier) instead of a half-rate max plus an FMA; ct.w holds w/2.  Eight independent
        // accumulation chains per row keep the FMA pipe busy.
        float score[C::ROWS_PER_TEAM];
        constexpr int NCHUNK = 2 * C::ROWS_PER_TEAM;            // 32-column chunks of this warp
        const uint32_t tbase = tmem_base + ((uint32_t)(lq * 32) << 16) + buf * C::N + team * C::ROWS_PER_TEAM * kHeads;
        uint32_t va[32], vb[32];
        float ap[4], an[4];
        auto fma_chunk = [&](const uint32_t (&v)[32], const float* wrow) {
          const float4* wp = reinterpret_cast<const float4*>(wrow);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float4 wv = wp[j];
            const float x0 = __uint_as_float(v[4 * j]), x1 = __uint_as_float(v[4 * j + 1]);
            const float x2 = __uint_as_float(v[4 * j + 2]), x3 = __uint_as_float(v[4 * j + 3]);
            ap[0] = fmaf(fabsf(x0), wv.x, ap[0]); an[0] = fmaf(x0, wv.x, an[0]);
            ap[1] = fmaf(fabsf(x1), wv.y, ap[1]); an[1] = fmaf(x1, wv.y, an[1]);
            ap[2] = fmaf(fabsf(x2), wv.z, ap[2]); an[2] = fmaf(x2, wv.z, an[2]);
            ap[3] = fmaf(fabsf(x3), wv.w, ap[3]); an[3] = fmaf(x3, wv.w, an[3]);
          }
        };
        ptx::tmem_ld_32x32_async(tbase, va);
#pragma unroll
        for (int c = 0; c < NCHUNK; ++c) {
          if (c & 1) ptx::tmem_wait_ld_regs(vb);                // chunk c has landed
          else ptx::tmem_wait_ld_regs(va);
          if (c + 1 < NCHUNK) {
            if (c & 1) ptx::tmem_ld_32x32_async(tbase + (c + 1) * 32, va);
            else ptx::tmem_ld_32x32_async(tbase + (c + 1) * 32, vb);
          }
          if ((c & 1) == 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { ap[i] = 0.f; an[i] = 0.f; }
          }
          const float* wrow = &ct.w[team * C::ROWS_PER_TEAM + (c >> 1)][(c & 1) * 32];
          if (c & 1) fma_chunk(vb, wrow);
          else fma_chunk(va, wrow);
          if (c & 1) score[c >> 1] = ((ap[0] + an[0]) + (ap[1] + an[1])) + ((ap[2] + an[2]) + (ap[3] + an[3]));
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ct.tmem_empty[buf]);
        // ---- survivors of this warp's 32 keys (key scale applied, Appendix A) go to the row queues
        const int qb = it % QD;
        (void)ptx::mbar_wait(&ct.s.sc_empty[qb], ((it / QD) & 1) ^ 1, abort_flag);
        const int s_key = t * TILE_KEYS + key_in_tile;
#pragma unroll
        for (int rl = 0; rl < C::ROWS_PER_TEAM; ++rl) {
          const int r = team * C::ROWS_PER_TEAM + rl;
          const uint32_t key = score_to_key(C::FP8 ? score[rl] * ksv : score[rl]);
          scan::push_survivors(ct.s, qb, r, lq, lane, s_key < n_vis[rl] && key > scan::row_threshold(ct.s, r, seq), key, s_key);
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ct.s.sc_full[qb]);
      }
      // (the rows' final exact select is the finisher warps' business: on to the next block)
    }
  } else if (warp < 2 + C::EPI_WARPS + C::SEL_WARPS) {
    // ------------------------------------------------------------------ append warps: one row each
    const int r = warp - 2 - C::EPI_WARPS;
    scan::append_role(ct.s, r, lane, Team{lane, 32, 3 + r}, rows, n_rows, n_blocks, sc, abort_flag);
  } else {
    // ------------------------------------------------------------------ finisher warps
    const int f = warp - 2 - C::EPI_WARPS - C::SEL_WARPS;
    constexpr int RPF = NROWS / C::FIN_WARPS;
    scan::finisher_role(ct.s, f * RPF, RPF, lane, rows, n_rows, n_blocks, sc, abort_flag);
  }
  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  if (threadIdx.x == 0 && ct.abort) set_status(sc.status, DEV_WAIT_EXPIRED);
  if (threadIdx.x == 0 && ct.s.abort_code) set_status(sc.status, ct.s.abort_code);
}

// ---------------------------------------------------------------------------- host side

template <int DT, int NROWS, int EPI = 1>
cudaError_t launch_one(const CUtensorMap& mk, const CUtensorMap& mq0, const CUtensorMap& mq1, const CUtensorMap& mks,
                       const RowDesc* rows, int n_rows, const ScanScratch& s, int sms, cudaStream_t st) {
  using C = Cfg<DT, NROWS, EPI>;
  auto kern = scan_select_tc_kernel<DT, NROWS, EPI>;
  static bool attr_set[kMaxDevices] = {};
  const size_t smem = smem_bytes<DT, NROWS, EPI>();
  if (cudaError_t e = opt_in_dynamic_smem(kern, smem, attr_set); e != cudaSuccess) return e;
  const int n_blocks = (n_rows + NROWS - 1) / NROWS;
  const int grid = n_blocks < sms ? n_blocks : sms;
  kern<<<grid, C::THREADS, smem, st>>>(mk, mq0, mq1, mks, rows, n_rows, s);
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D map over a row-major [rows, 128] operand tensor; box = 128 bytes x box_rows, 128B swizzle.
// row_stride: bytes between rows, 0 = dense (a multiple of 16 bytes otherwise: padded key-cache rows).
bool make_operand_map(CUtensorMap* m, const void* base, long long rows, int dtype, int box_rows, int row_stride) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const bool fp8 = dtype == DT_FP8;
  cuuint64_t dims[2] = {(cuuint64_t)kDim, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)(row_stride > 0 ? row_stride : kDim * (fp8 ? 1 : 2))};
  cuuint32_t box[2] = {(cuuint32_t)(fp8 ? 128 : 64), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 1-D map over an fp32 scale array; box = `box` scales (a TMA box holds at most 256 elements per dimension).
bool make_scale_map(CUtensorMap* m, const float* base, long long n, int box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[1] = {(cuuint64_t)n};
  cuuint64_t strides[1] = {0};
  cuuint32_t boxd[1] = {(cuuint32_t)box};
  cuuint32_t estr[1] = {1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 1, (void*)base, dims, strides, boxd, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


cudaError_t launch_scan_tc(const ScanOperands& op, const RowDesc* rows, int n_rows, int rows_per_block,
                           const ScanScratch& s, int sms, cudaStream_t st, bool fp32_head_sum) {
  if (n_rows <= 0) return cudaSuccess;
  CUtensorMap mk, mq0, mq1, mks;
  memset(&mks, 0, sizeof(mks));
  if (op.dtype == DT_FP8 && !make_scale_map(&mks, op.kscale, op.k_rows, TILE_KEYS)) return cudaErrorInvalidValue;
  if (!make_operand_map(&mk, op.kc, op.k_rows, op.dtype, TILE_KEYS, op.k_stride) ||
      !make_operand_map(&mq0, op.q, (long long)op.q_rows * kHeads, op.dtype, kHeads, 0) ||
      !make_operand_map(&mq1, op.proxy_q, (long long)(op.proxy_rows > 0 ? op.proxy_rows : 1) * kHeads, op.dtype, kHeads, 0))
    return cudaErrorInvalidValue;
  if (op.dtype == DT_FP8) {
    if (rows_per_block != 4) return launch_one<DT_FP8, 1>(mk, mq0, mq1, mks, rows, n_rows, s, sms, st);
    return fp32_head_sum ? launch_one<DT_FP8, 4, 0>(mk, mq0, mq1, mks, rows, n_rows, s, sms, st)
                         : launch_one<DT_FP8, 4, 1>(mk, mq0, mq1, mks, rows, n_rows, s, sms, st);
  }
  return rows_per_block == 4 ? launch_one<DT_BF16, 4>(mk, mq0, mq1, mks, rows, n_rows, s, sms, st)
                             : launch_one<DT_BF16, 1>(mk, mq0, mq1, mks, rows, n_rows, s, sms, st);
}

}  // namespace pivot
