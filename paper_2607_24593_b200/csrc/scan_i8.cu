// Kernels 2+3 for FP8 operands: the shared prefix scan (Eq. 5 / Eq. 1, FP8 form of Appendix A)
// with its gate-weighted head sum on the tensor core as an 8-bit integer contraction, and the
// streaming top-K select (Eq. 6 / Eq. 7) fused behind it.
//
// A unit of work is 128 keys (MMA M, one key per tensor-memory lane) by 3 rows x 64 heads (N = 192)
// by d = 128.  Per unit:
//   1. first MMA (kind::f8f6f4): X[128 keys x 192] = K8 . Q8^T, fp32, into one of two accumulator
//      buffers in tensor memory;
//   2. the ReLU warps (thread = key) read a row's 64 accumulators, take their maximum m, and write
//      round(255 ReLU(x) / m) as unsigned bytes, four to a column, into a separate packed region of
//      tensor memory (48 columns per unit); the accumulator buffer is free again at once;
//   3. second MMA (kind::i8, A operand = the packed bytes in tensor memory, B = the block's gates
//      as three signed base-128 digits per head in shared memory): S[128 keys x 9] = U . W^T,
//      exact 32-bit integer sums, into 16 columns beside the packed bytes;
//   4. the compact warps read the nine sums of their key, put the digits together, undo the two
//      scales (m / 255 per key and row, the gate unit per row), apply the key scale and the causal
//      cut and hand the survivors of the running threshold to the rows' append warps.
// Why this shape.  The second MMA's cost is its number of K steps (32 bytes of K each), whatever
// its N: bytes instead of bf16 halve it.  Keeping the packed operand outside the accumulator
// buffer lets the first MMA of the unit after next start as soon as the ReLU pass has read the
// buffer, instead of after the second MMA and the score read: the accumulator round trip no
// longer bounds the tile rate.  Three rows (not four) because tensor memory holds 512 columns:
// 2 x 192 accumulator columns + 2 x (48 packed + 16 sums).
// The 8-bit codes carry a relative error of at most 1/510 of the row's largest head term each;
// on the generator's data the head sum stays within 0.14 of the FP8 score tolerance.
//
// One persistent CTA per SM, 17 warps: 0 = TMA producer, 1 = MMA issuer + tensor-memory owner,
// 2-5 and 6-9 = two sets of ReLU warps taking alternate units (set = accumulator buffer), 10-13 =
// compact warps, 14-16 = one append warp per row.  At the end of a block the three 4-warp teams
// take the final exact selection of one row each.
#include <cuda.h>
#include <cuda_fp16.h>
#include <string.h>

#include "kernels.h"
#include "ptx.cuh"
#include "scan_common.cuh"
#include "segselect.cuh"

namespace pivot {
namespace {

// Cycle accounting of CTA 0 (builds with -DPIVOT_PROF only): where each role's time goes.
#ifdef PIVOT_PROF
__device__ unsigned long long g_scan_prof[64];
#define PROF_T0() const long long prof_t0 = clock64()
#define PROF_ADD(slot) do { if (blockIdx.x == 0 && lane == 0) atomicAdd(&g_scan_prof[slot], (unsigned long long)(clock64() - prof_t0)); } while (0)
#define PROF_WAIT(slot, expr) do { const long long prof_w = clock64(); (void)(expr); if (blockIdx.x == 0 && lane == 0) atomicAdd(&g_scan_prof[slot], (unsigned long long)(clock64() - prof_w)); } while (0)
#define PROF_COUNT(slot) do { if (blockIdx.x == 0 && lane == 0) atomicAdd(&g_scan_prof[slot], 1ull); } while (0)
#else
#define PROF_T0()
#define PROF_ADD(slot)
#define PROF_WAIT(slot, expr) (void)(expr)
#define PROF_COUNT(slot)
#endif

using scan::TILE_KEYS;
using scan::KS_SLOTS;
using scan::BlockIter;
using scan::block_tiles;

constexpr int NR = 3;                         // rows per block
constexpr int N1 = NR * kHeads;               // first MMA's N
constexpr int STAGES = 4;                     // key stages (16 KB each)
constexpr int QD = 4;                         // survivor-queue depth
constexpr int THREADS = 64 + (8 + 4 + NR) * 32;
constexpr int EPI_THREADS = (12 + NR) * 32;   // everybody behind the MMA: the block barrier
constexpr int STAGE_BYTES = TILE_KEYS * 128;
constexpr int QROW_BYTES = kHeads * 128;
constexpr int QBUF_BYTES = NR * QROW_BYTES;
constexpr int PK_BASE = 2 * N1;               // tensor-memory column of the first packed region
constexpr int PK_COLS = 64;                   // 48 packed columns + 16 sum columns
constexpr int PK_SUMS = 48;
constexpr int WMAT_BYTES = 4096;              // gate digits [16 x 192 B] as two K slabs of 16 rows x 128 B
constexpr uint32_t IDESC1 = ptx::make_idesc(0u, TILE_KEYS, N1);
constexpr uint32_t IDESC2 = ptx::make_idesc_u8s8(TILE_KEYS, 16);
constexpr float kPreScale = 1.0f / 512.0f;    // accumulators times 2^-9 fit fp16 (128 x 448 x 448 x 2^-9 < 65504)
constexpr int GATE_BITS = 20;                 // integer gates span +-2^20: three signed base-128 digits

struct Ctrl {
  alignas(1024) uint8_t wmat[WMAT_BYTES];
  alignas(128) float ks[KS_SLOTS][TILE_KEYS];   // key scales of the tiles in flight (TMA destination)
  float minv[2][NR][TILE_KEYS];                 // m / 255 of each key's row, per accumulator buffer
  float wscale[NR];                             // value of one unit of the row's integer gates
  uint64_t full[STAGES], empty[STAGES];
  uint64_t q_full[2], q_empty[2];
  uint64_t tmem_full[2];     // first MMA done                 (MMA -> ReLU set)
  uint64_t acc_empty[2];     // accumulator buffer read        (ReLU set -> MMA)
  uint64_t a_ready[2];       // packed bytes + minv written    (ReLU set -> MMA, compact)
  uint64_t s_ready[2];       // second MMA done                (MMA -> compact)
  uint64_t d_empty[2];       // sums and minv read             (compact -> MMA, ReLU set)
  uint64_t w_ready;          // the block's gate digits are in place
  uint64_t ks_full[KS_SLOTS];
  uint32_t tmem_base;
  int abort;
  scan::SelectCtrl<NR, QD> s;
};

constexpr size_t smem_bytes() { return 1024 + 2 * QBUF_BYTES + STAGES * STAGE_BYTES + sizeof(Ctrl); }
static_assert(smem_bytes() <= 232448, "shared memory budget");

__global__ void __launch_bounds__(THREADS, 1)
scan_select_i8_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q0,
                      const __grid_constant__ CUtensorMap tm_q1, const __grid_constant__ CUtensorMap tm_ks,
                      const RowDesc* __restrict__ rows, int n_rows, ScanScratch sc) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* qbuf = smem;                                   // 2 x QBUF_BYTES
  uint8_t* kring = smem + 2 * QBUF_BYTES;                 // STAGES x STAGE_BYTES
  Ctrl& ct = *reinterpret_cast<Ctrl*>(kring + STAGES * STAGE_BYTES);
  volatile int* abort_flag = &ct.abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_blocks = (n_rows + NR - 1) / NR;

  // A small launch whose rows are all dead leaves before any barrier or TMEM is set up.
  if (n_rows <= (int)blockDim.x) {
    const bool live = (int)threadIdx.x < n_rows && rows[threadIdx.x].K > 0 && rows[threadIdx.x].n_vis > 0;
    if (!__syncthreads_or(live)) return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&ct.full[s], 1); ptx::mbar_init(&ct.empty[s], 1); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ct.q_full[i], 1);
      ptx::mbar_init(&ct.q_empty[i], 1);
      ptx::mbar_init(&ct.tmem_full[i], 1);
      ptx::mbar_init(&ct.acc_empty[i], 4);
      ptx::mbar_init(&ct.a_ready[i], 4);
      ptx::mbar_init(&ct.s_ready[i], 1);
      ptx::mbar_init(&ct.d_empty[i], 4);
    }
    ptx::mbar_init(&ct.w_ready, 1);
    for (int i = 0; i < KS_SLOTS; ++i) ptx::mbar_init(&ct.ks_full[i], 1);
    for (int i = 0; i < QD; ++i) {
      ptx::mbar_init(&ct.s.sc_full[i], 4);
      ptx::mbar_init(&ct.s.sc_empty[i], NR);
    }
    ct.abort = 0;
    ct.s.abort_code = 0;
    for (int r = 0; r < NR; ++r) ct.s.thr[r] = 0u;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&ct.tmem_base, 512);
    ptx::tmem_relinquish();
  }
  // everything outside the diagonal blocks of the gate matrix stays zero
  for (int i = threadIdx.x; i < WMAT_BYTES / 16; i += blockDim.x) reinterpret_cast<uint4*>(ct.wmat)[i] = make_uint4(0, 0, 0, 0);
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
      ptx::prefetch_tensormap(&tm_ks);
      BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
      uint32_t it = 0, blk = 0;
      bool ok = true;
      for (int b = bi.next(); b >= 0 && ok; b = bi.next()) {
        int k_row0 = 0;
        const int ntiles = block_tiles(rows, n_rows, b, NR, &k_row0);
        if (ntiles == 0) continue;
        const int qb = blk & 1;
        ok = ptx::mbar_wait(&ct.q_empty[qb], ((blk >> 1) & 1) ^ 1, abort_flag, 64);
        if (!ok) break;
        int present = 0;
        for (int r = 0; r < NR; ++r) present += (b * NR + r < n_rows) ? 1 : 0;
        ptx::mbar_arrive_expect_tx(&ct.q_full[qb], present * QROW_BYTES);
        for (int r = 0; r < NR; ++r) {
          const int ri = b * NR + r;
          if (ri >= n_rows) continue;
          const CUtensorMap* tm = rows[ri].q_map ? &tm_q1 : &tm_q0;
          ptx::tma_load_2d(qbuf + qb * QBUF_BYTES + r * QROW_BYTES, tm, 0, rows[ri].q_row * kHeads, &ct.q_full[qb]);
        }
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int s = it % STAGES;
          ok = ptx::mbar_wait(&ct.empty[s], ((it / STAGES) & 1) ^ 1, abort_flag, 64);
          if (!ok) break;
          ptx::mbar_arrive_expect_tx(&ct.full[s], STAGE_BYTES);
          ptx::tma_load_2d(kring + s * STAGE_BYTES, &tm_k, 0, k_row0 + t * TILE_KEYS, &ct.full[s]);
          // The tile's key scales ride along into their own ring.  A slot is free again by
          // construction: this thread runs at most STAGES tiles ahead of the MMA and the MMA at
          // most four ahead of the compact warps, fewer than KS_SLOTS in total.
          const int ksl = it % KS_SLOTS;
          ptx::mbar_arrive_expect_tx(&ct.ks_full[ksl], TILE_KEYS * 4);
          ptx::tma_load_1d(&ct.ks[ksl][0], &tm_ks, k_row0 + t * TILE_KEYS, &ct.ks_full[ksl]);
        }
        ++blk;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
#ifdef PIVOT_PROF
      const int lane = 0;      // the elected thread does the accounting
#endif
      BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
      uint32_t it = 0, blk = 0;
      bool ok = true;
      // The second MMA of unit it-1 is issued right after the first MMA of unit it: its operand is
      // produced while that MMA runs.
      bool pend = false;
      uint32_t pend_it = 0, pend_blk = 0, w_blk = 0xffffffffu;
      const uint32_t w_addr = ptx::smem_u32(ct.wmat);
      auto issue_mma2 = [&]() -> bool {
        if (pend_blk != w_blk) {                 // first unit of a block: its gate digits must be in place
          if (!ptx::mbar_wait_poll(&ct.w_ready, pend_blk & 1, abort_flag)) return false;
          w_blk = pend_blk;
        }
        const int pb = pend_it & 1;
        const uint32_t ph = (pend_it >> 1) & 1;
        bool okw;
        PROF_WAIT(2, okw = ptx::mbar_wait_poll(&ct.d_empty[pb], ph ^ 1, abort_flag));   // sums of unit pend_it-2 read
        if (!okw) return false;
        PROF_WAIT(3, okw = ptx::mbar_wait_poll(&ct.a_ready[pb], ph, abort_flag));
        if (!okw) return false;
        ptx::tc_fence_after();
        const uint32_t pk = tmem_base + PK_BASE + pb * PK_COLS;
#pragma unroll
        for (int ks = 0; ks < N1 / 32; ++ks)     // 32 bytes of K per step: 8 packed columns, 32 bytes of W
          ptx::tc_mma_a_tmem_i8(pk + PK_SUMS, pk + ks * 8, ptx::smem_desc_sw128(w_addr + (ks >> 2) * 2048 + (ks & 3) * 32),
                                IDESC2, ks ? 1u : 0u);
        ptx::tc_commit(&ct.s_ready[pb]);
        return true;
      };
      for (int b = bi.next(); b >= 0 && ok; b = bi.next()) {
        int k_row0 = 0;
        const int ntiles = block_tiles(rows, n_rows, b, NR, &k_row0);
        if (ntiles == 0) continue;
        const int qb = blk & 1;
        ok = ptx::mbar_wait(&ct.q_full[qb], (blk >> 1) & 1, abort_flag, 32);
        if (!ok) break;
        const uint32_t q_addr = ptx::smem_u32(qbuf + qb * QBUF_BYTES);
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int s = it % STAGES;
          const int buf = it & 1;
          PROF_WAIT(0, ok = ptx::mbar_wait_poll(&ct.acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag));
          if (!ok) break;
          PROF_WAIT(1, ok = ptx::mbar_wait_poll(&ct.full[s], (it / STAGES) & 1, abort_flag));
          if (!ok) break;
          PROF_COUNT(4);
          ptx::tc_fence_after();
          const uint32_t k_addr = ptx::smem_u32(kring + s * STAGE_BYTES);
          const uint32_t d_tmem = tmem_base + buf * N1;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            ptx::tc_mma<true>(d_tmem, ptx::smem_desc_sw128(k_addr + ks * 32), ptx::smem_desc_sw128(q_addr + ks * 32), IDESC1,
                              ks ? 1u : 0u);
          ptx::tc_commit(&ct.empty[s]);       // key stage free once these MMAs are done
          ptx::tc_commit(&ct.tmem_full[buf]); // accumulator ready
          if (pend) { ok = issue_mma2(); if (!ok) break; }
          pend = true; pend_it = it; pend_blk = blk;
        }
        ptx::tc_commit(&ct.q_empty[qb]);
        ++blk;
      }
      if (pend && ok) (void)issue_mma2();
    }
  } else if (warp < 14) {
    // ------------------------------------------------------------------ ReLU sets and compact warps
    const int team = (warp - 2) >> 2;              // 0, 1: ReLU sets; 2: compact warps
    const int lq = warp & 3;                       // TMEM lane quarter this warp may access
    const int key_in_tile = lq * 32 + lane;
    const int tt = ((warp - 2) & 3) * 32 + lane;   // rank inside the team
    const Team tm{tt, 128, 1 + team};
    const Team blkbar{0, EPI_THREADS, 8};          // all of this branch and the append warps
    const uint32_t lane_base = tmem_base + ((uint32_t)(lq * 32) << 16);
    BlockIter bi(n_blocks, gridDim.x, blockIdx.x);
    uint32_t it = 0;
    // A failed wait never changes this role's control flow (the barriers below must stay matched);
    // once the abort flag is up every later wait returns at once.
    for (int b = bi.next(); b >= 0; b = bi.next()) {
      int k_row0 = 0;
      const int ntiles = block_tiles(rows, n_rows, b, NR, &k_row0);
      if (ntiles == 0) continue;
      const int present = n_rows - b * NR;         // rows of this block that exist (>= 1)
      if (team == 2) {
        // ---- gate digits of the block: warp r of the team takes row r (heads lane, lane + 32).
        //      The last second MMA of the previous block is through: its sums have been read.
        const int r = tt >> 5;
        if (r < NR) {
          const int ri = b * NR + r;
          float wv[2] = {0.f, 0.f};
          if (ri < n_rows && rows[ri].K > 0) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              wv[u] = rows[ri].w[lane + 32 * u];
              if (rows[ri].qscale) wv[u] = __fmul_rn(wv[u], rows[ri].qscale[lane + 32 * u]);
            }
          }
          const float wmax = __uint_as_float(__reduce_max_sync(0xffffffffu,
              max(__float_as_uint(fabsf(wv[0])), __float_as_uint(fabsf(wv[1])))));
          const float unit = wmax > 0.f ? wmax * (1.0f / (float)(1 << GATE_BITS)) : 0.f;
          const float inv = wmax > 0.f ? (float)(1 << GATE_BITS) / wmax : 0.f;
          if (lane == 0) ct.wscale[r] = unit;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int j = lane + 32 * u;
            const int W = __float2int_rn(wv[u] * inv);             // |W| <= 2^20
            const int d1 = (W + 8192 + (1 << 22)) / 16384 - 256;   // round(W / 2^14), floor division on a positive number
            const int rem = W - d1 * 16384;                        // -8192 .. 8191
            const int d2 = (rem + 64 + (1 << 14)) / 128 - 128;     // round(rem / 128)
            const int d3 = rem - d2 * 128;                         // -64 .. 63
            const int digit[3] = {d1, d2, d3};
            const int k = r * kHeads + j;                          // K index of (row, head)
            const int kk = k & 127;
#pragma unroll
            for (int t3 = 0; t3 < 3; ++t3) {
              const int n = r * 3 + t3;                            // N row: (row, digit)
              ct.wmat[(k >> 7) * 2048 + (n >> 3) * 1024 + (n & 7) * 128 + (((kk >> 4) ^ (n & 7)) << 4) + (kk & 15)] =
                  (uint8_t)(int8_t)digit[t3];
            }
          }
        }
        ptx::fence_proxy_async_smem();         // generic-proxy writes -> tensor-core reads
        tm.sync();
        if (tt == 0) ptx::mbar_arrive(&ct.w_ready);
        int nv[NR];
#pragma unroll
        for (int r2 = 0; r2 < NR; ++r2) {
          const int ri = b * NR + r2;
          nv[r2] = (ri < n_rows && rows[ri].K > 0) ? rows[ri].n_vis : 0;
        }
        float wsc[NR];
#pragma unroll
        for (int r2 = 0; r2 < NR; ++r2) wsc[r2] = ct.wscale[r2];
        // ---- compact warps: the nine integer sums of this thread's key -> three scores -> queues
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int buf = it & 1;
          const uint32_t ph = (it >> 1) & 1;
          const int ksl = it % KS_SLOTS;
          PROF_T0();
          PROF_WAIT(8, ptx::mbar_wait(&ct.ks_full[ksl], (it / KS_SLOTS) & 1, abort_flag));
          const float ksv = ct.ks[ksl][key_in_tile];
          PROF_WAIT(9, ptx::mbar_wait(&ct.a_ready[buf], ph, abort_flag));       // minv of this unit is visible
          float mi[NR];
#pragma unroll
          for (int r2 = 0; r2 < NR; ++r2) mi[r2] = ct.minv[buf][r2][key_in_tile];
          PROF_WAIT(10, ptx::mbar_wait(&ct.s_ready[buf], ph, abort_flag));
          ptx::tc_fence_after();
          uint32_t sv[16];         // column 3 r + t: sum with digit t of row r's gates
          ptx::tmem_ld_32x16(lane_base + PK_BASE + buf * PK_COLS + PK_SUMS, sv);
          ptx::tmem_wait_ld();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ct.d_empty[buf]);
          const int qb = it % QD;
          PROF_WAIT(11, ptx::mbar_wait(&ct.s.sc_empty[qb], ((it / QD) & 1) ^ 1, abort_flag));
          const int s_key = t * TILE_KEYS + key_in_tile;
#pragma unroll
          for (int r2 = 0; r2 < NR; ++r2) {
            const float T = fmaf((float)(int)sv[3 * r2], 16384.f, fmaf((float)(int)sv[3 * r2 + 1], 128.f, (float)(int)sv[3 * r2 + 2]));
            const uint32_t key = score_to_key(T * (mi[r2] * wsc[r2]) * ksv);
            scan::push_survivors(ct.s, qb, r2, lq, lane, s_key < nv[r2] && key > ct.s.thr[r2], key, s_key);
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ct.s.sc_full[qb]);
          if (lq == 0) { PROF_ADD(12); PROF_COUNT(13); }
        }
      } else {
        // ---- ReLU set `team`: units with it % 2 == team.  Thread = key: per row, 64 accumulators
        //      -> their maximum -> 64 unsigned bytes in 16 packed columns.
        const int buf = team;
        const uint32_t acc = lane_base + buf * N1;
        const uint32_t pk = lane_base + PK_BASE + buf * PK_COLS;
        for (int t = 0; t < ntiles; ++t, ++it) {
          if ((int)(it & 1) != team) continue;
          const uint32_t ph = (it >> 1) & 1;
          PROF_T0();
          PROF_WAIT(16 + team * 8, ptx::mbar_wait(&ct.tmem_full[buf], ph, abort_flag));
          ptx::tc_fence_after();
          uint32_t va[32], vb[32];
          ptx::tmem_ld_32x32_async(acc, va);
          ptx::tmem_ld_32x32_async(acc + 32, vb);
          // the packed region and the minv slots of this buffer: the sums of unit it-2 must have been read
          PROF_WAIT(17 + team * 8, ptx::mbar_wait(&ct.d_empty[buf], ph ^ 1, abort_flag));
#pragma unroll
          for (int r = 0; r < NR; ++r) {
            // ReLU, an exact power-of-two pre-scale (the largest accumulator, 128 x 448 x 448, must fit
            // fp16) and rounding to fp16 in pairs: the row's 64 values now take 32 registers and the
            // raw ones are free for the next row's loads
            uint32_t h[32];
            ptx::tmem_wait_ld_regs(va);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              ptx::relu_scale_pack_f16x2(__uint_as_float(va[4 * j]), __uint_as_float(va[4 * j + 1]), __uint_as_float(va[4 * j + 2]),
                                         __uint_as_float(va[4 * j + 3]), kPreScale, h[2 * j], h[2 * j + 1]);
            ptx::tmem_wait_ld_regs(vb);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              ptx::relu_scale_pack_f16x2(__uint_as_float(vb[4 * j]), __uint_as_float(vb[4 * j + 1]), __uint_as_float(vb[4 * j + 2]),
                                         __uint_as_float(vb[4 * j + 3]), kPreScale, h[16 + 2 * j], h[16 + 2 * j + 1]);
            if (r + 1 < NR) {                      // half of the next row's accumulators on their way
              ptx::tmem_ld_32x32_async(acc + (r + 1) * kHeads, va);
            } else {                               // all of the buffer has been read: the first MMA may refill it
              ptx::tc_fence_before();
              __syncwarp();
              if (lane == 0) ptx::mbar_arrive(&ct.acc_empty[buf]);
            }
            uint32_t mx[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
              mx[j] = ptx::max_f16x2(ptx::max_f16x2(h[j], h[8 + j]), ptx::max_f16x2(h[16 + j], h[24 + j]));
#pragma unroll
            for (int j = 0; j < 4; ++j) mx[j] = ptx::max_f16x2(mx[j], mx[4 + j]);
            const uint32_t m2 = ptx::max_f16x2(ptx::max_f16x2(mx[0], mx[1]), ptx::max_f16x2(mx[2], mx[3]));
            const __half2 mh = *reinterpret_cast<const __half2*>(&m2);
            const float m = fmaxf(__low2float(mh), __high2float(mh));      // largest pre-scaled head term of this key's row
            const bool have = r < present && m > 0.f;    // rows missing from a partial block: stale query bytes, anything
            // codes = round(h * s) with s rounded to fp16; the compact warps undo exactly that s
            const __half sh = __float2half_rn(have ? __fdividef(255.0f, m) : 0.f);
            const __half2 s2h = __half2half2(sh);
            const uint32_t s2 = *reinterpret_cast<const uint32_t*>(&s2h);
            const float s_used = __half2float(sh);
            uint32_t p8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) p8[j] = have ? ptx::quant4_u8_f16(h[2 * j], h[2 * j + 1], s2) : 0u;
            ptx::tmem_st_32x8(pk + r * 16, p8);
#pragma unroll
            for (int j = 0; j < 8; ++j) p8[j] = have ? ptx::quant4_u8_f16(h[16 + 2 * j], h[16 + 2 * j + 1], s2) : 0u;
            ptx::tmem_st_32x8(pk + r * 16 + 8, p8);
            if (r + 1 < NR) ptx::tmem_ld_32x32_async(acc + (r + 1) * kHeads + 32, vb);     // ... and the other half
            ct.minv[buf][r][key_in_tile] = (have && s_used > 0.f) ? __fdividef(1.0f / kPreScale, s_used) : 0.f;
          }
          ptx::tmem_wait_st();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ct.a_ready[buf]);
          if (lq == 0) { PROF_ADD(18 + team * 8); PROF_COUNT(19 + team * 8); }
        }
      }
      // ---- end of the block: team t takes the final exact selection of row t
      blkbar.sync();                               // append warps are done with the last tile
      {
        const int r = team;
        const int ri = b * NR + r;
        const bool live = ri < n_rows && rows[ri].K > 0;
        if (live) scan::final_select_row(ct.s, tm, r, rows[ri].K, rows[ri], sc);
      }
      blkbar.sync();                               // rows' histograms and segments may be reused
    }
  } else {
    // ------------------------------------------------------------------ append warps: one row each
    const int r = warp - 14;
    scan::append_role(ct.s, r, lane, Team{lane, 32, 4 + r}, Team{0, EPI_THREADS, 8}, rows, n_rows, n_blocks, sc, abort_flag);
  }
  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, 512);
  if (threadIdx.x == 0 && ct.abort) set_status(sc.status, DEV_WAIT_EXPIRED);
  if (threadIdx.x == 0 && ct.s.abort_code) set_status(sc.status, ct.s.abort_code);
}

}  // namespace

bool make_operand_map(CUtensorMap* m, const void* base, long long rows, int dtype, int box_rows);
bool make_scale_map(CUtensorMap* m, const float* base, long long n);

// Cycle counters of CTA 0 since the last call (all zeros unless built with -DPIVOT_PROF).
cudaError_t read_scan_prof(unsigned long long* out64_host) {
#ifdef PIVOT_PROF
  cudaError_t e = cudaMemcpyFromSymbol(out64_host, g_scan_prof, sizeof(unsigned long long) * 64);
  if (e != cudaSuccess) return e;
  static const unsigned long long zeros[64] = {};
  return cudaMemcpyToSymbol(g_scan_prof, zeros, sizeof(zeros));
#else
  for (int i = 0; i < 64; ++i) out64_host[i] = 0;
  return cudaSuccess;
#endif
}

cudaError_t launch_scan_i8(const ScanOperands& op, const RowDesc* rows, int n_rows, const ScanScratch& s, int sms,
                           cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  if (op.dtype != DT_FP8) return cudaErrorInvalidValue;
  CUtensorMap mk, mq0, mq1, mks;
  if (!make_scale_map(&mks, op.kscale, op.k_rows) || !make_operand_map(&mk, op.kc, op.k_rows, op.dtype, TILE_KEYS) ||
      !make_operand_map(&mq0, op.q, (long long)op.q_rows * kHeads, op.dtype, kHeads) ||
      !make_operand_map(&mq1, op.proxy_q, (long long)(op.proxy_rows > 0 ? op.proxy_rows : 1) * kHeads, op.dtype, kHeads))
    return cudaErrorInvalidValue;
  static bool attr_set[kMaxDevices] = {};
  const size_t smem = smem_bytes();
  if (cudaError_t e = opt_in_dynamic_smem(scan_select_i8_kernel, smem, attr_set); e != cudaSuccess) return e;
  const int n_blocks = (n_rows + NR - 1) / NR;
  const int grid = n_blocks < sms ? n_blocks : sms;
  scan_select_i8_kernel<<<grid, THREADS, smem, st>>>(mk, mq0, mq1, mks, rows, n_rows, s);
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace pivot
