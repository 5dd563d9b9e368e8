// Kernel 4: candidate gather + per-query re-score on tcgen05 tensor cores + fused top-k
// (Eq. 8-9).
//
// One group at a time per persistent CTA.  The group's m <= 4 member queries (m x 64 heads)
// form the MMA N side and stay in shared memory; the c candidate keys are gathered from the
// (L2-resident) key cache by two producer warps, 128 keys per tile, written straight into the
// 128-byte-swizzled K-major layout the tensor core reads (cp.async, 16 bytes at a time).  The
// epilogue is the scan's: one key per thread, ReLU, gate-weighted head sum, key scale.  Scores
// go to a per-CTA buffer, from which each member's exact top-k is selected and written out:
// by select warps while the next group is re-scored (FP8 prefill), by the epilogue warps after
// the group's last tile (bf16), or by a later kernel (the candidate chunks of a decode step).
//
// Warps: 0 = query TMA, 1 = MMA issuer + TMEM owner, 2-3 = gather producers, 4-11 = epilogue,
// 12-15 (EPI = 3) = select warps, one per member.
#include <cuda.h>

#include "kernels.h"
#include "ptx.cuh"
#include "segselect.cuh"

namespace pivot {
namespace {

constexpr int TILE_KEYS = 128;
constexpr int MAX_STAGES = 8;
constexpr int NMEM = 4;                       // members per MMA (N = 256)
constexpr int GATHER_WARPS = 2;       // each producer thread copies two rows of a tile
constexpr int EPI_WARPS = 8;
constexpr int SEL_WARPS = 4;
constexpr int N = NMEM * kHeads;
constexpr int TMEM_COLS = 2 * N;

// EPI: 0 = fp32 FMA head sum, scores as packed entries in the per-CTA global segments, each
// member's top-k by the epilogue teams after the group's tiles (bf16 operands; FP8 on request).
// FP8 otherwise takes the head sum on the tensor core and comes in two forms: 3 = prefill: the
// per-member top-k runs on four warps of their own, one group behind the tile loop; the score
// rows go through a double buffer in global memory (L2-resident, 2 x 4 x ScanScratch::rslots keys
// per CTA), so the tensor core and the gather keep running while a group's members are selected;
// every group of the launch has at most rslots candidates.  2 = the candidate chunks of a decode
// step: those leave packed entries for a later top-k kernel.  (1 = the default for bf16, same as 0.)
template <int DT, int EPI = 1>
struct RCfg {
  static constexpr bool FP8 = DT == DT_FP8;
  static constexpr bool OVL = EPI == 3;
  static constexpr int NSEL = OVL ? SEL_WARPS : 2;
  // 384 threads: 168 registers per thread; 512 (with the select warps): 128
  static constexpr int THREADS = (2 + GATHER_WARPS + EPI_WARPS + (OVL ? SEL_WARPS : 0)) * 32;
  static constexpr int KHALVES = FP8 ? 1 : 2;
  static constexpr int HALF_TILE_BYTES = TILE_KEYS * 128;
  static constexpr int STAGE_BYTES = KHALVES * HALF_TILE_BYTES;
  static constexpr int QROW_HALF_BYTES = kHeads * 128;
  static constexpr int QHALF_BYTES = NMEM * QROW_HALF_BYTES;
  static constexpr int QBUF_BYTES = KHALVES * QHALF_BYTES;
  // the next group's queries load while this one is re-scored, except where 2 x 64 KB of bf16
  // queries would leave no room for the select warps' histograms
  static constexpr int QBUFS = (OVL && !FP8) ? 1 : 2;
  static constexpr int STAGES = FP8 ? 6 : 2;
  static constexpr int LOOKAHEAD = FP8 ? 4 : 1;   // gather tiles in flight per producer thread
  static constexpr int ROW_BYTES = FP8 ? 128 : 256;
  static constexpr uint32_t IDESC = ptx::make_idesc(FP8 ? 0u : 1u, TILE_KEYS, N);
  // FP8: the gate-weighted head sum of Eq. 8 runs on the tensor core, as in the shared scan (a
  // second MMA over bf16 ReLU values written in place in tensor memory against a block-diagonal
  // gate matrix).  bf16 operands keep the fp32 FMA head sum.
  static constexpr bool MMA2 = FP8 && EPI != 0;
  static constexpr uint32_t IDESC2 = ptx::make_idesc(1u, TILE_KEYS, 16);
  static constexpr int TMEM_EMPTY_ARRIVALS = MMA2 ? 4 : EPI_WARPS;
};

constexpr int META_SLOTS = 8;     // key stages in flight (<= 6) + accumulator buffers (2)
static_assert(META_SLOTS >= 6 + 2, "meta ring");

// What the epilogue needs to know about a gathered key: its position and scale.
struct KeyMeta {
  int idx;       // key position, -1 for a padding slot
  float ks;      // key scale (1 for bf16)
};

// MMA2: the group's gate matrix, bf16, K-major with 128-byte swizzle, in the compact form the
// second MMA reads: 4 slabs (64 columns each) of 8 rows x 128 B -- row r = bf16 head of member r's
// effective gates (in slab r only), row 4 + r = their bf16 remainder -- followed by one 1 KB block
// of zeros that serves as rows 8..15 of every slab (the descriptor's stride between the two 8-row
// groups is set per slab).
constexpr int WMAT_BYTES = 5120;

template <bool MMA2, int NSEL = 2>
struct RCtrlT {
  alignas(1024) uint8_t wmat[MMA2 ? WMAT_BYTES : 16];
  uint64_t a_ready[2], s_ready[2], w_ready;      // MMA2 handshakes
  alignas(16) float w[MMA2 ? 1 : NMEM][kHeads];
  KeyMeta meta[META_SLOTS][TILE_KEYS];   // written by the gather warps, read by the epilogue
  uint64_t full[MAX_STAGES], empty[MAX_STAGES];
  uint64_t q_full[2], q_empty[2], tmem_full[2], tmem_empty[2];
  uint64_t g_ready[2];                           // a group's gates are staged (query warp -> score warps)
  alignas(16) float gstage[2][MMA2 ? NMEM * kHeads : 4];
  uint64_t k_full[2], k_free[2];                 // score rows of a group: score warps -> select warps
  uint32_t kstat[2][NMEM][4];                    // ... and each row's smallest / largest key and filled slots
  uint32_t tmem_base;
  int abort;
  SegSelSmem sel[NSEL];          // one per selecting team (EPI = 3: per select warp)
};

template <int DT, int EPI = 1>
constexpr size_t rsmem_bytes() {
  using C = RCfg<DT, EPI>;
  return 1024 + C::QBUFS * C::QBUF_BYTES + C::STAGES * C::STAGE_BYTES + sizeof(RCtrlT<C::MMA2, C::NSEL>);
}
static_assert(rsmem_bytes<DT_FP8, 0>() <= 232448 && rsmem_bytes<DT_FP8, 2>() <= 232448 &&
              rsmem_bytes<DT_FP8, 3>() <= 232448 && rsmem_bytes<DT_BF16, 3>() <= 232448 &&
              rsmem_bytes<DT_BF16>() <= 232448, "shared memory budget");

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int NPEND>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(NPEND) : "memory");
}

__device__ __forceinline__ int group_tiles(const GroupDesc& gd) {
  return gd.n_cand > 0 ? (gd.n_cand + TILE_KEYS - 1) / TILE_KEYS : 0;
}

template <int DT, int EPI>
__global__ void __launch_bounds__((RCfg<DT, EPI>::THREADS), 1)
refine_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const GroupDesc* __restrict__ groups, int n_groups,
                 int q_rows_total, ScanScratch sc) {
  using C = RCfg<DT, EPI>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* qbuf = smem;
  uint8_t* kring = smem + C::QBUFS * C::QBUF_BYTES;
  using RCtrl = RCtrlT<C::MMA2, C::NSEL>;
  RCtrl& ct = *reinterpret_cast<RCtrl*>(kring + C::STAGES * C::STAGE_BYTES);
  volatile int* abort_flag = &ct.abort;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      ptx::mbar_init(&ct.full[s], GATHER_WARPS);
      ptx::mbar_init(&ct.empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ct.q_full[i], 1);
      ptx::mbar_init(&ct.q_empty[i], 1);
      ptx::mbar_init(&ct.tmem_full[i], 1);
      ptx::mbar_init(&ct.tmem_empty[i], C::TMEM_EMPTY_ARRIVALS);
      ptx::mbar_init(&ct.a_ready[i], 4);
      ptx::mbar_init(&ct.s_ready[i], 1);
      ptx::mbar_init(&ct.k_full[i], C::MMA2 ? 4 : EPI_WARPS);   // every warp that writes score rows
      ptx::mbar_init(&ct.k_free[i], SEL_WARPS);
      ptx::mbar_init(&ct.g_ready[i], 1);
    }
    ptx::mbar_init(&ct.w_ready, 1);
    for (int i = 0; i < 2 * NMEM; ++i) {
      ct.kstat[i / NMEM][i % NMEM][0] = 0xffffffffu;
      ct.kstat[i / NMEM][i % NMEM][1] = 0u;
      ct.kstat[i / NMEM][i % NMEM][2] = 0u;
    }
    ct.abort = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&ct.tmem_base, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  if constexpr (C::MMA2)        // everything but the diagonal blocks of the gate matrix stays zero
    for (int i = threadIdx.x; i < WMAT_BYTES / 16; i += blockDim.x) reinterpret_cast<uint4*>(ct.wmat)[i] = make_uint4(0, 0, 0, 0);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = ct.tmem_base;
  // (a decode step launches this kernel so that the set-up above overlaps the kernel before it)
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ member-query TMA
    // ... and, for the tensor-core head sum, the group's effective gates: fetched here, up to two
    // groups ahead, into a small staging array, so that the warps that build the gate matrix at
    // the start of a group find them in shared memory instead of behind two global round trips.
    // (A staging slot is free when the query buffer of the same parity is: the group that used
    // it has issued its last MMA, and its gate matrix was built before its first.)
    const bool leader = ptx::elect_one();
    if (leader) ptx::prefetch_tensormap(&tm_q);
    uint32_t blk = 0;
    for (int gi = blockIdx.x; gi < n_groups; gi += gridDim.x) {
      const GroupDesc gd = groups[gi];
      if (group_tiles(gd) == 0) continue;
      const int qb = blk % C::QBUFS;
      if (!ptx::mbar_wait(&ct.q_empty[qb], ((blk / C::QBUFS) & 1) ^ 1, abort_flag, 128)) break;
      if (leader) {
        ptx::mbar_arrive_expect_tx(&ct.q_full[qb], gd.m * C::KHALVES * C::QROW_HALF_BYTES);
        for (int r = 0; r < gd.m; ++r)
          for (int h = 0; h < C::KHALVES; ++h)
            ptx::tma_load_2d(qbuf + qb * C::QBUF_BYTES + h * C::QHALF_BYTES + r * C::QROW_HALF_BYTES, &tm_q,
                             h * 64, (gd.q_row + r) * kHeads, &ct.q_full[qb]);
      }
      if constexpr (C::MMA2) {
        float wv[NMEM * kHeads / 32];
#pragma unroll
        for (int u = 0; u < NMEM * kHeads / 32; ++u) {
          const int i = u * 32 + lane, r = i >> 6, j = i & 63;
          wv[u] = 0.f;
          if (r < gd.m) {
            wv[u] = gd.w[r * kHeads + j];
            if (gd.qscale) wv[u] = __fmul_rn(wv[u], gd.qscale[r * kHeads + j]);
          }
        }
#pragma unroll
        for (int u = 0; u < NMEM * kHeads / 32; ++u) ct.gstage[blk & 1][u * 32 + lane] = wv[u];
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ct.g_ready[blk & 1]);
      }
      ++blk;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
      uint32_t it = 0, blk = 0;
      bool ok = true;
      // MMA2: the head sum of tile it-1 follows the first MMA of tile it (see the shared scan)
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
        if (pend_blk != w_blk) {                 // first tile of a group: its gate matrix must be in place
          bool okw;
          PW(3, okw = ptx::mbar_wait(&ct.w_ready, pend_blk & 1, abort_flag, 0))
          if (!okw) return false;
          w_blk = pend_blk;
        }
        const int pb = pend_it & 1;
        // no sleep between polls here or on the accumulator / key-stage waits below: this thread's
        // wake-up latency sits on the tile loop's critical path (four handoffs per tile)
        bool oka;
        PW(4, oka = ptx::mbar_wait_poll(&ct.a_ready[pb], (pend_it >> 1) & 1, abort_flag))
        if (!oka) return false;
        ptx::tc_fence_after();
        const uint32_t w_addr = ptx::smem_u32(ct.wmat);
        const uint32_t a_tmem = tmem_base + pb * N;
#pragma unroll
        for (int ks = 0; ks < 16; ++ks) {        // 16 bf16 of K per step: 8 TMEM columns, 32 bytes of W
          const int slab = ks >> 2;
          uint64_t d = ptx::smem_desc_sw128(w_addr + slab * 1024 + (ks & 3) * 32);
          d &= ~((uint64_t)0x3FFF << 32);        // rows 8..15 of the slab: the shared zero block
          d |= (uint64_t)(((4096 - slab * 1024) >> 4) & 0x3FFF) << 32;
          ptx::tc_mma_a_tmem_bf16(a_tmem + 128, a_tmem + ks * 8, d, C::IDESC2, ks ? 1u : 0u);
        }
        ptx::tc_commit(&ct.s_ready[pb]);
        return true;
      };
      for (int gi = blockIdx.x; gi < n_groups && ok; gi += gridDim.x) {
        const int ntiles = group_tiles(groups[gi]);
        if (ntiles == 0) continue;
        const int qb = blk % C::QBUFS;
        PW(0, ok = ptx::mbar_wait(&ct.q_full[qb], (blk / C::QBUFS) & 1, abort_flag, 32))
        if (!ok) break;
        const uint32_t q_addr = ptx::smem_u32(qbuf + qb * C::QBUF_BYTES);
        for (int t = 0; t < ntiles; ++t, ++it) {
          const int s = it % C::STAGES;
          const uint32_t ph = (it / C::STAGES) & 1;
          const int buf = it & 1;
          PW(1, ok = ptx::mbar_wait_poll(&ct.tmem_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag))
          if (!ok) break;
          PW(2, ok = ptx::mbar_wait_poll(&ct.full[s], ph, abort_flag))
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t k_addr = ptx::smem_u32(kring + s * C::STAGE_BYTES);
          const uint32_t d_tmem = tmem_base + buf * N;
#pragma unroll
          for (int h = 0; h < C::KHALVES; ++h)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t a = ptx::smem_desc_sw128(k_addr + h * C::HALF_TILE_BYTES + ks * 32);
              const uint64_t bq = ptx::smem_desc_sw128(q_addr + h * C::QHALF_BYTES + ks * 32);
              ptx::tc_mma<C::FP8>(d_tmem, a, bq, C::IDESC, (h | ks) ? 1u : 0u);
            }
          ptx::tc_commit(&ct.empty[s]);
          ptx::tc_commit(&ct.tmem_full[buf]);
          if constexpr (C::MMA2) {
            if (pend) { ok = issue_mma2(); if (!ok) break; }
            pend = true; pend_it = it; pend_blk = blk;
          }
        }
        if constexpr (C::MMA2) {                 // the group's last tile: nothing left to overlap it with
          if (pend && ok) ok = issue_mma2();
          pend = false;
        }
        ptx::tc_commit(&ct.q_empty[qb]);
        ++blk;
      }
#undef PW
      PIVOT_PROF_DO(if (C::OVL && C::MMA2) {
        pw[5] = clock64() - pstart;
        for (int i = 0; i < 6; ++i) prof_add(sc.status, PROF_REF_WAIT_QUERIES + i, pw[i]);
        prof_add(sc.status, PROF_REF_TILES, it);
      })
    }
  } else if (warp < 2 + GATHER_WARPS) {
    // ------------------------------------------------------------------ gather producers
    // Each gather warp fills 64 rows of a tile.  A lane looks up two of them (position, row in
    // the key tensor, scale: rows wrow0 + lane and wrow0 + 32 + lane); the copies themselves go
    // eight lanes to a row, one 16-byte chunk each, so that one warp instruction reads four whole
    // 128-byte lines (a lane-per-row copy would touch 32 lines for the same bytes and is bound
    // by the L1's tag rate).  Tiles are committed as cp.async groups; a tile is published
    // LOOKAHEAD tiles after it was issued.
    const int wrow0 = (warp - 2) * 64;
    const int sub = lane >> 3, chunk = lane & 7;
    uint32_t it = 0;          // tiles issued
    uint32_t pub = 0;         // tiles published
    bool ok = true;
    auto publish = [&](uint32_t p) {
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&ct.full[p % C::STAGES]);
    };
    for (int gi = blockIdx.x; gi < n_groups; gi += gridDim.x) {
      const GroupDesc gd = groups[gi];
      const int ntiles = group_tiles(gd);
      if (ntiles == 0) continue;
      const int krow_bytes = gd.k_stride > 0 ? gd.k_stride : C::ROW_BYTES;   // padded cache rows (32-bit: one wide multiply per address)
      // Candidate positions are fetched three tiles ahead, their rows in the key tensor (a
      // block-table lookup when the cache is paged) two tiles ahead and key scales one tile
      // ahead, so no round trip sits on this thread's issue path.
      const int pos_limit = gd.pos_max;
      auto load_idx = [&](int tile, int half) -> int {
        const int sl = tile * TILE_KEYS + wrow0 + half * 32 + lane;
        return (tile < ntiles && sl < gd.n_cand) ? __ldg(gd.cand + sl) : -1;
      };
      // A candidate position beyond the group's last member (gd.pos_max) cannot come from the scan; it
      // can come from a caller-supplied candidate set.  Such a slot is dropped like a padding slot and
      // the status word says so (tested in every build: the gather must never leave the cache).  The
      // test sits here, a pipeline stage after the load of the position, so that it does not wait
      // for that load.
      auto key_row = [&](int ix) -> int {      // -1: padding slot, or a page outside the pool
        if (ix > pos_limit || ix < -1) { set_status(sc.status, DEV_BOUNDS); return -1; }
        if (!gd.pages || ix < 0) return ix;
        const uint32_t pg = (uint32_t)__ldg(gd.pages + (ix >> 7));
        (void)PIVOT_BOUNDS(pg < (uint32_t)gd.n_pages, sc.status);     // checked build: a hole in the block table is reported
        return pg < (uint32_t)gd.n_pages ? (int)(pg * 128u + (uint32_t)(ix & 127)) : -1;
      };
      auto load_ks = [&](int row) -> float { return (gd.kscale && row >= 0) ? __ldg(gd.kscale + row) : 1.f; };
      int idx0[2] = {load_idx(0, 0), load_idx(0, 1)}, idx1[2] = {load_idx(1, 0), load_idx(1, 1)};
      int idx2[2] = {load_idx(2, 0), load_idx(2, 1)};
      int row0[2] = {key_row(idx0[0]), key_row(idx0[1])}, row1[2] = {key_row(idx1[0]), key_row(idx1[1])};
      float ks0[2] = {load_ks(row0[0]), load_ks(row0[1])};
      for (int t = 0; t < ntiles; ++t, ++it) {
        const int s = it % C::STAGES;
        const uint32_t ph = (it / C::STAGES) & 1;
        const int idx3[2] = {load_idx(t + 3, 0), load_idx(t + 3, 1)};
        const int row2[2] = {key_row(idx2[0]), key_row(idx2[1])};
        const float ks1[2] = {load_ks(row1[0]), load_ks(row1[1])};
        if (ok) ok = ptx::mbar_wait(&ct.empty[s], ph ^ 1, abort_flag, 64);   // whole warps wait here: sleep, do not spin
        int krow[2];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int row = wrow0 + half * 32 + lane;
          ct.meta[it % META_SLOTS][row] = KeyMeta{row0[half] < 0 ? -1 : idx0[half], ks0[half]};
          krow[half] = row0[half] < 0 ? 0 : row0[half];
          idx0[half] = idx1[half]; idx1[half] = idx2[half]; idx2[half] = idx3[half];
          row0[half] = row1[half]; row1[half] = row2[half];
          ks0[half] = ks1[half];
        }
        const uint32_t dst0 = ptx::smem_u32(kring + s * C::STAGE_BYTES);
#pragma unroll
        for (int i = 0; i < 16; ++i) {                 // four rows per pass
          const int rl = i * 4 + sub;                  // row inside this warp's 64
          const int kr = __shfl_sync(0xffffffffu, krow[i >> 3], rl & 31);
          const int row = wrow0 + rl;
          const uint8_t* src = (const uint8_t*)gd.kbase + (long long)kr * krow_bytes + chunk * 16;
          const uint32_t dst = dst0 + (uint32_t)row * 128u + (uint32_t)((chunk ^ (row & 7)) << 4);
#pragma unroll
          for (int h = 0; h < C::KHALVES; ++h) cp_async16(dst + h * C::HALF_TILE_BYTES, src + h * 128);
        }
        cp_async_commit();
        if (it + 1 - pub > (uint32_t)C::LOOKAHEAD) {
          cp_async_wait<C::LOOKAHEAD>();
          publish(pub++);
        }
      }
    }
    cp_async_wait<0>();
    while (pub < it) publish(pub++);
  } else if (C::OVL && warp >= 2 + GATHER_WARPS + EPI_WARPS) {
    // ------------------------------------------------------------------ select warps (EPI = 3)
    // Warp r takes member r's exact top-k of group n while the other warps re-score group n + 1.
    const int r = warp - (2 + GATHER_WARPS + EPI_WARPS);
    SegSelSmem& sel = ct.sel[r];
    const int RS = sc.rslots;                    // slots per score row
    const uint32_t* rk = sc.rkeys + (size_t)blockIdx.x * 2 * NMEM * RS;
    uint32_t blk = 0;
    for (int gi = blockIdx.x; gi < n_groups; gi += gridDim.x) {
      const GroupDesc gd = groups[gi];
      const int ntiles = min(group_tiles(gd), RS / TILE_KEYS);
      if (ntiles == 0) continue;
      const int kb = blk & 1;
      const uint32_t kph = (blk >> 1) & 1;
      ++blk;
      PIVOT_PROF_DO(const long long pt0 = clock64();)
      if (!ptx::mbar_wait(&ct.k_full[kb], kph, abort_flag, 64)) break;
      PIVOT_PROF_DO(const long long pt1 = clock64();)
      const uint32_t kmin = ct.kstat[kb][r][0], kmax = ct.kstat[kb][r][1], n_filled = ct.kstat[kb][r][2];
      __syncwarp();
      if (lane == 0) { ct.kstat[kb][r][0] = 0xffffffffu; ct.kstat[kb][r][1] = 0u; ct.kstat[kb][r][2] = 0u; }
      if (r < gd.m) {
        int32_t* out = gd.out + (size_t)r * gd.out_stride;
        float* outs = gd.out_score ? gd.out_score + (size_t)r * gd.out_stride : nullptr;
        const int n_valid = warp_row_topk(sel, rk + (size_t)(kb * NMEM + r) * RS, ntiles * TILE_KEYS, gd.cand,
                                          gd.n_cand, out, outs, gd.K, lane, kmin, kmax, n_filled);
        for (int i = n_valid + lane; i < gd.K; i += 32) {
          out[i] = -1;
          if (outs) outs[i] = -INFINITY;
        }
      }
      __syncwarp();
      PIVOT_PROF_DO(if (r == 0 && lane == 0) {
        prof_add(sc.status, PROF_REF_SEL_WAIT, pt1 - pt0);
        prof_add(sc.status, PROF_REF_SEL_WORK, clock64() - pt1);
        prof_add(sc.status, PROF_REF_SEL_GROUPS, 1);
      })
      if (lane == 0) ptx::mbar_arrive(&ct.k_free[kb]);     // this warp is through with the buffer
    }
  } else {
    // ------------------------------------------------------------------ epilogue + top-k
    const int ew = warp - (2 + GATHER_WARPS);
    const int team = ew >> 2;
    const int lq = warp & 3;
    const int key_in_tile = lq * 32 + lane;
    const int tt = (ew & 3) * 32 + lane;
    const Team tm{tt, 128, 1 + team};
    const Team all{ew * 32 + lane, EPI_WARPS * 32, 3};   // both teams
    SegSelSmem& sel = ct.sel[C::OVL ? 0 : team];
    const int wq = ew & 3;
    const int SEG = sc.cap >> 2;
    // per-CTA score segments: (member r, warp wq) -> cand64[cta][r][wq][0 .. SEG)
    const size_t cta_base = (size_t)blockIdx.x * NMEM * sc.cap;
    auto seg_off = [&](int r) { return cta_base + ((size_t)r * 4 + wq) * SEG; };
    uint32_t it = 0, blk = 0;
    const int RS = sc.rslots;
    uint32_t* const rk = C::OVL ? sc.rkeys + (size_t)blockIdx.x * 2 * NMEM * RS : nullptr;
    for (int gi = blockIdx.x; gi < n_groups; gi += gridDim.x) {
      const GroupDesc gd = groups[gi];
      const int ntiles = group_tiles(gd);
      if (ntiles == 0) continue;
      const int kb = blk & 1;                    // score-row buffer of this group (EPI = 3)
      const uint32_t kph = (blk >> 1) & 1;
      ++blk;
      if constexpr (C::MMA2) {
        // team 1 scores all four members (so both teams meet around the tile loop: the other team
        // selects from what it wrote) and writes the diagonal blocks of the gate matrix; the last
        // second MMA of the previous group is through (its scores have been read)
        all.sync();
        if (team == 1) {
          (void)ptx::mbar_wait(&ct.g_ready[kb], kph, abort_flag);   // staged by the query warp, usually long ago
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int i = tt + u * 128, r = i >> 6, j = i & 63;
            const float wv = ct.gstage[kb][i];
            const __nv_bfloat16 hi = __float2bfloat16_rn(wv);
            const __nv_bfloat16 lo = __float2bfloat16_rn(wv - __bfloat162float(hi));
            const uint32_t in_row = (j & 7) * 2;
            *reinterpret_cast<__nv_bfloat16*>(ct.wmat + r * 1024 + r * 128 + (((j >> 3) ^ (r & 7)) << 4) + in_row) = hi;
            *reinterpret_cast<__nv_bfloat16*>(ct.wmat + r * 1024 + (4 + r) * 128 + (((j >> 3) ^ ((4 + r) & 7)) << 4) + in_row) = lo;
          }
          ptx::fence_proxy_async_smem();         // generic-proxy writes -> tensor-core reads
          tm.sync();
          if (tt == 0) ptx::mbar_arrive(&ct.w_ready);
        }
      } else {
        tm.sync();
        const int rl = tt >> 6, jh = tt & 63;
        const int r = team * 2 + rl;
        float wv = 0.f;
        if (r < gd.m) {
          wv = gd.w[r * kHeads + jh];
          if (gd.qscale) wv = __fmul_rn(wv, gd.qscale[r * kHeads + jh]);
        }
        ct.w[r][jh] = 0.5f * wv;       // halved: see the ReLU identity in the tile loop
        tm.sync();
      }
      // One member row's result: a key never seen by the member (beyond its own position, or
      // before its own window in a chunk of per-query window slots: Appendix B) or a padding
      // slot counts as empty.
      uint32_t smn[NMEM], smx[NMEM], snv[NMEM];  // EPI = 3: this thread's share of the row statistics
#pragma unroll
      for (int r = 0; r < NMEM; ++r) { smn[r] = 0xffffffffu; smx[r] = 0u; snv[r] = 0u; }
      // (si: which of this thread's statistics slots the row uses -- a constant at every call)
      auto put = [&](int r, int si, int t, int slot, int idx, uint32_t key) {
        const int t_r = gd.first_pos + r;
        const bool seen = idx >= 0 && idx <= t_r && idx + gd.win_span > t_r;
        if constexpr (C::OVL) {        // key only, to this group's score-row buffer
          if (r < gd.m && slot < RS) {
            const uint32_t kv = seen ? key : 0u;
            rk[(size_t)(kb * NMEM + r) * RS + slot] = kv;
            smn[si] = (kv && kv < smn[si]) ? kv : smn[si];
            smx[si] = kv > smx[si] ? kv : smx[si];
            snv[si] += kv ? 1u : 0u;
          }
          return;
        }
        const entry_t e = seen ? make_entry(key, idx) : kPadEntry;
        if (gd.ent_out) {              // chunked mode: leave the entries for a later top-k
          if (r < gd.m && slot < gd.n_cand && PIVOT_BOUNDS(gd.slot0 + slot < gd.ent_stride, sc.status))
            gd.ent_out[(size_t)r * gd.ent_stride + gd.slot0 + slot] = e;
        } else if (r < gd.m && t * 32 + lane < SEG) {
          sc.cand64[seg_off(r) + t * 32 + lane] = e;   // entry t*32+lane of segment (r, lane quarter)
        }
      };
      if constexpr (C::MMA2) {
        if (team == 0) {
          // ---- ReLU warps: fp32 accumulator -> packed bf16 ReLU values, in place (thread = key)
          for (int t = 0; t < ntiles; ++t, ++it) {
            const int buf = it & 1;
            (void)ptx::mbar_wait(&ct.tmem_full[buf], (it >> 1) & 1, abort_flag);
            ptx::tc_fence_after();
            const uint32_t xb = tmem_base + ((uint32_t)(lq * 32) << 16) + buf * N;
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
              if ((c >> 1) >= gd.m) {                          // members missing from the group: zeros (warp-uniform)
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
          // ---- score warps: the four member scores of this thread's key
          if constexpr (C::OVL)        // the select warps are through with this buffer (two groups back)
            (void)ptx::mbar_wait(&ct.k_free[kb], kph ^ 1, abort_flag, 64);
          for (int t = 0; t < ntiles; ++t, ++it) {
            const int buf = it & 1;
            const int slot = t * TILE_KEYS + key_in_tile;
            (void)ptx::mbar_wait(&ct.s_ready[buf], (it >> 1) & 1, abort_flag);
            ptx::tc_fence_after();
            // position and scale of this thread's key, left in shared memory by the gather warps
            const KeyMeta mt = ct.meta[it % META_SLOTS][key_in_tile];
            uint32_t s8[8];            // columns r: sums with the gates' bf16 heads, 4 + r: with their remainders
            ptx::tmem_ld_32x8(tmem_base + ((uint32_t)(lq * 32) << 16) + buf * N + 128, s8);
            ptx::tmem_wait_ld();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ct.tmem_empty[buf]);
#pragma unroll
            for (int r = 0; r < NMEM; ++r) {
              const float sc_r = __uint_as_float(s8[r]) + __uint_as_float(s8[4 + r]);
              put(r, r, t, slot, mt.idx, score_to_key(gd.kscale ? sc_r * mt.ks : sc_r));
            }
          }
          if constexpr (C::OVL) {      // the group's score rows are complete: hand them over
#pragma unroll
            for (int r = 0; r < NMEM; ++r) {
              const uint32_t mn = __reduce_min_sync(0xffffffffu, smn[r]);
              const uint32_t mx = __reduce_max_sync(0xffffffffu, smx[r]);
              const uint32_t nv = __reduce_add_sync(0xffffffffu, snv[r]);
              if (lane == 0 && nv) {
                atomicMin(&ct.kstat[kb][r][0], mn);
                atomicMax(&ct.kstat[kb][r][1], mx);
                atomicAdd(&ct.kstat[kb][r][2], nv);
              }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ct.k_full[kb]);
          }
        }
        all.sync();
      } else {
      if constexpr (C::OVL)            // the select warps are through with this buffer (two groups back)
        (void)ptx::mbar_wait(&ct.k_free[kb], kph ^ 1, abort_flag, 64);
      for (int t = 0; t < ntiles; ++t, ++it) {
        const int buf = it & 1;
        const int slot = t * TILE_KEYS + key_in_tile;
        (void)ptx::mbar_wait(&ct.tmem_full[buf], (it >> 1) & 1, abort_flag);
        ptx::tc_fence_after();
        // position and scale of this thread's key, left in shared memory by the gather warps
        // (no global load here: it would queue behind nothing good next to the TMEM loads)
        const KeyMeta mt = ct.meta[it % META_SLOTS][key_in_tile];
        const int idx = mt.idx;
        const float ksv = mt.ks;
        float score[2];
#pragma unroll
        for (int rl = 0; rl < 2; ++rl) {
          const int r = team * 2 + rl;
          const uint32_t taddr = tmem_base + ((uint32_t)(lq * 32) << 16) + buf * N + r * kHeads;
          uint32_t v0[32], v1[32];
          ptx::tmem_ld_32x32(taddr, v0);
          ptx::tmem_ld_32x32(taddr + 32, v1);
          ptx::tmem_wait_ld();
          // w ReLU(x) = (w/2) x + (w/2) |x| (ct.w holds w/2): full-rate FMAs, eight chains
          float ap[4] = {0.f, 0.f, 0.f, 0.f}, an[4] = {0.f, 0.f, 0.f, 0.f};
          const float4* wp = reinterpret_cast<const float4*>(&ct.w[r][0]);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const float4 wa = wp[q4], wb = wp[8 + q4];
            const float x0 = __uint_as_float(v0[4 * q4]), x1 = __uint_as_float(v0[4 * q4 + 1]);
            const float x2 = __uint_as_float(v0[4 * q4 + 2]), x3 = __uint_as_float(v0[4 * q4 + 3]);
            const float y0 = __uint_as_float(v1[4 * q4]), y1 = __uint_as_float(v1[4 * q4 + 1]);
            const float y2 = __uint_as_float(v1[4 * q4 + 2]), y3 = __uint_as_float(v1[4 * q4 + 3]);
            ap[0] = fmaf(fabsf(x0), wa.x, ap[0]); an[0] = fmaf(x0, wa.x, an[0]);
            ap[1] = fmaf(fabsf(x1), wa.y, ap[1]); an[1] = fmaf(x1, wa.y, an[1]);
            ap[2] = fmaf(fabsf(x2), wa.z, ap[2]); an[2] = fmaf(x2, wa.z, an[2]);
            ap[3] = fmaf(fabsf(x3), wa.w, ap[3]); an[3] = fmaf(x3, wa.w, an[3]);
            ap[0] = fmaf(fabsf(y0), wb.x, ap[0]); an[0] = fmaf(y0, wb.x, an[0]);
            ap[1] = fmaf(fabsf(y1), wb.y, ap[1]); an[1] = fmaf(y1, wb.y, an[1]);
            ap[2] = fmaf(fabsf(y2), wb.z, ap[2]); an[2] = fmaf(y2, wb.z, an[2]);
            ap[3] = fmaf(fabsf(y3), wb.w, ap[3]); an[3] = fmaf(y3, wb.w, an[3]);
          }
          score[rl] = ((ap[0] + an[0]) + (ap[1] + an[1])) + ((ap[2] + an[2]) + (ap[3] + an[3]));
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ct.tmem_empty[buf]);
#pragma unroll
        for (int rl = 0; rl < 2; ++rl)
          put(team * 2 + rl, rl, t, slot, idx, score_to_key(gd.kscale ? score[rl] * ksv : score[rl]));
      }
      if constexpr (C::OVL) {          // this warp's share of its team's two score rows is complete
#pragma unroll
        for (int rl = 0; rl < 2; ++rl) {
          const int r = team * 2 + rl;
          const uint32_t mn = __reduce_min_sync(0xffffffffu, smn[rl]);
          const uint32_t mx = __reduce_max_sync(0xffffffffu, smx[rl]);
          const uint32_t nv = __reduce_add_sync(0xffffffffu, snv[rl]);
          if (lane == 0 && nv) {
            atomicMin(&ct.kstat[kb][r][0], mn);
            atomicMax(&ct.kstat[kb][r][1], mx);
            atomicAdd(&ct.kstat[kb][r][2], nv);
          }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ct.k_full[kb]);
      }
      tm.sync();
      }
      if (gd.ent_out || C::OVL) continue;
      // ---- per-member exact top-k over the candidate scores
#pragma unroll
      for (int rl = 0; rl < 2; ++rl) {
        const int r = team * 2 + rl;
        if (r >= gd.m) continue;
        int32_t* out = gd.out + (size_t)r * gd.out_stride;
        float* outs = gd.out_score ? gd.out_score + (size_t)r * gd.out_stride : nullptr;
        const int segcnt = min(ntiles * 32, SEG);
        const Seg seg{sc.cand64 + seg_off(r), segcnt};
        // 32 entries per lane (c <= 4096) fit the registers this kernel has; beyond that re-read
        const int n_valid = segcnt <= 32 * 32 ? seg_emit<true, 32>(tm, sel, seg, gd.n_cand, out, outs, gd.K)
                                              : seg_emit<false>(tm, sel, seg, gd.n_cand, out, outs, gd.K);
        for (int i = n_valid + tt; i < gd.K; i += 128) {
          out[i] = -1;
          if (outs) outs[i] = -INFINITY;
        }
        tm.sync();
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  if (threadIdx.x == 0 && ct.abort) set_status(sc.status, DEV_WAIT_EXPIRED);
}

template <int DT, int EPI = 1>
cudaError_t launch_one(const CUtensorMap& mq, const GroupDesc* groups, int n_groups, int q_rows,
                       const ScanScratch& s, int sms, cudaStream_t st, bool overlap_prev = false) {
  auto kern = refine_tc_kernel<DT, EPI>;
  static bool attr_set[kMaxDevices] = {};
  const size_t smem = rsmem_bytes<DT, EPI>();
  if (cudaError_t e = opt_in_dynamic_smem(kern, smem, attr_set); e != cudaSuccess) return e;
  const int grid = n_groups < sms ? n_groups : sms;
  ++launch_counter();
  return launch_kernel(kern, dim3(grid), dim3(RCfg<DT, EPI>::THREADS), smem, st, overlap_prev, mq, groups, n_groups, q_rows, s);
}

}  // namespace

bool make_operand_map(CUtensorMap* m, const void* base, long long rows, int dtype, int box_rows, int row_stride);

cudaError_t launch_refine_tc(const void* q, int q_rows, int dtype, const GroupDesc* groups, int n_groups,
                             const ScanScratch& s, int sms, cudaStream_t st, bool fp32_head_sum, bool chunked,
                             int max_cand, bool overlap_prev) {
  if (n_groups <= 0) return cudaSuccess;
  CUtensorMap mq;
  if (!make_operand_map(&mq, q, (long long)q_rows * kHeads, dtype, kHeads, 0)) return cudaErrorInvalidValue;
  // the select warps need the caller's score-row buffers, long enough for every group
  const bool rows_ok = s.rkeys && max_cand > 0 && max_cand <= s.rslots;
  if (dtype != DT_FP8)
    return rows_ok && !chunked ? launch_one<DT_BF16, 3>(mq, groups, n_groups, q_rows, s, sms, st)
                               : launch_one<DT_BF16>(mq, groups, n_groups, q_rows, s, sms, st);
  if (fp32_head_sum) return launch_one<DT_FP8, 0>(mq, groups, n_groups, q_rows, s, sms, st);
  if (chunked) return launch_one<DT_FP8, 2>(mq, groups, n_groups, q_rows, s, sms, st, overlap_prev);
  if (!rows_ok) return cudaErrorInvalidValue;
  return launch_one<DT_FP8, 3>(mq, groups, n_groups, q_rows, s, sms, st);
}

}  // namespace pivot
