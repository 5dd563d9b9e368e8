// Shared device helpers: score <-> order-preserving key, operand decoding, status word.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pivot {

constexpr int kHeads = 64;     // H_I
constexpr int kDim = 128;      // d
constexpr int DT_BF16 = 0;
constexpr int DT_FP8 = 1;

// Device status word values (first non-zero wins).
constexpr int DEV_OK = 0;
constexpr int DEV_WAIT_EXPIRED = 1;   // a bounded barrier wait ran out
constexpr int DEV_CAND_OVERFLOW = 2;  // a candidate buffer would have overflowed (logic error)
constexpr int DEV_BAD_POS = 3;        // decode: a sequence's pos0 lies outside [0, Lmax - g]; its rows are all -1
constexpr int DEV_BOUNDS = 4;         // PIVOT_DEBUG builds: an index, page or cursor failed its bounds check (access skipped)

// Cycle counters of a -DPIVOT_PROF build (the figures the profiles quote): 64-bit slots in the
// workspace head, behind the status word and the row counter (ints 8 .. 63), summed over all CTAs
// and calls until pivot_debug_counters reads and clears them.  An ordinary build has none of it.
enum ProfSlot {
  PROF_SCAN_WAIT_QUERIES = 0,   // shared scan, MMA-issuing thread: clocks waiting for the block's queries,
  PROF_SCAN_WAIT_ACC,           //   a free accumulator buffer,
  PROF_SCAN_WAIT_KEYS,          //   the key tile,
  PROF_SCAN_WAIT_GATES,         //   the block's gate matrix,
  PROF_SCAN_WAIT_RELU,          //   the packed ReLU operand of the second MMA,
  PROF_SCAN_TOTAL,              //   its whole loop; and
  PROF_SCAN_TILES,              //   tiles it issued
  PROF_REF_WAIT_QUERIES,        // re-score, MMA-issuing thread: the same seven
  PROF_REF_WAIT_ACC,
  PROF_REF_WAIT_KEYS,
  PROF_REF_WAIT_GATES,
  PROF_REF_WAIT_RELU,
  PROF_REF_TOTAL,
  PROF_REF_TILES,
  PROF_REF_SEL_WAIT,            // re-score, select warp of member 0: clocks waiting for a group's score rows,
  PROF_REF_SEL_WORK,            //   selecting; and
  PROF_REF_SEL_GROUPS,          //   groups selected
  PROF_DSEL_BOUNDARY,           // decode select, the CTA that takes the top-c: boundary bin off the histogram,
  PROF_DSEL_COLLECT,            //   collecting its share of the scores,
  PROF_DSEL_HANDOVER,           //   cluster barriers + reading the other CTAs' lists,
  PROF_DSEL_TOPK,               //   exact top-c of the collected entries; and
  PROF_DSEL_SEQS,               //   sequences
  PROF_DSCAN_PRODUCER_WAIT,     // decode scan: the key-TMA thread waiting for a free stage,
  PROF_DSCAN_MAX_TOTAL,         //   the MMA-issuing thread: the longest whole loop of any CTA (a maximum, not a sum),
  PROF_DSCAN_WAIT_ACC,          //   a free accumulator buffer,
  PROF_DSCAN_WAIT_KEYS,         //   the key tile,
  PROF_DSCAN_TOTAL,             //   its whole loop (from the end of the kernel's set-up); and
  PROF_DSCAN_TILES,             //   tiles
  PROF_SLOTS
};
static_assert(PROF_SLOTS <= 28, "the workspace head holds 28 counters");
#ifdef PIVOT_PROF
__device__ __forceinline__ void prof_add(int* status, int slot, long long v) {
  if (status) atomicAdd(reinterpret_cast<unsigned long long*>(status + 8) + slot, (unsigned long long)v);
}
__device__ __forceinline__ void prof_max(int* status, int slot, long long v) {
  if (status) atomicMax(reinterpret_cast<unsigned long long*>(status + 8) + slot, (unsigned long long)v);
}
#define PIVOT_PROF_DO(...) __VA_ARGS__
#else
#define PIVOT_PROF_DO(...)
#endif

// fp32 score -> uint32 key whose unsigned order equals the float order (-inf lowest).
__device__ __forceinline__ uint32_t score_to_key(float s) {
  uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_to_score(uint32_t k) {
  uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(b);
}

__device__ __forceinline__ float e4m3_to_float(uint8_t c) {
  __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
  return __half2float(__half(h));
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float(((uint32_t)b) << 16);
}

__device__ __forceinline__ void set_status(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// Checked build (-DPIVOT_DEBUG): indices the kernels derive themselves -- gathered candidate
// positions, block-table entries, score / entry slots -- are tested before use; a failed test
// records DEV_BOUNDS in the status word and the access is skipped.  Nothing traps.  (Positions
// that come from the caller are tested in every build.)
#ifdef PIVOT_DEBUG
__device__ __forceinline__ bool bounds_ok(bool ok, int* status) {
  if (!ok) set_status(status, DEV_BOUNDS);
  return ok;
}
#define PIVOT_BOUNDS(cond, status) ::pivot::bounds_ok((cond), (status))
#else
#define PIVOT_BOUNDS(cond, status) (true)
#endif

// One row of a scan: a (proxy or raw) query of H x d codes, its gates, and where the
// selection goes.  Filled by the host-side planner kernels.
struct RowDesc {
  const void* q;        // [H, d] codes
  const float* w;       // [H] gate
  const float* qscale;  // [H] or nullptr: effective gate = w * qscale (fp32 multiply)
  const void* kbase;    // key cache of this row's sequence [*, d]
  const float* kscale;  // [*] or nullptr
  int n_vis;            // keys 0 .. n_vis-1 are visible
  int K;                // entries to select
  int32_t* out;         // K entries (x out_rows copies, out_stride apart); -1 padded
  float* out_score;     // optional, same layout
  int out_rows;
  int out_stride;
  int q_map;            // which query tensor map holds q: 0 raw queries, 1 proxies
  int q_row;            // query row (units of H x d) inside that tensor
  int k_row0;           // first row of this sequence's keys inside the key-cache tensor
  // Paged key cache (decode): key tile t of this row is pool page pages[t]; nullptr = contiguous.
  const int32_t* pages = nullptr;
};

}  // namespace pivot
