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
