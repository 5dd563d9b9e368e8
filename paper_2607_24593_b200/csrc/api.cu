// C ABI of the library (see include/pivot.h): argument checks, workspace carving, and the
// launch sequence of Algorithm 1 -- proxy build (Eq. 4), planner, shared scan + streaming
// select (Eq. 5-7), gather + re-score + top-k (Eq. 8-9).
#include <stdio.h>
#include <string.h>

#include "../../include/pivot.h"
#include "api_internal.h"
#include "kernels.h"

using namespace pivot;

namespace {

constexpr int kMaxSel = 8192;
constexpr int kMaxDevices = 64;

#ifndef PIVOT_HOST_CHUNKS
#define PIVOT_HOST_CHUNKS 7
#endif
constexpr int kHostChunks = PIVOT_HOST_CHUNKS;   // query-row chunks of the host-buffer prefill pipeline

struct DeviceState {
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int sm_count = 0;
  int* last_status = nullptr;
  // host-buffer prefill: copy streams and events, created on first use
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_entry = nullptr, ev_in[kHostChunks + 2] = {}, ev_done[kHostChunks + 2] = {};
  // stage-timing events (created on this device on first use) and what the last call recorded
  cudaEvent_t ev[9] = {};
  bool ev_valid = false, ev_decode_scan = false;
};
DeviceState g_dev[kMaxDevices];
int g_last_cuda = 0;

int cur_device() {
  int d = 0;
  cudaGetDevice(&d);
  return (d >= 0 && d < kMaxDevices) ? d : 0;
}

int sm_count() {
  DeviceState& ds = g_dev[cur_device()];
  if (ds.sm_count == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, cur_device()) != cudaSuccess || n <= 0)
      n = 148;
    ds.sm_count = n;
  }
  return ds.sm_count;
}

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

int cand_cap(int kmax) {
  int cap = 2 * kmax;
  if (cap < kmax + 1024) cap = kmax + 1024;
  return (int)align_up((size_t)cap, 64);
}

#ifndef PIVOT_CAP_FACTOR
#define PIVOT_CAP_FACTOR 8
#endif
int tc_cap(int kmax) {
  size_t cap = (size_t)PIVOT_CAP_FACTOR * kmax;     // a tight running threshold admits about K (1 + ln(n / K)) entries
  if (cap < 8192) cap = 8192;
  return (int)align_up(cap, 256);
}

struct Carve {
  char* base;
  size_t off = 0;
  explicit Carve(void* p) : base((char*)p) {}
  template <typename T>
  T* take(size_t n) {
    T* p = (T*)(base + off);
    off = align_up(off + n * sizeof(T));
    return p;
  }
};

struct Workspace {
  int tc_cap;
  int* status;
  int* counter;
  void* proxy_q;
  float* proxy_w;
  int32_t* cand;
  RowDesc* rows;
  GroupDesc* groups;
  ScanScratch scan;
  size_t bytes;
};

// rows: scan-row slots; n_groups: groups (proxy rows / Refine groups).
Workspace carve_workspace(void* base, int rows, int n_groups, int c, int k) {
  Workspace w;
  Carve cv(base);
  const int kmax = c > k ? c : k;
  int* head = cv.take<int>(64);
  w.status = head;
  w.counter = head + 1;
  w.proxy_q = cv.take<uint16_t>((size_t)n_groups * kHeads * kDim);
  w.proxy_w = cv.take<float>((size_t)n_groups * kHeads);
  w.cand = cv.take<int32_t>((size_t)n_groups * c);
  w.rows = cv.take<RowDesc>((size_t)rows + n_groups);
  w.groups = cv.take<GroupDesc>((size_t)rows + n_groups);   // up to ceil(g/4) chunks per group
  // Candidate scratch.  Tensor-core kernels: one CTA per SM, 4 rows x cap packed entries each,
  // cap = 8 K (a tight running threshold admits about K (1 + ln(n / K)) entries per row; one
  // segment per epilogue warp, each able to hold K).
  // CUDA-core kernels: 4 CTAs per SM, two buffers of 2 K (key, index) pairs each.  The
  // region is sized for the larger of the two and shared.
  w.scan.n_cta = sm_count() * 4;
  w.scan.cap = cand_cap(kmax);
  w.tc_cap = tc_cap(kmax);
  const size_t simt_entries = (size_t)w.scan.n_cta * 2 * w.scan.cap;
  const size_t tc_entries = (size_t)sm_count() * 4 * 2 * w.tc_cap;     // two segments per row (alternate blocks)
  w.scan.cand64 = cv.take<unsigned long long>(simt_entries > tc_entries ? simt_entries : tc_entries);
  w.scan.cand_key = (uint32_t*)w.scan.cand64;
  w.scan.cand_idx = (int32_t*)w.scan.cand64 + simt_entries;
  w.scan.status = w.status;
  w.scan.counter = w.counter;
  w.scan.rslots = (c + 127) / 128 * 128;
  w.scan.rkeys = cv.take<uint32_t>((size_t)sm_count() * 2 * 4 * w.scan.rslots);
  w.bytes = cv.off;
  return w;
}

// The scratch as the tensor-core kernels see it: per-row capacity of packed entries.
ScanScratch tc_scratch(const Workspace& ws) {
  ScanScratch s = ws.scan;
  s.cap = ws.tc_cap;
  return s;
}

bool g_timing = false;
// Events belong to the device that was current when they were created: one set per device.
cudaEvent_t* timing_events() {
  DeviceState& ds = g_dev[cur_device()];
  if (!ds.ev[0])
    for (int i = 0; i < 9; ++i)
      if (cudaEventCreate(&ds.ev[i]) != cudaSuccess) { ds.ev[0] = nullptr; return nullptr; }
  return ds.ev;
}
inline void mark(int i, cudaStream_t st) {
  if (!g_timing) return;
  cudaEvent_t* ev = timing_events();
  if (!ev) return;
  cudaEventRecord(ev[i], st);
  if (i == 4) g_dev[cur_device()].ev_valid = true;
}

inline int check_cuda(cudaError_t e) { return pivot::record_cuda(e); }
inline int check_common(const pivot_tensor* q, const float* w, const pivot_tensor* kc, int H, int d, int c,
                        int k, int mode, const void* out) {
  return pivot::check_operands(q, w, kc, H, d, c, k, mode, out);
}

}  // namespace

namespace pivot {

int record_cuda(cudaError_t e) {
  if (e == cudaSuccess) return PIVOT_OK;
  g_last_cuda = (int)e;
  return PIVOT_ERR_CUDA;
}

int check_operands(const pivot_tensor* q, const float* w, const pivot_tensor* kc, int H, int d, int c,
                   int k, int mode, const void* out) {
  if (!q || !w || !kc || !out || !q->data || !kc->data) return PIVOT_ERR_INVALID_ARG;
  if (q->dtype != kc->dtype) return PIVOT_ERR_INVALID_ARG;
  if (q->dtype != PIVOT_BF16 && q->dtype != PIVOT_FP8_E4M3) return PIVOT_ERR_INVALID_ARG;
  if (q->dtype == PIVOT_FP8_E4M3 && (!q->scale || !kc->scale)) return PIVOT_ERR_INVALID_ARG;
  if (k < 1 || c < 1) return PIVOT_ERR_INVALID_ARG;
  if (mode != PIVOT_REUSE && mode != PIVOT_REFINE) return PIVOT_ERR_INVALID_ARG;
  if (mode == PIVOT_REFINE && k > c) return PIVOT_ERR_INVALID_ARG;
  if (((uintptr_t)q->data | (uintptr_t)kc->data) & 15) return PIVOT_ERR_INVALID_ARG;
  if (((uintptr_t)w | (uintptr_t)out | (uintptr_t)q->scale) & 3) return PIVOT_ERR_INVALID_ARG;
  if ((uintptr_t)kc->scale & 15) return PIVOT_ERR_INVALID_ARG;
  if (H != kHeads || d != kDim) return PIVOT_ERR_UNSUPPORTED;
  if (k > kMaxSel || c > kMaxSel) return PIVOT_ERR_UNSUPPORTED;
  // rows: queries dense; key rows dense or padded to a multiple of 16 bytes (below 2^31)
  const size_t row = (size_t)kDim * (q->dtype == PIVOT_FP8_E4M3 ? 1 : 2);
  if (q->stride_row != 0 && q->stride_row != (size_t)kHeads * row && q->stride_row != row) return PIVOT_ERR_UNSUPPORTED;
  if (kc->stride_row != 0 && (kc->stride_row < row || (kc->stride_row & 15) || kc->stride_row > (1u << 30)))
    return PIVOT_ERR_INVALID_ARG;
  return PIVOT_OK;
}

}  // namespace pivot

namespace {

// Bytes between key rows as the kernels take it: 0 for a dense cache.
int key_stride(const pivot_tensor* kc) {
  const size_t row = (size_t)kDim * (kc->dtype == PIVOT_FP8_E4M3 ? 1 : 2);
  return kc->stride_row == 0 || kc->stride_row == row ? 0 : (int)kc->stride_row;
}

int resolve_ws(const pivot_opts* o, size_t need, void** ws) {
  void* p = o && o->workspace ? o->workspace : g_dev[cur_device()].ws;
  size_t n = o && o->workspace ? o->workspace_bytes : g_dev[cur_device()].ws_bytes;
  if (!p || n < need || ((uintptr_t)p & 255)) return PIVOT_ERR_WORKSPACE;
  *ws = p;
  return PIVOT_OK;
}

int run_prefill(const pivot_tensor* q, const float* w, const pivot_tensor* kc, int L, int g, int c,
                int k, int mode, bool dense_only, int32_t* out_idx, cudaStream_t st,
                const pivot_opts* o) {
  const int nG = (L + g - 1) / g;
  const size_t need = pivot_workspace_bytes(L, nG, c, k);
  void* wsp = nullptr;
  int rc = resolve_ws(o, need, &wsp);
  if (rc) return rc;
  Workspace ws = carve_workspace(wsp, L, nG, c, k);
  g_dev[cur_device()].last_status = ws.status;

  int guard = (o && o->guard_len >= 0) ? o->guard_len : c;
  int first_group = guard <= 1 ? 0 : (guard - 1 + g - 1) / g;
  if (first_group > nG) first_group = nG;
  if (dense_only) first_group = nG;
  long long nd = (long long)first_group * g;      // rows below nd are scored densely
  if (nd > L) nd = L;
  // optional row range (chunked prefill): groups never straddle a chunk boundary
  int r0 = 0, r1 = L;
  if (o && (o->row_begin || o->row_end)) {
    r0 = o->row_begin; r1 = o->row_end;
    if (r0 < 0 || r1 <= r0 || r1 > L || r0 % g || (r1 % g && r1 != L)) return PIVOT_ERR_INVALID_ARG;
  }
  // local window (Appendix B): needs room in the candidate set and a scan of at least one key
  const int W = (o && !dense_only) ? o->W : 0;
  if (W < 0) return PIVOT_ERR_INVALID_ARG;
  if (W > 0 && (W + g - 1 >= c || guard < W + g || (o && o->impl == 1))) return PIVOT_ERR_INVALID_ARG;
  const int g_begin = r0 / g, g_end = (r1 + g - 1) / g;
  const int dense0 = r0 < nd ? r0 : (int)nd;
  const int dense1 = r1 < nd ? r1 : (int)nd;
  const int pg0 = g_begin > first_group ? g_begin : first_group;   // first proxy group of this call
  PrefillPlan p;
  p.q = q->data; p.w = w; p.qscale = q->scale;
  p.kc = kc->data; p.kscale = kc->scale;
  p.k_stride = key_stride(kc);
  if (p.k_stride && o && o->impl == 1) return PIVOT_ERR_UNSUPPORTED;
  p.proxy_q = ws.proxy_q; p.proxy_w = ws.proxy_w;
  p.cand = (o && o->dbg_cand) ? o->dbg_cand + (size_t)pg0 * c : ws.cand;
  p.cand_score = (o && o->dbg_cand_scores) ? o->dbg_cand_scores + (size_t)pg0 * c : nullptr;
  p.out = out_idx; p.out_score = o ? o->dbg_scores : nullptr;
  p.L = L; p.g = g; p.c = c; p.k = k; p.mode = mode; p.dtype = q->dtype;
  p.W = W;
  p.dense_begin = dense0;
  p.n_dense = dense1 - dense0;
  p.first_group = pg0;
  p.n_proxy = g_end > pg0 ? g_end - pg0 : 0;

  if ((rc = check_cuda(cudaMemsetAsync(ws.status, 0, 2 * sizeof(int), st)))) return rc;
  mark(0, st);
  launch_proxy_build(q->data, q->scale, w, ws.proxy_q, ws.proxy_w, L, g, pg0, p.n_proxy,
                     q->dtype, o ? o->pool : 0, st);
  mark(1, st);
  launch_plan_prefill(p, ws.rows, ws.groups, st);
  mark(2, st);
  if (o && o->impl == 1) {
    launch_scan_simt(ws.rows, p.n_dense + p.n_proxy, q->dtype, ws.scan, st);
  } else {
    ScanOperands op{kc->data, L, kc->scale, q->data, L, ws.proxy_q, p.n_proxy, q->dtype};
    op.k_stride = p.k_stride;
    if ((rc = check_cuda(launch_scan_tc(op, ws.rows, p.n_dense + p.n_proxy, 4, tc_scratch(ws), sm_count(), st,
                                        o && o->impl == 2))))
      return rc;
  }
  mark(3, st);
  if (mode == PIVOT_REFINE) {
    const int nd = p.n_proxy * group_chunks(g);
    if (o && o->impl == 1) launch_refine_simt(ws.groups, nd, q->dtype, ws.scan, st);
    else if ((rc = check_cuda(launch_refine_tc(q->data, L, q->dtype, ws.groups, nd, tc_scratch(ws), sm_count(), st,
                                               o && o->impl == 2, false, c))))
      return rc;
  }
  mark(4, st);
  return check_cuda(cudaGetLastError());
}

}  // namespace

extern "C" {

size_t pivot_workspace_bytes(int rows, int n_groups, int c, int k) {
  if (rows < 1 || n_groups < 1 || c < 1 || k < 1) return 0;
  return carve_workspace(nullptr, rows, n_groups, c, k).bytes;
}

size_t pivot_decode_workspace_bytes(int B, int Lmax, int g, int c, int k) {
  if (B < 1 || Lmax < 1 || g < 1 || c < 1 || k < 1) return 0;
  return pivot_workspace_bytes(B * g, B, c, k) + decode_fast_bytes(B, Lmax, g, c);
}

int pivot_set_workspace(void* workspace, size_t bytes) {
  if (workspace && ((uintptr_t)workspace & 255)) return PIVOT_ERR_INVALID_ARG;
  DeviceState& ds = g_dev[cur_device()];
  ds.ws = workspace;
  ds.ws_bytes = workspace ? bytes : 0;
  return PIVOT_OK;
}

int pivot_index_prefill_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L,
                           int H_I, int d, int g, int c, int k, int mode, int32_t* out_idx,
                           pivot_stream_t stream, const pivot_opts* opts) {
  int rc = check_common(q, w, kcache, H_I, d, c, k, mode, out_idx);
  if (rc) return rc;
  if (L < 1 || g < 1) return PIVOT_ERR_INVALID_ARG;
  if (opts && (opts->pool < 0 || opts->pool > 2 || opts->impl < 0 || opts->impl > 2))
    return PIVOT_ERR_INVALID_ARG;
  return run_prefill(q, w, kcache, L, g, c, k, mode, false, out_idx, (cudaStream_t)stream, opts);
}

int pivot_index_prefill(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L,
                        int H_I, int d, int g, int c, int k, int mode, int32_t* out_idx,
                        pivot_stream_t stream) {
  return pivot_index_prefill_ex(q, w, kcache, L, H_I, d, g, c, k, mode, out_idx, stream, nullptr);
}

int pivot_index_prefill_varlen(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                               const int32_t* cu_seqlens, int n_req, int H_I, int d, int g, int c, int k,
                               int mode, int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts) {
  int rc = check_common(q, w, kcache, H_I, d, c, k, mode, out_idx);
  if (rc) return rc;
  if (!cu_seqlens || n_req < 1 || g < 1 || cu_seqlens[0] != 0) return PIVOT_ERR_INVALID_ARG;
  if (opts && (opts->row_begin || opts->row_end || opts->dbg_cand || opts->dbg_scores || opts->dbg_cand_scores))
    return PIVOT_ERR_INVALID_ARG;
  const bool fp8 = q->dtype == PIVOT_FP8_E4M3;
  for (int i = 0; i < n_req; ++i) {
    if (cu_seqlens[i + 1] < cu_seqlens[i]) return PIVOT_ERR_INVALID_ARG;
    if (fp8 && (cu_seqlens[i] & 3)) return PIVOT_ERR_INVALID_ARG;
  }
  const size_t esz = fp8 ? 1 : 2;
  for (int i = 0; i < n_req; ++i) {
    const size_t r0 = (size_t)cu_seqlens[i];
    const int L = cu_seqlens[i + 1] - cu_seqlens[i];
    if (L == 0) continue;
    const size_t krow = kcache->stride_row ? kcache->stride_row : (size_t)d * esz;
    pivot_tensor tq{(const char*)q->data + r0 * H_I * d * esz, q->scale ? q->scale + r0 * H_I : nullptr, q->dtype, 0};
    pivot_tensor tk{(const char*)kcache->data + r0 * krow, kcache->scale ? kcache->scale + r0 : nullptr, q->dtype, kcache->stride_row};
    rc = pivot_index_prefill_ex(&tq, w + r0 * H_I, &tk, L, H_I, d, g, c, k, mode, out_idx + r0 * k, stream, opts);
    if (rc) return rc;
  }
  return PIVOT_OK;
}

int dense_index_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L, int H_I,
                   int d, int k, int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts) {
  int rc = check_common(q, w, kcache, H_I, d, k, k, PIVOT_REUSE, out_idx);
  if (rc) return rc;
  if (L < 1) return PIVOT_ERR_INVALID_ARG;
  return run_prefill(q, w, kcache, L, 1, k, k, PIVOT_REUSE, true, out_idx, (cudaStream_t)stream, opts);
}

int dense_index(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L, int H_I,
                int d, int k, int32_t* out_idx, pivot_stream_t stream) {
  return dense_index_ex(q, w, kcache, L, H_I, d, k, out_idx, stream, nullptr);
}

// One MTP decode step.  block_table == nullptr: kcache is [B, Lmax, d]; otherwise kcache is a
// pool of n_pages pages of 128 keys and block_table [B, Lmax / 128] names each sequence's pages.
static int run_decode(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, const int32_t* pos0,
                      int B, int Lmax, int H_I, int d, int g, int c, int k, int mode, int32_t* out_idx,
                      pivot_stream_t stream, const pivot_opts* o, const int32_t* block_table, int n_pages,
                      int dense_share = 0) {
  // dense_share > 0: the dense control -- B counts the step's queries, each planned as a sequence
  // of one member (g = 1) scanned with its own raw query; dense_share of them share a key cache
  int rc = check_common(q, w, kcache, H_I, d, c, k, mode, out_idx);
  if (rc) return rc;
  if (!pos0 || B < 1 || g < 1 || Lmax < g || Lmax < dense_share) return PIVOT_ERR_INVALID_ARG;
  // every sequence's scale row must start on a 16-byte boundary (TMA reads it in 128-scale tiles)
  if (q->dtype == PIVOT_FP8_E4M3 && (Lmax & 3)) return PIVOT_ERR_INVALID_ARG;
  if (o && (o->pool < 0 || o->pool > 2)) return PIVOT_ERR_INVALID_ARG;
  // local window, decode form (Appendix B): every query adds its own last W positions to the
  // pool, so W must cover the step (W >= g); Refine only
  const int W = o ? o->W : 0;
  if (W < 0 || (W > 0 && (mode != PIVOT_REFINE || W < g || W + g - 1 > kDecodeWinMax || o->impl == 1)))
    return PIVOT_ERR_INVALID_ARG;
  const int32_t* cand_in = o ? o->cand_in : nullptr;
  if (cand_in && (mode != PIVOT_REFINE || o->impl == 1 || dense_share || ((uintptr_t)cand_in & 3))) return PIVOT_ERR_INVALID_ARG;
  const bool paged = block_table != nullptr;
  if (paged && (n_pages < 1 || (Lmax & 127) || (o && o->impl == 1))) return PIVOT_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t base_bytes = pivot_workspace_bytes(B * g, B, c, k);
  const size_t need = base_bytes + decode_fast_bytes(B, Lmax, g, c);
  void* wsp = nullptr;
  if ((rc = resolve_ws(o, need, &wsp))) return rc;
  Workspace ws = carve_workspace(wsp, B * g, B, c, k);
  g_dev[cur_device()].last_status = ws.status;
  DecodePlan p;
  p.q = q->data; p.w = w; p.qscale = q->scale;
  p.kc = kcache->data; p.kscale = kcache->scale;
  p.k_stride = key_stride(kcache);
  if (p.k_stride && o && o->impl == 1) return PIVOT_ERR_UNSUPPORTED;
  p.pos0 = pos0;
  p.proxy_q = ws.proxy_q; p.proxy_w = ws.proxy_w;
  p.cand = cand_in ? const_cast<int32_t*>(cand_in) : (o && o->dbg_cand) ? o->dbg_cand : ws.cand;
  p.cand_score = (o && !cand_in) ? o->dbg_cand_scores : nullptr;
  p.out = out_idx; p.out_score = o ? o->dbg_scores : nullptr;
  p.B = B; p.Lmax = Lmax; p.g = g; p.c = c; p.k = k; p.mode = mode; p.dtype = q->dtype;
  p.guard_len = (o && o->guard_len >= 0) ? o->guard_len : c;
  // Paged: a short sequence's dense rows would need a contiguous prefix, so the guardrail is
  // off and short sequences take the proxy path with every visible key as a candidate.
  if (paged || dense_share) p.guard_len = 0;
  if (dense_share) { p.kv_share = dense_share; p.raw_q = true; }
  p.block_table = block_table;
  p.n_pages = n_pages;
  p.status = ws.status;
  p.W = W;
  const long long k_rows = paged ? (long long)n_pages * 128 : (long long)(dense_share ? B / dense_share : B) * Lmax;
  if ((rc = check_cuda(cudaMemsetAsync(ws.status, 0, 2 * sizeof(int), st)))) return rc;   // status, row counter
  mark(0, st);
  if (!dense_share && o && o->impl == 1)       // the tensor-core path builds the proxies inside its prepare kernel
    launch_proxy_build(q->data, q->scale, w, ws.proxy_q, ws.proxy_w, B * g, g, 0, B, q->dtype, o->pool, st);
  mark(1, st);
  if (o && o->impl == 1) launch_plan_decode(p, ws.rows, ws.groups, st);   // the tensor-core path plans inside its prepare kernel
  mark(2, st);
  if (o && o->impl == 1) {
    launch_scan_simt(ws.rows, B + B * g, q->dtype, ws.scan, st);
  } else {
    // proxy rows: key-tile-split scan, per-sequence select, chunked re-score, final top-k
    DecodeFast df;
    df.plan = p; df.pool = o ? o->pool : 0;
    df.prox = ws.rows; df.groups = ws.groups;
    df.kc = kcache->data; df.kscale = kcache->scale; df.q = q->data; df.proxy_q = dense_share ? q->data : ws.proxy_q;
    df.B = B; df.Lmax = Lmax; df.g = g; df.c = c; df.k = k; df.mode = mode; df.dtype = q->dtype;
    df.k_rows = k_rows;
    df.k_stride = p.k_stride;
    df.W = W;
    df.skip_scan = cand_in != nullptr;
    df.sms = sm_count();
    df.scratch = (char*)wsp + base_bytes;
    df.scratch_tc = tc_scratch(ws);
    df.status = ws.status;
    cudaEvent_t* tev = g_timing ? timing_events() : nullptr;
    df.ev_scan_begin = tev ? tev[6] : nullptr;
    df.ev_scan_end = tev ? tev[7] : nullptr;
    df.ev_select_end = tev ? tev[8] : nullptr;
    g_dev[cur_device()].ev_decode_scan = tev != nullptr;
    if ((rc = check_cuda(launch_decode_fast(df, st)))) return rc;
    // dense rows of guarded (short) sequences, if any: the generic scan, one row per block
    if (!paged) {
      ScanOperands op{kcache->data, k_rows, kcache->scale, q->data, B * g, ws.proxy_q, B, q->dtype};
      op.k_stride = p.k_stride;
      if ((rc = check_cuda(launch_scan_tc(op, ws.rows + B, B * g, 1, tc_scratch(ws), sm_count(), st)))) return rc;
    }
  }
  mark(3, st);
  if (mode == PIVOT_REFINE && o && o->impl == 1) {
    launch_refine_simt(ws.groups, B * group_chunks(g), q->dtype, ws.scan, st);
  }
  mark(4, st);
  return check_cuda(cudaGetLastError());
}

int pivot_index_decode_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                          const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int c, int k,
                          int mode, int32_t* out_idx, pivot_stream_t stream, const pivot_opts* o) {
  return run_decode(q, w, kcache, pos0, B, Lmax, H_I, d, g, c, k, mode, out_idx, stream, o, nullptr, 0);
}

int pivot_index_decode_paged(const pivot_tensor* q, const float* w, const pivot_tensor* kpages,
                             const int32_t* block_table, const int32_t* pos0, int B, int max_pages,
                             int n_pages, int H_I, int d, int g, int c, int k, int mode, int32_t* out_idx,
                             pivot_stream_t stream, const pivot_opts* o) {
  if (!block_table || max_pages < 1 || max_pages > (1 << 23)) return PIVOT_ERR_INVALID_ARG;
  return run_decode(q, w, kpages, pos0, B, max_pages * 128, H_I, d, g, c, k, mode, out_idx, stream, o,
                    block_table, n_pages);
}

int pivot_index_decode(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                       const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int c, int k,
                       int mode, int32_t* out_idx, pivot_stream_t stream) {
  return pivot_index_decode_ex(q, w, kcache, pos0, B, Lmax, H_I, d, g, c, k, mode, out_idx, stream,
                               nullptr);
}

int dense_index_decode_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, const int32_t* pos0,
                          int B, int Lmax, int H_I, int d, int g, int k, int32_t* out_idx, pivot_stream_t stream,
                          const pivot_opts* o) {
  if (B < 1 || g < 1 || (long long)B * g > (1 << 24)) return PIVOT_ERR_INVALID_ARG;
  if (o && (o->impl == 1 || o->W)) return PIVOT_ERR_INVALID_ARG;
  // Every query of the step as a sequence of one member on the key-split decode path: Reuse with
  // g = 1 and the raw query as its own scan row is Eq. 1 + TopK (c plays no part).
  return run_decode(q, w, kcache, pos0, B * g, Lmax, H_I, d, 1, k, k, PIVOT_REUSE, out_idx, stream, o, nullptr, 0, g);
}

int dense_index_decode(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, const int32_t* pos0,
                       int B, int Lmax, int H_I, int d, int g, int k, int32_t* out_idx, pivot_stream_t stream) {
  return dense_index_decode_ex(q, w, kcache, pos0, B, Lmax, H_I, d, g, k, out_idx, stream, nullptr);
}

int pivot_merge_topk(const float* scores, const int32_t* idx, int n_seg, int seg_len, const int32_t* seg_offset, int K,
                     int32_t* out_idx, float* out_scores, pivot_stream_t stream) {
  if (!scores || !idx || !out_idx || n_seg < 1 || seg_len < 1 || K < 1) return PIVOT_ERR_INVALID_ARG;
  if (K > kMaxSel || (long long)n_seg * seg_len > (1 << 24)) return PIVOT_ERR_UNSUPPORTED;
  if (((uintptr_t)scores | (uintptr_t)idx | (uintptr_t)out_idx | (uintptr_t)seg_offset | (uintptr_t)out_scores) & 3)
    return PIVOT_ERR_INVALID_ARG;
  DeviceState& ds = g_dev[cur_device()];
  const size_t need = 256 + (size_t)n_seg * seg_len * sizeof(unsigned long long);
  if (!ds.ws || ds.ws_bytes < need) return PIVOT_ERR_WORKSPACE;
  return check_cuda(launch_merge_topk(scores, idx, n_seg, seg_len, seg_offset, (unsigned long long*)((char*)ds.ws + 256), K,
                                      out_idx, out_scores, (cudaStream_t)stream));
}

int pivot_debug_wait_expiry(unsigned long long limit_ns, pivot_stream_t stream) {
  if (limit_ns < 1000ull || limit_ns > 1000000000ull) return PIVOT_ERR_INVALID_ARG;      // 1 us .. 1 s
  DeviceState& ds = g_dev[cur_device()];
  if (!ds.ws || ds.ws_bytes < 256) return PIVOT_ERR_WORKSPACE;
  int* status = (int*)ds.ws;                     // the status word is the first word of every workspace
  ds.last_status = status;
  cudaStream_t st = (cudaStream_t)stream;
  int rc = check_cuda(cudaMemsetAsync(status, 0, sizeof(int), st));
  if (rc) return rc;
  return check_cuda(launch_wait_expiry_probe(status, limit_ns, st));
}

int pivot_debug_mma_model(long long* out_device, pivot_stream_t stream) {
  if (!out_device || ((uintptr_t)out_device & 7)) return PIVOT_ERR_INVALID_ARG;
  return check_cuda(launch_mma_model_probe(out_device, (cudaStream_t)stream));
}

int pivot_debug_key_stream(const void* keys_device, int n_keys, int ctas, int tiles, int stages, int mode,
                           long long* out_device, pivot_stream_t stream) {
  if (!keys_device || !out_device || ((uintptr_t)keys_device & 15) || ((uintptr_t)out_device & 7)) return PIVOT_ERR_INVALID_ARG;
  return check_cuda(launch_key_stream_probe(keys_device, n_keys, ctas, tiles, stages, mode, out_device, (cudaStream_t)stream));
}

size_t pivot_prefill_host_arena_bytes(int L, int H_I, int d, int g, int c, int k, int dtype) {
  if (L < 1 || g < 1 || H_I < 1 || d < 1) return 0;
  const size_t esz = dtype == PIVOT_FP8_E4M3 ? 1 : 2;
  size_t n = 0;
  n += align_up((size_t)L * H_I * d * esz);   // q
  n += align_up((size_t)L * H_I * 4);         // q scale
  n += align_up((size_t)L * H_I * 4);         // w
  n += align_up((size_t)L * d * esz);         // k
  n += align_up((size_t)L * 4);               // k scale
  n += align_up((size_t)L * k * 4);           // out
  n += pivot_workspace_bytes(L, (L + g - 1) / g, c, k);
  return n;
}

int pivot_index_prefill_host(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L,
                             int H_I, int d, int g, int c, int k, int mode, int32_t* out_idx,
                             void* arena, size_t arena_bytes, pivot_stream_t stream) {
  if (!q || !w || !kcache || !out_idx || !arena || L < 1 || g < 1) return PIVOT_ERR_INVALID_ARG;
  // every argument check of the device entry point runs here, before the first copy is enqueued
  int rc = check_common(q, w, kcache, H_I, d, c, k, mode, out_idx);
  if (rc) return rc;
  if (key_stride(kcache)) return PIVOT_ERR_UNSUPPORTED;          // host arrays are copied as dense blocks
  if (((uintptr_t)arena & 255) || arena_bytes < pivot_prefill_host_arena_bytes(L, H_I, d, g, c, k, q->dtype))
    return PIVOT_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const bool fp8 = q->dtype == PIVOT_FP8_E4M3;
  const size_t esz = fp8 ? 1 : 2;
  DeviceState& ds = g_dev[cur_device()];
  if (!ds.copy_in) {
    if ((rc = check_cuda(cudaStreamCreateWithFlags(&ds.copy_in, cudaStreamNonBlocking)))) return rc;
    if ((rc = check_cuda(cudaStreamCreateWithFlags(&ds.copy_out, cudaStreamNonBlocking)))) return rc;
    if ((rc = check_cuda(cudaEventCreateWithFlags(&ds.ev_entry, cudaEventDisableTiming)))) return rc;
    for (int i = 0; i < kHostChunks + 2; ++i) {
      if ((rc = check_cuda(cudaEventCreateWithFlags(&ds.ev_in[i], cudaEventDisableTiming)))) return rc;
      if ((rc = check_cuda(cudaEventCreateWithFlags(&ds.ev_done[i], cudaEventDisableTiming)))) return rc;
    }
  }
  // From here on copies are in flight on three streams: an error return must not leave them
  // running on the caller's pinned buffers and arena.
  auto body = [&]() -> int {
  Carve cv(arena);
  char* dq = cv.take<char>((size_t)L * H_I * d * esz);
  float* dqs = cv.take<float>((size_t)L * H_I);
  float* dw = cv.take<float>((size_t)L * H_I);
  void* dk = cv.take<char>((size_t)L * d * esz);
  float* dks = cv.take<float>((size_t)L);
  int32_t* dout = cv.take<int32_t>((size_t)L * k);
  void* dws = (char*)arena + cv.off;

  // Row chunks: whole groups, at least 8192 rows each, at most kHostChunks of them.
  const int nG = (L + g - 1) / g;
  int n_chunks = L / 8192;
  n_chunks = n_chunks < 1 ? 1 : (n_chunks > kHostChunks ? kHostChunks : n_chunks);
  const int chunk_rows = ((nG + n_chunks - 1) / n_chunks) * g;
  n_chunks = (L + chunk_rows - 1) / chunk_rows;

  // The copy-in stream may not touch the arena before earlier work on `stream` has left it.
  if ((rc = check_cuda(cudaEventRecord(ds.ev_entry, st)))) return rc;
  if ((rc = check_cuda(cudaStreamWaitEvent(ds.copy_in, ds.ev_entry, 0)))) return rc;
  // keys and their scales: every chunk needs all of them; small, ahead of the first chunk on
  // the compute stream
  if ((rc = check_cuda(cudaMemcpyAsync(dk, kcache->data, (size_t)L * d * esz, cudaMemcpyHostToDevice, st)))) return rc;
  if (fp8 && (rc = check_cuda(cudaMemcpyAsync(dks, kcache->scale, (size_t)L * 4, cudaMemcpyHostToDevice, st)))) return rc;
  // Order of the chunks: a chunk's cost grows with its position in the request (longer prefixes)
  // while its copies do not.  In row order the first chunks finish long before the next input
  // has arrived; back to front, the last (cheap) chunks finish faster than their results can
  // leave.  Alternating the two ends (last, first, last but one, second, ...) keeps both the
  // compute stream and the copy-out stream fed.  The chunk taken first and the chunk taken last
  // go in two halves: nothing overlaps the first input copy and the last result copy, so those
  // two are kept short (more chunks throughout cost more in kernel ramps and tails than they save).
  struct Piece { int r0, r1; };
  Piece piece[kHostChunks + 2];
  int n_pieces = 0;
  for (int j = 0; j < n_chunks; ++j) {
    const int i = (j & 1) ? j / 2 : n_chunks - 1 - j / 2;
    const int r0 = i * chunk_rows, r1 = (r0 + chunk_rows < L) ? r0 + chunk_rows : L;
    // a quarter first (the first input copy) resp. last (the last result copy)
#ifndef PIVOT_HOST_SPLIT
#define PIVOT_HOST_SPLIT 4
#endif
    const int mid = j == 0 ? r0 + (r1 - r0) / PIVOT_HOST_SPLIT / g * g : r1 - (r1 - r0) / PIVOT_HOST_SPLIT / g * g;
    if ((j == 0 || j == n_chunks - 1) && n_chunks >= 4 && mid > r0 && mid < r1) {
      piece[n_pieces++] = Piece{r0, mid};
      piece[n_pieces++] = Piece{mid, r1};
    } else {
      piece[n_pieces++] = Piece{r0, r1};
    }
  }
  // queries: piece by piece on the copy-in stream
  const size_t qrow = (size_t)H_I * d * esz;
  for (int j = 0; j < n_pieces; ++j) {
    const int i = j;
    const int r0 = piece[j].r0, r1 = piece[j].r1;
    // a chunk's queries, gates and query scales travel together
    if ((rc = check_cuda(cudaMemcpyAsync(dw + (size_t)r0 * H_I, w + (size_t)r0 * H_I, (size_t)(r1 - r0) * H_I * 4,
                                         cudaMemcpyHostToDevice, ds.copy_in))))
      return rc;
    if (fp8 && (rc = check_cuda(cudaMemcpyAsync(dqs + (size_t)r0 * H_I, q->scale + (size_t)r0 * H_I,
                                                (size_t)(r1 - r0) * H_I * 4, cudaMemcpyHostToDevice, ds.copy_in))))
      return rc;
    if ((rc = check_cuda(cudaMemcpyAsync(dq + (size_t)r0 * qrow, (const char*)q->data + (size_t)r0 * qrow,
                                         (size_t)(r1 - r0) * qrow, cudaMemcpyHostToDevice, ds.copy_in))))
      return rc;
    if ((rc = check_cuda(cudaEventRecord(ds.ev_in[i], ds.copy_in)))) return rc;
  }
  pivot_tensor tq{dq, fp8 ? dqs : nullptr, q->dtype, 0};
  pivot_tensor tk{dk, fp8 ? dks : nullptr, q->dtype, 0};
  for (int j = 0; j < n_pieces; ++j) {
    const int i = j;
    const int r0 = piece[j].r0, r1 = piece[j].r1;
    pivot_opts o;
    memset(&o, 0, sizeof(o));
    o.guard_len = -1;
    o.workspace = dws;
    o.workspace_bytes = arena_bytes - cv.off;
    if (n_pieces > 1) { o.row_begin = r0; o.row_end = r1; }
    if ((rc = check_cuda(cudaStreamWaitEvent(st, ds.ev_in[i], 0)))) return rc;
    rc = pivot_index_prefill_ex(&tq, dw, &tk, L, H_I, d, g, c, k, mode, dout, stream, &o);
    if (rc) return rc;
    if ((rc = check_cuda(cudaEventRecord(ds.ev_done[i], st)))) return rc;
    if ((rc = check_cuda(cudaStreamWaitEvent(ds.copy_out, ds.ev_done[i], 0)))) return rc;
    if ((rc = check_cuda(cudaMemcpyAsync(out_idx + (size_t)r0 * k, dout + (size_t)r0 * k, (size_t)(r1 - r0) * k * 4,
                                         cudaMemcpyDeviceToHost, ds.copy_out))))
      return rc;
  }
  if ((rc = check_cuda(cudaStreamSynchronize(st)))) return rc;
  return check_cuda(cudaStreamSynchronize(ds.copy_out));
  };
  rc = body();
  if (rc) {
    cudaStreamSynchronize(ds.copy_in);
    cudaStreamSynchronize(st);
    cudaStreamSynchronize(ds.copy_out);
  }
  return rc;
}

int pivot_device_status(pivot_stream_t stream, int* status) {
  if (!status) return PIVOT_ERR_INVALID_ARG;
  int* p = g_dev[cur_device()].last_status;
  *status = 0;
  if (!p) return PIVOT_OK;
  int rc = check_cuda(cudaStreamSynchronize((cudaStream_t)stream));
  if (rc) return rc;
  if ((rc = check_cuda(cudaMemcpy(status, p, sizeof(int), cudaMemcpyDeviceToHost)))) return rc;
  if (*status) rc = check_cuda(cudaMemset(p, 0, sizeof(int)));     // read and cleared
  return rc;
}

int pivot_debug_counters(pivot_stream_t stream, unsigned long long* out, int n) {
#ifdef PIVOT_PROF
  if (!out || n < 1 || n > 28) return PIVOT_ERR_INVALID_ARG;
  int* p = g_dev[cur_device()].last_status;
  if (!p) return PIVOT_ERR_WORKSPACE;
  int rc = check_cuda(cudaStreamSynchronize((cudaStream_t)stream));
  if (rc) return rc;
  if ((rc = check_cuda(cudaMemcpy(out, p + 8, (size_t)n * 8, cudaMemcpyDeviceToHost)))) return rc;
  return check_cuda(cudaMemset(p + 8, 0, 28 * 8));                   // read and cleared
#else
  (void)stream; (void)out; (void)n;
  return PIVOT_ERR_UNSUPPORTED;                                        // the library was built without -DPIVOT_PROF
#endif
}

int pivot_stage_timing(int enable) {
  if (enable && !timing_events()) { (void)check_cuda(cudaGetLastError()); return PIVOT_ERR_CUDA; }
  g_timing = enable != 0;
  for (DeviceState& ds : g_dev) { ds.ev_valid = false; ds.ev_decode_scan = false; }
  return PIVOT_OK;
}

int pivot_stage_times(float* ms, int n) {
  DeviceState& ds = g_dev[cur_device()];
  if (!ms || n < 5 || !ds.ev_valid) return PIVOT_ERR_INVALID_ARG;
  cudaEvent_t* ev = ds.ev;
  int rc = check_cuda(cudaEventSynchronize(ev[4]));
  if (rc) return rc;
  for (int i = 0; i < 4; ++i)
    if ((rc = check_cuda(cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1])))) return rc;
  if ((rc = check_cuda(cudaEventElapsedTime(&ms[4], ev[0], ev[4])))) return rc;
  if (n >= 6) {
    ms[5] = 0.f;
    if (ds.ev_decode_scan && (rc = check_cuda(cudaEventElapsedTime(&ms[5], ev[6], ev[7])))) return rc;
  }
  if (n >= 7) {
    ms[6] = 0.f;
    if (ds.ev_decode_scan && (rc = check_cuda(cudaEventElapsedTime(&ms[6], ev[7], ev[8])))) return rc;
  }
  return PIVOT_OK;
}

long long pivot_launch_count_reset(void) {
  long long n = launch_counter();
  launch_counter() = 0;
  return n;
}

const char* pivot_status_str(int code) {
  switch (code) {
    case PIVOT_OK: return "ok";
    case PIVOT_ERR_INVALID_ARG: return "invalid argument";
    case PIVOT_ERR_UNSUPPORTED:
      return "unsupported: shape (H_I must be 64, d 128, k and c at most 8192), layout, or an entry point this build does not carry";
    case PIVOT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case PIVOT_ERR_CUDA: return "CUDA runtime error (see pivot_last_cuda_error)";
    case PIVOT_ERR_DEVICE: return "device-side condition recorded in the status word";
    default: return "unknown status";
  }
}

int pivot_last_cuda_error(void) { return g_last_cuda; }

}  // extern "C"
