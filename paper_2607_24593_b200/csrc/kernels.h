// Host-callable launchers of the library's kernels (internal header).
#pragma once
#include <utility>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace pivot {

constexpr int kMembersPerDesc = 4;
inline int group_chunks(int g) { return (g + kMembersPerDesc - 1) / kMembersPerDesc; }

// One group's fine step (Eq. 8-9): m members re-score the candidate list.
struct GroupDesc {
  const void* q;        // first member [m, H, d] codes, members contiguous
  const float* w;       // [m, H]
  const float* qscale;  // [m, H] or nullptr
  const void* kbase;
  const float* kscale;
  int k_stride = 0;     // bytes between key rows (0: dense)
  const int32_t* cand;  // candidate key positions, valid entries first
  int n_cand;           // valid candidates (0: group is skipped)
  int m;                // members (at most kMembersPerDesc per descriptor)
  int K;                // entries to select per member
  int first_pos;        // position of the first member (slot i sits at first_pos + i)
  int q_row;            // row of the first member inside the raw query tensor (units of H x d)
  int32_t* out;         // [m, out_stride]
  float* out_score;     // optional
  int out_stride;
  // Chunked mode (decode): when ent_out is set the kernel does not select; member r's packed
  // entries go to ent_out[r * ent_stride + slot0 + slot] for a later top-k over the whole list.
  unsigned long long* ent_out;
  int ent_stride;
  int slot0;
  // Paged key cache (decode): kbase / kscale are the page pool and key position s lives in pool
  // row pages[s / 128] * 128 + s % 128; pages == nullptr means one contiguous cache.
  const int32_t* pages = nullptr;
  int n_pages = 0;      // pages in the pool (entries outside [0, n_pages) are treated as holes)
  // Per-query window slots (decode form of Appendix B): the member at position t takes a slot
  // only if t - win_span < position <= t.  The default never excludes anything below t.
  int win_span = 1 << 30;
  // Largest key position a candidate of this group may name (the group's last member); the
  // gather drops anything beyond it and reports DEV_BOUNDS.
  int pos_max = 0x7fffffff;
};

constexpr int kDecodeWinMax = 512;      // most window slots (W + g - 1) of a decode step

constexpr int kDecodeCandChunk = 512;   // candidates per re-score work item in decode

// One query's re-scored candidates (packed entries) awaiting the final top-k.
struct EntryList {
  const unsigned long long* list;
  int n;
  int K;
  int32_t* out;
  float* out_score;
};

// Geometry of a prefill-shaped call, shared by the planner kernels.
struct PrefillPlan {
  const void* q; const float* w; const float* qscale;   // raw per-query operands
  const void* kc; const float* kscale;                  // key cache
  int k_stride = 0;                                     // bytes between key rows (0: dense)
  void* proxy_q; float* proxy_w;                        // [nP, H, d], [nP, H]
  int32_t* cand; float* cand_score;                     // [nP, c] (Refine)
  int32_t* out; float* out_score;                       // [L, k]
  int L, g, c, k, mode, dtype;
  int W;            // local window (Appendix B); 0 = off
  int dense_begin;  // first densely scored row of this call
  int n_dense;      // rows dense_begin .. dense_begin+n_dense-1 are scored densely (guarded groups or dense control)
  int first_group;  // first group taking the proxy path
  int n_proxy;      // groups on the proxy path
};

struct DecodePlan {
  const void* q; const float* w; const float* qscale;   // [B, g, H, d] ...
  const void* kc; const float* kscale;                  // [B, Lmax, d], [B, Lmax]
  int k_stride = 0;                                     // bytes between key rows (0: dense)
  const int32_t* pos0;
  void* proxy_q; float* proxy_w;                        // [B, H, d], [B, H]
  int32_t* cand; float* cand_score;                     // [B, c]
  int32_t* out; float* out_score;                       // [B, g, k]
  int B, Lmax, g, c, k, mode, dtype, guard_len;
  const int32_t* block_table = nullptr;                 // paged cache: [B, Lmax / 128] pool pages
  int n_pages = 0;
  int W = 0;                                            // per-query local window (Appendix B, decode form)
  int* status = nullptr;                                // device status word (a bad pos0 is reported there)
  // Dense control (Eq. 1 per query): every query of the step is planned as a sequence of its own
  // with one member.  kv_share consecutive plan slots then share one key cache: slot b reads cache
  // b / kv_share and sits at position pos0[b / kv_share] + b % kv_share.  raw_q: the scan rows
  // are the raw queries themselves (no proxy is built); the planner leaves their effective gates
  // fl32(w * qscale) in proxy_w.
  int kv_share = 1;
  bool raw_q = false;
};

struct ScanScratch {
  uint32_t* cand_key;   // [n_cta][2][cap]   (CUDA-core kernels: separate key / index arrays)
  int32_t* cand_idx;    // [n_cta][2][cap]
  unsigned long long* cand64;   // the same memory seen as packed 64-bit entries (tensor-core kernels)
  int cap;
  int n_cta;
  int* status;
  int* counter;         // dynamic row scheduler
  uint32_t* rkeys = nullptr;   // re-score: [SMs][2][4][rslots] score keys between the tile loop and the select warps
  int rslots = 0;              // ... slots per row: the candidate budget rounded up to whole 128-key tiles
};

void launch_proxy_build(const void* q, const float* qscale, const float* w, void* proxy_q,
                        float* proxy_w, int rows, int g, int first_group, int n_proxy, int dtype,
                        int pool, cudaStream_t st);
void launch_plan_prefill(const PrefillPlan& p, RowDesc* rows, GroupDesc* groups, cudaStream_t st);
void launch_plan_decode(const DecodePlan& p, RowDesc* rows, GroupDesc* groups, cudaStream_t st);
// Decode proxies need the guard test on device (pos0 lives there): rows of guarded sequences
// get K = 0 and are skipped.
void launch_scan_simt(const RowDesc* rows, int n_rows, int dtype, const ScanScratch& s, cudaStream_t st);
void launch_refine_simt(const GroupDesc* groups, int n_groups, int dtype, const ScanScratch& s, cudaStream_t st);

// Operand tensors of a tensor-core scan, for the TMA tensor maps.
struct ScanOperands {
  const void* kc; long long k_rows;        // key cache [k_rows, d]
  const float* kscale;                     // [k_rows] (FP8) or nullptr
  const void* q; int q_rows;               // raw queries [q_rows, H, d]
  const void* proxy_q; int proxy_rows;     // proxies [proxy_rows, H, d]
  int dtype;
  int k_stride = 0;                        // bytes between key rows (0: dense)
};
// rows_per_block consecutive scan rows share one key stream (4 in prefill, 1 in decode).
// fp32_head_sum: keep the gate-weighted head sum in fp32 FMAs even where the tensor-core form
// (FP8, four rows per block) is available.
// fp32_head_sum: keep the gate-weighted head sum in fp32 FMAs even where the tensor-core form
// (FP8, four rows per block) is available.
cudaError_t launch_scan_tc(const ScanOperands& op, const RowDesc* rows, int n_rows, int rows_per_block,
                           const ScanScratch& s, int sms, cudaStream_t st, bool fp32_head_sum = false);

cudaError_t launch_refine_tc(const void* q, int q_rows, int dtype, const GroupDesc* groups, int n_groups,
                             const ScanScratch& s, int sms, cudaStream_t st, bool fp32_head_sum = false,
                             bool chunked = false, int max_cand = 0, bool overlap_prev = false);

// Decode fast path: key-tile-split scan -> per-sequence select -> chunked re-score -> top-k.
struct DecodeFast {
  DecodePlan plan;            // the call's geometry: the prepare kernel plans the sequences itself
  int pool = 0;               // proxy aggregation (the prepare kernel builds the proxies)
  RowDesc* prox;              // [B + B * g] row slots; [0, B) = proxy rows (K = 0: guarded sequence, skipped)
  GroupDesc* groups;          // [B * group_chunks(g)]
  const void* kc; const float* kscale; const void* q; const void* proxy_q;
  int B, Lmax, g, c, k, mode, dtype, sms;
  long long k_rows;           // rows of the key tensor (B * Lmax, or pool pages * 128 when paged)
  int k_stride = 0;           // bytes between key rows (0: dense)
  int W = 0;                  // per-query local window (Appendix B, decode form); Refine only
  bool skip_scan = false;     // the candidate sets come from the caller: no scan, no top-c select
  void* scratch;              // decode_fast_bytes(...) bytes
  ScanScratch scratch_tc;     // candidate scratch of the re-score kernel
  int* status;
  cudaEvent_t ev_scan_begin, ev_scan_end;   // optional: recorded around the scan kernel
  cudaEvent_t ev_select_end = nullptr;      // ... and behind the per-sequence select
};
size_t decode_fast_bytes(int B, int Lmax, int g, int c);
cudaError_t launch_decode_fast(const DecodeFast& d, cudaStream_t st);

long long& launch_counter();
// Top-K of the union of n_seg candidate lists (see pivot_merge_topk); entries = scratch for n_seg * seg_len packed entries.
cudaError_t launch_merge_topk(const float* scores, const int32_t* idx, int n_seg, int seg_len, const int32_t* seg_offset,
                              unsigned long long* entries, int K, int32_t* out_idx, float* out_scores, cudaStream_t st);

// Diagnostic: a kernel whose bounded waits run out after limit_ns (see debug_probe.cu).
cudaError_t launch_wait_expiry_probe(int* status, unsigned long long limit_ns, cudaStream_t st);
// Diagnostic: tensor-pipe / tensor-memory / hand-over timings of one SM (see debug_probe.cu); out = 256 slots.
cudaError_t launch_mma_model_probe(long long* out, cudaStream_t st);
// Diagnostic: rate at which all SMs together can pull the scan's 16 KB key tiles out of L2.
cudaError_t launch_key_stream_probe(const void* keys, int n_keys, int ctas, int tiles, int stages, int mode, long long* out,
                                    cudaStream_t st);

// The opt-in to more than 48 KB of dynamic shared memory is an attribute of (function, device):
// remembered per device, so that a process driving several GPUs sets it on each of them.
constexpr int kMaxDevices = 64;
template <typename Kern>
inline cudaError_t opt_in_dynamic_smem(Kern kern, size_t bytes, bool (&done)[kMaxDevices]) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < kMaxDevices;
  if (tracked && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && tracked) done[dev] = true;
  return e;
}

// Launch with programmatic stream serialisation (`overlap`): the kernel may start before its
// predecessor in the stream has finished and must call ptx::grid_dependency_wait() before it
// touches anything the predecessor writes or reads.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(std::forward<Args>(args))...);
}

}  // namespace pivot
