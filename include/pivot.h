/*
 * pivot.h -- C ABI of the PIVOT group-shared indexer for NVIDIA B200 (sm_100a).
 *
 * The library produces, for every query token t, the index set T_t (k key positions) that a
 * DSA-style sparse attention operator consumes.  It implements
 *   - the dense lightning indexer  I_{t,s} = sum_j w_{t,j} ReLU(q_{t,j} . k_s), s <= t   (Eq. 1)
 *     followed by T_t = TopK(I_{t,:}, k), and
 *   - PIVOT (Algorithm 1): per group of g nearby queries one mean proxy (Eq. 4), one shared
 *     prefix scan cut at the group's first position (Eq. 5), then either the proxy top-k for
 *     the whole group (Reuse, Eq. 6) or a top-c candidate set (Eq. 7) re-scored by every member
 *     with its own query and gate and reduced to a per-query top-k (Refine, Eq. 8-9).
 * Groups are fixed-size runs of consecutive positions in prefill (Eq. 2) and the queries of one
 * multi-token-prediction step in decode (Eq. 3).  Groups whose visible prefix is shorter than
 * guard_len (default c) are scored densely per member (short-group guardrail of Algorithm 1).
 *
 * Conventions
 *   - Positions are 0-indexed; query t sees keys 0..t inclusive.
 *   - All pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     The library never allocates or frees device memory; scratch comes from the caller's
 *     workspace (pivot_workspace_bytes / pivot_set_workspace, or the *_ex forms).
 *   - All work is enqueued on `stream`; no entry point synchronises unless documented.
 *   - Index output rows are SETS in unspecified order, no duplicates, every entry <= t.  When
 *     fewer than k keys are visible (dense / guarded rows only) the valid entries come first
 *     and the remainder is -1.
 *   - Supported shapes: H_I = 64 indexer heads, d = 128, 1 <= k <= c <= 8192 (Refine) or
 *     1 <= k <= 8192 (Reuse / dense).  Anything else returns PIVOT_ERR_UNSUPPORTED.
 *   - Return value: PIVOT_OK or a positive error code; argument errors are detected on the host
 *     before any launch.  Device-side conditions (a bounded wait that expired) are recorded in
 *     a status word readable with pivot_device_status; kernels never trap.
 */
#ifndef PIVOT_H_
#define PIVOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* pivot_stream_t; /* a cudaStream_t */

enum { PIVOT_BF16 = 0, PIVOT_FP8_E4M3 = 1 };
enum { PIVOT_REUSE = 0, PIVOT_REFINE = 1 };
enum { PIVOT_POOL_MEAN = 0, PIVOT_POOL_FIRST = 1, PIVOT_POOL_LAST = 2 };
enum {
  PIVOT_OK = 0,
  PIVOT_ERR_INVALID_ARG = 1,
  PIVOT_ERR_UNSUPPORTED = 2,
  PIVOT_ERR_WORKSPACE = 3,   /* no workspace set, or too small */
  PIVOT_ERR_CUDA = 4,        /* a CUDA runtime call failed; see pivot_last_cuda_error */
  PIVOT_ERR_DEVICE = 5       /* device status word non-zero (pivot_device_status) */
};
/* Values of the device status word (pivot_device_status); the first condition of a call wins. */
enum {
  PIVOT_DEV_OK = 0,
  PIVOT_DEV_WAIT_EXPIRED = 1,  /* a bounded wait inside a kernel ran out; the kernel ended early, results invalid */
  PIVOT_DEV_CAND_OVERFLOW = 2, /* a candidate buffer would have overflowed (internal error; the entry was dropped) */
  PIVOT_DEV_BAD_POS = 3,       /* decode: some pos0[b] outside [0, Lmax - g]; that sequence's rows are all -1 */
  PIVOT_DEV_BOUNDS = 4         /* checked builds (-DPIVOT_DEBUG) only: an index failed a bounds check, access skipped */
};

/*
 * A quantised operand.
 *   data   row-major storage: bf16 bit patterns (2 B) or e4m3 codes (1 B).
 *          queries: [L, H_I, d] (decode: [B, g, H_I, d]); key cache: [L, d] (decode: [B, Lmax, d]).
 *   scale  NULL for bf16.  FP8: one fp32 scale per d-vector -- queries [L, H_I]
 *          (decode [B, g, H_I]), keys [L] (decode [B, Lmax]); value = code * scale.
 *   dtype  PIVOT_BF16 or PIVOT_FP8_E4M3; q and kcache must agree.
 *   stride_row  bytes from one row of d elements to the next; 0 = dense (d * element size).  Key
 *          caches may be padded (a serving engine's cache rows often carry more than the indexer
 *          key): any multiple of 16 bytes >= the dense row size.  Queries must be dense.  The scale
 *          arrays are always dense.  Not available with impl = 1 or the host-buffer entry point.
 * data must be 16-byte aligned; the key-cache scale 16-byte aligned, the query scale 4-byte.
 */
typedef struct pivot_tensor {
  const void* data;
  const float* scale;
  int dtype;
  size_t stride_row;
} pivot_tensor;

/*
 * Options of the *_ex entry points.  Zero-initialise, then set what is needed.
 *   guard_len     groups with fewer visible keys than this are scored densely per member;
 *                 -1 selects the default c (Algorithm 1 tests t0 < c).  0 disables the guardrail.
 *   pool          proxy aggregation: mean (Eq. 4) or the first / last member (the paper's ablation).
 *   dbg_cand      optional [n_groups, c] int32: candidate set of every group (Refine; rows of
 *                 guarded groups are left untouched).  Unordered.
 *   dbg_scores    optional fp32 buffer receiving the score that ranked each emitted index:
 *                 same shape as out_idx ([rows, k]; -inf beside a -1 index).  For Refine these are
 *                 the per-query re-scores (Eq. 8), for Reuse the proxy scores (Eq. 5), for dense
 *                 and guarded rows Eq. 1.
 *   dbg_cand_scores optional [n_groups, c] fp32: proxy score (Eq. 5) of each dbg_cand entry.
 *   workspace     scratch of at least pivot_workspace_bytes(...) bytes, 256-byte aligned.
 *   impl          0: tensor-core kernels (tcgen05; the product path).  In FP8 prefill the shared
 *                 scan also takes the gate-weighted head sum of Eq. 5 on the tensor core: ReLU
 *                 values rounded to bf16, gates carried as two bf16 terms, fp32 accumulation -- a
 *                 relative score error of about 2^-9, inside the FP8 acceptance band.
 *                 2: the same kernels with that head sum in fp32 FMAs (slower; the scores then
 *                 differ from exact arithmetic by fp32 summation order only).
 *                 1: the plain CUDA-core kernels that compute the same thing one key per thread
 *                 -- a slow on-device cross-check, not a fallback: nothing selects it
 *                 automatically.
 *   row_begin, row_end  prefill / dense only: index just the query rows row_begin .. row_end-1 of
 *                 the request (chunked prefill; the other rows of out_idx are left untouched).
 *                 Both 0 = all rows.  row_begin must be a multiple of g, row_end a multiple of g
 *                 or L.  Tensor arguments keep their full-request shapes; a chunk's result is the
 *                 same as the corresponding rows of one whole call (groups never straddle chunks).
 *   W             local window of Appendix B (0 = off, the default; the paper's setting is 4).
 *                 Prefill: the proxy scan of a group at t0 then ranks the keys s <= t0 - W
 *                 only.  Refine: the proxy fills c - (W + m - 1) candidate slots (m = members of
 *                 the group) and the last W + m - 1 slots hold the window positions
 *                 t0-W+1 .. t0+m-1 in ascending order; every member re-scores all slots and
 *                 ignores window slots beyond its own position.  Reuse: the shared top-k comes
 *                 from the shortened scan.  Needs W + g - 1 < c and a guardrail of at least
 *                 W + g (the default c is).
 *                 Decode (Refine only): the pool is still the proxy's top-c over s <= pos0, and
 *                 the query at t re-scores pool U [t-W+1, t] (duplicates counted once).  Needs
 *                 W >= g (the window then covers the keys written inside the step) and
 *                 W + g - 1 <= 512.  Sequences under the guardrail are scored densely as usual.
 *                 Not available with impl = 1.
 *   cand_in       decode, Refine only: a candidate set supplied from outside, [B, c] int32 on the
 *                 device, valid entries first (min(c, pos0[b] + 1) of them).  The call then skips the
 *                 shared scan and the top-c select (Eq. 5, Eq. 7) and runs Eq. 8-9 on these
 *                 candidates -- the second half of a step whose scan was split over several GPUs
 *                 (pivot_merge_topk builds the set).  Sequences under the guardrail are still
 *                 scored densely and ignore it.  NULL (the default): the call scans.
 */
typedef struct pivot_opts {
  int guard_len;
  int pool;
  int32_t* dbg_cand;
  float* dbg_scores;
  float* dbg_cand_scores;
  void* workspace;
  size_t workspace_bytes;
  int impl;
  int row_begin, row_end;
  int W;
  const int32_t* cand_in;
} pivot_opts;

/* Bytes of scratch a prefill / dense call with these sizes needs: rows = L, n_groups = ceil(L/g)
 * (L for dense_index).  Depends on the device's SM count (queried once).  Decode calls need
 * pivot_decode_workspace_bytes. */
size_t pivot_workspace_bytes(int rows, int n_groups, int c, int k);

/* Scratch of a decode call (adds the per-key score array and histograms of the decode path). */
size_t pivot_decode_workspace_bytes(int B, int Lmax, int g, int c, int k);

/* Registers the scratch buffer used by the short entry points below on the current device.
 * The buffer stays owned by the caller and must outlive those calls.  Calls that share one
 * workspace must not overlap on the GPU. */
int pivot_set_workspace(void* workspace, size_t bytes);

/*
 * Prefill (Algorithm 1 with the grouping of Eq. 2) over one request of L positions.
 *   q, kcache  operands as described at pivot_tensor; w is the gate [L, H_I] fp32 (the raw gate
 *              times any positive constant; for FP8 NOT pre-multiplied by the query scale).
 *   g          group size (>= 1; g = 1 is the dense indexer, Appendix A).
 *   c, k       candidate budget and selection size; Refine needs k <= c.
 *   mode       PIVOT_REUSE or PIVOT_REFINE.
 *   out_idx    [L, k] int32.
 */
int pivot_index_prefill(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                        int L, int H_I, int d, int g, int c, int k, int mode,
                        int32_t* out_idx, pivot_stream_t stream);
int pivot_index_prefill_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                           int L, int H_I, int d, int g, int c, int k, int mode,
                           int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts);

/*
 * Batched prefill of several requests packed back to back (the request boundaries of Eq. 2:
 * groups and causal prefixes never cross from one request into the next).
 *   cu_seqlens   HOST array [n_req + 1], non-decreasing, cu_seqlens[0] = 0: request i owns rows
 *                cu_seqlens[i] .. cu_seqlens[i+1]-1 of q / w / kcache / out_idx (total rows =
 *                cu_seqlens[n_req]).  With FP8 every request must start on a multiple of 4 rows
 *                (the key-scale rows are read in 16-byte units); empty requests are allowed.
 *   out_idx      [total rows, k]; positions are relative to the start of the row's own request.
 * Each request is indexed by the prefill path above, one after the other on `stream`, sharing
 * one workspace sized for the longest request (opts->workspace, else the registered one).
 * opts may be NULL; row_begin / row_end and the debug buffers are not available here.
 */
int pivot_index_prefill_varlen(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                               const int32_t* cu_seqlens, int n_req, int H_I, int d, int g, int c, int k,
                               int mode, int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts);

/*
 * Decode (Algorithm 1 with the grouping of Eq. 3): B independent sequences, each contributing
 * the g queries of one MTP step at positions pos0[b] .. pos0[b]+g-1.
 *   q       [B, g, H_I, d]; w [B, g, H_I]; kcache [B, Lmax, d] (+ scale [B, Lmax]); sequence b's
 *           cache must hold keys 0 .. pos0[b]+g-1.
 *   pos0    [B] int32, device.  The proxy scan is cut at pos0[b] (inclusive).  Must lie in
 *           [0, Lmax - g]; a sequence whose pos0 does not is not indexed: its g output rows are
 *           filled with -1 and the status word reads PIVOT_DEV_BAD_POS (nothing is read out of
 *           range, nothing traps).
 *   Lmax    rows per sequence in kcache; with FP8 it must be a multiple of 4 (each sequence's
 *           scale row then starts on a 16-byte boundary).
 *   out_idx [B, g, k] int32.
 */
int pivot_index_decode(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                       const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int c, int k,
                       int mode, int32_t* out_idx, pivot_stream_t stream);
int pivot_index_decode_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                          const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int c, int k,
                          int mode, int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts);

/*
 * Decode over a PAGED key cache (the layout a serving engine's block manager keeps; the method
 * itself, Algorithm 1 with the grouping of Eq. 3, is unchanged).
 *   kpages       the page pool: data [n_pages * 128, d] (+ scale [n_pages * 128]); a page holds
 *                128 consecutive key positions of one sequence.
 *   block_table  [B, max_pages] int32, device: block_table[b][p] is the pool page holding keys
 *                128 p .. 128 p + 127 of sequence b.  Entries for pages past pos0[b] + g - 1 are
 *                never read.  An entry outside [0, n_pages) faults nothing: its keys read as
 *                zeros in the scan and are dropped as holes by the re-score.
 *   pos0, q, w, out_idx, c, k, mode   as in pivot_index_decode; returned positions are LOGICAL
 *                key positions of the sequence.
 * Differences from the contiguous form: the short-sequence guardrail is off (opts->guard_len is
 * ignored) -- a sequence with fewer than c visible keys takes the proxy path with every visible
 * key as a candidate, so Refine is still exact for it over the keys up to pos0 -- and
 * opts->impl = 1 is rejected.  Workspace: pivot_decode_workspace_bytes(B, max_pages * 128, ...).
 */
int pivot_index_decode_paged(const pivot_tensor* q, const float* w, const pivot_tensor* kpages,
                             const int32_t* block_table, const int32_t* pos0, int B, int max_pages,
                             int n_pages, int H_I, int d, int g, int c, int k, int mode,
                             int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts);

/*
 * TopK (Eq. 7) over the union of several partial candidate lists: the merge step of one decode
 * sequence whose key axis was split over GPUs -- every part scans its own key range into a local
 * top-c with proxy scores (pivot_index_decode in Reuse mode with k = c on that range, positions
 * relative to the range), the parts are exchanged, and the global top-c is the top-c of their union
 * (a key of the global top-c is in the top-c of its own range).
 *   scores, idx   [n_seg, seg_len] fp32 / int32, device: part p's entries; idx < 0 marks an empty slot.
 *   seg_offset    [n_seg] int32, device, or NULL: added to the positions of part p (its range's first key).
 *   K             entries to keep (at most 8192); order (score desc, position asc), as everywhere.
 *   out_idx       [K] int32, valid entries first, then -1; out_scores [K] fp32 or NULL.
 * Uses the registered workspace (at least 256 + 8 * n_seg * seg_len bytes).
 */
int pivot_merge_topk(const float* scores, const int32_t* idx, int n_seg, int seg_len, const int32_t* seg_offset,
                     int K, int32_t* out_idx, float* out_scores, pivot_stream_t stream);

/*
 * Dense control: Eq. 1 + TopK for every query of a request (prefill form) -- the O(L^2) indexer
 * PIVOT replaces, run by the same kernels with one row per query.  out_idx [L, k].
 */
int dense_index(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                int L, int H_I, int d, int k, int32_t* out_idx, pivot_stream_t stream);
int dense_index_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                   int L, int H_I, int d, int k, int32_t* out_idx, pivot_stream_t stream,
                   const pivot_opts* opts);

/*
 * Dense control, decode form: Eq. 1 + TopK for each of the g queries of one MTP step (the grouping
 * of Eq. 3) of B sequences -- what a DSA decode step costs without PIVOT.  Arguments as in
 * pivot_index_decode (contiguous cache); the query at position pos0[b] + i ranks keys
 * 0 .. pos0[b] + i of sequence b.  Runs on the same key-split kernels as pivot_index_decode, every
 * query as a scan row of its own (its raw codes, effective gate fl32(w * qscale)): the g rows of a
 * sequence stream that sequence's keys one after the other.  out_idx [B, g, k] int32.  Workspace:
 * pivot_decode_workspace_bytes(B * g, Lmax, 1, k, k).  opts: dbg_scores, workspace.
 */
int dense_index_decode(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                       const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int k,
                       int32_t* out_idx, pivot_stream_t stream);
int dense_index_decode_ex(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                          const int32_t* pos0, int B, int Lmax, int H_I, int d, int g, int k,
                          int32_t* out_idx, pivot_stream_t stream, const pivot_opts* opts);

/*
 * dense_index without any caller-provided scratch (no counterpart in the paper: this is a
 * deployment convenience, not part of the method).  For hosts that may not allocate device
 * memory -- a plugin inside a server that owns the device heap, code bound to a framework's
 * memory pool -- the scratch comes from an 8 MiB array built into the library image (every GPU
 * that loads the library holds it until the process exits).  Same arguments and result as
 * dense_index; q, w, kcache, out_idx are device pointers as usual.
 *   Limits: L <= 4096 and k <= 512, else PIVOT_ERR_WORKSPACE.  Runs on a reduced grid, so it is
 *   slower than dense_index.
 *   The first call on a device looks up the array's device address; make that call before any
 *   stream capture.  Calls never allocate or free.
 *   All calls on a device share the array (it keeps the previous call's contents; what must
 *   start at zero is cleared on `stream`): calls that overlap on the GPU race -- run them on
 *   one stream, or order them otherwise.  pivot_device_status does not cover this entry point.
 */
int dense_index_static(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                       int L, int H_I, int d, int k, int32_t* out_idx, pivot_stream_t stream);

/*
 * Host-buffer form of pivot_index_prefill: every tensor pointer (q, w, kcache, out_idx) is HOST
 * memory (pinned, else the copies are neither asynchronous nor fast).  The call copies the inputs
 * into `arena` (device, at least pivot_prefill_host_arena_bytes(...) bytes, which includes the
 * workspace), runs the device path and copies out_idx back; it returns after everything has
 * finished.  Keys and key scales go first; queries, gates and query scales then travel in row
 * chunks on a copy stream of the library's own while earlier chunks are indexed on `stream`
 * (row_begin / row_end of pivot_opts) and their results return on a second copy stream, so the
 * PCIe transfers in both directions overlap the kernels.  Chunks are taken alternately from the
 * end and the start of the request (late rows cost the most compute per byte copied).  The first call on a device creates the two copy streams and
 * their events (kept until the process exits).
 */
size_t pivot_prefill_host_arena_bytes(int L, int H_I, int d, int g, int c, int k, int dtype);
int pivot_index_prefill_host(const pivot_tensor* q, const float* w, const pivot_tensor* kcache,
                             int L, int H_I, int d, int g, int c, int k, int mode,
                             int32_t* out_idx, void* arena, size_t arena_bytes,
                             pivot_stream_t stream);

/* Reads (and clears) the device status word of the workspace last used on this device after
 * synchronising `stream`.  0 = no device-side condition, else a PIVOT_DEV_* value. */
int pivot_device_status(pivot_stream_t stream, int* status);

/*
 * Diagnostic (no counterpart in the paper): runs a one-block kernel whose threads wait, through the
 * library's own bounded-wait routines, for a barrier that nothing completes, with a limit of
 * limit_ns nanoseconds (1 us .. 1 s) instead of the library's 4 s.  The waits run out, the kernel
 * returns normally and pivot_device_status then reads PIVOT_DEV_WAIT_EXPIRED -- the path every
 * tensor-core kernel here takes instead of hanging should one of its hand-shakes ever break.
 * Uses the status word of the registered workspace (pivot_set_workspace; PIVOT_ERR_WORKSPACE if
 * there is none).  The GPU context stays usable; later calls are unaffected.
 */
int pivot_debug_wait_expiry(unsigned long long limit_ns, pivot_stream_t stream);

/*
 * Diagnostic (no counterpart in the paper): times, on one SM, the tensor-core instruction streams
 * the shared scan (Eq. 5) and the re-score (Eq. 8) are built from -- the 128 x 256 x 128 FP8
 * product, the head-sum product with its A operand in tensor memory in several operand widths,
 * both interleaved -- alone and while other warps keep the tensor-memory port busy, plus the
 * latency of a warp-to-warp mbarrier hand-over.  out_device: 256 int64 slots in device memory,
 * clocks per tile; `bench.py --mma-model` prints them with their labels.  Operands are zeros: this
 * measures time only.
 */
int pivot_debug_mma_model(long long* out_device, pivot_stream_t stream);

/*
 * Diagnostic (no counterpart in the paper): `ctas` CTAs each pull `tiles` consecutive 16 KB key
 * tiles (the shared scan's TMA box: 128 FP8 keys) of keys_device [n_keys, 128] (device, n_keys a
 * multiple of 128, L2-sized) through `stages` shared-memory stages and discard them: the rate at
 * which L2 feeds the key stream of Eq. 5's scan to all SMs at once.  mode 0: one TMA stream per CTA
 * (stages 1..12); mode 1: two independent TMA streams; mode 2: a TMA stream plus a stream of 16-byte
 * cp.async copies by four warps (stages 1..6 each); mode 3: one stream whose tiles are issued as
 * four 32-key boxes by one thread; mode 4: the same boxes issued by four lanes.  out_device[2 cta], [2 cta + 1] = clocks per tile
 * of the CTA's first / second stream (int64, device, 2 * ctas slots).
 */
int pivot_debug_key_stream(const void* keys_device, int n_keys, int ctas, int tiles, int stages, int mode,
                           long long* out_device, pivot_stream_t stream);

/*
 * Diagnostic (no counterpart in the paper): cycle counters of a library built with -DPIVOT_PROF
 * (`python -m paper_2607_24593_b200.build --variant prof -DPIVOT_PROF`), summed over all CTAs and
 * calls since the last read: where the thread that issues the tensor-core instructions of Eq. 5's
 * scan and of Eq. 8's re-score waits, how long the re-score's select warps take for Eq. 9, and the
 * phases of the decode step's top-c select (Eq. 7).  out (host) receives the first n <= 28 slots
 * (ProfSlot in csrc/common.cuh) of the workspace last used on this device and the slots are
 * cleared; the first read after a workspace is registered returns whatever the memory held.
 * Synchronises on `stream`.  PIVOT_ERR_UNSUPPORTED in an ordinary build, PIVOT_ERR_WORKSPACE
 * before any call.
 */
int pivot_debug_counters(pivot_stream_t stream, unsigned long long* out, int n);

/*
 * Per-stage timing, off by default.  While enabled, every call records CUDA events on its own
 * stream around its stages; pivot_stage_times synchronises on the last call's final event and
 * returns elapsed milliseconds: ms[0] proxy build (Eq. 4), ms[1] planner, ms[2] shared scan +
 * streaming select (Eq. 5-7, and the dense rows), ms[3] gather + re-score + top-k (Eq. 8-9),
 * ms[4] the whole call.  n must be at least 5; with n >= 6, ms[5] is the key-streaming scan kernel
 * of the last decode call (0 if the last call was not a decode call) and, with n >= 7, ms[6] its
 * per-sequence top-c select kernel (Eq. 6 / Eq. 7).  For decode calls ms[2] covers scan, select,
 * re-score and top-k together.  Not thread-safe.
 */
int pivot_stage_timing(int enable);
int pivot_stage_times(float* ms, int n);

/* Kernel launches issued by the library since the last call of this function (host counter). */
long long pivot_launch_count_reset(void);

const char* pivot_status_str(int code);
int pivot_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PIVOT_H_ */
