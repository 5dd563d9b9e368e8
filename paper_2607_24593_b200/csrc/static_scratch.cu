// dense_index_static: the dense indexer (Eq. 1 + TopK) for callers that cannot allocate.
//
// Some hosts of this library may not call cudaMalloc at all: a plugin running inside an
// inference server that owns the whole device heap, or code that runs under a memory-pool
// policy where every device allocation must come from the framework.  For them this entry
// point runs the same tensor-core scan + streaming select as dense_index, but takes its scratch
// (row descriptors, candidate segments, status word) from a fixed array that is part of the
// library image instead of a caller workspace.  The price is a size limit and a smaller grid.
//
// The array lives in device memory of every GPU that loads the library, until the process
// exits.  Its name is only a host-side handle: the device address is looked up once per device
// with cudaGetSymbolAddress (first call on that device) and that address is what the kernels get.
#include "../../include/pivot.h"
#include "api_internal.h"
#include "kernels.h"

using namespace pivot;

namespace {

constexpr size_t kStaticBytes = (size_t)8 << 20;          // 8 MiB per GPU
constexpr int kStaticMaxL = 4096;
constexpr int kStaticMaxK = 512;
constexpr int kStaticCtas = 24;                           // grid cap: 24 x 4 rows x 2 segments x 4096 entries x 8 B = 6 MiB
// (4096 entries per row = eight warp segments of 512 = the largest k this entry point accepts)
constexpr int kStaticCap = 4096;                          // candidate entries per row
constexpr int kMaxDev = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

void* g_scratch_ptr[kMaxDev];   // device address of the array, per device (nullptr: not looked up yet)

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int dense_index_static(const pivot_tensor* q, const float* w, const pivot_tensor* kcache, int L,
                                  int H_I, int d, int k, int32_t* out_idx, pivot_stream_t stream) {
  // the same argument checks as dense_index (pointers, operand types, alignment, shapes)
  if (int rc = check_operands(q, w, kcache, H_I, d, k, k, PIVOT_REUSE, out_idx)) return rc;
  if (L < 1) return PIVOT_ERR_INVALID_ARG;
  if (L > kStaticMaxL || k > kStaticMaxK) return PIVOT_ERR_WORKSPACE;   // beyond the built-in scratch
  cudaStream_t st = (cudaStream_t)stream;

  int dev = 0;
  if (int rc = record_cuda(cudaGetDevice(&dev))) return rc;
  if (dev < 0 || dev >= kMaxDev) return PIVOT_ERR_UNSUPPORTED;
  if (!g_scratch_ptr[dev]) {       // one-time set-up on this device (do it before any stream capture)
    void* p = nullptr;
    if (int rc = record_cuda(cudaGetSymbolAddress(&p, g_static_scratch))) return rc;
    if (!p) return PIVOT_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  char* base = (char*)g_scratch_ptr[dev];
  size_t off = 0;
  int* status = (int*)(base + off);                     off += 256;
  RowDesc* rows = (RowDesc*)(base + off);               off += up256(sizeof(RowDesc) * (size_t)kStaticMaxL);
  unsigned long long* cand = (unsigned long long*)(base + off);
  off += (size_t)kStaticCtas * 4 * 2 * kStaticCap * sizeof(unsigned long long);   // two segments per row
  if (off > kStaticBytes) return PIVOT_ERR_WORKSPACE;

  // The array keeps whatever the previous call left: the status word must start at zero; row
  // descriptors are rewritten for rows 0..L-1 and candidate cursors start at zero in registers.
  if (int rc = record_cuda(cudaMemsetAsync(status, 0, 2 * sizeof(int), st))) return rc;

  PrefillPlan p;
  p.q = q->data; p.w = w; p.qscale = q->scale;
  p.kc = kcache->data; p.kscale = kcache->scale;
  p.proxy_q = nullptr; p.proxy_w = nullptr; p.cand = nullptr; p.cand_score = nullptr;
  p.out = out_idx; p.out_score = nullptr;
  p.L = L; p.g = 1; p.c = k; p.k = k; p.mode = 0; p.dtype = q->dtype;
  p.W = 0; p.dense_begin = 0; p.n_dense = L; p.first_group = L; p.n_proxy = 0;
  launch_plan_prefill(p, rows, nullptr, st);

  ScanScratch sc;
  sc.cand_key = nullptr; sc.cand_idx = nullptr;
  sc.cand64 = cand;
  sc.cap = kStaticCap;
  sc.n_cta = kStaticCtas;
  sc.status = status;
  sc.counter = status + 1;
  // the proxy tensor map needs some valid address; no row refers to it
  ScanOperands op{kcache->data, L, kcache->scale, q->data, L, q->data, 1, q->dtype};
  {
    const size_t row = (size_t)kDim * (kcache->dtype == PIVOT_FP8_E4M3 ? 1 : 2);
    op.k_stride = kcache->stride_row == 0 || kcache->stride_row == row ? 0 : (int)kcache->stride_row;
  }
  if (int rc = record_cuda(launch_scan_tc(op, rows, L, 4, sc, kStaticCtas, st))) return rc;
  return record_cuda(cudaGetLastError());
}
