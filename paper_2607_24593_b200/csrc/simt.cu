// CUDA-core (no tensor core) scan + select and gather + re-score kernels.
//
// These are the plain, easily checked producers of the same streams the tensor-core kernels
// emit: one thread scores one key against one row (Eq. 1 / Eq. 5 / Eq. 8) with fp32 FMAs in a
// fixed order, then the streaming top-K machinery (filter by the running threshold, append to
// the candidate buffer, exact radix compaction when it fills) keeps the K best.
#include "kernels.h"
#include "select.cuh"

namespace pivot {

constexpr int SIMT_THREADS = 256;

struct RowSmem {
  alignas(16) float q[kHeads][kDim];   // decoded query codes (read as float4)
  float w[kHeads];         // effective gate
  SelectSmem sel;
  uint32_t count;          // entries in the current candidate buffer
  int row;                 // scheduler hand-off
};

__device__ __forceinline__ void load_row_operands(RowSmem& sm, const void* q, const float* w,
                                                  const float* qscale, int dtype) {
  for (int i = threadIdx.x; i < kHeads * kDim; i += SIMT_THREADS) {
    float v = dtype == DT_FP8 ? e4m3_to_float(reinterpret_cast<const uint8_t*>(q)[i])
                              : bf16_bits_to_float(reinterpret_cast<const uint16_t*>(q)[i]);
    (&sm.q[0][0])[i] = v;
  }
  if (threadIdx.x < kHeads)
    sm.w[threadIdx.x] = qscale ? __fmul_rn(w[threadIdx.x], qscale[threadIdx.x]) : w[threadIdx.x];
}

// Score of key s against the row staged in sm (Eq. 1 with the FP8 form of Appendix A).
__device__ __forceinline__ float score_one(const RowSmem& sm, const void* kbase,
                                           const float* kscale, int s, int dtype) {
  float kv[kDim];
  if (dtype == DT_FP8) {
    const uint4* p = reinterpret_cast<const uint4*>((const uint8_t*)kbase + (size_t)s * kDim);
#pragma unroll
    for (int c = 0; c < kDim / 16; ++c) {
      uint4 v = p[c];
      uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) kv[c * 16 + j * 4 + e] = e4m3_to_float((wv[j] >> (8 * e)) & 0xff);
    }
  } else {
    const uint4* p = reinterpret_cast<const uint4*>((const uint16_t*)kbase + (size_t)s * kDim);
#pragma unroll
    for (int c = 0; c < kDim / 8; ++c) {
      uint4 v = p[c];
      uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        kv[c * 8 + j * 2] = bf16_bits_to_float(wv[j] & 0xffff);
        kv[c * 8 + j * 2 + 1] = bf16_bits_to_float(wv[j] >> 16);
      }
    }
  }
  float total = 0.f;
  for (int h = 0; h < kHeads; ++h) {
    float dot = 0.f;
    const float4* qh = reinterpret_cast<const float4*>(&sm.q[h][0]);
#pragma unroll
    for (int i = 0; i < kDim / 4; ++i) {
      float4 qv = qh[i];
      dot = fmaf(qv.x, kv[4 * i], dot);
      dot = fmaf(qv.y, kv[4 * i + 1], dot);
      dot = fmaf(qv.z, kv[4 * i + 2], dot);
      dot = fmaf(qv.w, kv[4 * i + 3], dot);
    }
    total = fmaf(sm.w[h], fmaxf(dot, 0.f), total);
  }
  if (kscale) total *= kscale[s];
  return total;
}

// Appends the entries flagged `take` (one per thread) to the candidate buffer.
__device__ __forceinline__ void append(RowSmem& sm, uint32_t* ckey, int32_t* cidx, bool take,
                                       uint32_t key, int32_t idx) {
  const int lane = threadIdx.x & 31;
  uint32_t m = __ballot_sync(0xffffffffu, take);
  if (m) {
    uint32_t pos = 0;
    const int leader = __ffs(m) - 1;
    if (lane == leader) pos = atomicAdd(&sm.count, (uint32_t)__popc(m));
    pos = __shfl_sync(0xffffffffu, pos, leader);
    if (take) {
      uint32_t p = pos + __popc(m & ((1u << lane) - 1u));
      ckey[p] = key;
      cidx[p] = idx;
    }
  }
}

__device__ __forceinline__ void emit(const RowSmem&, const Team& tm, int32_t* out, float* out_score,
                                     int n_valid, int K, int out_rows, int out_stride) {
  // pad the first row, then replicate it (Reuse shares one set across the group)
  for (int i = n_valid + tm.tid; i < K; i += tm.nthr) {
    out[i] = -1;
    if (out_score) out_score[i] = -INFINITY;
  }
  tm.sync();
  for (int r = 1; r < out_rows; ++r)
    for (int i = tm.tid; i < K; i += tm.nthr) {
      out[(size_t)r * out_stride + i] = out[i];
      if (out_score) out_score[(size_t)r * out_stride + i] = out_score[i];
    }
}

__global__ void __launch_bounds__(SIMT_THREADS)
scan_select_simt_kernel(const RowDesc* __restrict__ rows, int n_rows, int dtype, ScanScratch sc) {
  __shared__ RowSmem sm;
  const Team tm{(int)threadIdx.x, SIMT_THREADS, 0};
  uint32_t* kbuf[2] = {sc.cand_key + (size_t)blockIdx.x * 2 * sc.cap,
                       sc.cand_key + (size_t)blockIdx.x * 2 * sc.cap + sc.cap};
  int32_t* ibuf[2] = {sc.cand_idx + (size_t)blockIdx.x * 2 * sc.cap,
                      sc.cand_idx + (size_t)blockIdx.x * 2 * sc.cap + sc.cap};
  // longest rows first: row ids are handed out from the top
  for (int it = blockIdx.x; it < n_rows; it += gridDim.x) {
    const RowDesc rd = rows[n_rows - 1 - it];
    if (rd.K <= 0) continue;
    __syncthreads();
    load_row_operands(sm, rd.q, rd.w, rd.qscale, dtype);
    if (threadIdx.x == 0) sm.count = 0;
    __syncthreads();
    int cur = 0;
    bool have_tau = false;
    uint32_t tau = 0;
    for (int base = 0; base < rd.n_vis; base += SIMT_THREADS) {
      if ((int)sm.count + SIMT_THREADS > sc.cap) {        // compaction: keep the exact top-K
        const int n = (int)sm.count;
        __syncthreads();
        team_select_topk(tm, sm.sel, kbuf[cur], ibuf[cur], n, rd.K, kbuf[cur ^ 1], ibuf[cur ^ 1],
                         nullptr, &sm.sel.hist[0]);
        tau = sm.sel.hist[0];
        have_tau = true;
        __syncthreads();
        if (threadIdx.x == 0) sm.count = (uint32_t)rd.K;
        cur ^= 1;
        __syncthreads();
      }
      const int s = base + threadIdx.x;
      bool take = false;
      uint32_t key = 0;
      if (s < rd.n_vis) {
        key = score_to_key(score_one(sm, rd.kbase, rd.kscale, s, dtype));
        // keys arrive in index order, so an equal key loses the tie-break against the buffer
        take = !have_tau || key > tau;
      }
      append(sm, kbuf[cur], ibuf[cur], take, key, s);
      __syncthreads();
    }
    const int n = (int)sm.count;
    int n_valid = n;
    if (n > rd.K) {
      team_select_topk(tm, sm.sel, kbuf[cur], ibuf[cur], n, rd.K, nullptr, rd.out, rd.out_score, nullptr);
      n_valid = rd.K;
    } else {
      for (int i = threadIdx.x; i < n; i += SIMT_THREADS) {
        rd.out[i] = ibuf[cur][i];
        if (rd.out_score) rd.out_score[i] = key_to_score(kbuf[cur][i]);
      }
    }
    __syncthreads();
    emit(sm, tm, rd.out, rd.out_score, n_valid, rd.K, rd.out_rows, rd.out_stride);
  }
}

void launch_scan_simt(const RowDesc* rows, int n_rows, int dtype, const ScanScratch& s, cudaStream_t st) {
  if (n_rows <= 0) return;
  const int grid = n_rows < s.n_cta ? n_rows : s.n_cta;
  scan_select_simt_kernel<<<grid, SIMT_THREADS, 0, st>>>(rows, n_rows, dtype, s);
  ++launch_counter();
}

// Gather + re-score + per-query top-k (Eq. 8-9): one block per group, members in turn.
__global__ void __launch_bounds__(SIMT_THREADS)
refine_simt_kernel(const GroupDesc* __restrict__ groups, int n_groups, int dtype, ScanScratch sc) {
  __shared__ RowSmem sm;
  const Team tm{(int)threadIdx.x, SIMT_THREADS, 0};
  uint32_t* kbuf = sc.cand_key + (size_t)blockIdx.x * 2 * sc.cap;
  int32_t* ibuf = sc.cand_idx + (size_t)blockIdx.x * 2 * sc.cap;
  const size_t esz = dtype == DT_FP8 ? 1 : 2;
  for (int gi = blockIdx.x; gi < n_groups; gi += gridDim.x) {
    const GroupDesc gd = groups[gi];
    if (gd.n_cand <= 0) continue;
    for (int i = 0; i < gd.m; ++i) {
      __syncthreads();
      load_row_operands(sm, (const char*)gd.q + (size_t)i * kHeads * kDim * esz, gd.w + i * kHeads,
                        gd.qscale ? gd.qscale + i * kHeads : nullptr, dtype);
      __syncthreads();
      for (int j = threadIdx.x; j < gd.n_cand; j += SIMT_THREADS) {
        const int s = gd.cand[j];
        kbuf[j] = score_to_key(score_one(sm, gd.kbase, gd.kscale, s, dtype));
        ibuf[j] = s;
      }
      __syncthreads();
      int32_t* out = gd.out + (size_t)i * gd.out_stride;
      float* outs = gd.out_score ? gd.out_score + (size_t)i * gd.out_stride : nullptr;
      int n_valid = gd.n_cand;
      if (gd.n_cand > gd.K) {
        team_select_topk(tm, sm.sel, kbuf, ibuf, gd.n_cand, gd.K, nullptr, out, outs, nullptr);
        n_valid = gd.K;
      } else {
        for (int j = threadIdx.x; j < gd.n_cand; j += SIMT_THREADS) {
          out[j] = ibuf[j];
          if (outs) outs[j] = key_to_score(kbuf[j]);
        }
      }
      __syncthreads();
      emit(sm, tm, out, outs, n_valid, gd.K, 1, gd.out_stride);
    }
  }
}

void launch_refine_simt(const GroupDesc* groups, int n_groups, int dtype, const ScanScratch& s, cudaStream_t st) {
  if (n_groups <= 0) return;
  const int grid = n_groups < s.n_cta ? n_groups : s.n_cta;
  refine_simt_kernel<<<grid, SIMT_THREADS, 0, st>>>(groups, n_groups, dtype, s);
  ++launch_counter();
}

}  // namespace pivot
