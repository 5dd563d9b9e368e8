// Device-side planners shared by the planner kernels and the decode path's fused prepare kernel.
#pragma once
#include "kernels.h"

namespace pivot {

// The fine-step kernels take at most kMembersPerDesc members per descriptor (the MMA N side is
// 4 x 64 heads); a larger group is split into chunks that share the candidate list.  Chunk
// slots without members get n_cand = 0 and are skipped.
__device__ __forceinline__ void put_group_chunks(GroupDesc* slots, const GroupDesc& full, int g, int dtype) {
  const size_t esz = dtype == DT_FP8 ? 1 : 2;
  const int chunks = (g + kMembersPerDesc - 1) / kMembersPerDesc;
  for (int ch = 0; ch < chunks; ++ch) {
    GroupDesc gd = full;
    const int first = ch * kMembersPerDesc;
    const int m = full.m - first;
    gd.m = m < kMembersPerDesc ? (m > 0 ? m : 0) : kMembersPerDesc;
    if (gd.m == 0) gd.n_cand = 0;
    gd.q = (const char*)full.q + (size_t)first * kHeads * kDim * esz;
    gd.w = full.w + (size_t)first * kHeads;
    gd.qscale = full.qscale ? full.qscale + (size_t)first * kHeads : nullptr;
    gd.first_pos = full.first_pos + first;
    gd.q_row = full.q_row + first;
    gd.out = full.out + (size_t)first * full.out_stride;
    gd.out_score = full.out_score ? full.out_score + (size_t)first * full.out_stride : nullptr;
    slots[ch] = gd;
  }
}

// Decode, one sequence: scan-row slot b is sequence b's proxy row; slots B + b*g + i are its dense rows.
// Exactly one of the two kinds is live per sequence (the guard test runs here because pos0
// lives on the device); dead slots get K = 0 and are skipped by the kernels.
// The cache of a sequence holds Lmax rows and the step reads keys 0 .. pos0 + g - 1: a pos0 outside
// [0, Lmax - g] would send the scan past the sequence's rows (into the next sequence, or past the
// block table).  Such a sequence gets no live slot at all, the status word reports DEV_BAD_POS, and
// the function returns false so that the caller fills the sequence's output rows with -1.
__device__ __forceinline__ bool plan_decode_sequence(const DecodePlan& p, int b, RowDesc* rows, GroupDesc* groups) {
  const size_t esz = p.dtype == DT_FP8 ? 1 : 2;
  const size_t qrow = (size_t)kHeads * kDim * esz;
  const int cb = b / p.kv_share;                 // whose key cache (and pos0) this slot uses
  const int p_in = p.pos0[cb];
  const int step = p.g > p.kv_share ? p.g : p.kv_share;          // queries of the MTP step
  const bool bad = p_in < 0 || p_in > p.Lmax - step;
  if (bad) set_status(p.status, DEV_BAD_POS);
  const int p0 = bad ? 0 : p_in + b % p.kv_share;
  const int n0 = p0 + 1;
  const bool guarded = n0 < p.guard_len;
  // Paged cache: descriptors point at the page pool and carry the sequence's block-table row.
  const bool paged = p.block_table != nullptr;
  const int32_t* pages = paged ? p.block_table + (size_t)cb * (p.Lmax / 128) : nullptr;
  const size_t krow = p.k_stride > 0 ? (size_t)p.k_stride : kDim * esz;                       // bytes per key row
  const void* kb = paged ? p.kc : (const char*)p.kc + (size_t)cb * p.Lmax * krow;
  const float* ksb = !p.kscale ? nullptr : paged ? p.kscale : p.kscale + (size_t)cb * p.Lmax;
  int32_t* outb = p.out + (size_t)b * p.g * p.k;
  float* outsb = p.out_score ? p.out_score + (size_t)b * p.g * p.k : nullptr;
  RowDesc r;
  r.q = (const char*)(p.raw_q ? p.q : p.proxy_q) + (size_t)b * qrow;
  r.w = p.proxy_w + (size_t)b * kHeads;
  r.qscale = nullptr;
  r.kbase = kb;
  r.kscale = ksb;
  r.n_vis = n0;
  r.q_map = p.raw_q ? 0 : 1; r.q_row = b; r.k_row0 = paged ? 0 : cb * p.Lmax;
  r.pages = pages;
  GroupDesc gd;
  gd.pages = pages;
  gd.n_pages = p.n_pages;
  gd.q = (const char*)p.q + (size_t)b * p.g * qrow;
  gd.w = p.w + (size_t)b * p.g * kHeads;
  gd.qscale = p.qscale ? p.qscale + (size_t)b * p.g * kHeads : nullptr;
  gd.kbase = kb;
  gd.kscale = ksb;
  gd.k_stride = p.k_stride;
  gd.cand = p.cand + (size_t)b * p.c;
  gd.n_cand = 0;
  gd.m = p.g;
  gd.K = p.k;
  gd.first_pos = p0;
  gd.pos_max = p0 + p.g - 1;
  gd.q_row = b * p.g;
  gd.out = outb;
  gd.out_score = outsb;
  gd.out_stride = p.k;
  gd.ent_out = nullptr; gd.ent_stride = 0; gd.slot0 = 0;
  if (guarded || bad) {
    r.K = 0; r.out = nullptr; r.out_score = nullptr; r.out_rows = 0; r.out_stride = 0;
  } else if (p.mode == 0) {
    r.K = p.k; r.out = outb; r.out_score = outsb; r.out_rows = p.g; r.out_stride = p.k;
  } else {
    r.K = p.c; r.out = p.cand + (size_t)b * p.c;
    r.out_score = p.cand_score ? p.cand_score + (size_t)b * p.c : nullptr;
    r.out_rows = 1; r.out_stride = p.c;
    gd.n_cand = min(p.c, n0);
  }
  rows[b] = r;
  put_group_chunks(groups + (size_t)b * ((p.g + kMembersPerDesc - 1) / kMembersPerDesc), gd, p.g, p.dtype);
  for (int i = 0; i < p.g; ++i) {
    RowDesc dr;
    dr.q = (const char*)p.q + ((size_t)b * p.g + i) * qrow;
    dr.w = p.w + ((size_t)b * p.g + i) * kHeads;
    dr.qscale = p.qscale ? p.qscale + ((size_t)b * p.g + i) * kHeads : nullptr;
    dr.kbase = kb;
    dr.kscale = ksb;
    dr.n_vis = p0 + i + 1;
    dr.K = (guarded && !bad) ? p.k : 0;
    dr.out = outb + (size_t)i * p.k;
    dr.out_score = outsb ? outsb + (size_t)i * p.k : nullptr;
    dr.out_rows = 1;
    dr.out_stride = p.k;
    dr.q_map = 0; dr.q_row = b * p.g + i; dr.k_row0 = cb * p.Lmax;
    rows[p.B + b * p.g + i] = dr;
  }
  return !bad;
}

// Dense control: the scan row of slot b is the raw query b, whose effective gate fl32(w * qscale)
// (Appendix A: the gate absorbs the query scale) goes where a proxy's gate would be.
__device__ __forceinline__ void raw_query_gates(const DecodePlan& p, int b, int tid, int nthreads) {
  for (int j = tid; j < kHeads; j += nthreads) {
    const size_t i = (size_t)b * kHeads + j;
    p.proxy_w[i] = p.qscale ? __fmul_rn(p.w[i], p.qscale[i]) : p.w[i];
  }
}

// Output rows of a sequence that was not indexed (bad pos0): every entry -1 (scores -inf).
__device__ __forceinline__ void fill_decode_rows_empty(const DecodePlan& p, int b, int tid, int nthreads) {
  for (int i = tid; i < p.g * p.k; i += nthreads) {
    p.out[(size_t)b * p.g * p.k + i] = -1;
    if (p.out_score) p.out_score[(size_t)b * p.g * p.k + i] = -INFINITY;
  }
}

}  // namespace pivot
