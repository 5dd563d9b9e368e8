// Planner kernels: turn a call's geometry into row descriptors (one per scan row) and group
// descriptors (one per Refine group).  Grouping follows Eq. 2 (prefill) and Eq. 3 (decode);
// the short-group guardrail of Algorithm 1 decides which rows are dense.
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

// Scan-row order for prefill: rows [0, n_dense) are dense rows (row i = query i), rows
// [n_dense, n_dense + n_proxy) are proxy rows.
__global__ void plan_prefill_kernel(PrefillPlan p, RowDesc* rows, GroupDesc* groups) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const size_t esz = p.dtype == DT_FP8 ? 1 : 2;
  const size_t qrow = (size_t)kHeads * kDim * esz;
  if (i < p.n_dense) {
    const int t = p.dense_begin + i;      // query row (= position) of this dense row
    RowDesc r;
    r.q = (const char*)p.q + (size_t)t * qrow;
    r.w = p.w + (size_t)t * kHeads;
    r.qscale = p.qscale ? p.qscale + (size_t)t * kHeads : nullptr;
    r.kbase = p.kc;
    r.kscale = p.kscale;
    r.n_vis = t + 1;
    r.K = p.k;
    r.out = p.out + (size_t)t * p.k;
    r.out_score = p.out_score ? p.out_score + (size_t)t * p.k : nullptr;
    r.out_rows = 1;
    r.out_stride = p.k;
    r.q_map = 0; r.q_row = t; r.k_row0 = 0;
    rows[i] = r;
  } else if (i < p.n_dense + p.n_proxy) {
    const int pr = i - p.n_dense;
    const int t0 = (p.first_group + pr) * p.g;
    const int m = min(p.g, p.L - t0);
    RowDesc r;
    r.q = (const char*)p.proxy_q + (size_t)pr * qrow;
    r.w = p.proxy_w + (size_t)pr * kHeads;
    r.qscale = nullptr;
    r.kbase = p.kc;
    r.kscale = p.kscale;
    // With a local window the proxy ranks s <= t0 - W only (Appendix B); the window itself is
    // appended to the candidate set below.
    r.n_vis = p.W > 0 ? max(t0 - p.W + 1, 0) : t0 + 1;
    r.q_map = 1; r.q_row = pr; r.k_row0 = 0;
    if (p.mode == 0) {   // Reuse: the proxy top-k goes to every member (Eq. 6)
      r.K = p.k;
      r.out = p.out + (size_t)t0 * p.k;
      r.out_score = p.out_score ? p.out_score + (size_t)t0 * p.k : nullptr;
      r.out_rows = m;
      r.out_stride = p.k;
    } else {             // Refine: top-c candidate set (Eq. 7)
      const int w_g = p.W > 0 ? p.W + m - 1 : 0;      // slots reserved for the window union
      r.K = p.c - w_g;
      r.out = p.cand + (size_t)pr * p.c;
      for (int j = 0; j < w_g; ++j) {                 // t0-W+1 .. t0+m-1, ascending
        const int s = t0 - p.W + 1 + j;
        p.cand[(size_t)pr * p.c + (p.c - w_g) + j] = s >= 0 ? s : -1;
        if (p.cand_score) p.cand_score[(size_t)pr * p.c + (p.c - w_g) + j] = __int_as_float(0x7fc00000);
      }
      r.out_score = p.cand_score ? p.cand_score + (size_t)pr * p.c : nullptr;
      r.out_rows = 1;
      r.out_stride = p.c;
      GroupDesc gd;
      gd.q = (const char*)p.q + (size_t)t0 * qrow;
      gd.w = p.w + (size_t)t0 * kHeads;
      gd.qscale = p.qscale ? p.qscale + (size_t)t0 * kHeads : nullptr;
      gd.kbase = p.kc;
      gd.kscale = p.kscale;
      gd.cand = r.out;
      gd.n_cand = p.W > 0 ? p.c : min(p.c, r.n_vis);   // with a window every slot is read (pads are skipped)
      gd.m = m;
      gd.K = p.k;
      gd.first_pos = t0;
      gd.q_row = t0;
      gd.out = p.out + (size_t)t0 * p.k;
      gd.out_score = p.out_score ? p.out_score + (size_t)t0 * p.k : nullptr;
      gd.out_stride = p.k;
      gd.ent_out = nullptr; gd.ent_stride = 0; gd.slot0 = 0;
      const int chunks = (p.g + kMembersPerDesc - 1) / kMembersPerDesc;
      put_group_chunks(groups + (size_t)pr * chunks, gd, p.g, p.dtype);
    }
    rows[i] = r;
  }
}

void launch_plan_prefill(const PrefillPlan& p, RowDesc* rows, GroupDesc* groups, cudaStream_t st) {
  const int n = p.n_dense + p.n_proxy;
  if (n <= 0) return;
  plan_prefill_kernel<<<(n + 255) / 256, 256, 0, st>>>(p, rows, groups);
  ++launch_counter();
}

// Decode: scan-row slot b is sequence b's proxy row; slots B + b*g + i are its dense rows.
// Exactly one of the two kinds is live per sequence (the guard test runs here because pos0
// lives on the device); dead slots get K = 0 and are skipped by the kernels.
__global__ void plan_decode_kernel(DecodePlan p, RowDesc* rows, GroupDesc* groups) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.B) return;
  const size_t esz = p.dtype == DT_FP8 ? 1 : 2;
  const size_t qrow = (size_t)kHeads * kDim * esz;
  const int p0 = p.pos0[b];
  const int n0 = p0 + 1;
  const bool guarded = n0 < p.guard_len;
  // Paged cache: descriptors point at the page pool and carry the sequence's block-table row.
  const bool paged = p.block_table != nullptr;
  const int32_t* pages = paged ? p.block_table + (size_t)b * (p.Lmax / 128) : nullptr;
  const void* kb = paged ? p.kc : (const char*)p.kc + (size_t)b * p.Lmax * kDim * esz;
  const float* ksb = !p.kscale ? nullptr : paged ? p.kscale : p.kscale + (size_t)b * p.Lmax;
  int32_t* outb = p.out + (size_t)b * p.g * p.k;
  float* outsb = p.out_score ? p.out_score + (size_t)b * p.g * p.k : nullptr;
  RowDesc r;
  r.q = (const char*)p.proxy_q + (size_t)b * qrow;
  r.w = p.proxy_w + (size_t)b * kHeads;
  r.qscale = nullptr;
  r.kbase = kb;
  r.kscale = ksb;
  r.n_vis = n0;
  r.q_map = 1; r.q_row = b; r.k_row0 = paged ? 0 : b * p.Lmax;
  r.pages = pages;
  GroupDesc gd;
  gd.pages = pages;
  gd.n_pages = p.n_pages;
  gd.q = (const char*)p.q + (size_t)b * p.g * qrow;
  gd.w = p.w + (size_t)b * p.g * kHeads;
  gd.qscale = p.qscale ? p.qscale + (size_t)b * p.g * kHeads : nullptr;
  gd.kbase = kb;
  gd.kscale = ksb;
  gd.cand = p.cand + (size_t)b * p.c;
  gd.n_cand = 0;
  gd.m = p.g;
  gd.K = p.k;
  gd.first_pos = p0;
  gd.q_row = b * p.g;
  gd.out = outb;
  gd.out_score = outsb;
  gd.out_stride = p.k;
  gd.ent_out = nullptr; gd.ent_stride = 0; gd.slot0 = 0;
  if (guarded) {
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
    dr.K = guarded ? p.k : 0;
    dr.out = outb + (size_t)i * p.k;
    dr.out_score = outsb ? outsb + (size_t)i * p.k : nullptr;
    dr.out_rows = 1;
    dr.out_stride = p.k;
    dr.q_map = 0; dr.q_row = b * p.g + i; dr.k_row0 = b * p.Lmax;
    rows[p.B + b * p.g + i] = dr;
  }
}

void launch_plan_decode(const DecodePlan& p, RowDesc* rows, GroupDesc* groups, cudaStream_t st) {
  plan_decode_kernel<<<(p.B + 127) / 128, 128, 0, st>>>(p, rows, groups);
  ++launch_counter();
}

}  // namespace pivot
