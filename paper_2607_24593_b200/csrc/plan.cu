// Planner kernels: turn a call's geometry into row descriptors (one per scan row) and group
// descriptors (one per Refine group).  Grouping follows Eq. 2 (prefill) and Eq. 3 (decode);
// the short-group guardrail of Algorithm 1 decides which rows are dense.
#include "kernels.h"
#include "plan.cuh"

namespace pivot {

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
      gd.k_stride = p.k_stride;
      gd.cand = r.out;
      gd.n_cand = p.W > 0 ? p.c : min(p.c, r.n_vis);   // with a window every slot is read (pads are skipped)
      gd.m = m;
      gd.K = p.k;
      gd.first_pos = t0;
      gd.pos_max = t0 + m - 1;
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

__global__ void plan_decode_kernel(DecodePlan p, RowDesc* rows, GroupDesc* groups) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.B) return;
  if (!plan_decode_sequence(p, b, rows, groups)) fill_decode_rows_empty(p, b, 0, 1);
  if (p.raw_q) raw_query_gates(p, b, 0, 1);
}

void launch_plan_decode(const DecodePlan& p, RowDesc* rows, GroupDesc* groups, cudaStream_t st) {
  plan_decode_kernel<<<(p.B + 127) / 128, 128, 0, st>>>(p, rows, groups);
  ++launch_counter();
}

}  // namespace pivot
