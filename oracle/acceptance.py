"""Acceptance rule that compares index sets / scores produced elsewhere with the oracle's.
TEST INFRASTRUCTURE ONLY (used by tests, the smoke check and the benchmark's parity probe).

Index sets must equal the oracle's except for keys whose oracle score lies within the score
tolerance of the K-th threshold (either side): there the two selections may differ, because
the other implementation ranks by its own fp32 / low-precision scores.  Scores must agree as
|a - b| <= atol + rtol * |b| with rtol = 2e-2 (FP8) or 5e-3 (bf16) and atol = 1e-3.

Refine is checked in two conditional stages so that a swap at the c-th threshold cannot pass
for (or hide) an error of the fine step: (i) the candidate set against the proxy scores
(Eq. 5 / Eq. 7); (ii) each member's final set against the oracle's Eq. 8-9 evaluated on the
candidate set that was actually produced.
"""
from __future__ import annotations

import dataclasses

import numpy as np

from . import pivot_oracle as po

ATOL = 1e-3
RTOL = {"bf16": 5e-3, "fp8": 2e-2}


@dataclasses.dataclass
class Tally:
    rows: int = 0
    exact_rows: int = 0          # rows whose set equals the oracle's own selection
    band_swaps: int = 0          # entries that differ but lie inside the tolerance band
    scores_checked: int = 0
    max_score_err: float = 0.0   # max |gpu - oracle| / (atol + rtol |oracle|)

    def merge(self, o: "Tally"):
        self.rows += o.rows
        self.exact_rows += o.exact_rows
        self.band_swaps += o.band_swaps
        self.scores_checked += o.scores_checked
        self.max_score_err = max(self.max_score_err, o.max_score_err)


def check_selection(got_idx, scores, index, K, rtol, tally: Tally, what="", got_scores=None):
    """got_idx: K int32 entries (-1 padded) chosen among `index` (key positions, ascending or
    not) whose oracle scores are `scores`.  Asserts validity and the band rule."""
    index = np.asarray(index, dtype=np.int64)
    n = len(index)
    want_n = min(K, n)
    got = np.asarray(got_idx, dtype=np.int64)
    valid = got[:want_n]
    assert (got[want_n:] == -1).all(), f"{what}: entries beyond the {want_n} visible keys must be -1"
    assert (valid >= 0).all(), f"{what}: -1 among the first {want_n} entries"
    assert len(np.unique(valid)) == want_n, f"{what}: duplicate indices"
    pos = {int(s): j for j, s in enumerate(index)}
    try:
        slots = np.array([pos[int(s)] for s in valid], dtype=np.int64)
    except KeyError as e:
        raise AssertionError(f"{what}: index {e} is not among the allowed keys") from None
    tally.rows += 1
    want = po.top_set(scores, K, index)
    if set(want.tolist()) == set(valid.tolist()):
        tally.exact_rows += 1
    elif want_n < n:
        order = np.sort(scores)[::-1]
        tau = order[want_n - 1]
        tol = ATOL + rtol * abs(tau)
        chosen = np.zeros(n, bool)
        chosen[slots] = True
        lo = scores[chosen].min()
        hi = scores[~chosen].max()
        assert lo >= tau - tol, f"{what}: selected a key scoring {lo} below threshold {tau} - {tol}"
        assert hi <= tau + tol, f"{what}: missed a key scoring {hi} above threshold {tau} + {tol}"
        tally.band_swaps += len(set(valid.tolist()) - set(want.tolist()))
    else:
        raise AssertionError(f"{what}: all {n} keys must be selected")
    if got_scores is not None:
        gs = np.asarray(got_scores, dtype=np.float64)[:want_n]
        ref = scores[slots]
        err = np.abs(gs - ref) / (ATOL + rtol * np.abs(ref))
        tally.scores_checked += want_n
        tally.max_score_err = max(tally.max_score_err, float(err.max()) if want_n else 0.0)
        assert (err <= 1.0).all(), f"{what}: score mismatch, worst {err.max():.3f} x tolerance"
        pad = np.asarray(got_scores)[want_n:]
        assert np.all(np.isneginf(pad)), f"{what}: padded scores must be -inf"


def check_group(x: dict, kd, kscale, members, *, c, k, mode, guard_len, out_idx, out_scores=None,
                cand=None, cand_scores=None, q_rows=None, pool="mean", W=0, per_query_window=False) -> Tally:
    """Checks one group's rows of out_idx ([m, k]) (and candidates [c]) against the oracle.

    With a local window (Appendix B, W > 0) the proxy part of the candidate set is checked
    against the shortened scan, the window slots must hold t0-W+1 .. t0+m-1 in ascending order,
    and every member is checked on the slots it may see (positions <= its own).
    per_query_window (decode form): `cand` is the pool of c entries, checked as for W = 0, and
    each member is checked on the produced pool united with its own window [t-W+1, t]."""
    rtol = RTOL[x["dtype"]]
    t = Tally()
    r = po.pivot_group(x, members, kd, kscale, c=c, k=k, mode=mode, guard_len=guard_len, pool=pool,
                       q_rows=q_rows, W=W, per_query_window=per_query_window)
    W_own = W if per_query_window else 0
    if per_query_window:
        W = 0                      # pool and scan are those of the plain method
    m = len(r.members)
    if r.guarded:
        for i, tq in enumerate(r.members):
            check_selection(out_idx[i], r.member_scores[i], np.arange(tq + 1), k, rtol, t,
                            f"dense row t={tq}", None if out_scores is None else out_scores[i])
        return t
    n0 = r.t0 + 1 if W == 0 else max(r.t0 - W + 1, 0)      # keys the proxy scan ranks
    if mode == po.MODE_REUSE:
        for i, tq in enumerate(r.members):
            check_selection(out_idx[i], r.proxy_scores, np.arange(n0), k, rtol, t,
                            f"reuse row t={tq}", None if out_scores is None else out_scores[i])
            assert sorted(out_idx[i].tolist()) == sorted(out_idx[0].tolist()), "reuse rows must share one set"
        return t
    assert cand is not None, "Refine parity needs the candidate set"
    w_g = W + m - 1 if W > 0 else 0
    cp = c - w_g                                            # slots filled by the proxy scan
    check_selection(cand[:cp], r.proxy_scores, np.arange(n0), cp, rtol, t, f"candidates t0={r.t0}",
                    None if cand_scores is None else cand_scores[:cp])
    C = np.asarray(cand[: min(cp, n0)], dtype=np.int64)
    if w_g:
        win = np.arange(max(r.t0 - W + 1, 0), r.t0 + m, dtype=np.int64)
        got_win = np.asarray(cand[cp:], dtype=np.int64)
        assert np.array_equal(got_win[got_win >= 0], win), f"window slots of group t0={r.t0}"
        C = np.concatenate([C, win])
    rows = r.members if q_rows is None else np.asarray(q_rows)
    qs = None if x["qscale"] is None else x["qscale"][rows]
    qd, weff = po.member_operands(x["q"][rows], qs, x["w"][rows], x["dtype"])
    for i, tq in enumerate(r.members):
        Ci = C
        if W_own:
            win = np.arange(max(int(tq) - W_own + 1, 0), int(tq) + 1, dtype=np.int64)
            Ci = np.concatenate([C, np.setdiff1d(win, C)])
        s, _, ok = po.refine_on_candidates(qd[i], weff[i], kd, kscale, Ci, k, t_member=int(tq) if w_g else None)
        check_selection(out_idx[i], s[ok], Ci[ok], k, rtol, t, f"refine row t={tq}",
                        None if out_scores is None else out_scores[i])
    return t


def check_prefill(x: dict, *, g, c, k, mode, guard_len, out_idx, out_scores=None, cand=None,
                  cand_scores=None, groups=None, pool="mean", W=0) -> Tally:
    L = x["q"].shape[0]
    kd = po.decode_operand(x["k"], x["dtype"])
    allg = po.prefill_groups(L, g)
    total = Tally()
    for gi in (range(len(allg)) if groups is None else groups):
        mem = allg[gi]
        total.merge(check_group(
            x, kd, x["kscale"], mem, c=c, k=k, mode=mode, guard_len=guard_len,
            out_idx=out_idx[mem], out_scores=None if out_scores is None else out_scores[mem],
            cand=None if cand is None else cand[gi],
            cand_scores=None if cand_scores is None else cand_scores[gi], pool=pool, W=W))
    return total


def check_dense(x: dict, *, k, out_idx, out_scores=None, rows=None) -> Tally:
    L = x["q"].shape[0]
    res = po.dense_index(x, k=k, rows=rows)
    t = Tally()
    for tq, (s, _) in res.items():
        check_selection(out_idx[tq], s, np.arange(tq + 1), k, RTOL[x["dtype"]], t, f"dense row t={tq}",
                        None if out_scores is None else out_scores[tq])
    return t


def check_decode(x: dict, *, c, k, mode, guard_len, out_idx, out_scores=None, cand=None,
                 cand_scores=None, seqs=None, W=0) -> Tally:
    B, g = x["q"].shape[0], x["q"].shape[1]
    total = Tally()
    for b in (range(B) if seqs is None else seqs):
        p0 = int(x["pos0"][b])
        nk = p0 + g
        kd = po.decode_operand(x["k"][b, :nk], x["dtype"])
        ks = None if x["kscale"] is None else x["kscale"][b, :nk]
        xb = dict(dtype=x["dtype"], q=x["q"][b], qscale=None if x["qscale"] is None else x["qscale"][b],
                  w=x["w"][b])
        total.merge(check_group(
            xb, kd, ks, np.arange(p0, p0 + g), c=c, k=k, mode=mode, guard_len=guard_len,
            out_idx=out_idx[b], out_scores=None if out_scores is None else out_scores[b],
            cand=None if cand is None else cand[b],
            cand_scores=None if cand_scores is None else cand_scores[b], q_rows=np.arange(g),
            W=W, per_query_window=W > 0))
    return total
