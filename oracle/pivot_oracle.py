"""CPU oracle for the PIVOT group-shared indexer.  TEST INFRASTRUCTURE ONLY.

Plain numpy, float64 arithmetic after the operands are decoded, one obvious loop per step of
the paper's Algorithm 1.  It shares no code with the CUDA path and must never be imported by
the product package; only tests, the smoke check and the benchmark's CPU-baseline leg use it.

What it computes, with the passage each function follows:
  indexer_scores      Eq. 1 (dense lightning-indexer score), FP8 form of Appendix A
  top_set             TopK of Eq. 1 / 6 / 7 / 9, total order (score desc, index asc)
  build_proxy         Eq. 4 (per-head mean of queries and gates over the group)
  pivot_group         Algorithm 1, one group: guardrail, Eq. 5 scan, Eq. 6 Reuse, Eq. 7-9 Refine,
                      local window of Appendix B when W > 0 (prefill form: one shared candidate
                      set with reserved window slots; decode form: pool united with each query's
                      own window)
  refine_on_candidates Eq. 8-9 on a candidate set supplied from outside
  pivot_prefill / pivot_decode / dense_index   drivers over groups (Eq. 2 / Eq. 3 grouping)

PIVOT approximates the dense indexer, so this oracle is the algorithm's steps in the paper's
order, not the dense definition -- except for g = 1 and for guarded (short) groups, where it is
the dense definition itself.

Readings taken where the paper is silent:
  * positions are 0-indexed here; a query at t sees keys s <= t (inclusive);
  * the proxy scan is cut at the group's first position t0, n0 = t0 + 1 keys visible;
  * guardrail: dense per member iff n0 < guard_len (default c), for both variants;
  * a short last group averages over its actual size;
  * fewer than k visible keys: the valid indices first, then -1;
  * ties: (score desc, index asc);
  * the proxy is formed from de-quantised queries in fp32, summed in member order, scaled by
    fl32(1/m), then rounded back to the storage type (bf16: RN-even; e4m3: fresh per-head scale
    a/448 with a = max(amax, 1e-4), RN-even, saturating), the new scale folded into the proxy
    gate -- these are the rounding points of a kernel that must feed a low-precision scan;
  * the key scale multiplies after the head sum (Appendix A).

Pins: every function is pinned by tests that do not call it to produce their expectation
(hand-worked example, torch einsum/topk restatement, g = 1 identity, c >= n0 identity,
identical-member identity, coverage identity, brute-force select, codec tables; first / last
pooling against the dense indexer's row of that member; the rounded proxy against the exact
fp64 mean inside the score band).  The prefill window variant is pinned by its reduction to the
dense definition over [0, t] when the proxy part and the window slots together hold every
visible key, and by a torch restatement of its slot layout; the decode window variant by the
same reduction and by a set-membership restatement of "pool united with the query's own
window".  Parity unpinned: only the reading that the short-group guardrail also applies to
Reuse (Algorithm 1 tests it before the variant branch; nothing else in the paper fixes it).
"""
from __future__ import annotations

import dataclasses

import numpy as np

MODE_REUSE = 0
MODE_REFINE = 1

# --------------------------------------------------------------------------- storage codecs


def bf16_decode(u16: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64 (exact)."""
    bits = u16.astype(np.uint32) << np.uint32(16)
    return bits.view(np.float32).astype(np.float64)


def bf16_encode(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    return ((bits + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def _e4m3_table() -> np.ndarray:
    """All 256 e4m3 (finite-only variant, bias 7) values; codes 0x7F / 0xFF are NaN."""
    t = np.empty(256, np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            v = np.nan
        elif e == 0:
            v = (m / 8.0) * 2.0 ** -6
        else:
            v = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[code] = sign * v
    return t


E4M3_TABLE = _e4m3_table()
_E4M3_POS = E4M3_TABLE[:0x7F].copy()          # codes 0 .. 0x7E, ascending, max 448
E4M3_MAX = 448.0


def e4m3_decode(u8: np.ndarray) -> np.ndarray:
    return E4M3_TABLE[u8]


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """float32 -> e4m3 codes: round to nearest, ties to the even code, saturate at +-448."""
    xf = np.asarray(x, dtype=np.float32).astype(np.float64)
    mag = np.minimum(np.abs(xf), E4M3_MAX)
    hi = np.searchsorted(_E4M3_POS, mag, side="left")          # POS[hi-1] < mag <= POS[hi]
    hi = np.minimum(hi, len(_E4M3_POS) - 1)
    lo = np.maximum(hi - 1, 0)
    mid = 0.5 * (_E4M3_POS[lo] + _E4M3_POS[hi])
    pick_hi = (mag > mid) | ((mag == mid) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    code = np.where(np.signbit(xf), code | np.uint8(0x80), code).astype(np.uint8)
    return code


def decode_operand(codes: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_decode(codes) if dtype == "bf16" else e4m3_decode(codes)


# --------------------------------------------------------------------------- Eq. 1 and TopK


def indexer_scores(qd: np.ndarray, weff: np.ndarray, kd: np.ndarray, kscale) -> np.ndarray:
    """Eq. 1: I_s = sum_j w_j * ReLU(q_j . k_s) for every key row of kd.

    qd [H, d] decoded query codes, weff [H] gate (already times the query scale for FP8),
    kd [n, d] decoded key codes, kscale [n] or None (Appendix A: the key scale multiplies
    the head sum).  float64 throughout.
    """
    dots = kd @ qd.T                       # [n, H]
    s = np.maximum(dots, 0.0) @ weff.astype(np.float64)
    if kscale is not None:
        s = s * kscale.astype(np.float64)
    return s


def top_set(scores: np.ndarray, k: int, index: np.ndarray | None = None) -> np.ndarray:
    """Indices of the k largest scores, ordered by (score desc, index asc).

    `index` maps slots to key positions (defaults to 0..n-1); ties break on the key position.
    Returns min(k, n) key positions.
    """
    n = scores.shape[0]
    idx = np.arange(n, dtype=np.int64) if index is None else np.asarray(index, dtype=np.int64)
    order = np.lexsort((idx, -scores))
    return idx[order[:k]]


def _pad(ids: np.ndarray, k: int) -> np.ndarray:
    out = np.full(k, -1, np.int32)
    out[: len(ids)] = ids
    return out


# --------------------------------------------------------------------------- Eq. 4 proxy


def member_operands(q_codes: np.ndarray, qscale, w: np.ndarray, dtype: str):
    """Per-query operands of Eq. 1 / Eq. 8: decoded codes [.., H, d] and effective gate
    fl32(w * qscale) (FP8; Appendix A: the gate absorbs the query scale) or w (bf16)."""
    qd = decode_operand(q_codes, dtype)
    if dtype == "fp8":
        weff = (w.astype(np.float32) * qscale.astype(np.float32)).astype(np.float32)
    else:
        weff = w.astype(np.float32)
    return qd, weff


def build_proxy(q_codes: np.ndarray, qscale, w: np.ndarray, dtype: str, pool: str = "mean"):
    """Eq. 4: proxy query and gate of one group.

    q_codes [m, H, d], qscale [m, H] or None, w [m, H].  Returns (proxy codes [H, d] in the
    storage type, proxy effective gate [H] float32).  pool = "mean" (the paper's choice),
    "first" or "last" (the ablation's endpoint proxies).
    """
    m = q_codes.shape[0]
    if dtype == "fp8":
        x = e4m3_decode(q_codes).astype(np.float32) * qscale.astype(np.float32)[..., None]
    else:
        x = bf16_decode(q_codes).astype(np.float32)
    wf = w.astype(np.float32)
    if pool == "first":
        qbar, wbar = x[0].copy(), wf[0].copy()
    elif pool == "last":
        qbar, wbar = x[m - 1].copy(), wf[m - 1].copy()
    else:
        acc, wacc = x[0].copy(), wf[0].copy()
        for i in range(1, m):                      # member order, fp32
            acc = (acc + x[i]).astype(np.float32)
            wacc = (wacc + wf[i]).astype(np.float32)
        inv_m = np.float32(1.0) / np.float32(m)
        qbar = (acc * inv_m).astype(np.float32)
        wbar = (wacc * inv_m).astype(np.float32)
    if dtype == "bf16":
        return bf16_encode(qbar), wbar
    a = np.maximum(np.abs(qbar).max(axis=-1), np.float32(1e-4)).astype(np.float32)   # [H]
    sbar = (a / np.float32(448.0)).astype(np.float32)
    inv = (np.float32(448.0) / a).astype(np.float32)
    codes = e4m3_encode((qbar * inv[:, None]).astype(np.float32))
    return codes, (wbar * sbar).astype(np.float32)


# --------------------------------------------------------------------------- Algorithm 1


@dataclasses.dataclass
class GroupResult:
    t0: int
    members: np.ndarray                 # query positions of the group
    guarded: bool                       # True: dense per member (short-group guardrail)
    T: np.ndarray                       # [m, k] int32, -1 padded
    C: np.ndarray | None = None         # candidate positions (Refine), score order
    proxy_scores: np.ndarray | None = None   # [n0] float64, Eq. 5
    member_scores: np.ndarray | None = None  # Refine: [m, |C|] float64 (Eq. 8); guarded: list of [t+1]
    C_mask: np.ndarray | None = None    # [m, |C|] bool, False where a window slot lies beyond t
    member_C: list | None = None        # decode window form: each member's own candidate positions


def refine_on_candidates(qd, weff, kd_all, kscale_all, C: np.ndarray, k: int, t_member=None):
    """Eq. 8-9 for one query on a given candidate set C (key positions).

    Returns (scores over C [len(C)] float64, T = top-k positions).  Slots with C > t_member
    (only possible for window slots) are excluded.
    """
    C = np.asarray(C, dtype=np.int64)
    ks = None if kscale_all is None else kscale_all[C]
    s = indexer_scores(qd, weff, kd_all[C], ks)
    if t_member is not None:
        ok = C <= t_member
    else:
        ok = np.ones(len(C), bool)
    T = top_set(s[ok], k, C[ok])
    return s, T, ok


def pivot_group(x: dict, members: np.ndarray, kd: np.ndarray, kscale, *, c: int, k: int, mode: int,
                guard_len: int | None = None, W: int = 0, pool: str = "mean",
                q_rows: np.ndarray | None = None, per_query_window: bool = False) -> GroupResult:
    """Algorithm 1 for one group.

    per_query_window selects the decode form of Appendix B's local window: the scan and the
    pool C are those of W = 0, and the member at t refines over C united with [t-W+1, t].

    x: dict with "dtype", "q" [.., H, d] codes, "qscale", "w" indexed by q_rows (defaults to
    `members`, the query positions; decode passes slot indices instead).  kd / kscale: decoded
    key cache rows 0 .. (at least) max(members).
    """
    dtype = x["dtype"]
    members = np.asarray(members, dtype=np.int64)
    rows = members if q_rows is None else np.asarray(q_rows)
    m = len(members)
    t0 = int(members[0])
    n0 = t0 + 1
    guard = c if guard_len is None else guard_len
    qs = None if x["qscale"] is None else x["qscale"][rows]
    qd, weff = member_operands(x["q"][rows], qs, x["w"][rows], dtype)

    if n0 < guard:                                   # short-group guardrail: dense per member
        T = np.empty((m, k), np.int32)
        ms = []
        for i, t in enumerate(members):
            s = indexer_scores(qd[i], weff[i], kd[: t + 1], None if kscale is None else kscale[: t + 1])
            T[i] = _pad(top_set(s, k), k)
            ms.append(s)
        return GroupResult(t0, members, True, T, member_scores=ms)

    pq_codes, pweff = build_proxy(x["q"][rows], qs, x["w"][rows], dtype, pool)        # Eq. 4
    pqd = decode_operand(pq_codes, dtype)
    # Eq. 5: one scan, cut at the group's first position (prefill form of the window: t0 - W,
    # the window part then covers the rest without duplicates)
    n_scan = n0 if (W == 0 or per_query_window) else max(t0 - W + 1, 0)
    pscores = indexer_scores(pqd, pweff, kd[:n_scan], None if kscale is None else kscale[:n_scan])

    if mode == MODE_REUSE:                           # Eq. 6: the proxy top-k serves every member
        S = top_set(pscores, k)
        T = np.tile(_pad(S, k), (m, 1))
        return GroupResult(t0, members, False, T, proxy_scores=pscores)

    # Refine.  Eq. 7 candidate set; with a window, the proxy fills c - w_g slots and the
    # union of the members' windows [t0-W+1, t0+m-1] takes the rest (Appendix B).
    if W > 0 and per_query_window:
        # decode form: every query keeps the pool and adds its own W most recent positions
        C = top_set(pscores, c)
        T = np.empty((m, k), np.int32)
        ms, member_C = [], []
        for i, t in enumerate(members):
            win = np.arange(max(int(t) - W + 1, 0), int(t) + 1, dtype=np.int64)
            Ci = np.concatenate([C, win[~np.isin(win, C)]])          # duplicates counted once
            s, Ti, _ = refine_on_candidates(qd[i], weff[i], kd, kscale, Ci, k)
            T[i] = _pad(Ti, k)
            ms.append(s)
            member_C.append(Ci)
        return GroupResult(t0, members, False, T, C=C, proxy_scores=pscores, member_scores=ms, member_C=member_C)
    if W == 0:
        C = top_set(pscores, c)
    else:
        w_g = W + m - 1
        win = np.arange(max(t0 - W + 1, 0), t0 + m, dtype=np.int64)
        C = np.concatenate([top_set(pscores, c - w_g), win])
    T = np.empty((m, k), np.int32)
    ms = np.empty((m, len(C)), np.float64)
    masks = np.empty((m, len(C)), bool)
    for i, t in enumerate(members):                  # Eq. 8-9 per member
        s, Ti, ok = refine_on_candidates(qd[i], weff[i], kd, kscale, C, k, t_member=int(t))
        ms[i], masks[i] = s, ok
        T[i] = _pad(Ti, k)
    return GroupResult(t0, members, False, T, C=C, proxy_scores=pscores, member_scores=ms, C_mask=masks)


def prefill_groups(L: int, g: int):
    """Eq. 2: contiguous groups of g positions; the last may be short."""
    return [np.arange(t0, min(t0 + g, L), dtype=np.int64) for t0 in range(0, L, g)]


def pivot_prefill(x: dict, *, g: int, c: int, k: int, mode: int, guard_len=None, W: int = 0,
                  pool: str = "mean", groups=None):
    """Algorithm 1 over one request (prefill).  `groups`: indices of the groups to evaluate
    (default all).  Returns {group index: GroupResult}."""
    L = x["q"].shape[0]
    kd = decode_operand(x["k"], x["dtype"])
    allg = prefill_groups(L, g)
    sel = range(len(allg)) if groups is None else groups
    return {gi: pivot_group(x, allg[gi], kd, x["kscale"], c=c, k=k, mode=mode,
                            guard_len=guard_len, W=W, pool=pool) for gi in sel}


def pivot_decode(x: dict, *, c: int, k: int, mode: int, guard_len=None, W: int = 0,
                 pool: str = "mean", seqs=None):
    """Algorithm 1 in decode (Eq. 3): sequence b's group is its g queries at positions
    pos0_b .. pos0_b + g - 1, scanned against that sequence's own key cache, cut at pos0_b.
    Returns {b: GroupResult}."""
    B, g = x["q"].shape[0], x["q"].shape[1]
    if W and W < g:
        raise ValueError("the decode window must cover the step: W >= g (Appendix B)")
    out = {}
    for b in (range(B) if seqs is None else seqs):
        p0 = int(x["pos0"][b])
        nk = p0 + g
        kd = decode_operand(x["k"][b, :nk], x["dtype"])
        ks = None if x["kscale"] is None else x["kscale"][b, :nk]
        xb = dict(dtype=x["dtype"], q=x["q"][b], qscale=None if x["qscale"] is None else x["qscale"][b],
                  w=x["w"][b])
        out[b] = pivot_group(xb, np.arange(p0, p0 + g), kd, ks, c=c, k=k, mode=mode,
                             guard_len=guard_len, W=W, pool=pool, q_rows=np.arange(g),
                             per_query_window=True)
    return out


def dense_index(x: dict, *, k: int, rows=None):
    """Eq. 1 + TopK for each query row t over keys [0, t].  Returns {t: (scores [t+1], T [k])}."""
    L = x["q"].shape[0]
    kd = decode_operand(x["k"], x["dtype"])
    out = {}
    for t in (range(L) if rows is None else rows):
        qs = None if x["qscale"] is None else x["qscale"][t]
        qd, weff = member_operands(x["q"][t], qs, x["w"][t], x["dtype"])
        s = indexer_scores(qd, weff, kd[: t + 1], None if x["kscale"] is None else x["kscale"][: t + 1])
        out[t] = (s, _pad(top_set(s, k), k))
    return out


def assemble(results: dict, L: int, k: int, fill: int = -2) -> np.ndarray:
    """Stack GroupResults into an [L, k] index table (rows of groups not evaluated = fill)."""
    out = np.full((L, k), fill, np.int32)
    for r in results.values():
        out[r.members] = r.T
    return out
