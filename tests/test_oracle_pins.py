"""Pins for the CPU oracle: each test derives its expectation from something other than the
function under test -- a hand-worked example, torch's own casts / einsum / topk, a brute-force
select, or an identity the paper states (g = 1 recovers the dense indexer, Appendix A)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import pivot_oracle as po
from paper_2607_24593_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden", "worked_example.json")


def tiny(L=96, H=4, d=8, dtype="bf16", seed=3):
    return inputs.make_prefill(L, H, d, dtype=dtype, seed=seed, threads=1).codes()


# ----------------------------------------------------------------------------- codecs

def test_e4m3_table_hand_values():
    t = po.E4M3_TABLE
    assert t[0x00] == 0.0 and t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9
    assert t[0x08] == 2.0 ** -6 and t[0x38] == 1.0 and t[0x3C] == 1.5
    assert t[0x7E] == 448.0 and t[0xFE] == -448.0 and t[0xB8] == -1.0
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF])


def test_e4m3_table_matches_torch():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    ok = ~np.isnan(ref)
    assert ok.sum() == 254
    np.testing.assert_array_equal(po.E4M3_TABLE[ok], ref[ok])


def test_e4m3_encode_roundtrip_and_saturation():
    codes = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], np.uint8)
    vals = po.e4m3_decode(codes).astype(np.float32)
    back = po.e4m3_encode(vals)
    np.testing.assert_array_equal(po.e4m3_decode(back), po.e4m3_decode(codes))   # -0 == +0
    assert po.e4m3_encode(np.float32([1e9, -1e9, 449.0, 464.0])).tolist() == [0x7E, 0xFE, 0x7E, 0x7E]
    # ties go to the even code: 1.0625 is midway between 1.0 (0x38) and 1.125 (0x39)
    assert po.e4m3_encode(np.float32([1.0625, 1.1875])).tolist() == [0x38, 0x3A]


def test_e4m3_encode_matches_torch_cast():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(500000) * 100, rng.standard_normal(500000) * 0.01,
                        rng.uniform(-448, 448, 100000)]).astype(np.float32)
    x = np.clip(x, -448, 448)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = po.e4m3_encode(x)
    np.testing.assert_array_equal(po.e4m3_decode(got), po.e4m3_decode(ref))


def test_bf16_codec_matches_torch():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(po.bf16_encode(x), ref)
    np.testing.assert_array_equal(po.bf16_decode(ref), torch.from_numpy(x).to(torch.bfloat16).double().numpy())


# ----------------------------------------------------------------------------- hand-worked example

def _gold_inputs(fp8: bool):
    g = json.load(open(GOLD))
    keys = np.array(g["keys"], np.float32)
    L, H, d = 6, 2, 2
    q = np.zeros((L, H, d), np.float32)
    w = np.ones((L, H), np.float32)
    for t in ("4", "5"):
        q[int(t)] = np.array(g["q"][t], np.float32)
        w[int(t)] = np.array(g["w"][t], np.float32)
    if not fp8:
        x = dict(dtype="bf16", q=po.bf16_encode(q).reshape(q.shape), qscale=None, w=w,
                 k=po.bf16_encode(keys).reshape(keys.shape), kscale=None)
    else:
        # codes hold 2x the value with a query scale of 0.5; keys carry the fixture's scales
        qs = np.full((L, H), 0.5, np.float32)
        x = dict(dtype="fp8", q=po.e4m3_encode(q * 2).reshape(q.shape), qscale=qs, w=w,
                 k=po.e4m3_encode(keys).reshape(keys.shape), kscale=np.array(g["fp8_kscale"], np.float32))
    return g, x


def test_worked_example_bf16():
    g, x = _gold_inputs(False)
    pq, pw = po.build_proxy(x["q"][[4, 5]], None, x["w"][[4, 5]], "bf16")
    np.testing.assert_array_equal(po.bf16_decode(pq), np.array(g["proxy_q"], np.float64))
    np.testing.assert_array_equal(pw, np.array(g["proxy_w"], np.float32))
    kd = po.decode_operand(x["k"], "bf16")
    r = po.pivot_group(x, np.array([4, 5]), kd, None, c=3, k=2, mode=po.MODE_REUSE, guard_len=0)
    np.testing.assert_allclose(r.proxy_scores, g["proxy_scores"], rtol=0, atol=0)
    assert po.top_set(r.proxy_scores, 5).tolist() == g["proxy_order"]
    assert r.T.tolist() == [g["reuse_k2"], g["reuse_k2"]]
    r = po.pivot_group(x, np.array([4, 5]), kd, None, c=3, k=2, mode=po.MODE_REFINE)
    assert not r.guarded                       # n0 = 5 >= c = 3
    assert r.C.tolist() == g["refine_c3_candidates"]
    np.testing.assert_array_equal(r.member_scores, [g["refine_scores"]["4"], g["refine_scores"]["5"]])
    assert r.T.tolist() == [g["refine_k2"]["4"], g["refine_k2"]["5"]]
    s, T = po.dense_index(x, k=3, rows=[5])[5]
    np.testing.assert_array_equal(s, g["dense_scores_5"])
    assert T.tolist() == g["dense_k3_5"]


def test_worked_example_fp8_scales():
    g, x = _gold_inputs(True)
    kd = po.decode_operand(x["k"], "fp8")
    r = po.pivot_group(x, np.array([4, 5]), kd, x["kscale"], c=3, k=2, mode=po.MODE_REUSE, guard_len=0)
    np.testing.assert_allclose(r.proxy_scores, g["fp8_proxy_scores"], rtol=1e-6)
    assert po.top_set(r.proxy_scores, 5).tolist() == g["fp8_proxy_order"]
    # member 5 dense scores: the fixture's bf16 values times the key scales
    s, _ = po.dense_index(x, k=3, rows=[5])[5]
    np.testing.assert_allclose(s, np.array(g["dense_scores_5"]) * np.array(g["fp8_kscale"]), rtol=1e-12)


def test_guardrail_boundary():
    """Dense iff n0 < c (1-indexed t0 < c in Algorithm 1): the group starting at position
    c - 1 (n0 = c) runs the proxy path, the one before it is dense."""
    x = tiny(L=40, H=2, d=4)
    res = po.pivot_prefill(x, g=2, c=8, k=4, mode=po.MODE_REFINE)
    for gi, r in res.items():
        assert r.guarded == (r.t0 + 1 < 8)
    assert res[3].guarded and res[3].t0 == 6          # n0 = 7 < 8
    assert res[4].t0 == 8 and not res[4].guarded
    res1 = po.pivot_prefill(x, g=1, c=8, k=4, mode=po.MODE_REFINE)
    assert res1[6].guarded and not res1[7].guarded    # t0 = 7: n0 = 8 = c runs PIVOT


# ----------------------------------------------------------------------------- library restatement

def _torch_dense(x, k):
    """Dense indexer with torch ops only (einsum / relu / tril mask / topk), fp64."""
    if x["dtype"] == "bf16":
        q = torch.from_numpy(x["q"].view(np.int16)).view(torch.bfloat16).double()
        kk = torch.from_numpy(x["k"].view(np.int16)).view(torch.bfloat16).double()
        w = torch.from_numpy(x["w"]).double()
        ks = torch.ones(kk.shape[0], dtype=torch.float64)
    else:
        q = torch.from_numpy(x["q"]).view(torch.float8_e4m3fn).double()
        kk = torch.from_numpy(x["k"]).view(torch.float8_e4m3fn).double()
        w = (torch.from_numpy(x["w"]) * torch.from_numpy(x["qscale"])).double()
        ks = torch.from_numpy(x["kscale"]).double()
    dots = torch.einsum("thd,sd->ths", q, kk)
    I = (torch.relu(dots) * w[:, :, None]).sum(1) * ks[None, :]
    L = q.shape[0]
    I = I.masked_fill(torch.ones(L, L).triu(1).bool(), float("-inf"))
    return I, [set(torch.topk(I[t], min(k, t + 1)).indices.tolist()) for t in range(L)]


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_dense_matches_torch_restatement(dtype):
    x = tiny(L=80, H=4, d=8, dtype=dtype)
    I, sets = _torch_dense(x, 7)
    res = po.dense_index(x, k=7)
    for t in range(80):
        s, T = res[t]
        np.testing.assert_allclose(s, I[t, : t + 1].numpy(), rtol=1e-12, atol=1e-15)
        assert set(T[T >= 0].tolist()) == sets[t]
        assert (T[min(7, t + 1):] == -1).all()


def test_single_head_reduces_to_gemv_topk():
    """H = 1 with a positive gate: ranking by the score equals ranking by the dot product."""
    x = tiny(L=64, H=1, d=8)
    q = po.bf16_decode(x["q"])[:, 0]
    kk = po.bf16_decode(x["k"])
    res = po.dense_index(x, k=5, rows=[63])
    dots = kk @ q[63]
    pos = np.flatnonzero(dots > 0)
    assert len(pos) >= 5
    want = pos[np.argsort(-dots[pos], kind="stable")][:5]
    assert res[63][1].tolist() == want.tolist()


def test_top_set_vs_bruteforce_argmax():
    rng = np.random.default_rng(5)
    for n in (1, 2, 7, 33, 64):
        s = rng.integers(0, 6, n).astype(np.float64)       # many ties
        for k in (1, 3, n):
            left = s.copy()
            want = []
            for _ in range(min(k, n)):
                j = int(np.argmax(left))                  # first occurrence = lowest index
                want.append(j)
                left[j] = -np.inf
            assert po.top_set(s, k).tolist() == want


# ----------------------------------------------------------------------------- identities of the method

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_group_of_one_is_the_dense_indexer(dtype, mode):
    """Appendix A: group size one recovers the per-query indexer exactly.  For bf16 the proxy
    of one member is the member bit for bit; for fp8 the re-quantised proxy equals the member
    because the scale is recomputed from values that already sit on the e4m3 grid."""
    x = tiny(L=72, H=4, d=8, dtype=dtype)
    _, sets = _torch_dense(x, 6)
    for guard in (None, 0):
        res = po.pivot_prefill(x, g=1, c=12, k=6, mode=mode, guard_len=guard)
        for t in range(72):
            T = res[t].T[0]
            if mode == po.MODE_REUSE or res[t].guarded or t + 1 <= 12:
                assert set(T[T >= 0].tolist()) == sets[t], (t, guard)
            else:      # Refine, c < n0: top-k of the top-c of the same scores = the top-k
                assert set(T.tolist()) == sets[t]


def test_refine_with_c_covering_prefix_is_dense_on_prefix():
    x = tiny(L=64, H=4, d=8)
    I, _ = _torch_dense(x, 5)
    res = po.pivot_prefill(x, g=4, c=64, k=5, mode=po.MODE_REFINE, guard_len=0)
    for gi, r in res.items():
        if r.t0 + 1 < 5:
            continue
        for i, t in enumerate(r.members):
            want = set(torch.topk(I[t, : r.t0 + 1], 5).indices.tolist())     # restricted to [0, t0]
            assert set(r.T[i].tolist()) == want


def test_c_equal_k_refine_equals_reuse():
    x = tiny(L=64, H=4, d=8)
    a = po.pivot_prefill(x, g=4, c=6, k=6, mode=po.MODE_REFINE)
    b = po.pivot_prefill(x, g=4, c=6, k=6, mode=po.MODE_REUSE)
    for gi in a:
        for i in range(len(a[gi].members)):
            assert set(a[gi].T[i].tolist()) == set(b[gi].T[i].tolist())
            if not a[gi].guarded:
                assert set(a[gi].T[i].tolist()) == set(a[gi].C.tolist())


def test_identical_members_make_reuse_refine_dense_agree():
    x = tiny(L=64, H=4, d=8)
    for t0 in range(0, 64, 4):                # copy the first member over its group
        x["q"][t0:t0 + 4] = x["q"][t0]
        x["w"][t0:t0 + 4] = x["w"][t0]
    I, _ = _torch_dense(x, 5)
    for mode in (po.MODE_REUSE, po.MODE_REFINE):
        res = po.pivot_prefill(x, g=4, c=10, k=5, mode=mode, guard_len=0)
        for r in res.values():
            if r.t0 + 1 < 10:
                continue
            want = set(torch.topk(I[r.t0, : r.t0 + 1], 5).indices.tolist())
            for i in range(4):
                assert set(r.T[i].tolist()) == want


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_containment_and_coverage(dtype):
    x = tiny(L=160, H=4, d=8, dtype=dtype)
    I, _ = _torch_dense(x, 8)
    res = po.pivot_prefill(x, g=4, c=16, k=8, mode=po.MODE_REFINE)
    for r in res.values():
        for i, t in enumerate(r.members):
            T = r.T[i]
            valid = T[T >= 0]
            assert len(set(valid.tolist())) == len(valid) == min(8, t + 1)
            assert valid.max() <= t
            if r.guarded:
                continue
            assert set(valid.tolist()) <= set(r.C.tolist()) and r.C.max() <= r.t0 and len(r.C) == 16
            D = set(torch.topk(I[t, : r.t0 + 1], 8).indices.tolist())
            # any key of the dense top-k (over the proxy's prefix) that made it into C is selected
            assert set(valid.tolist()) & D == set(r.C.tolist()) & D


def test_power_of_two_rescaling_leaves_sets_unchanged():
    x = tiny(L=96, H=4, d=8)
    y = dict(x)
    y["q"] = po.bf16_encode(po.bf16_decode(x["q"]).astype(np.float32) * np.float32(4.0)).reshape(x["q"].shape)
    y["w"] = x["w"] * np.float32(0.125)
    for mode in (po.MODE_REUSE, po.MODE_REFINE):
        a = po.pivot_prefill(x, g=4, c=16, k=8, mode=mode)
        b = po.pivot_prefill(y, g=4, c=16, k=8, mode=mode)
        for gi in a:
            np.testing.assert_array_equal(a[gi].T, b[gi].T)


def test_short_last_group_averages_over_its_size():
    x = tiny(L=23, H=2, d=4)
    r = po.pivot_prefill(x, g=4, c=4, k=2, mode=po.MODE_REUSE, groups=[5])[5]
    assert r.members.tolist() == [20, 21, 22]
    pq, pw = po.build_proxy(x["q"][20:23], None, x["w"][20:23], "bf16")
    want_w = ((x["w"][20] + x["w"][21]) + x["w"][22]) * (np.float32(1) / np.float32(3))
    np.testing.assert_array_equal(pw, want_w.astype(np.float32))
    assert r.T.shape == (3, 2)


def test_window_reduces_and_contains():
    """W = 0 is the plain candidate set; with W > 0 each member keeps its W most recent keys
    among the candidates and the candidate count stays c (Appendix B)."""
    x = tiny(L=96, H=4, d=8)
    a = po.pivot_prefill(x, g=4, c=24, k=8, mode=po.MODE_REFINE, W=0)
    b = po.pivot_prefill(x, g=4, c=24, k=8, mode=po.MODE_REFINE, W=4)
    for gi, r in b.items():
        if r.guarded:
            np.testing.assert_array_equal(r.T, a[gi].T)
            continue
        assert len(r.C) == 24 and len(set(r.C.tolist())) == 24
        for i, t in enumerate(r.members):
            assert set(range(t - 3, t + 1)) <= set(r.C[r.C_mask[i]].tolist())
            assert r.T[i].max() <= t


def test_decode_group_equals_prefill_group_on_same_tensors():
    """Eq. 3 vs Eq. 2: a decode group at pos0 is the prefill group starting at pos0."""
    x = tiny(L=64, H=4, d=8, dtype="fp8")
    g, p0 = 2, 40
    xd = dict(dtype="fp8", q=x["q"][None, p0:p0 + g], qscale=x["qscale"][None, p0:p0 + g],
              w=x["w"][None, p0:p0 + g], k=x["k"][None], kscale=x["kscale"][None],
              pos0=np.array([p0], np.int32))
    a = po.pivot_decode(xd, c=12, k=6, mode=po.MODE_REFINE)[0]
    b = po.pivot_prefill(x, g=g, c=12, k=6, mode=po.MODE_REFINE, groups=[p0 // g])[p0 // g]
    np.testing.assert_array_equal(a.T, b.T)
    np.testing.assert_array_equal(a.C, b.C)


def _decode_view(x, p0, g):
    return dict(dtype=x["dtype"], q=x["q"][None, p0:p0 + g],
                qscale=None if x["qscale"] is None else x["qscale"][None, p0:p0 + g],
                w=x["w"][None, p0:p0 + g], k=x["k"][None],
                kscale=None if x["kscale"] is None else x["kscale"][None], pos0=np.array([p0], np.int32))


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_decode_window_covering_everything_is_the_dense_indexer(dtype):
    """Decode form of Appendix B: with the pool holding every key up to pos0 (c >= pos0 + 1) and
    W >= g, pool united with [t-W+1, t] is the whole visible prefix of t, so every query of the
    step must get the dense indexer's set (torch restatement), including the keys written
    inside the step, which the pool cannot hold."""
    x = tiny(L=80, H=4, d=8, dtype=dtype)
    g, p0, k = 3, 50, 9
    _, sets = _torch_dense(x, k)
    r = po.pivot_decode(_decode_view(x, p0, g), c=64, k=k, mode=po.MODE_REFINE, guard_len=0, W=3)[0]
    assert not r.guarded
    for i in range(g):
        assert set(r.T[i].tolist()) == sets[p0 + i]
    # without the window the later queries cannot see the step's own keys
    r0 = po.pivot_decode(_decode_view(x, p0, g), c=64, k=k, mode=po.MODE_REFINE, guard_len=0)[0]
    assert r0.T.max() <= p0


def test_decode_window_is_pool_united_with_own_window():
    """Set-membership restatement: each query's result is the top-k, by its own dense scores
    (torch restatement), over exactly pool U [t-W+1, t] -- a recent key outside the pool is
    eligible for the queries whose window covers it and for no other."""
    x = tiny(L=96, H=4, d=8, dtype="bf16", seed=5)
    g, p0, c, k, W = 3, 80, 10, 6, 4
    I, _ = _torch_dense(x, k)
    r = po.pivot_decode(_decode_view(x, p0, g), c=c, k=k, mode=po.MODE_REFINE, guard_len=0, W=W)[0]
    pool = set(r.C.tolist())
    assert len(pool) == c and max(pool) <= p0
    r_plain = po.pivot_decode(_decode_view(x, p0, g), c=c, k=k, mode=po.MODE_REFINE, guard_len=0)[0]
    np.testing.assert_array_equal(r.C, r_plain.C)                  # the pool is the plain method's
    for i in range(g):
        t = p0 + i
        allowed = sorted(pool | set(range(t - W + 1, t + 1)))
        sc = I[t, allowed].numpy()
        order = sorted(range(len(allowed)), key=lambda j: (-sc[j], allowed[j]))[:k]
        assert set(r.T[i].tolist()) == {allowed[j] for j in order}
        assert sorted(r.member_C[i].tolist()) == allowed
    with pytest.raises(ValueError):
        po.pivot_decode(_decode_view(x, p0, g), c=c, k=k, mode=po.MODE_REFINE, guard_len=0, W=2)   # W < g


def test_acceptance_rule_decode_window_accepts_the_oracle_and_rejects_a_stale_row():
    from oracle import acceptance as acc
    x = inputs.make_decode(3, 2, 200, 400, dtype="bf16", seed=9).codes()
    c, k, W = 64, 24, 4
    res = po.pivot_decode(x, c=c, k=k, mode=po.MODE_REFINE, guard_len=0, W=W)
    out = np.stack([res[b].T for b in range(3)])
    cand = np.stack([res[b].C for b in range(3)]).astype(np.int32)
    t = acc.check_decode(x, c=c, k=k, mode=po.MODE_REFINE, guard_len=0, out_idx=out, cand=cand, W=W)
    assert t.rows > 0 and t.exact_rows == t.rows
    plain = po.pivot_decode(x, c=c, k=k, mode=po.MODE_REFINE, guard_len=0)
    differs = [b for b in range(3) if not np.array_equal(np.sort(plain[b].T), np.sort(res[b].T))]
    assert differs, "the window must change at least one row of this case"
    bad = out.copy()
    bad[differs[0]] = plain[differs[0]].T                           # result computed without the window
    with pytest.raises(AssertionError):
        acc.check_decode(x, c=c, k=k, mode=po.MODE_REFINE, guard_len=0, out_idx=bad, cand=cand, W=W)


# ---------------------------------------------------------------- acceptance rule with a local window

def test_acceptance_rule_with_window_accepts_the_oracle_and_rejects_mutations():
    """The window form of the acceptance check (Appendix B) passes on the oracle's own output,
    and fails when a window slot is wrong or a member selects a key beyond its own position."""
    from oracle import acceptance as acc
    from paper_2607_24593_b200 import inputs
    L, g, c, k, W = 120, 4, 32, 12, 3
    x = inputs.make_prefill(L, dtype="bf16", seed=3).codes()
    res = po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, W=W)
    out = np.full((L, k), -1, np.int32)
    cand = np.full((len(res), c), -1, np.int32)
    for gi, r in res.items():
        out[r.members] = r.T
        if r.C is not None:
            cand[gi, : len(r.C)] = r.C
    t = acc.check_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=None, out_idx=out, cand=cand, W=W)
    assert t.rows > 0 and t.exact_rows == t.rows
    gi = len(res) - 1                       # a group past the guardrail
    r = res[gi]
    assert not r.guarded
    bad = cand.copy()
    bad[gi, c - 1] -= 1                     # last window slot must be t0 + m - 1
    with pytest.raises(AssertionError):
        acc.check_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=None, out_idx=out, cand=bad, W=W, groups=[gi])
    bad_out = out.copy()
    first = int(r.members[0])
    bad_out[first, 0] = first + 1           # a key the first member may not see
    with pytest.raises(AssertionError):
        acc.check_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=None, out_idx=bad_out, cand=cand, W=W, groups=[gi])


# ---------------------------------------------------------------- pooling variants, prefill window, proxy rounding

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_first_and_last_pooling_reduce_to_a_member_row_of_the_dense_indexer(dtype):
    """Endpoint proxies of the pooling ablation: with pool = "first" the proxy IS the group's first
    query, whose visible prefix is exactly the scan's [0, t0], so Reuse must return the dense
    indexer's top-k of row t0 (torch restatement); with pool = "last" it is the last member's
    query scored over [0, t0] only.  (bf16: the proxy is the member bit for bit; fp8: values that
    already sit on the e4m3 grid re-quantise to themselves.)"""
    L, g, k = 72, 4, 6
    x = tiny(L=L, H=4, d=8, dtype=dtype)
    I, sets = _torch_dense(x, k)
    first = po.pivot_prefill(x, g=g, c=12, k=k, mode=po.MODE_REUSE, guard_len=0, pool="first")
    last = po.pivot_prefill(x, g=g, c=12, k=k, mode=po.MODE_REUSE, guard_len=0, pool="last")
    mean = po.pivot_prefill(x, g=g, c=12, k=k, mode=po.MODE_REUSE, guard_len=0)
    differs = 0
    for gi in first:
        t0, tl = int(first[gi].t0), int(first[gi].members[-1])
        if t0 + 1 < k:
            continue
        for T in first[gi].T:
            assert set(T.tolist()) == sets[t0]
        want_last = set(torch.topk(I[tl, : t0 + 1], k).indices.tolist())
        for T in last[gi].T:
            assert set(T.tolist()) == want_last
        differs += set(mean[gi].T[0].tolist()) != sets[t0]
    assert differs > 0, "mean pooling must differ from the first-member proxy somewhere in this case"
    # Refine with the first-member proxy: the candidate set is row t0's dense top-c
    r = po.pivot_prefill(x, g=g, c=12, k=k, mode=po.MODE_REFINE, guard_len=0, pool="first", groups=[10])[10]
    assert set(r.C.tolist()) == set(torch.topk(I[r.t0, : r.t0 + 1], 12).indices.tolist())


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("g,W", [(4, 4), (4, 2), (3, 5)])
def test_prefill_window_covering_everything_is_the_dense_indexer(dtype, g, W):
    """Prefill form of Appendix B: the proxy part ranks s <= t0 - W and fills c - (W + m - 1) slots,
    the window union [t0 - W + 1, t0 + m - 1] takes the rest.  With the guardrail off and
    c - (W + m - 1) >= t0 - W + 1 the two parts together hold every key up to t0 + m - 1, each
    member masks the slots beyond its own position, and so every member must get the dense
    indexer's top-k over [0, t] (torch restatement) -- including the keys of its own group, which
    the plain method (W = 0) cannot reach."""
    L, k, c = 61, 5, 80
    x = tiny(L=L, H=4, d=8, dtype=dtype)
    _, sets = _torch_dense(x, k)
    res = po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=0, W=W)
    reached_own_group = 0
    for r in res.values():
        assert not r.guarded
        m = len(r.members)
        assert len(r.C) == min(c, r.t0 + m) and sorted(r.C.tolist()) == list(range(r.t0 + m))
        for i, t in enumerate(r.members):
            T = r.T[i]
            assert set(T[T >= 0].tolist()) == sets[t], (r.t0, i)
            assert (T[min(k, t + 1):] == -1).all()
            reached_own_group += int(T.max() > r.t0)
    assert reached_own_group > 0
    plain = po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=0, W=0)
    assert all(r.T.max() <= r.t0 for r in plain.values())


def test_prefill_window_slot_layout_with_a_short_candidate_budget():
    """The same form when the proxy part does NOT cover its prefix: the last W + m - 1 slots are
    the window positions in ascending order, the first c - (W + m - 1) are the top of the proxy
    scores over s <= t0 - W (recomputed here from build_proxy + torch), and no slot repeats."""
    L, g, c, k, W = 96, 4, 24, 8, 4
    x = tiny(L=L, H=4, d=8)
    kk = torch.from_numpy(x["k"].view(np.int16)).view(torch.bfloat16).double()
    res = po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, W=W)
    checked = 0
    for r in res.values():
        if r.guarded:
            continue
        m, t0 = len(r.members), r.t0
        w_g = W + m - 1
        assert r.C[c - w_g:].tolist() == list(range(t0 - W + 1, t0 + m))
        pq, pw = po.build_proxy(x["q"][r.members], None, x["w"][r.members], "bf16")
        pqt = torch.from_numpy(pq.view(np.int16)).view(torch.bfloat16).double()
        n_scan = t0 - W + 1
        s = (torch.relu(kk[:n_scan] @ pqt.T) * torch.from_numpy(pw).double()).sum(1)
        want = set(torch.topk(s, c - w_g).indices.tolist())
        assert set(r.C[: c - w_g].tolist()) == want
        assert len(set(r.C.tolist())) == c
        checked += 1
    assert checked > 5


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_rounded_proxy_stays_inside_the_score_band_of_the_exact_mean(dtype):
    """Eq. 4 is real-valued; the oracle rounds the mean proxy back to the storage type (the rounding
    points of a kernel that feeds a low-precision scan).  This bounds that reading from the oracle's
    side: Eq. 5 scores of the rounded proxy against those of the unrounded fp64 mean of the
    de-quantised members, at the real head count and width, stay inside the acceptance band."""
    from oracle import acceptance as acc
    L, g = 640, 4
    x = inputs.make_prefill(L, dtype=dtype, seed=17, threads=1).codes()
    kd = po.decode_operand(x["k"], dtype)
    ks = x["kscale"]
    worst = 0.0
    for t0 in (128, 300, 636):
        rows = np.arange(t0, t0 + g)
        qs = None if x["qscale"] is None else x["qscale"][rows]
        pq, pw = po.build_proxy(x["q"][rows], qs, x["w"][rows], dtype)
        s_round = po.indexer_scores(po.decode_operand(pq, dtype), pw, kd[: t0 + 1], None if ks is None else ks[: t0 + 1])
        qd = po.decode_operand(x["q"][rows], dtype)
        if dtype == "fp8":
            qd = qd * qs.astype(np.float64)[..., None]
        qbar = qd.mean(axis=0)                                    # exact Eq. 4, fp64
        wbar = x["w"][rows].astype(np.float64).mean(axis=0)
        s_exact = np.maximum(kd[: t0 + 1] @ qbar.T, 0.0) @ wbar
        if ks is not None:
            s_exact = s_exact * ks[: t0 + 1].astype(np.float64)
        err = np.abs(s_round - s_exact) / (acc.ATOL + acc.RTOL[dtype] * np.abs(s_exact))
        worst = max(worst, float(err.max()))
    assert worst <= 1.0, worst
