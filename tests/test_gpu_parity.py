"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded
inputs, element by element, under the acceptance rule of oracle/acceptance.py."""
import os
import numpy as np
import pytest
import torch

from oracle import acceptance as acc
from oracle import pivot_oracle as po
from paper_2607_24593_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pv():
    from paper_2607_24593_b200 import binding
    return binding


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def _report(name, t):
    print(f"\n[{name}] rows={t.rows} exact={t.exact_rows} band_swaps={t.band_swaps} "
          f"scores={t.scores_checked} worst_score_err={t.max_score_err:.3f} x tol")


# ---------------------------------------------------------------- small prefill, all groups

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
@pytest.mark.parametrize("seed", [20260724, 11, 12])
def test_prefill_small_full_parity(pv, gu, dtype, mode, seed):
    """Config 1: L=2048, g=4, k=256, c=512 -- every group against the oracle."""
    L, g, c, k = 2048, 4, 512, 256
    x = inputs.make_prefill(L, dtype=dtype, seed=seed)
    out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out,
                          out_scores=sc, cand=cand, cand_scores=cs)
    _report(f"prefill {dtype} mode={mode} seed={seed}", t)
    # Every row passed the band rule above.  How many rows are the oracle's set exactly: nearly all
    # with fp32 head sums; the FP8 scan sums heads on the tensor core with bf16 ReLU values, so keys
    # within ~2^-9 of the cut may trade places (inside the band) in a good part of the rows.
    assert t.exact_rows >= (0.5 if dtype == "fp8" else 0.95) * t.rows
    assert t.max_score_err <= (0.25 if dtype == "fp8" else 1.0)
    if dtype == "fp8":       # the fp32 head-sum form of the same kernels
        out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, impl=pv.IMPL_TENSOR_CORE_FP32_HEAD_SUM)
        t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out,
                              out_scores=sc, cand=cand, cand_scores=cs)
        _report(f"prefill fp8 (fp32 head sum) mode={mode} seed={seed}", t)
        assert t.exact_rows >= 0.95 * t.rows


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_cuda_core_cross_check_kernels_against_the_oracle(pv, gu, dtype, mode):
    """impl = 1: the plain CUDA-core kernels (one key per thread, radix select) that the library
    keeps as an on-device cross-check -- config 1, every group against the oracle."""
    L, g, c, k = 2048, 4, 512, 256
    x = inputs.make_prefill(L, dtype=dtype, seed=20260724)
    out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, impl=pv.IMPL_CUDA_CORE)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out,
                          out_scores=sc, cand=cand, cand_scores=cs)
    _report(f"CUDA-core kernels {dtype} mode={mode}", t)
    assert t.exact_rows >= 0.95 * t.rows
    # and the tensor-core path returns the same sets up to the band swaps both are allowed
    ref, _, _, _ = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, impl=pv.IMPL_TENSOR_CORE_FP32_HEAD_SUM)
    same = (_sorted_rows_np(out) == _sorted_rows_np(ref)).all(axis=1).mean()
    assert same >= 0.9


def _sorted_rows_np(a):
    return np.sort(a, axis=1)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_dense_small_full_parity(pv, gu, dtype):
    L, k = 1536, 256
    x = inputs.make_prefill(L, dtype=dtype, seed=5)
    out, sc = gu.run_dense(x, k=k)
    t = acc.check_dense(x.codes(), k=k, out_idx=out, out_scores=sc)
    _report(f"dense {dtype}", t)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("L,g,c,k,guard", [
    (1000, 4, 512, 256, None),     # ragged last tile
    (1027, 3, 300, 77, None),      # odd sizes, short last group (m = 1)
    (517, 8, 128, 128, 0),         # c == k, guardrail off: early groups see fewer than c keys
    (260, 5, 64, 16, 1),           # tiny selection
    (130, 1, 32, 8, None),         # g = 1
    (64, 4, 512, 256, None),       # everything guarded, fewer keys than k
    (1, 4, 8, 4, None),            # single token
    (700, 3, 101, 37, None),       # odd sizes: output rows not 16-byte aligned, g does not divide L
])
def test_prefill_edge_shapes(pv, gu, dtype, L, g, c, k, guard):
    x = inputs.make_prefill(L, dtype=dtype, seed=L)
    for mode in (po.MODE_REUSE, po.MODE_REFINE):
        out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, guard_len=guard)
        t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=guard, out_idx=out,
                              out_scores=sc, cand=cand, cand_scores=cs)
        _report(f"edge L={L} g={g} c={c} k={k} {dtype} mode={mode}", t)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_prefill_candidate_budget_above_4096(pv, gu, dtype):
    """c above 4096 (and not a multiple of the tile): the re-score's score rows are longer than
    4096 slots with a ragged last tile, the scan selects more than 4096 per row."""
    L, g, c, k = 9000, 4, 5000, 2500
    x = inputs.make_prefill(L, dtype=dtype, seed=32)
    out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE)
    nG = (L + g - 1) // g
    groups = [0, 1, 1249, 1250, 1251, 1500, 2000, nG - 1]           # guarded, at the guardrail, proxy groups
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                          out_scores=sc, cand=cand, cand_scores=cs, groups=groups)
    _report(f"large c {dtype}", t)
    plain, _, _, _ = gu.run_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, debug=False)
    assert np.array_equal(np.sort(plain, axis=1), np.sort(out, axis=1))


def _random_configs(n, seed):
    rng = np.random.default_rng(seed)
    cfgs = []
    while len(cfgs) < n:
        L = int(rng.integers(1, 1400))
        g = int(rng.integers(1, 10))
        k = int(rng.integers(1, 300))
        c = int(k + rng.integers(0, 400))
        mode = int(rng.integers(0, 2))
        dtype = ("bf16", "fp8")[int(rng.integers(0, 2))]
        guard = (None, 0, int(rng.integers(1, c + 50)))[int(rng.integers(0, 3))]
        W = 0
        if rng.integers(0, 3) == 0:                              # a third of the cases with a local window
            W = int(rng.integers(1, 9))
            eff_guard = c if guard is None else guard
            if W + g - 1 >= c or eff_guard < W + g:
                continue
        pool = ("mean", "first", "last")[int(rng.integers(0, 3))]
        cfgs.append((L, g, c, k, mode, dtype, guard, W, pool))
    return cfgs


@pytest.mark.parametrize("cfg", _random_configs(28, 20260724), ids=lambda c: "L{}-g{}-c{}-k{}-m{}-{}-gd{}-W{}-{}".format(*c))
def test_prefill_random_small_configs(pv, gu, cfg):
    """Seeded random shapes (lengths, group sizes, budgets, guardrails, windows, pooling, both
    operand types and variants): the whole request against the oracle."""
    L, g, c, k, mode, dtype, guard, W, pool = cfg
    x = inputs.make_prefill(L, dtype=dtype, seed=1000 + L)
    pools = {"mean": pv.POOL_MEAN, "first": pv.POOL_FIRST, "last": pv.POOL_LAST}
    out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, guard_len=guard, pool=pools[pool], W=W)
    acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=guard, out_idx=out, out_scores=sc,
                      cand=cand, cand_scores=cs, pool=pool, W=W)


@pytest.mark.parametrize("cfg", [
    (5802, 1, 2378, 1105, 72, 5, "last"),      # guardrail far below c: rows with fewer valid candidates than k
    (900, 4, 64, 64, None, 3, "mean"),         # c == k: the window slots a member may not see leave it short of k
])
def test_window_rows_with_fewer_candidates_than_k_are_padded(pv, gu, cfg):
    """bf16 Refine with a local window: a member whose visible candidates number fewer than k
    gets them all, and -1 after them (the row's tail must not keep what the buffer held)."""
    L, g, c, k, guard, W, pool = cfg
    pools = {"mean": pv.POOL_MEAN, "last": pv.POOL_LAST}
    x = inputs.make_prefill(L, dtype="bf16", seed=5)
    out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=guard, pool=pools[pool], W=W)
    assert (out >= -1).all()                                   # the -7 the buffer was filled with is gone everywhere
    nG = (L + g - 1) // g
    groups = sorted({0, 1, 20, 100 // g, 613 // g, nG // 2, nG - 1})
    acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=po.MODE_REFINE, guard_len=guard, out_idx=out, out_scores=sc,
                      cand=cand, cand_scores=cs, pool=pool, W=W, groups=groups)


def test_group_of_one_equals_dense_on_gpu(pv, gu):
    """Appendix A: g = 1 recovers the dense indexer -- on the GPU outputs themselves."""
    x = inputs.make_prefill(700, dtype="bf16", seed=9)
    a, _, _, _ = gu.run_prefill(x, g=1, c=128, k=64, mode=po.MODE_REUSE)
    b, _ = gu.run_dense(x, k=64)
    for t in range(700):
        assert set(a[t].tolist()) == set(b[t].tolist())


def test_ties_all_equal_scores(pv, gu):
    """Zero gates make every score 0: the total order falls back to the lowest indices."""
    x = inputs.make_prefill(900, dtype="bf16", seed=4)
    x.w.zero_()
    out, sc, cand, cs = gu.run_prefill(x, g=4, c=256, k=128, mode=po.MODE_REFINE)
    for t in range(900):
        n = min(128, t + 1)
        assert sorted(out[t, :n].tolist()) == list(range(n))
        assert (out[t, n:] == -1).all()


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_heavy_ties_few_distinct_keys(pv, gu, dtype):
    """Eight distinct key vectors repeated over the whole cache: every row's scores take at most eight
    values, so the c-th and k-th thresholds always sit inside a tie class of hundreds of keys -- the
    boundary bins of the scan's finisher, of the re-score's select warps and of their narrowing rounds
    are as crowded as they get.  Checked with the acceptance rule (any member of a tie class within
    the tolerance of the threshold is a valid pick) and, where every score is equal, exactly."""
    L, g, c, k = 2600, 4, 700, 300
    x = inputs.make_prefill(L, dtype=dtype, seed=41)
    x.k[:] = x.k[:8].repeat((L + 7) // 8, 1)[:L]
    if x.kscale is not None:
        x.kscale[:] = x.kscale[:8].repeat((L + 7) // 8)[:L]
    for mode in (po.MODE_REUSE, po.MODE_REFINE):
        out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode)
        nG = (L + g - 1) // g
        groups = [0, 1, 174, 175, 176, 300, 449, nG - 1]
        t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out, out_scores=sc,
                              cand=cand, cand_scores=cs, groups=groups)
        _report(f"heavy ties {dtype} mode={mode}", t)
        # no duplicates, nothing from the future, full rows once enough keys are visible
        for tq in (299, 300, 1234, L - 1):
            row = out[tq]
            vis = row[row >= 0]
            assert len(set(vis.tolist())) == len(vis) == min(k, tq + 1) and vis.max() <= tq


def test_pool_variants(pv, gu):
    x = inputs.make_prefill(600, dtype="fp8", seed=8)
    for pool, name in ((pv.POOL_FIRST, "first"), (pv.POOL_LAST, "last")):
        out, sc, cand, cs = gu.run_prefill(x, g=4, c=128, k=64, mode=po.MODE_REFINE, pool=pool)
        acc.check_prefill(x.codes(), g=4, c=128, k=64, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                          out_scores=sc, cand=cand, cand_scores=cs, pool=name)


# ---------------------------------------------------------------- decode

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_decode_small_parity(pv, gu, dtype, mode):
    x = inputs.make_decode(6, 2, 300, 3000, dtype=dtype, seed=21)
    out, sc, cand, cs = gu.run_decode(x, c=512, k=256, mode=mode)     # mixes guarded and proxy sequences
    t = acc.check_decode(x.codes(), c=512, k=256, mode=mode, guard_len=None, out_idx=out, out_scores=sc,
                         cand=cand, cand_scores=cs)
    _report(f"decode {dtype} mode={mode}", t)


def test_decode_ties_beyond_the_select_list(pv, gu):
    """Zero gates make all scores equal: with more visible keys than the select's shared-memory
    list holds, the boundary bin is the whole sequence and one CTA refines it down to the
    position bits -- the total order must still return the lowest positions."""
    x = inputs.make_decode(2, 2, 20000, 24000, dtype="bf16", seed=29)
    x.w.zero_()
    out, _, cand, _ = gu.run_decode(x, c=512, k=256, mode=po.MODE_REFINE)
    for b in range(2):
        assert sorted(cand[b].tolist()) == list(range(512))
        for i in range(2):
            assert sorted(out[b, i].tolist()) == list(range(256))


def test_decode_cache_rows_not_a_multiple_of_four(pv):
    """bf16 caches may have any Lmax: the per-sequence score rows are padded inside the library."""
    x = inputs.make_decode(3, 2, 700, 1200, dtype="bf16", seed=30)
    Lmax = x.k.shape[1] - 3                                      # 1213: odd
    k = x.k[:, :Lmax].contiguous().cuda()
    q, w, pos0 = x.q.cuda(), x.w.cuda(), x.pos0.cuda()
    out = torch.full((3, 2, 128), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_decode(q, w, k, pos0, 3, Lmax, 64, 128, 2, 256, 128, pv.REFINE, out)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    ref = torch.full((3, 2, 128), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_decode(q, w, x.k.cuda(), pos0, 3, x.k.shape[1], 64, 128, 2, 256, 128, pv.REFINE, ref)
    torch.cuda.synchronize()
    assert torch.equal(torch.sort(out, dim=2).values, torch.sort(ref, dim=2).values)


def test_decode_more_than_1024_sequences(pv, gu):
    """Batch sizes beyond one block's worth of sequences in the setup kernel."""
    x = inputs.make_decode(1100, 2, 40, 200, dtype="bf16", seed=31)
    out, sc, cand, cs = gu.run_decode(x, c=32, k=16, mode=po.MODE_REFINE)
    t = acc.check_decode(x.codes(), c=32, k=16, mode=po.MODE_REFINE, guard_len=None, out_idx=out, out_scores=sc,
                         cand=cand, cand_scores=cs, seqs=[0, 5, 511, 1023, 1024, 1025, 1099])
    assert t.rows > 0


def _random_decode_configs(n, seed):
    rng = np.random.default_rng(seed)
    cfgs = []
    while len(cfgs) < n:
        B = int(rng.integers(1, 7))
        g = int(rng.integers(1, 6))
        lo = int(rng.integers(1, 1500))
        hi = lo + int(rng.integers(0, 1500))
        k = int(rng.integers(1, 200))
        c = int(k + rng.integers(0, 300))
        mode = int(rng.integers(0, 2))
        dtype = ("bf16", "fp8")[int(rng.integers(0, 2))]
        paged = bool(rng.integers(0, 3) == 0)
        guard = 0 if paged else (None, 0, int(rng.integers(1, c + 50)))[int(rng.integers(0, 3))]
        W = 0
        if mode == 1 and rng.integers(0, 3) == 0:
            W = int(g + rng.integers(0, 12))
        cfgs.append((B, g, lo, hi, c, k, mode, dtype, guard, W, paged))
    return cfgs


@pytest.mark.parametrize("cfg", _random_decode_configs(20, 20260725),
                         ids=lambda c: "B{}-g{}-n{}..{}-c{}-k{}-m{}-{}-gd{}-W{}-pg{}".format(*c))
def test_decode_random_small_configs(pv, gu, cfg):
    """Seeded random decode steps (batch, MTP width, prefix lengths, budgets, guardrails, window,
    contiguous or paged cache, both operand types and variants) against the oracle."""
    B, g, lo, hi, c, k, mode, dtype, guard, W, paged = cfg
    x = inputs.make_decode(B, g, lo, hi, dtype=dtype, seed=2000 + lo)
    if paged:
        out, sc, cand, cs = gu.run_decode_paged(x, c=c, k=k, mode=mode, seed=lo, W=W)
    else:
        out, sc, cand, cs = gu.run_decode(x, c=c, k=k, mode=mode, guard_len=guard, W=W)
    acc.check_decode(x.codes(), c=c, k=k, mode=mode, guard_len=guard, out_idx=out, out_scores=sc,
                     cand=cand, cand_scores=cs, W=W)


def test_decode_group_of_four(pv, gu):
    x = inputs.make_decode(3, 4, 2000, 2600, dtype="fp8", seed=22)
    out, sc, cand, cs = gu.run_decode(x, c=256, k=128, mode=po.MODE_REFINE)
    acc.check_decode(x.codes(), c=256, k=128, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                     out_scores=sc, cand=cand, cand_scores=cs)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_decode_paged_matches_contiguous(pv, gu, dtype, mode):
    """Paged key cache: same step as the contiguous cache with the guardrail off, page by page
    scattered over a pool -- oracle parity, and the same positions as the contiguous call."""
    x = inputs.make_decode(5, 2, 200, 3000, dtype=dtype, seed=23)     # some sequences shorter than c
    out, sc, cand, cs = gu.run_decode_paged(x, c=512, k=256, mode=mode, seed=5)
    t = acc.check_decode(x.codes(), c=512, k=256, mode=mode, guard_len=0, out_idx=out, out_scores=sc,
                         cand=cand, cand_scores=cs)
    _report(f"decode paged {dtype} mode={mode}", t)
    ref, _, rcand, _ = gu.run_decode(x, c=512, k=256, mode=mode, guard_len=0)
    assert np.array_equal(np.sort(out, axis=2), np.sort(ref, axis=2))
    if cand is not None:
        assert np.array_equal(np.sort(cand, axis=1), np.sort(rcand, axis=1))


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("g,W", [(2, 4), (4, 4), (3, 64)])
def test_decode_local_window_parity(pv, gu, dtype, g, W):
    """Decode form of the local window (Appendix B): pool of c from the scan up to pos0, each
    query re-scores pool U [t-W+1, t]; mixes guarded (dense) and proxy sequences."""
    x = inputs.make_decode(5, g, 300, 2600, dtype=dtype, seed=26)
    out, sc, cand, cs = gu.run_decode(x, c=512, k=256, mode=po.MODE_REFINE, W=W)
    t = acc.check_decode(x.codes(), c=512, k=256, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                         out_scores=sc, cand=cand, cand_scores=cs, W=W)
    _report(f"decode window {dtype} g={g} W={W}", t)
    # the step's own keys are reachable now: the last query's newest key is its own position
    ref, _, _, _ = gu.run_decode(x, c=512, k=256, mode=po.MODE_REFINE)
    p0 = x.pos0.numpy()
    assert all(ref[b].max() <= p0[b] or p0[b] + 1 < 512 for b in range(5))
    assert any(out[b, g - 1].max() > p0[b] for b in range(5))


def test_decode_local_window_paged_matches_contiguous(pv, gu):
    x = inputs.make_decode(4, 2, 700, 2600, dtype="fp8", seed=27)
    out, _, cand, _ = gu.run_decode_paged(x, c=512, k=256, mode=po.MODE_REFINE, seed=7, W=4)
    ref, _, rcand, _ = gu.run_decode(x, c=512, k=256, mode=po.MODE_REFINE, guard_len=0, W=4)
    assert np.array_equal(np.sort(out, axis=2), np.sort(ref, axis=2))
    assert np.array_equal(np.sort(cand, axis=1), np.sort(rcand, axis=1))


def test_decode_local_window_argument_errors(pv):
    x = inputs.make_decode(2, 4, 300, 600, dtype="bf16", seed=28)
    q, w, k, pos0 = x.q.cuda(), x.w.cuda(), x.k.cuda(), x.pos0.cuda()
    out = torch.empty((2, 4, 64), dtype=torch.int32, device="cuda")
    args = (q, w, k, pos0, 2, k.shape[1], 64, 128, 4, 128, 64)
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_decode(*args, pv.REFINE, out, W=3)              # W < g
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_decode(*args, pv.REUSE, out, W=4)               # Reuse has no candidate set to widen
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_decode(*args, pv.REFINE, out, W=510)            # W + g - 1 > 512


def test_decode_paged_bad_page_is_a_hole(pv, gu):
    """A block-table entry outside the pool faults nothing: the page's keys are never returned by
    Refine (the scan sees zeros there, the re-score drops them)."""
    x = inputs.make_decode(2, 2, 1500, 2000, dtype="fp8", seed=24)
    out, _, _, _ = gu.run_decode_paged(x, c=512, k=256, mode=po.MODE_REFINE, seed=6, bad_entry=(1, 3))
    hole = (out[1] >= 3 * 128) & (out[1] < 4 * 128)
    assert not hole.any()
    assert (out[0] >= 0).all()


def test_decode_paged_argument_errors(pv):
    x = inputs.make_decode(2, 2, 300, 600, dtype="bf16", seed=25)
    q, w, k, pos0 = x.q.cuda(), x.w.cuda(), x.k.cuda(), x.pos0.cuda()
    B, g = 2, 2
    mp = k.shape[1] // 128
    pool = k[:, : mp * 128].reshape(B * mp * 128, 128).contiguous()
    bt = torch.arange(B * mp, dtype=torch.int32, device="cuda").reshape(B, mp)
    out = torch.empty((B, g, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_decode_paged(q, w, pool, bt, pos0, B, mp, 0, 64, 128, g, 128, 64, pv.REFINE, out)   # empty pool
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_decode_paged(q, w, pool, bt, pos0, B, mp, B * mp, 64, 128, g, 128, 64, pv.REFINE, out,
                                    impl=pv.IMPL_CUDA_CORE)


# ---------------------------------------------------------------- dense control of a decode step

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("g", [1, 2, 4, 5])
def test_dense_decode_control_against_the_oracle(pv, dtype, g):
    """dense_index_decode: Eq. 1 + TopK for every query of an MTP step.  The query at pos0 + i of
    sequence b is row pos0 + i of the dense indexer over that sequence's cache: compared with the
    oracle's dense rows, scores included."""
    B, k = 5, 96
    x = inputs.make_decode(B, g, 40, 1500, dtype=dtype, seed=61)        # some sequences with fewer keys than k
    d = {n: (None if getattr(x, n) is None else getattr(x, n).cuda()) for n in ("q", "qscale", "w", "k", "kscale", "pos0")}
    Lmax = x.k.shape[1]
    out = torch.full((B, g, k), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((B, g, k), float("nan"), dtype=torch.float32, device="cuda")
    pv.dense_index_decode(d["q"], d["w"], d["k"], d["pos0"], B, Lmax, 64, 128, g, k, out, q_scale=d["qscale"],
                          k_scale=d["kscale"], dbg_scores=sc)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    out, sc = out.cpu().numpy(), sc.cpu().numpy()
    xc = x.codes()
    t = acc.Tally()
    for b in range(B):
        p0 = int(xc["pos0"][b])
        nk = p0 + g
        # the step's queries placed at rows pos0 .. pos0 + g - 1 of a request over this sequence's keys
        H, dd = xc["q"].shape[2], xc["q"].shape[3]
        q = np.zeros((nk, H, dd), xc["q"].dtype)
        w = np.zeros((nk, H), np.float32)
        q[p0:] = xc["q"][b]
        w[p0:] = xc["w"][b]
        qs = None
        if xc["qscale"] is not None:
            qs = np.ones((nk, H), np.float32)
            qs[p0:] = xc["qscale"][b]
        xb = dict(dtype=dtype, q=q, qscale=qs, w=w, k=xc["k"][b, :nk],
                  kscale=None if xc["kscale"] is None else xc["kscale"][b, :nk])
        o = np.full((nk, k), -1, np.int32)
        s = np.full((nk, k), -np.inf, np.float32)
        o[p0:], s[p0:] = out[b], sc[b]
        t.merge(acc.check_dense(xb, k=k, out_idx=o, out_scores=s, rows=range(p0, nk)))
    _report(f"dense decode {dtype} g={g}", t)
    assert t.rows == B * g


def test_decode_bad_pos0_is_reported_not_read(pv, gu):
    """pos0 outside [0, Lmax - g]: the sequence is not indexed (rows of -1), the status word says so,
    the other sequences are unaffected, and a following call is clean."""
    x = inputs.make_decode(4, 2, 600, 1500, dtype="fp8", seed=62)
    d = gu.to_cuda(x)
    Lmax = x.k.shape[1]
    good, _, _, _ = gu.run_decode(x, c=256, k=128, mode=po.MODE_REFINE)
    for bad_value in (-1, Lmax - 1, Lmax + 5000):
        pos = x.pos0.clone()
        pos[1] = bad_value
        out = torch.full((4, 2, 128), -7, dtype=torch.int32, device="cuda")
        pv.pivot_index_decode(d["q"], d["w"], d["k"], pos.cuda(), 4, Lmax, 64, 128, 2, 256, 128, pv.REFINE, out,
                              q_scale=d["qscale"], k_scale=d["kscale"])
        torch.cuda.synchronize()
        assert pv.pivot_device_status() == pv.DEV_BAD_POS
        assert pv.pivot_device_status() == 0                           # read and cleared
        o = out.cpu().numpy()
        assert (o[1] == -1).all()
        for b in (0, 2, 3):
            assert np.array_equal(np.sort(o[b], axis=1), np.sort(good[b], axis=1))
        dn = torch.full((4, 2, 128), -7, dtype=torch.int32, device="cuda")
        pv.dense_index_decode(d["q"], d["w"], d["k"], pos.cuda(), 4, Lmax, 64, 128, 2, 128, dn, q_scale=d["qscale"],
                              k_scale=d["kscale"])
        torch.cuda.synchronize()
        assert pv.pivot_device_status() == pv.DEV_BAD_POS
        assert (dn[1] == -1).all() and (dn[0] >= 0).all()
    again, _, _, _ = gu.run_decode(x, c=256, k=128, mode=po.MODE_REFINE)
    assert np.array_equal(np.sort(again, axis=2), np.sort(good, axis=2))


# ---------------------------------------------------------------- padded key-cache rows (pivot_tensor.stride_row)

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_prefill_with_padded_key_cache_rows(pv, gu, dtype, mode):
    """A key cache whose rows sit in a wider buffer (a serving engine's cache row carries more than the
    indexer key): passed as a strided view, scanned through the TMA map's row stride and gathered by
    the re-score with the same stride -- oracle parity, and the same sets as the dense copy."""
    L, g, c, k = 1500, 4, 256, 128
    x = inputs.make_prefill(L, dtype=dtype, seed=81)
    d = gu.to_cuda(x)
    pad = 48 if dtype == "fp8" else 24                      # elements: 176-byte / 304-byte rows (multiples of 16)
    wide = torch.full((L, 128 + pad), 0x7e if dtype == "fp8" else 1.0, dtype=torch.uint8 if dtype == "fp8" else d["k"].dtype,
                      device="cuda")
    if dtype == "fp8":
        wide = wide.view(torch.float8_e4m3fn)
    wide[:, :128] = d["k"]
    kview = wide[:, :128]
    assert not kview.is_contiguous()
    nG = (L + g - 1) // g
    out = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((L, k), float("nan"), dtype=torch.float32, device="cuda")
    cand = torch.full((nG, c), -7, dtype=torch.int32, device="cuda") if mode == pv.REFINE else None
    cs = torch.full((nG, c), float("nan"), dtype=torch.float32, device="cuda") if mode == pv.REFINE else None
    pv.pivot_index_prefill(d["q"], d["w"], kview, L, 64, 128, g, c, k, mode, out, q_scale=d["qscale"], k_scale=d["kscale"],
                           dbg_scores=sc, dbg_cand=cand, dbg_cand_scores=cs)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    f = lambda t_: None if t_ is None else t_.cpu().numpy()
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=f(out), out_scores=f(sc),
                          cand=f(cand), cand_scores=f(cs))
    _report(f"padded key rows {dtype} mode={mode}", t)
    dense, _, _, _ = gu.run_prefill(x, g=g, c=c, k=k, mode=mode)
    assert np.array_equal(np.sort(f(out), axis=1), np.sort(dense, axis=1))
    with pytest.raises(pv.PivotError, match="unsupported"):
        pv.pivot_index_prefill(d["q"], d["w"], kview, L, 64, 128, g, c, k, mode, out, q_scale=d["qscale"],
                               k_scale=d["kscale"], impl=pv.IMPL_CUDA_CORE)


def test_decode_with_padded_key_cache_rows(pv, gu):
    x = inputs.make_decode(4, 2, 300, 2500, dtype="fp8", seed=82)
    d = gu.to_cuda(x)
    B, Lmax = x.k.shape[0], x.k.shape[1]
    wide = torch.full((B, Lmax, 160), 0x7e, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    wide[:, :, :128] = d["k"]
    kview = wide[:, :, :128]
    out = torch.full((B, 2, 128), -7, dtype=torch.int32, device="cuda")
    cand = torch.full((B, 256), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_decode(d["q"], d["w"], kview, d["pos0"], B, Lmax, 64, 128, 2, 256, 128, pv.REFINE, out,
                          q_scale=d["qscale"], k_scale=d["kscale"], dbg_cand=cand)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    acc.check_decode(x.codes(), c=256, k=128, mode=po.MODE_REFINE, guard_len=None, out_idx=out.cpu().numpy(),
                     cand=cand.cpu().numpy())
    ref, _, _, _ = gu.run_decode(x, c=256, k=128, mode=po.MODE_REFINE)
    assert np.array_equal(np.sort(out.cpu().numpy(), axis=2), np.sort(ref, axis=2))


# ---------------------------------------------------------------- one decode sequence, key axis split

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("world", [2, 3, 5])
def test_decode_key_split_matches_the_single_call_and_the_oracle(pv, gu, dtype, world):
    """The multi-GPU form of one decode sequence (its scan split along the keys, one exchange of c
    (score, position) pairs per rank, merge, Eq. 8-9), with the ranks' parts run one after the other
    on this GPU: same candidate set and index sets as one call, and the oracle agrees."""
    from paper_2607_24593_b200 import sharded
    c, k, g = 512, 256, 2
    x = inputs.make_decode(1, g, 5000, 9000, dtype=dtype, seed=71)
    d = gu.to_cuda(x)
    Lmax = x.k.shape[1]
    p0 = int(x.pos0[0])
    parts = [sharded.decode_keysplit_local(d["q"], d["w"], d["k"], p0, Lmax, 64, 128, c, rank=r, world=world,
                                           q_scale=d["qscale"], k_scale=d["kscale"]) for r in range(world)]
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    all_sc = torch.stack([p[0] for p in parts]).contiguous()
    all_ix = torch.stack([p[1] for p in parts]).contiguous()
    offsets = torch.tensor([p[2] for p in parts], dtype=torch.int32, device="cuda")
    out = torch.full((1, g, k), -7, dtype=torch.int32, device="cuda")
    cand = torch.full((1, c), -7, dtype=torch.int32, device="cuda")
    sharded.decode_keysplit_finish(d["q"], d["w"], d["k"], d["pos0"], Lmax, 64, 128, c, k, out, all_sc, all_ix, offsets,
                                   q_scale=d["qscale"], k_scale=d["kscale"], cand_out=cand)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    ref, _, rcand, _ = gu.run_decode(x, c=c, k=k, mode=po.MODE_REFINE, guard_len=0)
    assert np.array_equal(np.sort(cand.cpu().numpy(), axis=1), np.sort(rcand, axis=1))
    assert np.array_equal(np.sort(out.cpu().numpy(), axis=2), np.sort(ref, axis=2))
    t = acc.check_decode(x.codes(), c=c, k=k, mode=po.MODE_REFINE, guard_len=0, out_idx=out.cpu().numpy(),
                         cand=cand.cpu().numpy())
    assert t.rows == 1 + g


def test_merge_topk_ties_and_empty_slots(pv):
    """pivot_merge_topk: (score desc, position asc) over the union, empty slots skipped, offsets added."""
    sc = torch.tensor([[3.0, 1.0, 1.0, 0.0], [1.0, 3.0, 2.0, 9.0]], dtype=torch.float32, device="cuda")
    ix = torch.tensor([[0, 5, 2, -1], [1, 0, 3, -1]], dtype=torch.int32, device="cuda")
    off = torch.tensor([0, 100], dtype=torch.int32, device="cuda")
    out = torch.full((5,), -7, dtype=torch.int32, device="cuda")
    osc = torch.zeros(5, dtype=torch.float32, device="cuda")
    pv.pivot_merge_topk(sc, ix, 5, out, osc, seg_offset=off)
    torch.cuda.synchronize()
    got = sorted(zip((-osc).tolist(), out.tolist()))
    assert [p for _, p in got] == [0, 100, 103, 2, 5]          # 3.0 @0, 3.0 @100, 2.0 @103, then the 1.0 tie: 2, 5 (101 is sixth)
    out7 = torch.full((7,), -7, dtype=torch.int32, device="cuda")
    pv.pivot_merge_topk(sc, ix, 7, out7, seg_offset=off)
    torch.cuda.synchronize()
    assert sorted(out7.tolist()) == [-1, 0, 2, 5, 100, 101, 103]


# ---------------------------------------------------------------- bounds checks

def test_candidate_from_the_caller_outside_the_sequence_is_dropped_and_reported(pv, gu):
    """pivot_opts.cand_in is the one place where key positions come from outside: an entry beyond the
    sequence must not be gathered (the read would leave the cache); it is dropped and the status word
    reads DEV_BOUNDS.  The other rows are unaffected."""
    x = inputs.make_decode(2, 2, 1500, 2000, dtype="fp8", seed=83)
    d = gu.to_cuda(x)
    Lmax = x.k.shape[1]
    ref, _, rcand, _ = gu.run_decode(x, c=256, k=128, mode=po.MODE_REFINE, guard_len=0)
    cand = torch.from_numpy(rcand).cuda().contiguous()
    out = torch.full((2, 2, 128), -7, dtype=torch.int32, device="cuda")
    run = lambda: pv.pivot_index_decode(d["q"], d["w"], d["k"], d["pos0"], 2, Lmax, 64, 128, 2, 256, 128, pv.REFINE, out,
                                        q_scale=d["qscale"], k_scale=d["kscale"], guard_len=0, cand_in=cand)
    run()
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    assert np.array_equal(np.sort(out.cpu().numpy(), axis=2), np.sort(ref, axis=2))
    bad = int(cand[1, 7])
    cand[1, 7] = 5_000_000                        # far outside the cache
    run()
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == pv.DEV_BOUNDS
    o = out.cpu().numpy()
    assert np.array_equal(np.sort(o[0], axis=1), np.sort(ref[0], axis=1))
    assert (o[1] != 5_000_000).all() and (o[1] >= -1).all()
    assert set(o[1, 0][o[1, 0] >= 0].tolist()) <= set(rcand[1].tolist()) - {bad}


def test_checked_build_runs_the_small_parity_cases_clean():
    """The -DPIVOT_DEBUG build of the same sources (bounds checks on gathered positions, block-table
    entries, score and entry slots; a failed check sets DEV_BOUNDS and skips the access): small
    prefill / decode / paged cases in a process of its own -- oracle parity and a clean status word."""
    import os
    import subprocess
    import sys
    from paper_2607_24593_b200 import build
    lib = build.build_variant("debug", ["-DPIVOT_DEBUG"])
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = """
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import torch, gpu_util
from oracle import acceptance as acc, pivot_oracle as po
from paper_2607_24593_b200 import binding as pv, inputs
assert pv.LIB_PATH.endswith('libpivot_debug.so')
for dtype in ('bf16', 'fp8'):
    x = inputs.make_prefill(1100, dtype=dtype, seed=91)
    for mode in (po.MODE_REUSE, po.MODE_REFINE):
        out, sc, cand, cs = gpu_util.run_prefill(x, g=4, c=256, k=128, mode=mode, W=4 if mode else 0)
        acc.check_prefill(x.codes(), g=4, c=256, k=128, mode=mode, guard_len=None, out_idx=out, out_scores=sc, cand=cand,
                          cand_scores=cs, W=4 if mode else 0)
    xd = inputs.make_decode(3, 2, 300, 2600, dtype=dtype, seed=92)
    out, sc, cand, cs = gpu_util.run_decode(xd, c=256, k=128, mode=po.MODE_REFINE, W=4)
    acc.check_decode(xd.codes(), c=256, k=128, mode=po.MODE_REFINE, guard_len=None, out_idx=out, out_scores=sc, cand=cand,
                     cand_scores=cs, W=4)
    out, sc, cand, cs = gpu_util.run_decode_paged(xd, c=256, k=128, mode=po.MODE_REFINE, seed=3)
    acc.check_decode(xd.codes(), c=256, k=128, mode=po.MODE_REFINE, guard_len=0, out_idx=out, out_scores=sc, cand=cand,
                     cand_scores=cs)
print('checked build ok')
""" % (root, os.path.join(root, "tests"))
    env = dict(os.environ, PIVOT_LIB=os.path.basename(lib))
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "checked build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


# ---------------------------------------------------------------- bounded device waits

def test_bounded_wait_runs_out_and_reports_without_hanging(pv, gu):
    """Failure detection: the kernels' barrier waits are bounded.  A diagnostic kernel waits -- through
    the library's own wait routines, limit 1 ms -- on a barrier nothing completes: it must return,
    the status word must read DEV_WAIT_EXPIRED, and the next ordinary call must be clean."""
    import time
    x = inputs.make_prefill(600, dtype="fp8", seed=63)
    gu.run_prefill(x, g=4, c=128, k=64, mode=po.MODE_REFINE)           # registers a workspace
    t0 = time.perf_counter()
    pv.pivot_debug_wait_expiry(1_000_000)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert pv.pivot_device_status() == pv.DEV_WAIT_EXPIRED
    assert dt < 1.0, f"the bounded wait took {dt:.3f} s"
    assert pv.pivot_device_status() == 0                               # cleared by the read
    out, sc, cand, cs = gu.run_prefill(x, g=4, c=128, k=64, mode=po.MODE_REFINE)
    acc.check_prefill(x.codes(), g=4, c=128, k=64, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                      out_scores=sc, cand=cand, cand_scores=cs)
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_debug_wait_expiry(10)                                  # below 1 us
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_debug_wait_expiry(5_000_000_000)                       # above 1 s


# ---------------------------------------------------------------- argument errors (host side)

def test_counters_entry_point_is_refused_by_an_ordinary_build(pv):
    """pivot_debug_counters belongs to the -DPIVOT_PROF build (bench.py --counters); the library the
    tests load carries no counters and says so instead of returning the workspace head's bytes."""
    if os.path.basename(os.environ.get("PIVOT_LIB", "libpivot.so")) == "libpivot_prof.so":
        pytest.skip("counters build loaded")
    with pytest.raises(pv.PivotError, match="unsupported|not supported"):
        pv.pivot_debug_counters()


def test_argument_errors(pv):
    x = inputs.make_prefill(64, dtype="bf16", seed=1)
    q, w, k = x.q.cuda(), x.w.cuda(), x.k.cuda()
    out = torch.empty((64, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_prefill(q, w, k, 64, 64, 128, 4, 4, 8, pv.REFINE, out)      # k > c
    with pytest.raises(pv.PivotError, match="unsupported"):
        pv.pivot_index_prefill(q, w, k, 64, 32, 128, 4, 16, 8, pv.REFINE, out)     # H_I != 64
    with pytest.raises(pv.PivotError, match="workspace"):
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        pv.pivot_index_prefill(q, w, k, 64, 64, 128, 4, 16, 8, pv.REFINE, out, workspace=small)


# ---------------------------------------------------------------- chunked prefill / host pipeline

def _sorted_rows(a):
    return np.sort(a, axis=1)


def _oracle_check_plain(gu, x, plain_out, *, g, c, k, mode, groups=None, what=""):
    """Acceptance rule on the index rows of a call made WITHOUT debug buffers.  Refine's two-stage
    check needs the candidate sets the kernels produced: they come from a second call on the same
    inputs that asks for them (every key's score is computed independently of the launch shape, so
    both calls rank the same candidates; if they did not, stage two would fail here)."""
    out_d, sc_d, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=plain_out,
                          cand=cand, cand_scores=cs, groups=groups)
    _report(what or "plain call vs oracle", t)
    assert t.rows > 0
    return t


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_plain_call_matches_the_call_with_debug_buffers(pv, gu, dtype):
    """The oracle parity tests pass score / candidate buffers, which take other store paths in
    the kernels than a caller's plain call: both must return the same sets."""
    L, g, c, k = 2500, 4, 512, 256
    x = inputs.make_prefill(L, dtype=dtype, seed=78)
    dbg, _, _, _ = gu.run_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE)
    plain, _, _, _ = gu.run_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, debug=False)
    assert np.array_equal(_sorted_rows(plain), _sorted_rows(dbg))


def test_two_streams_with_their_own_workspaces(pv):
    """Two requests indexed at the same time on two streams, each call with its own workspace
    (pivot_opts.workspace): same results as one after the other."""
    L, g, c, k = 6000, 4, 512, 256
    xs = [inputs.make_prefill(L, dtype="fp8", seed=80 + i) for i in range(2)]
    dev = [dict(q=x.q.cuda(), w=x.w.cuda(), k=x.k.cuda(), qs=x.qscale.cuda(), ks=x.kscale.cuda()) for x in xs]
    nG = (L + g - 1) // g
    ws = [torch.empty(pv.pivot_workspace_bytes(L, nG, c, k), dtype=torch.uint8, device="cuda") for _ in range(2)]
    serial = []
    for d, wsp in zip(dev, ws):
        o = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
        pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, 64, 128, g, c, k, pv.REFINE, o, q_scale=d["qs"],
                               k_scale=d["ks"], workspace=wsp)
        serial.append(o)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]
    both = [torch.full((L, k), -7, dtype=torch.int32, device="cuda") for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(3):
        for d, wsp, st, o in zip(dev, ws, streams, both):
            pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, 64, 128, g, c, k, pv.REFINE, o, st, q_scale=d["qs"],
                                   k_scale=d["ks"], workspace=wsp)
    torch.cuda.synchronize()
    for a, b in zip(serial, both):
        assert np.array_equal(_sorted_rows(a.cpu().numpy()), _sorted_rows(b.cpu().numpy()))


def test_sharded_request_blocks_match_whole_call(pv, gu):
    """The multi-GPU form of one request (row blocks dealt to ranks in snake order), with the
    ranks' shares indexed one after the other on this GPU: together they give the whole call."""
    from paper_2607_24593_b200 import sharded
    L, g, c, k = 3000, 4, 256, 128
    x = inputs.make_prefill(L, dtype="fp8", seed=79)
    q, w, kk, qs, ks = x.q.cuda(), x.w.cuda(), x.k.cuda(), x.qscale.cuda(), x.kscale.cuda()
    whole = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_prefill(q, w, kk, L, 64, 128, g, c, k, pv.REFINE, whole, q_scale=qs, k_scale=ks)
    parts = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    covered = 0
    for rank in range(3):
        mine = sharded.pivot_index_prefill_sharded(q, w, kk, L, 64, 128, g, c, k, pv.REFINE, parts, rank=rank, world=3,
                                                   block_rows=400, q_scale=qs, k_scale=ks)
        covered += sum(r1 - r0 for r0, r1 in mine)
    torch.cuda.synchronize()
    assert covered == L and pv.pivot_device_status() == 0
    assert np.array_equal(_sorted_rows(parts.cpu().numpy()), _sorted_rows(whole.cpu().numpy()))
    _oracle_check_plain(gu, x, parts.cpu().numpy(), g=g, c=c, k=k, mode=po.MODE_REFINE, what="sharded row blocks")


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
def test_prefill_row_ranges_match_whole_call(pv, gu, dtype, mode):
    """Chunks of query rows (row_begin / row_end) give the rows of one whole call: same sets
    (the order inside a row is free), rows outside the chunk untouched."""
    L, g, c, k = 1900, 4, 256, 64
    x = inputs.make_prefill(L, dtype=dtype, seed=77)
    q, w, kk = x.q.cuda(), x.w.cuda(), x.k.cuda()
    sc = dict(q_scale=None if x.qscale is None else x.qscale.cuda(),
              k_scale=None if x.kscale is None else x.kscale.cuda())
    whole = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_prefill(q, w, kk, L, 64, 128, g, c, k, mode, whole, **sc)
    parts = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    bounds = [0, 128, 260, 1000, 1524, L]          # chunks inside, across and past the guardrail (c = 256)
    for r0, r1 in zip(bounds[:-1], bounds[1:]):
        before = parts.clone()
        pv.pivot_index_prefill(q, w, kk, L, 64, 128, g, c, k, mode, parts, rows=(r0, r1), **sc)
        torch.cuda.synchronize()
        assert pv.pivot_device_status() == 0
        untouched = torch.ones(L, dtype=torch.bool, device="cuda")
        untouched[r0:r1] = False
        assert torch.equal(parts[untouched], before[untouched])
    assert np.array_equal(_sorted_rows(parts.cpu().numpy()), _sorted_rows(whole.cpu().numpy()))
    _oracle_check_plain(gu, x, parts.cpu().numpy(), g=g, c=c, k=k, mode=mode, what=f"row ranges {dtype} mode={mode}")
    for bad in [(2, 8), (0, 6), (8, 8), (0, L + 4), (-4, 8)]:
        with pytest.raises(pv.PivotError, match="invalid"):
            pv.pivot_index_prefill(q, w, kk, L, 64, 128, g, c, k, mode, parts, rows=bad, **sc)


def test_prefill_host_pipeline_matches_device_call(pv, gu):
    """The host-buffer entry point (chunked copies overlapping the kernels) returns what the
    device entry point returns for the same request; large enough for several chunks."""
    L, g, c, k = 20000, 4, 512, 128
    x = inputs.make_prefill(L, dtype="fp8", seed=5)
    dev = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_prefill(x.q.cuda(), x.w.cuda(), x.k.cuda(), L, 64, 128, g, c, k, pv.REFINE, dev,
                           q_scale=x.qscale.cuda(), k_scale=x.kscale.cuda())
    torch.cuda.synchronize()
    pin = lambda t: t.contiguous().pin_memory()
    hq, hw, hk, hqs, hks = pin(x.q), pin(x.w), pin(x.k), pin(x.qscale), pin(x.kscale)
    hout = torch.full((L, k), -7, dtype=torch.int32).pin_memory()
    arena = torch.empty(pv.pivot_prefill_host_arena_bytes(L, 64, 128, g, c, k, pv.FP8_E4M3), dtype=torch.uint8, device="cuda")
    for _ in range(2):          # second call: the arena and the copy streams are reused
        hout.fill_(-7)
        pv.pivot_index_prefill_host(hq, hw, hk, L, 64, 128, g, c, k, pv.REFINE, hout, arena, q_scale=hqs, k_scale=hks)
        assert np.array_equal(_sorted_rows(hout.numpy()), _sorted_rows(dev.cpu().numpy()))
    nG = L // g
    groups = sorted({0, 127, 128, 129, 2499, 2500, 2501, nG // 2, nG - 1} |
                    set(np.random.default_rng(5).integers(0, nG, 12).tolist()))      # chunk edges at multiples of 2500 groups
    _oracle_check_plain(gu, x, hout.numpy(), g=g, c=c, k=k, mode=po.MODE_REFINE, groups=groups, what="host pipeline")


# ---------------------------------------------------------------- local window (Appendix B)

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("mode", [po.MODE_REUSE, po.MODE_REFINE])
@pytest.mark.parametrize("g,W", [(4, 4), (8, 3), (3, 1)])
def test_prefill_local_window_parity(pv, gu, dtype, mode, g, W):
    """W > 0: shortened proxy scan, window slots at the end of the candidate set, per-member
    causal mask over the window -- every group against the oracle's Appendix B steps."""
    L, c, k = 1000 + g - 1, 256, 96          # short last group
    x = inputs.make_prefill(L, dtype=dtype, seed=31)
    out, scores, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, W=W)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out, out_scores=scores,
                          cand=cand, cand_scores=cs, W=W)
    _report(f"window {dtype} mode={mode} g={g} W={W}", t)
    assert t.rows > 0


def test_local_window_argument_errors(pv):
    x = inputs.make_prefill(256, dtype="bf16", seed=1)
    q, w, k = x.q.cuda(), x.w.cuda(), x.k.cuda()
    out = torch.empty((256, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_prefill(q, w, k, 256, 64, 128, 4, 16, 8, pv.REFINE, out, W=13)        # W + g - 1 >= c
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_prefill(q, w, k, 256, 64, 128, 4, 16, 8, pv.REFINE, out, W=4, guard_len=4)   # guardrail < W + g
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_prefill(q, w, k, 256, 64, 128, 4, 16, 8, pv.REFINE, out, W=-1)


# ---------------------------------------------------------------- packed requests (Eq. 2 boundaries)

@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_prefill_varlen_equals_per_request_calls(pv, gu, dtype):
    """Requests packed back to back give, row for row, what separate calls give: groups and causal
    prefixes stop at the request boundaries, positions are relative to the request."""
    lens = [700, 0, 1028, 300]            # starts at multiples of 4 (FP8 scale rows), one empty request
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    g, c, k, mode = 4, 256, 64, pv.REFINE
    xs = [inputs.make_prefill(n, dtype=dtype, seed=100 + i) if n else None for i, n in enumerate(lens)]
    cat = lambda name: torch.cat([getattr(x, name) for x in xs if x is not None]).cuda()
    q, w, kk = cat("q"), cat("w"), cat("k")
    sc = dict(q_scale=cat("qscale"), k_scale=cat("kscale")) if dtype == "fp8" else {}
    packed = torch.full((int(cu[-1]), k), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_prefill_varlen(q, w, kk, cu, 64, 128, g, c, k, mode, packed, **sc)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    for i, x in enumerate(xs):
        if x is None:
            continue
        one = torch.full((lens[i], k), -7, dtype=torch.int32, device="cuda")
        s1 = dict(q_scale=x.qscale.cuda(), k_scale=x.kscale.cuda()) if dtype == "fp8" else {}
        pv.pivot_index_prefill(x.q.cuda(), x.w.cuda(), x.k.cuda(), lens[i], 64, 128, g, c, k, mode, one, **s1)
        got = packed[cu[i]:cu[i + 1]].cpu().numpy()
        assert np.array_equal(_sorted_rows(got), _sorted_rows(one.cpu().numpy())), f"request {i}"
        assert got.max() < lens[i]
        _oracle_check_plain(gu, x, got, g=g, c=c, k=k, mode=po.MODE_REFINE, what=f"packed request {i} {dtype}")
    if dtype == "fp8":
        with pytest.raises(pv.PivotError, match="invalid"):
            pv.pivot_index_prefill_varlen(q, w, kk, [0, 702, int(cu[-1])], 64, 128, g, c, k, mode, packed, **sc)
    with pytest.raises(pv.PivotError, match="invalid"):
        pv.pivot_index_prefill_varlen(q, w, kk, [0, 800, 400], 64, 128, g, c, k, mode, packed, **sc)
