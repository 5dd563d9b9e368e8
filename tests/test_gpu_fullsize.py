"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the CUDA
path runs the whole request, the oracle re-computes a seeded sample of groups one by one
(groups are independent, so sampled parity is exact per group): first and last proxy group,
the guardrail boundary, tile-edge positions, and a random rest."""
import numpy as np
import pytest
import torch

from oracle import acceptance as acc
from oracle import pivot_oracle as po
from paper_2607_24593_b200 import inputs

pytestmark = pytest.mark.gpu

_cache = {}


def _inputs(L, dtype):
    if (L, dtype) not in _cache:
        _cache.clear()                      # one big request at a time
        _cache[(L, dtype)] = inputs.make_prefill(L, dtype=dtype)
    return _cache[(L, dtype)]


def _sample_groups(L, g, c, n_random, seed):
    nG = (L + g - 1) // g
    first = (c - 1 + g - 1) // g            # first group on the proxy path
    picks = {0, 1, first - 1, first, first + 1, nG - 1, nG - 2}
    for pos in (127, 128, 129, 4095, 4096, 4224, L // 2 - 1, L // 2, L - 129):
        picks.add(min(max(pos // g, 0), nG - 1))
    rng = np.random.default_rng(seed)
    picks.update(rng.integers(0, nG, n_random).tolist())
    return sorted(p for p in picks if 0 <= p < nG)


def _run_and_check(L, dtype, g, c, k, mode, n_random):
    import gpu_util
    x = _inputs(L, dtype)
    out, sc, cand, cs = gpu_util.run_prefill(x, g=g, c=c, k=k, mode=mode)
    groups = _sample_groups(L, g, c, n_random, seed=L + g + mode)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=out, out_scores=sc,
                          cand=cand, cand_scores=cs, groups=groups)
    print(f"\n[L={L} {dtype} g={g} mode={mode}] groups={len(groups)} rows={t.rows} exact={t.exact_rows} "
          f"band_swaps={t.band_swaps} worst_score_err={t.max_score_err:.3f} x tol")
    # properties that hold at any size, on every row
    assert (out < np.arange(L)[:, None] + 1).all(), "an index beyond the query position"
    full = out[k - 1:]                      # rows with at least k visible keys
    assert (full >= 0).all()
    srt = np.sort(full[:: max(1, len(full) // 4096)], axis=1)
    assert (np.diff(srt, axis=1) > 0).all(), "duplicate index in a row"
    return t


@pytest.mark.parametrize("mode", [po.MODE_REFINE, po.MODE_REUSE])
def test_config2_prefill_32k_bf16(mode):
    _run_and_check(32768, "bf16", 4, 4096, 2048, mode, n_random=24)


def test_config2_dense_32k_bf16_sampled_rows():
    import gpu_util
    L, k = 32768, 2048
    x = _inputs(L, "bf16")
    out, sc = gpu_util.run_dense(x, k=k)
    rows = [0, 1, 127, 128, 2047, 2048, 2049, 4095, 4096, 16383, 16384, 32767] + \
        np.random.default_rng(3).integers(0, L, 12).tolist()
    t = acc.check_dense(x.codes(), k=k, out_idx=out, out_scores=sc, rows=sorted(set(rows)))
    print(f"\n[dense 32k bf16] rows={t.rows} exact={t.exact_rows} band_swaps={t.band_swaps}")


@pytest.mark.parametrize("g,mode", [(4, po.MODE_REFINE), (4, po.MODE_REUSE), (8, po.MODE_REFINE)])
def test_config3_prefill_128k_fp8(g, mode):
    _run_and_check(131072, "fp8", g, 4096, 2048, mode, n_random=20)


def _rows_equal_as_sets(a: torch.Tensor, b: torch.Tensor) -> bool:
    return bool((torch.sort(a, dim=1).values == torch.sort(b, dim=1).values).all().item())


def test_config3_plain_call_and_host_pipeline_at_full_size():
    """The headline configuration exactly as bench.py times it: the call WITHOUT debug buffers
    (other store paths in the kernels: staged 16-byte index rows, candidates in the workspace) and
    the host-buffer pipeline in its row chunks.  Both must return, row for row, the sets of the
    call with debug buffers, and those are checked against the oracle on the sampled groups."""
    import gpu_util
    from paper_2607_24593_b200 import binding as pv
    L, g, c, k, mode = 131072, 4, 4096, 2048, po.MODE_REFINE
    x = _inputs(L, "fp8")
    d = gpu_util.to_cuda(x)
    nG = L // g
    dbg = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    cand = torch.full((nG, c), -7, dtype=torch.int32, device="cuda")
    cs = torch.full((nG, c), float("nan"), dtype=torch.float32, device="cuda")
    pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, 64, 128, g, c, k, mode, dbg, q_scale=d["qscale"],
                           k_scale=d["kscale"], dbg_cand=cand, dbg_cand_scores=cs)
    plain = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, 64, 128, g, c, k, mode, plain, q_scale=d["qscale"],
                           k_scale=d["kscale"])
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    assert _rows_equal_as_sets(plain, dbg)
    groups = _sample_groups(L, g, c, 12, seed=99)
    t = acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=None, out_idx=plain.cpu().numpy(),
                          cand=cand.cpu().numpy(), cand_scores=cs.cpu().numpy(), groups=groups)
    print(f"\n[128K plain call] groups={len(groups)} rows={t.rows} exact={t.exact_rows} band_swaps={t.band_swaps}")
    del cand, cs, dbg
    # host pipeline (seven chunks at this size, the first and the last cut once more)
    pv.pivot_set_workspace(None)
    del d
    torch.cuda.empty_cache()
    pin = lambda t_: t_.contiguous().pin_memory()
    hq, hw, hk, hqs, hks = pin(x.q), pin(x.w), pin(x.k), pin(x.qscale), pin(x.kscale)
    hout = torch.full((L, k), -7, dtype=torch.int32).pin_memory()
    arena = torch.empty(pv.pivot_prefill_host_arena_bytes(L, 64, 128, g, c, k, pv.FP8_E4M3), dtype=torch.uint8, device="cuda")
    pv.pivot_index_prefill_host(hq, hw, hk, L, 64, 128, g, c, k, mode, hout, arena, q_scale=hqs, k_scale=hks)
    assert _rows_equal_as_sets(hout.cuda(), plain)
    del arena
    torch.cuda.empty_cache()


def test_config5_prefill_256k_fp8_refine():
    _run_and_check(262144, "fp8", 4, 4096, 2048, po.MODE_REFINE, n_random=12)


def test_prefill_512k_fp8_refine_beyond_the_benchmark_sizes():
    """Four times the headline length (4.3 GB of queries, 131072 groups): sizes and offsets past
    the benchmark's, same launch path."""
    _run_and_check(524288, "fp8", 4, 4096, 2048, po.MODE_REFINE, n_random=2)
    _cache.clear()


def test_config4_decode_mtp_groups():
    """32 sequences, prefix lengths uniform in [64K, 128K], FP8 cache, g = 2, Refine."""
    import gpu_util
    _cache.clear()
    x = inputs.make_decode(32, 2, 65536, 131072, dtype="fp8")
    out, sc, cand, cs = gpu_util.run_decode(x, c=4096, k=2048, mode=po.MODE_REFINE)
    t = acc.check_decode(x.codes(), c=4096, k=2048, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                         out_scores=sc, cand=cand, cand_scores=cs, seqs=[0, 1, 7, 15, 16, 30, 31])
    print(f"\n[decode cfg4] rows={t.rows} exact={t.exact_rows} band_swaps={t.band_swaps} "
          f"worst_score_err={t.max_score_err:.3f} x tol")
    pos0 = x.pos0.numpy()
    for b in range(32):
        for i in range(2):
            assert out[b, i].min() >= 0 and out[b, i].max() <= pos0[b] + i
            assert len(np.unique(out[b, i])) == 2048


def test_decode_million_key_sequences():
    """Two sequences of about a million keys each (eight times the benchmark's longest)."""
    import gpu_util
    x = inputs.make_decode(2, 2, 900000, 1048000, dtype="fp8", seed=41)
    out, sc, cand, cs = gpu_util.run_decode(x, c=4096, k=2048, mode=po.MODE_REFINE)
    t = acc.check_decode(x.codes(), c=4096, k=2048, mode=po.MODE_REFINE, guard_len=None, out_idx=out,
                         out_scores=sc, cand=cand, cand_scores=cs)
    assert t.rows == 6          # per sequence: the candidate set and its two queries
