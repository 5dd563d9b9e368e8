"""dense_index_static: the entry point for callers that are not allowed to allocate device
memory (its scratch is an array inside the library).  Checked through the C ABI against
dense_index on the same inputs, twice in a row with different sizes so that the second call
runs on whatever the first one left in the shared array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import acceptance as acc
from paper_2607_24593_b200 import inputs

pytestmark = pytest.mark.gpu


def _both(pv, x, L, k):
    q, w, kc = x.q.cuda(), x.w.cuda(), x.k.cuda()
    qs = None if x.qscale is None else x.qscale.cuda()
    ks = None if x.kscale is None else x.kscale.cuda()
    ref = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    got = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    pv.dense_index(q, w, kc, L, 64, 128, k, ref, q_scale=qs, k_scale=ks)
    before = torch.cuda.memory_allocated()
    pv.dense_index_static(q, w, kc, L, 64, 128, k, got, q_scale=qs, k_scale=ks)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    return ref.cpu().numpy(), got.cpu().numpy()


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_static_scratch_matches_dense_index_twice(dtype):
    from paper_2607_24593_b200 import binding as pv
    for L, k, seed in ((1500, 128, 31), (700, 256, 32)):          # two calls in a row
        x = inputs.make_prefill(L, dtype=dtype, seed=seed)
        ref, got = _both(pv, x, L, k)
        # same kernel, same scores: the selected sets must be identical row by row
        np.testing.assert_array_equal(np.sort(got, axis=1), np.sort(ref, axis=1))
        for t in (0, 1, k - 1, k, L - 1):
            n = min(k, t + 1)
            assert (np.sort(got[t])[k - n:] >= 0).all() and (got[t] <= t).all()
        # and against the CPU oracle (Eq. 1 + TopK), under the acceptance rule of the other tests
        rows = sorted({0, 1, k - 1, k, 127, 128, L // 2, L - 1} | set(np.random.default_rng(seed).integers(0, L, 24).tolist()))
        tally = acc.check_dense(x.codes(), k=k, out_idx=got, rows=rows)
        assert tally.rows == len(rows)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_static_scratch_at_its_size_limits(dtype):
    """L = 4096 and k = 512: the largest request the built-in scratch is sized for."""
    from paper_2607_24593_b200 import binding as pv
    L, k = 4096, 512
    x = inputs.make_prefill(L, dtype=dtype, seed=33)
    ref, got = _both(pv, x, L, k)
    np.testing.assert_array_equal(np.sort(got, axis=1), np.sort(ref, axis=1))
    rows = [0, 511, 512, 513, 2047, 4095]
    tally = acc.check_dense(x.codes(), k=k, out_idx=got, rows=rows)
    assert tally.rows == len(rows)


def test_static_scratch_rejects_oversize():
    from paper_2607_24593_b200 import binding as pv
    x = inputs.make_prefill(64, dtype="bf16", seed=1)
    q, w, kc = x.q.cuda(), x.w.cuda(), x.k.cuda()
    out = torch.empty((64, 1024), dtype=torch.int32, device="cuda")
    with pytest.raises(pv.PivotError, match="workspace"):
        pv.dense_index_static(q, w, kc, 64, 64, 128, 1024, out)          # k beyond the built-in scratch
    out2 = torch.empty((5000, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(pv.PivotError, match="workspace"):
        pv.dense_index_static(q, w, kc, 5000, 64, 128, 16, out2)        # L beyond it (checked before any access)
