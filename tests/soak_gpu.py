"""Randomised parity soak (run by hand on a GPU machine; pytest does not collect it):

    python tests/soak_gpu.py [seed] [seconds] [decode length scale]

draws prefill and decode configurations at random from the seed -- lengths, group sizes, budgets,
guardrails, local windows, pooling, operand types, contiguous or paged caches -- runs each through
the C ABI and checks sampled groups (prefill) or the whole step (decode) against the oracle with
the acceptance rule.  Prints every failing configuration and a final count; exit status 1 if any.
"""
import sys, time, traceback
import os
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT); sys.path.insert(0, os.path.join(ROOT, 'tests'))
import numpy as np
import gpu_util as gu
from oracle import acceptance as acc, pivot_oracle as po
from paper_2607_24593_b200 import inputs, binding as pv
rng = np.random.default_rng(int(sys.argv[1]) if len(sys.argv) > 1 else 7)
pools = {"mean": pv.POOL_MEAN, "first": pv.POOL_FIRST, "last": pv.POOL_LAST}
DEC_MAX = int(sys.argv[3]) if len(sys.argv) > 3 else 6000        # decode prefix lengths up to about twice this
fails = 0
t0 = time.time()
n = 0
while time.time() - t0 < float(sys.argv[2]) if len(sys.argv) > 2 else 300:
    L = int(rng.integers(1, 9000)); g = int(rng.integers(1, 12)); k = int(rng.integers(1, 1200)); c = int(k + rng.integers(0, 1500))
    mode = int(rng.integers(0, 2)); dtype = ("bf16", "fp8")[int(rng.integers(0, 2))]
    guard = (None, 0, int(rng.integers(1, c + 50)))[int(rng.integers(0, 3))]
    W = 0
    if rng.integers(0, 3) == 0:
        W = int(rng.integers(1, 9)); eg = c if guard is None else guard
        if W + g - 1 >= c or eg < W + g: continue
    pool = ("mean", "first", "last")[int(rng.integers(0, 3))]
    cfg = (L, g, c, k, mode, dtype, guard, W, pool)
    try:
        x = inputs.make_prefill(L, dtype=dtype, seed=int(rng.integers(1, 1 << 30)))
        out, sc, cand, cs = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, guard_len=guard, pool=pools[pool], W=W)
        nG = (L + g - 1) // g
        groups = sorted(set(rng.integers(0, nG, 12).tolist() + [0, nG - 1]))
        acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=guard, out_idx=out, out_scores=sc, cand=cand,
                          cand_scores=cs, pool=pool, W=W, groups=groups)
        # the same request through other forms of the call: fp32 head sum, two row chunks, dense control
        import torch
        if dtype == "fp8" and rng.integers(0, 3) == 0:
            o2 = gu.run_prefill(x, g=g, c=c, k=k, mode=mode, guard_len=guard, pool=pools[pool], W=W, impl=2)
            acc.check_prefill(x.codes(), g=g, c=c, k=k, mode=mode, guard_len=guard, out_idx=o2[0], out_scores=o2[1],
                              cand=o2[2], cand_scores=o2[3], pool=pool, W=W, groups=groups)
        if nG > 1 and rng.integers(0, 2) == 0:
            d = gu.to_cuda(x)
            cut = int(rng.integers(1, nG)) * g
            parts = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
            for rows_ in ((0, cut), (cut, L)):
                pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, 64, 128, g, c, k, mode, parts, q_scale=d["qscale"],
                                       k_scale=d["kscale"], guard_len=guard, pool=pools[pool], W=W, rows=rows_)
            torch.cuda.synchronize()
            assert np.array_equal(np.sort(parts.cpu().numpy(), axis=1), np.sort(out, axis=1)), "row chunks differ from the whole call"
        if L <= 3000 and rng.integers(0, 3) == 0:
            do, ds = gu.run_dense(x, k=k)
            acc.check_dense(x.codes(), k=k, out_idx=do, out_scores=ds, rows=sorted(set(rng.integers(0, L, 10).tolist() + [0, L - 1])))
    except Exception as e:
        fails += 1
        print("FAIL prefill", cfg, repr(e)[:300]); traceback.print_exc(limit=2)
    n += 1
    # a decode step
    B = int(rng.integers(1, 9)); gd = int(rng.integers(1, 7)); lo = int(rng.integers(1, DEC_MAX)); hi = lo + int(rng.integers(0, DEC_MAX))
    kd = int(rng.integers(1, 600)); cd = int(kd + rng.integers(0, 900)); md = int(rng.integers(0, 2)); paged = bool(rng.integers(0, 3) == 0)
    gdl = 0 if paged else (None, 0, int(rng.integers(1, cd + 50)))[int(rng.integers(0, 3))]
    Wd = int(gd + rng.integers(0, 12)) if (md == 1 and rng.integers(0, 3) == 0) else 0
    cfg = (B, gd, lo, hi, cd, kd, md, dtype, gdl, Wd, paged)
    try:
        xd = inputs.make_decode(B, gd, lo, hi, dtype=dtype, seed=int(rng.integers(1, 1 << 30)))
        if paged: o = gu.run_decode_paged(xd, c=cd, k=kd, mode=md, seed=lo, W=Wd)
        else: o = gu.run_decode(xd, c=cd, k=kd, mode=md, guard_len=gdl, W=Wd)
        acc.check_decode(xd.codes(), c=cd, k=kd, mode=md, guard_len=gdl, out_idx=o[0], out_scores=o[1], cand=o[2], cand_scores=o[3], W=Wd)
    except Exception as e:
        fails += 1
        print("FAIL decode", cfg, repr(e)[:300]); traceback.print_exc(limit=2)
    n += 1
print("cases", n, "fails", fails, "seconds", round(time.time() - t0))
sys.exit(1 if fails else 0)
