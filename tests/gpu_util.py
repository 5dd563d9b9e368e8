"""Helpers for the GPU parity tests: run the library on seeded tensors, return numpy results."""
import numpy as np
import torch

from paper_2607_24593_b200 import binding as pv


def to_cuda(x):
    d = {}
    for name in ("q", "qscale", "w", "k", "kscale", "pos0"):
        t = getattr(x, name)
        d[name] = None if t is None else t.cuda()
    return d


def run_prefill(x, *, g, c, k, mode, guard_len=None, pool=pv.POOL_MEAN, debug=True, W=0, impl=0):
    d = to_cuda(x)
    L, H, dd = x.q.shape
    nG = (L + g - 1) // g
    out = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((L, k), float("nan"), dtype=torch.float32, device="cuda") if debug else None
    cand = torch.full((nG, c), -7, dtype=torch.int32, device="cuda") if debug and mode == pv.REFINE else None
    cs = torch.full((nG, c), float("nan"), dtype=torch.float32, device="cuda") if cand is not None else None
    pv.pivot_index_prefill(d["q"], d["w"], d["k"], L, H, dd, g, c, k, mode, out, q_scale=d["qscale"],
                           k_scale=d["kscale"], guard_len=guard_len, pool=pool, dbg_cand=cand,
                           dbg_scores=scores, dbg_cand_scores=cs, W=W, impl=impl)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    f = lambda t: None if t is None else t.cpu().numpy()
    return f(out), f(scores), f(cand), f(cs)


def run_dense(x, *, k):
    d = to_cuda(x)
    L, H, dd = x.q.shape
    out = torch.full((L, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((L, k), float("nan"), dtype=torch.float32, device="cuda")
    pv.dense_index(d["q"], d["w"], d["k"], L, H, dd, k, out, q_scale=d["qscale"], k_scale=d["kscale"],
                   dbg_scores=scores)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    return out.cpu().numpy(), scores.cpu().numpy()


def run_decode(x, *, c, k, mode, guard_len=None):
    d = to_cuda(x)
    B, g, H, dd = x.q.shape
    Lmax = x.k.shape[1]
    out = torch.full((B, g, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((B, g, k), float("nan"), dtype=torch.float32, device="cuda")
    cand = torch.full((B, c), -7, dtype=torch.int32, device="cuda") if mode == pv.REFINE else None
    cs = torch.full((B, c), float("nan"), dtype=torch.float32, device="cuda") if cand is not None else None
    pv.pivot_index_decode(d["q"], d["w"], d["k"], d["pos0"], B, Lmax, H, dd, g, c, k, mode, out,
                          q_scale=d["qscale"], k_scale=d["kscale"], guard_len=guard_len, dbg_cand=cand,
                          dbg_scores=scores, dbg_cand_scores=cs)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    f = lambda t: None if t is None else t.cpu().numpy()
    return f(out), f(scores), f(cand), f(cs)
