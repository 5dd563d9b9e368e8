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


def run_decode(x, *, c, k, mode, guard_len=None, W=0):
    d = to_cuda(x)
    B, g, H, dd = x.q.shape
    Lmax = x.k.shape[1]
    out = torch.full((B, g, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((B, g, k), float("nan"), dtype=torch.float32, device="cuda")
    cand = torch.full((B, c), -7, dtype=torch.int32, device="cuda") if mode == pv.REFINE else None
    cs = torch.full((B, c), float("nan"), dtype=torch.float32, device="cuda") if cand is not None else None
    pv.pivot_index_decode(d["q"], d["w"], d["k"], d["pos0"], B, Lmax, H, dd, g, c, k, mode, out,
                          q_scale=d["qscale"], k_scale=d["kscale"], guard_len=guard_len, dbg_cand=cand,
                          dbg_scores=scores, dbg_cand_scores=cs, W=W)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    f = lambda t: None if t is None else t.cpu().numpy()
    return f(out), f(scores), f(cand), f(cs)


def run_decode_paged(x, *, c, k, mode, seed=0, bad_entry=None, W=0):
    """The same decode step over a paged copy of x's key cache: pages scattered over a pool by a
    seeded permutation, spare pool pages filled with large codes (a wrong page read shows up)."""
    d = to_cuda(x)
    B, g, H, dd = x.q.shape
    Lmax = x.k.shape[1]
    mp = (Lmax + 127) // 128
    gen = torch.Generator().manual_seed(seed)
    n_pages = B * mp + 5
    perm = torch.randperm(n_pages, generator=gen)[: B * mp].to(torch.int32).reshape(B, mp)
    kd = d["k"]
    kb = kd.view(torch.uint8)                          # [B, Lmax, row bytes]
    pool_b = torch.full((n_pages * 128, kb.shape[2]), 0x7e if kd.element_size() == 1 else 0x40,
                        dtype=torch.uint8, device="cuda")
    ks = d["kscale"]
    pool_s = torch.full((n_pages * 128,), 7.0, dtype=torch.float32, device="cuda") if ks is not None else None
    for b in range(B):
        for p_ in range(mp):
            n = min(128, Lmax - p_ * 128)
            r0 = int(perm[b, p_]) * 128
            pool_b[r0:r0 + n] = kb[b, p_ * 128:p_ * 128 + n]
            if ks is not None:
                pool_s[r0:r0 + n] = ks[b, p_ * 128:p_ * 128 + n]
    pool = pool_b.view(kd.dtype)
    bt = perm.clone()
    if bad_entry is not None:
        bt[bad_entry] = n_pages + 3
    bt = bt.cuda()
    out = torch.full((B, g, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((B, g, k), float("nan"), dtype=torch.float32, device="cuda")
    cand = torch.full((B, c), -7, dtype=torch.int32, device="cuda") if mode == pv.REFINE else None
    cs = torch.full((B, c), float("nan"), dtype=torch.float32, device="cuda") if cand is not None else None
    pv.pivot_index_decode_paged(d["q"], d["w"], pool, bt, d["pos0"], B, mp, n_pages, H, dd, g, c, k, mode, out,
                                q_scale=d["qscale"], k_scale=pool_s, dbg_cand=cand, dbg_scores=scores,
                                dbg_cand_scores=cs, W=W)
    torch.cuda.synchronize()
    assert pv.pivot_device_status() == 0
    f = lambda t: None if t is None else t.cpu().numpy()
    return f(out), f(scores), f(cand), f(cs)
