"""Seeded synthetic indexer tensors (queries, gates, key cache) for tests and benchmarks.

This module only *draws inputs*: it holds none of the indexer's arithmetic (no scores, no
proxy, no selection).  Both the CUDA path and the CPU oracle are fed from here, so they see
identical bytes.  Storage casts (fp32 -> bf16, fp32 -> e4m3) use torch's CPU casts.

Recipe (stands in for the indexer activations of a DSA model on long prompts):
  keys     k_s = z_s / sqrt(d), z ~ N(0, I_d); each position is an outlier with probability
           0.02 (iid) and then gets + 4*u, u one shared random unit vector per key cache.
           This gives the long-tailed score profile the paper reports (observation O3).
  queries  every (head, channel) follows a stationary AR(1) along the position axis:
           q_0 ~ N(0, 1/(d(1-rho^2))), q_t = rho*q_{t-1} + eps_t, eps ~ N(0, 1/d) (variance),
           rho = 0.9, fp32 recursion, one rounding to bf16.  Neighbouring queries therefore
           overlap in what they select (observation O1).
  gates    w_{t,h} = |N(0,1)| / sqrt(H).
  fp8      the bf16 tensors are re-quantised to e4m3 with one fp32 scale per 128-vector:
           scale = max(amax, 1e-4) / 448, code = RN(x / scale); keys get one scale per
           position, queries one per (position, head).

Random streams are Philox counters keyed by (seed, tensor id, chunk index); a tensor is drawn
in chunks of CHUNK positions so the bytes do not depend on how many threads draw it.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

CHUNK = 4096          # positions per random-stream chunk (part of the recipe)
RHO = 0.9
OUTLIER_P = 0.02
OUTLIER_GAIN = 4.0
DEFAULT_SEED = 20260724

_TID_KEYS, _TID_OUTLIER, _TID_DIR, _TID_Q, _TID_Q0, _TID_W, _TID_LEN = range(7)


def _rng(seed: int, tensor_id: int, chunk: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) + tensor_id, (stream << 32) + chunk]))


def _chunks(n: int):
    return [(c, c * CHUNK, min(n, (c + 1) * CHUNK)) for c in range((n + CHUNK - 1) // CHUNK)]


def _pool_map(fn, items, threads: int):
    if threads <= 1 or len(items) <= 1:
        return [fn(it) for it in items]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(fn, items))


@dataclasses.dataclass
class IndexerTensors:
    """Host tensors of one indexer call.  `dtype` is "bf16" or "fp8".

    q      [L, H, d]  torch.bfloat16 or torch.float8_e4m3fn   (decode: [B, g, H, d])
    qscale [L, H]     float32 or None                         (decode: [B, g, H])
    w      [L, H]     float32                                 (decode: [B, g, H])
    k      [L, d]     storage dtype                           (decode: [B, Lmax, d])
    kscale [L]        float32 or None                         (decode: [B, Lmax])
    pos0   None, or int32 [B]: first query position of each decode group
    """
    dtype: str
    q: torch.Tensor
    qscale: torch.Tensor | None
    w: torch.Tensor
    k: torch.Tensor
    kscale: torch.Tensor | None
    pos0: torch.Tensor | None = None

    def codes(self):
        """Raw storage bits as numpy arrays (uint16 for bf16, uint8 for e4m3) plus scales."""
        view = torch.int16 if self.dtype == "bf16" else torch.uint8
        npdt = np.uint16 if self.dtype == "bf16" else np.uint8
        qc = self.q.view(view).numpy().view(npdt)
        kc = self.k.view(view).numpy().view(npdt)
        return dict(
            dtype=self.dtype, q=qc, qscale=None if self.qscale is None else self.qscale.numpy(),
            w=self.w.numpy(), k=kc, kscale=None if self.kscale is None else self.kscale.numpy(),
            pos0=None if self.pos0 is None else self.pos0.numpy())


def _draw_keys(n: int, d: int, seed: int, stream: int, threads: int) -> torch.Tensor:
    """fp32 keys [n, d] following the key recipe above."""
    u = _rng(seed, _TID_DIR, 0, stream).standard_normal(d).astype(np.float32)
    u /= np.float32(np.sqrt(np.sum(u.astype(np.float64) ** 2)))
    out = np.empty((n, d), np.float32)

    def fill(item):
        c, lo, hi = item
        z = _rng(seed, _TID_KEYS, c, stream).standard_normal((hi - lo, d), dtype=np.float32)
        z *= np.float32(1.0 / np.sqrt(d))
        hit = _rng(seed, _TID_OUTLIER, c, stream).random(hi - lo) < OUTLIER_P
        z[hit] += np.float32(OUTLIER_GAIN) * u
        out[lo:hi] = z

    _pool_map(fill, _chunks(n), threads)
    return torch.from_numpy(out)


def _draw_queries(n: int, H: int, d: int, seed: int, stream: int, threads: int) -> torch.Tensor:
    """bf16 queries [n, H, d]: stationary AR(1) along the first axis, per (head, channel)."""
    C = H * d
    out = torch.empty((n, C), dtype=torch.bfloat16)
    sd = np.float32(1.0 / np.sqrt(d))
    chunks = _chunks(n)

    def draw(item):
        c, lo, hi = item
        e = _rng(seed, _TID_Q, c, stream).standard_normal((hi - lo, C), dtype=np.float32)
        e *= sd
        return e

    state = _rng(seed, _TID_Q0, 0, stream).standard_normal(C, dtype=np.float32)
    state *= np.float32(1.0 / np.sqrt(d * (1.0 - RHO * RHO)))
    rho = np.float32(RHO)
    # draw chunks a few at a time (bounded memory), run the recursion serially
    step = max(1, threads)
    for base in range(0, len(chunks), step):
        batch = chunks[base:base + step]
        drawn = _pool_map(draw, batch, threads)
        for (c, lo, hi), e in zip(batch, drawn):
            if lo == 0:
                e[0] = state          # position 0 is the stationary draw itself
                start = 1
            else:
                start = 0
            for i in range(start, hi - lo):
                state = rho * state + e[i]
                e[i] = state
            out[lo:hi] = torch.from_numpy(e).to(torch.bfloat16)
    return out.view(n, H, d)


def _draw_gates(n: int, H: int, seed: int, stream: int) -> torch.Tensor:
    out = np.empty((n, H), np.float32)
    for c, lo, hi in _chunks(n):
        z = _rng(seed, _TID_W, c, stream).standard_normal((hi - lo, H), dtype=np.float32)
        out[lo:hi] = np.abs(z) * np.float32(1.0 / np.sqrt(H))
    return torch.from_numpy(out)


def quantize_e4m3(x: torch.Tensor):
    """x [..., d] (any float dtype) -> (e4m3 codes [..., d], fp32 scale [...]) with one scale
    per trailing vector: scale = max(amax, 1e-4)/448, code = RN(x/scale)."""
    xf = x.float()
    amax = xf.abs().amax(dim=-1).clamp_min(1e-4)
    scale = amax / 448.0
    codes = (xf / scale.unsqueeze(-1)).clamp(-448.0, 448.0).to(torch.float8_e4m3fn)
    return codes, scale.contiguous()


def _quantize_chunked(x: torch.Tensor, rows_per_chunk: int = 8192):
    n = x.shape[0]
    codes = torch.empty(x.shape, dtype=torch.float8_e4m3fn)
    scale = torch.empty(x.shape[:-1], dtype=torch.float32)
    for lo in range(0, n, rows_per_chunk):
        c, s = quantize_e4m3(x[lo:lo + rows_per_chunk])
        codes[lo:lo + rows_per_chunk] = c
        scale[lo:lo + rows_per_chunk] = s
    return codes, scale


def make_prefill(L: int, H: int = 64, d: int = 128, dtype: str = "bf16",
                 seed: int = DEFAULT_SEED, threads: int = 8) -> IndexerTensors:
    """One request of L positions: queries, gates and keys at every position."""
    assert dtype in ("bf16", "fp8")
    k = _draw_keys(L, d, seed, 0, threads).to(torch.bfloat16)
    q = _draw_queries(L, H, d, seed, 0, threads)
    w = _draw_gates(L, H, seed, 0)
    if dtype == "bf16":
        return IndexerTensors("bf16", q, None, w, k, None)
    q8, qs = _quantize_chunked(q)
    k8, ks = quantize_e4m3(k)
    return IndexerTensors("fp8", q8, qs, w, k8, ks)


def make_decode(B: int, g: int, len_lo: int, len_hi: int, H: int = 64, d: int = 128,
                dtype: str = "fp8", seed: int = DEFAULT_SEED, threads: int = 8) -> IndexerTensors:
    """B independent sequences, each with a key cache and one MTP group of g queries.

    The visible-prefix length n0_b = pos0_b + 1 is a uniform integer in [len_lo, len_hi];
    sequence b's cache holds keys 0 .. pos0_b + g - 1 (later rows of the [B, Lmax, d]
    buffer are zero), Lmax = len_hi + g rounded up to a multiple of 64.
    """
    assert dtype in ("bf16", "fp8")
    n0 = _rng(seed, _TID_LEN, 0).integers(len_lo, len_hi + 1, size=B).astype(np.int64)
    Lmax = (len_hi + g + 63) // 64 * 64       # rows per sequence, rounded up (alignment of the scale rows)
    st = torch.bfloat16 if dtype == "bf16" else torch.float8_e4m3fn
    k = torch.zeros((B, Lmax, d), dtype=torch.bfloat16).to(st)
    ks = None if dtype == "bf16" else torch.zeros((B, Lmax), dtype=torch.float32)
    q = torch.empty((B, g, H, d), dtype=st)
    qs = None if dtype == "bf16" else torch.empty((B, g, H), dtype=torch.float32)
    w = torch.empty((B, g, H), dtype=torch.float32)
    for b in range(B):
        nk = int(n0[b]) + g - 1
        kb = _draw_keys(nk, d, seed, 1 + b, threads).to(torch.bfloat16)
        qb = _draw_queries(g, H, d, seed, 1 + b, 1)
        w[b] = _draw_gates(g, H, seed, 1 + b)
        if dtype == "bf16":
            k[b, :nk] = kb
            q[b] = qb
        else:
            k8, s8 = quantize_e4m3(kb)
            k[b, :nk] = k8
            ks[b, :nk] = s8
            q8, q8s = quantize_e4m3(qb)
            q[b] = q8
            qs[b] = q8s
    pos0 = torch.from_numpy((n0 - 1).astype(np.int32))
    return IndexerTensors(dtype, q, qs, w, k, ks, pos0)
