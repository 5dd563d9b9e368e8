"""One prefill request over several GPUs (one process per GPU, torch.distributed for the plumbing).

Groups are independent given the key cache (Eq. 2, Eq. 5: every group scans the shared keys with
its own proxy), so the query rows of a request are cut into blocks of whole groups and dealt to the
ranks; each rank indexes its blocks with the chunked-prefill form of the library
(`pivot_opts.row_begin / row_end`) against its own copy of the key cache, and the index sets are
exchanged once at the end if every rank needs all of them.  There is no collective on the data
path of the kernels.

A block's cost grows with its position (later rows scan longer prefixes), so the blocks are dealt
in snake order -- rank r gets blocks r, 2P-1-r, 2P+r, ... -- which pairs a cheap block with an
expensive one.

This module only decides who indexes which rows and moves results; the indexing itself is
`binding.pivot_index_prefill` (or any callable with the same `rows=` contract, which is how the
CPU test drives it without a GPU).
"""
from __future__ import annotations

from typing import Callable, List, Sequence, Tuple

import torch
import torch.distributed as dist

Block = Tuple[int, int]


def row_blocks(L: int, g: int, block_rows: int = 8192) -> List[Block]:
    """Blocks [r0, r1) of whole groups covering rows 0 .. L-1 (the last may be short)."""
    if L < 1 or g < 1 or block_rows < 1:
        raise ValueError("L, g and block_rows must be positive")
    br = max(g, block_rows // g * g)
    return [(r0, min(r0 + br, L)) for r0 in range(0, L, br)]


def owner(block: int, world: int) -> int:
    """Rank that indexes block number `block` (snake order over the ranks)."""
    rnd, pos = divmod(block, world)
    return pos if rnd % 2 == 0 else world - 1 - pos


def my_blocks(L: int, g: int, world: int, rank: int, block_rows: int = 8192) -> List[Block]:
    return [b for i, b in enumerate(row_blocks(L, g, block_rows)) if owner(i, world) == rank]


def block_cost(block: Block) -> float:
    """Relative scan cost of a block: sum over its rows of the prefix length (the causal ramp)."""
    r0, r1 = block
    return 0.5 * (r1 - r0) * (r0 + r1 + 1)


def index_my_rows(index_rows: Callable[[Block], None], L: int, g: int, world: int, rank: int,
                  block_rows: int = 8192) -> List[Block]:
    """Calls index_rows((r0, r1)) for every block of this rank; returns those blocks."""
    mine = my_blocks(L, g, world, rank, block_rows)
    for b in mine:
        index_rows(b)
    return mine


def pivot_index_prefill_sharded(q, w, kcache, L, H_I, d, g, c, k, mode, out_idx, *, rank: int, world: int,
                                block_rows: int = 8192, stream=None, **kw) -> List[Block]:
    """Indexes this rank's share of the request's rows into out_idx ([L, k], the other rows are
    left untouched).  q / w / kcache hold the whole request on every rank (the queries of rows a
    rank does not own are never read, so they may be left uninitialised there)."""
    from . import binding as pv

    def run(b: Block):
        pv.pivot_index_prefill(q, w, kcache, L, H_I, d, g, c, k, mode, out_idx, stream, rows=b, **kw)

    return index_my_rows(run, L, g, world, rank, block_rows)


def all_gather_rows(out_idx: torch.Tensor, L: int, g: int, world: int, rank: int, block_rows: int = 8192,
                    group=None) -> torch.Tensor:
    """After every rank has indexed its blocks: fills the other ranks' rows of out_idx ([L, k]) on
    every rank with one all-gather of the ranks' packed rows.  Works on CPU (gloo) and GPU (nccl)
    tensors alike."""
    blocks = row_blocks(L, g, block_rows)
    k = out_idx.shape[1]
    rows_of = [[b for i, b in enumerate(blocks) if owner(i, world) == r] for r in range(world)]
    cap = max(sum(r1 - r0 for r0, r1 in bl) for bl in rows_of)
    send = torch.full((cap, k), -1, dtype=out_idx.dtype, device=out_idx.device)
    at = 0
    for r0, r1 in rows_of[rank]:
        send[at:at + r1 - r0] = out_idx[r0:r1]
        at += r1 - r0
    recv = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(recv, send, group=group)
    for r in range(world):
        if r == rank:
            continue
        at = 0
        for r0, r1 in rows_of[r]:
            out_idx[r0:r1] = recv[r][at:at + r1 - r0]
            at += r1 - r0
    return out_idx


def imbalance(L: int, g: int, world: int, block_rows: int = 8192) -> float:
    """Slowest rank's share of the scan cost over the mean share (1.0 = perfectly balanced)."""
    blocks = row_blocks(L, g, block_rows)
    cost = [0.0] * world
    for i, b in enumerate(blocks):
        cost[owner(i, world)] += block_cost(b)
    return max(cost) / (sum(cost) / world)


# ------------------------------------------------------------------------------------------------
# One decode sequence over several GPUs: the key axis of the shared scan is split.
#
# The scan of Eq. 5 is a score per key, so key ranges are independent; a key of the global top-c
# (Eq. 7) is in the top-c of its own range.  Every rank holds the sequence's key cache, scans its
# own range into a local top-c with proxy scores, the (score, position) lists are exchanged once
# (c pairs per rank), every rank merges them into the same global candidate set, and Eq. 8-9 run
# on that set (on the owner, or on every rank alike).  The exchange is the only collective.

def key_ranges(n_visible: int, world: int, tile: int = 128) -> List[Block]:
    """Rank r scans keys [k0, k1) of the n_visible keys: whole 128-key tiles dealt evenly, the last
    range ends at n_visible; ranks beyond the tile count get an empty range."""
    if n_visible < 1 or world < 1:
        raise ValueError("n_visible and world must be positive")
    tiles = (n_visible + tile - 1) // tile
    per = (tiles + world - 1) // world
    out = []
    for r in range(world):
        t0, t1 = min(r * per, tiles), min((r + 1) * per, tiles)
        out.append((t0 * tile, min(t1 * tile, n_visible)) if t1 > t0 else (n_visible, n_visible))
    return out


def gather_candidate_lists(scores: torch.Tensor, idx: torch.Tensor, world: int, group=None):
    """All-gather of the ranks' local lists ([c] each) into [world, c] tensors on every rank."""
    all_sc = [torch.empty_like(scores) for _ in range(world)]
    all_ix = [torch.empty_like(idx) for _ in range(world)]
    dist.all_gather(all_sc, scores, group=group)
    dist.all_gather(all_ix, idx, group=group)
    return torch.stack(all_sc), torch.stack(all_ix)


def decode_keysplit_local(q, w, kcache, pos0: int, Lmax, H_I, d, c, *, rank: int, world: int, stream=None,
                          q_scale=None, k_scale=None):
    """This rank's part of the scan of ONE sequence (q [1, g, H, d], kcache [1, Lmax, d]): the local
    top-c of the proxy scores over its key range.  Returns (scores [c] fp32, positions [c] int32
    relative to the range, -1 padded, range start)."""
    from . import binding as pv
    g = q.shape[1]
    k0, k1 = key_ranges(pos0 + 1, world)[rank]
    dev = q.device
    sc = torch.full((c,), float("-inf"), dtype=torch.float32, device=dev)
    ix = torch.full((c,), -1, dtype=torch.int32, device=dev)
    if k1 > k0:
        out = torch.empty((1, g, c), dtype=torch.int32, device=dev)
        osc = torch.empty((1, g, c), dtype=torch.float32, device=dev)
        view = kcache[:, k0:]                              # one sequence: the range is a contiguous view
        vks = None if k_scale is None else k_scale[:, k0:]
        p0 = torch.tensor([k1 - k0 - 1], dtype=torch.int32, device=dev)
        # Reuse with k = c on the range: the proxy of the step's g queries, its top-c and their scores
        pv.pivot_index_decode(q, w, view, p0, 1, Lmax - k0, H_I, d, g, c, c, pv.REUSE, out, stream, q_scale=q_scale,
                              k_scale=vks, guard_len=0, dbg_scores=osc)
        sc, ix = osc[0, 0].contiguous(), out[0, 0].contiguous()
    return sc, ix, k0


def decode_keysplit_finish(q, w, kcache, pos0_dev, Lmax, H_I, d, c, k, out_idx, all_scores, all_idx, offsets, *,
                           stream=None, q_scale=None, k_scale=None, cand_out=None):
    """Merge of the gathered lists ([world, c]) into the global candidate set, then Eq. 8-9 on it.
    offsets [world] int32 (device): first key of each rank's range."""
    from . import binding as pv
    cand = cand_out if cand_out is not None else torch.empty((1, c), dtype=torch.int32, device=q.device)
    pv.pivot_merge_topk(all_scores, all_idx, c, cand, seg_offset=offsets, stream=stream)
    g = q.shape[1]
    pv.pivot_index_decode(q, w, kcache, pos0_dev, 1, Lmax, H_I, d, g, c, k, pv.REFINE, out_idx, stream, q_scale=q_scale,
                          k_scale=k_scale, guard_len=0, cand_in=cand)
    return cand


def pivot_index_decode_keysplit(q, w, kcache, pos0: int, Lmax, H_I, d, c, k, out_idx, *, rank: int, world: int,
                                group=None, stream=None, q_scale=None, k_scale=None):
    """One MTP decode step of ONE sequence with its scan split over `world` ranks (one process per
    GPU, each holding the sequence's key cache).  Every rank returns the same out_idx [1, g, k]."""
    sc, ix, _ = decode_keysplit_local(q, w, kcache, pos0, Lmax, H_I, d, c, rank=rank, world=world, stream=stream,
                                      q_scale=q_scale, k_scale=k_scale)
    all_sc, all_ix = gather_candidate_lists(sc, ix, world, group) if world > 1 else (sc[None], ix[None])
    offsets = torch.tensor([r[0] for r in key_ranges(pos0 + 1, world)], dtype=torch.int32, device=q.device)
    pos0_dev = torch.tensor([pos0], dtype=torch.int32, device=q.device)
    decode_keysplit_finish(q, w, kcache, pos0_dev, Lmax, H_I, d, c, k, out_idx, all_sc.contiguous(), all_ix.contiguous(),
                           offsets, stream=stream, q_scale=q_scale, k_scale=k_scale)
    return out_idx
