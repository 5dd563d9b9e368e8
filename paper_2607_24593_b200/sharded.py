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
