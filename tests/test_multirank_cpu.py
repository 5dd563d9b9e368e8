"""N > 1 host logic on CPU (gloo, world size 2): every rank indexes its own request -- no
data-path collective -- and the job's throughput is the units of all ranks over the slowest
rank's time.  Uses the oracle as the per-rank worker so no GPU is needed."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from oracle import pivot_oracle as po
    from paper_2607_24593_b200 import inputs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L, g, c, k = 256, 4, 32, 16
    x = inputs.make_prefill(L, 4, 8, dtype="bf16", seed=bench.rank_seed(rank), threads=1)
    res = po.pivot_prefill(x.codes(), g=g, c=c, k=k, mode=po.MODE_REFINE)
    out = po.assemble(res, L, k)
    my_ms = 10.0 * (rank + 1)                       # pretend rank 1 is slower
    slowest = bench.max_over_ranks(my_ms, dist)
    digest = torch.tensor([float(out[out >= 0].sum())], dtype=torch.float64)
    both = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(both, digest)
    if rank == 0:
        ret["slowest"] = slowest
        ret["value"] = bench.job_throughput(world, L, slowest)
        ret["digests"] = [float(b.item()) for b in both]
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_index_independent_requests():
    with mp.Manager() as m:
        ret = m.dict()
        port = 29500 + (os.getpid() % 2000)
        mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
        assert ret["slowest"] == 20.0                       # max over ranks, not the mean
        assert abs(ret["value"] - 2 * 256 / 20e-3) < 1e-6   # all ranks' tokens over the slowest time
        assert ret["digests"][0] != ret["digests"][1]       # different requests per rank


# ---------------------------------------------------------------- one request sharded over the ranks

def test_row_blocks_cover_the_request_and_balance():
    from paper_2607_24593_b200 import sharded
    for L, g, world, br in [(131072, 4, 8, 8192), (1000, 3, 2, 64), (7, 4, 4, 8), (50000, 8, 3, 4096)]:
        blocks = sharded.row_blocks(L, g, br)
        assert blocks[0][0] == 0 and blocks[-1][1] == L
        assert all(a[1] == b[0] for a, b in zip(blocks[:-1], blocks[1:]))
        assert all(r0 % g == 0 for r0, _ in blocks)                       # whole groups
        seen = sorted(b for r in range(world) for b in sharded.my_blocks(L, g, world, r, br))
        assert seen == blocks                                             # every block has exactly one owner
    assert [sharded.owner(i, 4) for i in range(10)] == [0, 1, 2, 3, 3, 2, 1, 0, 0, 1]
    assert sharded.imbalance(131072, 4, 8) < 1.01                         # snake order pairs cheap with expensive blocks
    assert sharded.imbalance(131072, 4, 8) < sum(
        sharded.block_cost(b) for i, b in enumerate(sharded.row_blocks(131072, 4)) if i % 8 == 7) / (
        sum(sharded.block_cost(b) for b in sharded.row_blocks(131072, 4)) / 8)   # plain cyclic is worse


def _shard_worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import pivot_oracle as po
    from paper_2607_24593_b200 import inputs, sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L, g, c, k, br = 300, 4, 32, 16, 40
    x = inputs.make_prefill(L, 4, 8, dtype="bf16", seed=5, threads=1).codes()      # the same request on every rank
    out = torch.full((L, k), -7, dtype=torch.int32)

    def index_rows(b):                      # stands in for the library's chunked prefill (rows=(r0, r1))
        r0, r1 = b
        res = po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE, groups=range(r0 // g, (r1 + g - 1) // g))
        for gr in res.values():
            out[torch.from_numpy(gr.members)] = torch.from_numpy(gr.T)

    mine = sharded.index_my_rows(index_rows, L, g, world, rank, br)
    untouched = torch.ones(L, dtype=torch.bool)
    for r0, r1 in mine:
        untouched[r0:r1] = False
    assert (out[untouched] == -7).all()     # a rank writes its own rows only
    sharded.all_gather_rows(out, L, g, world, rank, br)
    if rank == 0:
        ret["out"] = out.numpy().copy()
    dist.barrier()
    dist.destroy_process_group()


def test_one_request_sharded_over_two_ranks_matches_one_process():
    from oracle import pivot_oracle as po
    from paper_2607_24593_b200 import inputs
    with mp.Manager() as m:
        ret = m.dict()
        port = 31500 + (os.getpid() % 2000)
        mp.spawn(_shard_worker, args=(2, port, ret), nprocs=2, join=True)
        got = ret["out"]
    L, g, c, k = 300, 4, 32, 16
    x = inputs.make_prefill(L, 4, 8, dtype="bf16", seed=5, threads=1).codes()
    want = po.assemble(po.pivot_prefill(x, g=g, c=c, k=k, mode=po.MODE_REFINE), L, k)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------- one decode sequence, key axis split over the ranks

def test_key_ranges_cover_the_prefix_in_whole_tiles():
    from paper_2607_24593_b200 import sharded
    for n, world in [(1, 1), (1, 4), (127, 2), (128, 2), (129, 2), (100000, 8), (70001, 3), (300, 5)]:
        rs = sharded.key_ranges(n, world)
        assert len(rs) == world and rs[0][0] == 0 and max(r[1] for r in rs) == n
        prev = 0
        for k0, k1 in rs:
            assert k0 <= k1 and (k1 == k0 or (k0 == prev and k0 % 128 == 0))    # contiguous, tile-aligned starts
            prev = max(prev, k1)
        assert sum(k1 - k0 for k0, k1 in rs) == n


def _keysplit_worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import pivot_oracle as po
    from paper_2607_24593_b200 import inputs, sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    c = 48
    x = inputs.make_decode(1, 2, 900, 1000, 4, 8, dtype="bf16", seed=11, threads=1).codes()     # the same sequence on every rank
    p0 = int(x["pos0"][0])
    rows = np.arange(2)
    pq, pw = po.build_proxy(x["q"][0][rows], None, x["w"][0][rows], "bf16")                     # Eq. 4: same proxy everywhere
    kd = po.decode_operand(x["k"][0, : p0 + 1], "bf16")
    k0, k1 = sharded.key_ranges(p0 + 1, world)[rank]
    sc = torch.full((c,), float("-inf"), dtype=torch.float64)
    ix = torch.full((c,), -1, dtype=torch.int32)
    if k1 > k0:                                   # the oracle stands in for the library's scan of this range
        s = po.indexer_scores(po.decode_operand(pq, "bf16"), pw, kd[k0:k1], None)
        top = po.top_set(s, c)                     # positions relative to the range
        sc[: len(top)] = torch.from_numpy(s[top])
        ix[: len(top)] = torch.from_numpy(top.astype(np.int32))
    all_sc, all_ix = sharded.gather_candidate_lists(sc, ix, world)
    offs = np.array([r[0] for r in sharded.key_ranges(p0 + 1, world)])
    pos = (all_ix.numpy().astype(np.int64) + offs[:, None]).ravel()
    val = all_sc.numpy().ravel()
    keep = all_ix.numpy().ravel() >= 0
    merged = po.top_set(val[keep], c, pos[keep])
    if rank == 0:
        ret["merged"] = merged.tolist()
        ret["p0"] = p0
    dist.barrier()
    dist.destroy_process_group()


def test_key_split_merge_of_two_ranks_is_the_single_process_candidate_set():
    """Eq. 7 over a key axis split in two: the merge of the ranks' local top-c lists (one
    all-gather of c pairs per rank) is the oracle's top-c over the whole prefix."""
    from oracle import pivot_oracle as po
    from paper_2607_24593_b200 import inputs
    with mp.Manager() as m:
        ret = m.dict()
        port = 33500 + (os.getpid() % 2000)
        mp.spawn(_keysplit_worker, args=(2, port, ret), nprocs=2, join=True)
        merged, p0 = ret["merged"], ret["p0"]
    x = inputs.make_decode(1, 2, 900, 1000, 4, 8, dtype="bf16", seed=11, threads=1).codes()
    r = po.pivot_decode(x, c=48, k=16, mode=po.MODE_REFINE, guard_len=0)[0]
    assert p0 == int(x["pos0"][0])
    assert merged == r.C.tolist()                 # same set, same (score desc, position asc) order
