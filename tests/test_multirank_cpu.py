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
