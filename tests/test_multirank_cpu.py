"""The N > 1 path of the benchmark on CPU ranks (gloo, world size 2): token split with a
distinct seeded batch per rank, max-over-ranks of the timings, whole-job throughput."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        x = bench.rank_batch(2, 64, 32, rank)
        local_ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 slower on the first, faster on the second
        mx = bench.max_over_ranks(local_ms)
        dist.barrier()
        gathered = [None] * world
        dist.all_gather_object(gathered, float(x.sum()))
        out.put((rank, mx, gathered, bench.job_throughput(world, 64, 4, mx[0])))
    finally:
        dist.destroy_process_group()


def test_token_split_and_max_over_ranks():
    world, port = 2, 29500 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, gathered, tput in res:
        assert mx == [15.0, 3.0]                                  # slowest rank decides, on every rank
        assert gathered[0] != gathered[1]                         # ranks run different batches
        assert tput == 2 * 64 * 4 / 15e-3                         # all ranks' tokens over the slowest time
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]         # single process: identity
    assert np.array_equal(bench.rank_batch(2, 8, 16, 1), bench.rank_batch(2, 8, 16, 1))
