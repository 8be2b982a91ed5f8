"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, no GPU.

The path has no data-path collective (every rank compresses its own replica); what the ranks share
is the timing rule: the job takes as long as its slowest rank, and the value is all ranks' units
over that time.
"""
import os
import sys

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
    ms = [10.0 + 5.0 * rank, 40.0 - 3.0 * rank]            # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(ms, world, "cpu")
    layers = bench.rank_layers(rank)
    gathered = [None] * world
    dist.all_gather_object(gathered, layers)
    if rank == 0:
        out.put((got, gathered, bench.job_throughput(world, 4, 1000, got[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_share_only_the_timing_rule():
    world, port = 2, 29611 + os.getpid() % 500
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got, gathered, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [15.0, 40.0]                              # element-wise maximum over the ranks
    assert len(set(gathered[0]) | set(gathered[1])) == len(gathered[0]) + len(gathered[1])   # disjoint replicas
    assert abs(value - 2 * 4 * 1000 / 15e-3) < 1e-6        # both ranks' units over the slowest rank's time
