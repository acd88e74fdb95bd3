"""Multi-rank bookkeeping of bench.py on CPU: two gloo ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2608_01651_b200 import inputs
    wl = bench.rank_workload(inputs.workload("c3", B=2, H=2), rank)
    parents, accepted = inputs.make_trees(wl)
    times = [10.0 + rank, 5.0 - rank, 1.0, 0.0]
    red = bench.max_over_ranks(times, world, "cpu")
    dist.barrier()
    out[rank] = (wl.seed, parents.tobytes(), red, bench.job_nodes_per_step(wl, world))
    dist.destroy_process_group()


def test_two_ranks_shard_by_request_and_take_the_slowest_time():
    world = 2
    port = 29500 + (os.getpid() % 1000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    (s0, p0, r0, n0), (s1, p1, r1, n1) = res[0], res[1]
    assert s0 != s1 and p0 != p1            # each rank draws its own requests
    assert r0 == r1 == [11.0, 5.0, 1.0, 0.0]  # element-wise max over ranks, same on every rank
    assert n0 == n1 == 2 * 64 * 1 * world     # weak scaling: units add up over ranks


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, "cpu") == [1.5, 2.5]
