"""The N > 1 path of bench.py on CPU: two gloo ranks reduce their step times with max-over-ranks and
turn them into whole-job throughput (independent replicas, no data-path collective)."""
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
    ms = bench.max_over_ranks(2.0 + rank, world, "cpu")       # rank 1 is the slow one
    out[rank] = (ms, bench.job_throughput(2.0 * 8192 ** 3, ms, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_their_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29533, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 3.0 and res[1][0] == 3.0
    expect = 2 * 2.0 * 8192 ** 3 / 3.0e-3 / 1e12
    assert abs(res[0][1] - expect) < 1e-9 * expect and res[0][1] == res[1][1]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5, 1, "cpu") == 1.5
    assert abs(bench.job_throughput(2e12, 1000.0, 1) - 2.0) < 1e-12
