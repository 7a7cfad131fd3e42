"""The N > 1 aggregation of bench.py (independent replicas, no data-path collective): the job's time is the
max over ranks and the value is the sum of the ranks' work over that time.  Two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + rank                       # seconds: rank 1 is the slower replica
    slowest = bench.slowest_rank(mine, world, "cpu")
    out[rank] = (slowest, bench.whole_job_rate(64, 10, world, slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, 29531 + os.getpid() % 1000, out), nprocs=world, join=True)
        assert out[0] == out[1] == (3.0, 2 * 64 * 10 / 3.0)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank(1.5, 1, "cpu") == 1.5
    assert bench.whole_job_rate(64, 100, 1, 0.5) == 12800.0
