"""N > 1 host logic on CPU: two gloo ranks reduce their timings the way bench.py
does (max of the elapsed times, sum of the records)."""
import os
import sys

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
    elapsed, e2e, total = bench.reduce_over_ranks(dist, 10.0 + 5.0 * rank, 100.0 - rank, 1000 + rank,
                                                  torch.device("cpu"))
    out[rank] = (elapsed, e2e, total)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_records():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29512, out), nprocs=2, join=True)
    for r in range(2):
        assert out[r] == (15.0, 100.0, 2001)
