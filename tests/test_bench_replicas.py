"""Multi-rank bookkeeping of bench.py on CPU: the replicas exchange no data; the only collective is the MAX
over ranks of the timings (gloo, world_size 2)."""
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
    dev_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 30.0 - 7.0 * rank], dist)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (dev_ms, e2e_ms, bench.replicas_value(world, 1000, dev_ms / 5))


def test_timings_are_the_max_over_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
    for rank in range(world):
        dev_ms, e2e_ms, value = out[rank]
        assert dev_ms == 15.0 and e2e_ms == 30.0            # slowest rank of each timing
        assert abs(value - 2 * 1000 / (3.0e-3)) < 1e-6      # two replicas, 3 ms per step
