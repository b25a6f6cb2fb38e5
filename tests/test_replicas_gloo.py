"""The multi-GPU path of bench.py has no data-path collective (rows are independent, every
rank runs a replica); what it shares is the timing rule: the job's time is the maximum over
ranks and its throughput the sum of the replicas' work over that time.  Checked here with two
gloo ranks on CPU."""
import os
import sys

import pytest
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
    mine = 2.0 + rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(mine, world)
    # every rank must agree on the aggregate line's numbers
    value = bench.aggregate_throughput(10 ** 9, 4, ms, world)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_time_is_max_over_ranks_and_value_is_the_aggregate():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 3.0
    assert value == pytest.approx(2 * 4 * 1e9 / 3e-3 / 1e9)


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.aggregate_throughput(7_430_000_000, 100, 146.9, 1) == pytest.approx(5057.9, rel=1e-3)
