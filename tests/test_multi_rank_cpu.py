"""The N > 1 path of the benchmark on CPU: independent replicas, one process per rank, combined by the
maximum of the ranks' times (gloo, world size 2)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, torch.device("cpu"))
    dist.barrier()
    out[rank] = (slowest, bench.aggregate_value(1e9, 4, slowest, world))
    dist.destroy_process_group()


def test_replicas_are_combined_by_the_slowest_rank():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        slowest, value = out[0]
    assert slowest == 15.0
    # two replicas, 4 steps of 1 GB each in 15 ms: 2 * 4 GB / 0.015 s
    assert abs(value - 2 * 4 * 1e9 / 0.015 / 1e9) < 1e-6


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.workload("per_tensor")[2] == 25557032 and len(bench.workload("per_tensor")[4]) == 161
