"""The multi-GPU leg of bench.py runs independent replicas (the path has no exchange step); its only
cross-rank logic is the aggregation of the measurements, checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    res = bench.aggregate_replicas(10.0 + 5 * rank, 0.5 - 0.1 * rank, 800.0 + rank, world, "cpu")
    if rank == 0:
        torch.save(list(res), out)
    dist.destroy_process_group()


def test_replica_aggregation_with_two_gloo_ranks(tmp_path):
    out = str(tmp_path / "agg.pt")
    mp.spawn(_worker, args=(2, 29591, out), nprocs=2, join=True)
    total_ms, e2e_s, rows = torch.load(out)
    assert total_ms == 15.0 and e2e_s == 0.5 and rows == 1601.0      # slowest rank's times, summed rows
    import bench
    assert bench.aggregate_replicas(1.0, 2.0, 3.0, 1, "cpu") == (1.0, 2.0, 3.0)
