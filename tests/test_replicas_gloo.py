"""The path does not shard (one GPU, no collectives), so `bench.py --gpus N` runs N independent replicas and only the
timing is combined across ranks: job time = MAX over ranks, job work = N x per-replica work. This checks that
combination with two gloo ranks on the CPU."""
import os
import sys

import pytest
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
    # rank 0 needs 100 ms for its 10 steps, rank 1 needs 250 ms: the job took 250 ms
    mine = [100.0, 400.0] if rank == 0 else [250.0, 300.0]
    ms, vals = bench.replica_aggregate(mine, flops_per_replica_step=2.0e12, steps=10, world=world)
    dist.barrier()
    if rank == 0:
        torch.save({"ms": ms, "vals": vals}, out)
    dist.destroy_process_group()


def test_replica_timing_is_max_over_ranks(tmp_path):
    out = str(tmp_path / "r.pt")
    port = 29500 + os.getpid() % 500
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["ms"] == [250.0, 400.0]
    # 2 replicas x 2 TFLOP per step / (25 ms per step) = 160 TFLOP/s ; e2e: / 40 ms = 100 TFLOP/s
    assert r["vals"] == pytest.approx([160.0, 100.0])


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms, vals = bench.replica_aggregate([50.0], 1.0e12, 5, 1)
    assert ms == [50.0] and vals == pytest.approx([100.0])
