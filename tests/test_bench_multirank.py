"""The N > 1 path of the benchmark: replicas only, whole-job time = max over ranks, work = sum over ranks.
Two CPU processes on the gloo backend exercise the same aggregation the NCCL run uses."""
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
    ms, kept, dense = bench.aggregate_over_ranks(10.0 + rank, 100.0 * (rank + 1), 1000.0, "cpu")
    out[rank] = (ms, kept, dense)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1] == (11.0, 300.0, 2000.0)      # max of the times, sum of the work


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.0, 5.0, 7.0) == (3.0, 5.0, 7.0)


def test_reference_arm_prints_only_on_rank_zero(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    args = type("A", (), {"steps": 1, "warmup": 0, "gpus": 2, "workload": "mlp2048_row"})()
    bench.run_reference(args, bench.WORKLOADS["mlp2048_row"])
    assert capsys.readouterr().out == ""
