"""The N > 1 path of bench.py on CPU: two gloo ranks run independent replicas (the contraction path has
no exchange step), the job time is the slowest rank's, and the value is the sum over replicas."""
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
    my_ms = 2.0 + rank                       # rank 1 is the slow one
    job_ms = bench.max_over_ranks(my_ms, dist, "cpu")
    value = bench.aggregate_value(1_000_000_000, job_ms, world)
    dist.barrier()
    if rank == 0:
        torch.save({"job_ms": job_ms, "value": value}, out)
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_sum_throughput(tmp_path):
    out = str(tmp_path / "r.pt")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["job_ms"] == 3.0
    assert abs(r["value"] - 2 * 1e9 / 3.0 / 1e6) < 1e-9


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(1.25, None, "cpu") == 1.25
    assert bench.aggregate_value(2_000_000, 1.0, 1) == 2.0
