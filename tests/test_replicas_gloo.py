"""The multi-GPU protocol of the benchmark (independent replicas, barrier, max-over-ranks time)
on two gloo ranks on CPU."""
import os

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_39813_b200 import harness
    ms = 10.0 + 5.0 * rank                     # rank 1 is the slow replica
    dist.barrier()
    worst = harness.max_over_ranks(ms)
    value = harness.replica_throughput(1000, 4, world, worst)
    out[rank] = (worst, value)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_timing_two_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    worst, value = out[0]
    assert worst == 15.0
    assert value == pytest.approx(2 * 1000 * 4 / 0.015)


def test_single_process_is_identity():
    from paper_2609_39813_b200 import harness
    assert harness.max_over_ranks(3.5) == 3.5
    assert harness.replica_throughput(10, 2, 1, 1000.0) == 20.0
