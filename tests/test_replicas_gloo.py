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


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher environment starts two ranks itself (one process
    per GPU on a GPU machine; here the timing protocol alone, on gloo) and rank 0 prints one line."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--selftest-replicas"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_max"] == 20.0           # the slower of the two ranks
    assert line["value"] == pytest.approx(2 * 1000 / 0.020)
