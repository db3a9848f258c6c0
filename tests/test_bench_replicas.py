"""The benchmark's multi-rank logic (replicas only: max of the times, sum of the work) on two
gloo ranks on CPU."""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    total_ms, e2e_ms, inter = bench.combine_ranks(dist, torch.device("cpu"), 10.0 + rank, 20.0 - rank, 100 * (rank + 1))
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (total_ms, e2e_ms, inter)


def test_two_replicas_take_max_time_and_sum_work():
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(2):
        assert out[r] == (11.0, 20.0, 300.0)


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.combine_ranks(None, None, 1.5, 2.5, 7) == (1.5, 2.5, 7.0)
