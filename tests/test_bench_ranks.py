"""The multi-replica bookkeeping of bench.py on CPU: two gloo ranks, no GPU.

The path does not shard, so N GPUs run N independent replicas; what the ranks
exchange is one scalar (the elapsed time, MAX over ranks)."""
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
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")
    value = bench.aggregate_gbs(world, 2e9, slowest)
    out.put((rank, slowest, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]                    # MAX over ranks on both
    assert got[0][2] == got[1][2] == pytest.approx(2 * 2e9 / 15e-3 / 1e9)


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_gbs(1, 1e9, 1.0) == pytest.approx(1000.0)
    m = [1, 1, 0, 1]
    # byte models: streaming schedule vs Gram-first for K = 4, fp32
    assert bench.schedule_bytes(m, 4, 10, 4) == ((8 + 4) + (8 + 8) + (8 + 0) + (8 + 4)) * 10
    assert bench.gram_first_bytes(m, 4, 10, 4) == ((4 + 3) * 4 + 4) * 10
