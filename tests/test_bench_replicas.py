"""N > 1 in bench.py means independent replicas (the method ranks one global list
on one GPU; nothing is exchanged). What is shared is the timing rule: the slowest
rank's time, the sum of the work. Checked here with two gloo ranks on the CPU."""
import os
import sys

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0           # rank 1 is the slow one
    value, ms_per_step = bench.replica_throughput(local_ms, steps=10, n_params=1000, world=world)
    out.put((rank, value, ms_per_step))
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_use_the_slowest_rank_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms in got:
        assert ms == pytest.approx(25.0)                         # 250 ms / 10 steps on every rank
        assert value == pytest.approx(2 * 1000 / 25e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.replica_throughput(50.0, steps=5, n_params=10, world=1)
    assert ms == pytest.approx(10.0) and value == pytest.approx(1000.0)
