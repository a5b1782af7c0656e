"""N > 1 path of the benchmark on CPU: replicas only, no data-path collective.  Two gloo ranks
time different amounts of work; every rank must see the slowest rank's time and the whole-job
value must count both replicas' units over that time."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms_local = 10.0 * (rank + 1)                     # rank 1 is twice as slow
    ms = bench.max_over_ranks(ms_local, dist, device="cpu")
    value = bench.aggregate_value(units_per_rank_step=128, steps=5, ms_max=ms, world=world)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, ms, value))


def test_two_replicas_report_max_time_and_total_units():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in out:
        assert ms == 20.0
        assert value == pytest.approx(2 * 128 * 5 / 0.020)


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None) == 3.5
    assert bench.aggregate_value(1024, 10, 50.0, 1) == pytest.approx(1024 * 10 / 0.05)
