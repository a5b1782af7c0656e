"""Column-sharded mix: the partition (host logic) and, with two gloo ranks on CPU, the claim it rests on: the update
is independent per column (Eqs. 4-5), so shards computed separately and concatenated are the whole result, exactly,
with nothing exchanged between ranks."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_partition_properties():
    from paper_2102_06280_b200.sharding import column_shards
    for d, world in [(1048576, 8), (1048576, 3), (8228, 2), (7, 1), (4206624, 5), (12, 3)]:
        sh = column_shards(d, world)
        assert len(sh) == world and sh[0][0] == 0 and sh[-1][1] == d
        for (a0, a1), (b0, b1) in zip(sh, sh[1:]):
            assert a1 == b0 and a0 < a1 and b0 % 4 == 0
        widths = [c1 - c0 for c0, c1 in sh]
        assert max(widths) - min(widths) <= 4 + (4 - d % 4) % 4
    with pytest.raises(ValueError):
        column_shards(8, 3)            # only two 4-column units
    with pytest.raises(ValueError):
        column_shards(0, 1)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    from oracle import dbw_oracle as orc
    from paper_2102_06280_b200.sharding import column_shards
    from workloads import configs as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.make_workload(4, d=1000)                       # the mix-only workload's graph, 1000 columns
    X = wl.gaussian_rows(w.init_seed, range(w.N), w.d)
    G = wl.gaussian_rows(wl.external_gradient_seed(w), range(w.N), w.d, scale=0.01)
    t = wl.arrival_times(w, 1)[0]
    b = wl.uniform_backups(w, 1)[0]
    kept = orc.select_fastest(w.rowptr, w.col, t, b)       # replicated on every rank
    ws, we = orc.mixing_weights(w.rowptr, w.col, b, kept, orc.UNIFORM)
    c0, c1 = column_shards(w.d, world)[rank]
    mine = orc.mix_update(w.rowptr, w.col, X[:, c0:c1], G[:, c0:c1], ws, we, w.lr)
    parts = [None] * world
    dist.all_gather_object(parts, (c0, c1, mine))          # test plumbing only: the method exchanges nothing
    if rank == 0:
        whole = orc.mix_update(w.rowptr, w.col, X, G, ws, we, w.lr)
        glued = np.concatenate([p[2] for p in sorted(parts, key=lambda p: p[0])], axis=1)
        q.put(bool(np.array_equal(glued, whole)) and [p[:2] for p in parts] == column_shards(w.d, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_compute_disjoint_shards_that_glue_to_the_whole():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    ok = q.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
