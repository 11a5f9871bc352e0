"""Job-sharded curve construction (paper Section 5.2: curves "can be computed in parallel ... cached") on CPU:
the tile bounds partition the jobs in order, and two / three gloo ranks that each fill their own tile of per-job
rows end up, after the all-gather, with the same full tables as a single rank that fills everything; the
agreement check tells identical assignments from differing ones.  The rows are filled with a pattern derived
from the job index (no arithmetic of the method is involved)."""
import os
import socket

import numpy as np
import pytest

from paper_2408_08586_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("J,world", [(16384, 8), (1000, 3), (7, 8), (0, 4), (5, 1), (64, 2), (65, 2)])
def test_tiles_partition_the_jobs_in_order(J, world):
    t = sharding.tiles_cover(J, world)
    assert t[0, 0] == 0 and t[:, 1].sum() == J
    assert np.array_equal(t[1:, 0], np.cumsum(t[:, 1])[:-1])            # contiguous, ascending
    assert t[:, 1].max() - t[:, 1].min() <= 1 and t[:, 1].max() == sharding.tile_capacity(J, world)
    assert np.all(np.diff(t[:, 1]) <= 0)                                # the larger tiles come first


def _pattern(start, count, n, dtype):
    import torch
    rows = torch.arange(start, start + count, dtype=torch.int64).view(-1, 1) * 1000 + torch.arange(n, dtype=torch.int64).view(1, -1)
    return rows.reshape(-1).to(dtype)


def _rank_main(rank, world, port, J, out):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows = {"feas": (5, torch.int32), "cv": (12, torch.float32), "cp": (12, torch.int32)}

    def compute(start, count, bufs):
        for k, (n, dt) in rows.items():
            bufs[k][: count * n] = _pattern(start, count, n, dt)

    full = sharding.sharded_tables(compute, J, world, rank, rows, "cpu")
    ok = all(torch.equal(full[k], _pattern(0, J, n, dt)) for k, (n, dt) in rows.items())
    same = torch.arange(100, dtype=torch.uint8)
    agree_same = sharding.assignments_agree(same, world)
    differ = same.clone()
    differ[17] = rank                                                   # one byte differs between the ranks
    agree_diff = sharding.assignments_agree(differ, world)
    out.put((rank, ok, agree_same, agree_diff))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,J", [(2, 64), (2, 65), (3, 10), (2, 1)])
def test_ranks_gather_the_tables_of_a_single_rank(world, J):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, J, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ok, agree_same, agree_diff in got:
        assert ok and agree_same and not agree_diff


def test_single_rank_needs_no_process_group():
    import torch
    rows = {"cv": (3, torch.float32)}
    full = sharding.sharded_tables(lambda s, c, b: b["cv"].__setitem__(slice(0, c * 3), _pattern(s, c, 3, torch.float32)), 9, 1, 0, rows, "cpu")
    assert torch.equal(full["cv"], _pattern(0, 9, 3, torch.float32))
    assert sharding.assignments_agree(torch.zeros(4, dtype=torch.uint8), 1)
