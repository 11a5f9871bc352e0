"""Host logic of bench.py and of the multi-GPU arrangement, on CPU: two gloo ranks exercise the
reductions (max over ranks of the time, sum over ranks of the work), the per-rank workloads are
independent draws of the same recipe, and the byte accounting of the roofline is what the design
notes state."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.make_workload("paper-scale", rank=rank)
    ms = 10.0 + 5.0 * rank                                   # rank 1 is the slow one
    work = float(len(cfg["jobs"]["P"]) * 1344 * 24)
    total_ms = bench.reduce_max_ms(ms, world)
    total_work = bench.reduce_sum(work, world)
    out.put((rank, total_ms, total_work, float(cfg["jobs"]["P"][0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_work_by_sum():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, w0, p0), (r1, ms1, w1, p1) = got
    assert ms0 == ms1 == 15.0                                # the job is as slow as its slowest rank
    assert w0 == w1 == 2 * 64 * 1344 * 24                    # every rank contributes its own batch
    assert p0 != p1                                          # independent draws: another seed per rank


def test_rank_workloads_follow_the_same_recipe_with_their_own_seed():
    a = bench.make_workload("paper-scale", rank=0)
    b = bench.make_workload("paper-scale", rank=3)
    again = bench.make_workload("paper-scale", rank=0)
    assert np.array_equal(a["jobs"]["P"], again["jobs"]["P"])
    assert not np.array_equal(a["jobs"]["P"], b["jobs"]["P"])
    assert a["n_nodes"] == b["n_nodes"] and np.array_equal(a["c_levels"], b["c_levels"])
    assert bench.shard_seed_offset(0) == 0 and bench.shard_seed_offset(2) == 200
    from paper_2408_08586_b200 import workloads
    assert workloads.CONFIGS["paper-scale"]["seed"] == 1     # the table of configs is left untouched


def test_algorithmic_byte_counts():
    J, P, C, G, M = 16384, 2640, 24, 9, 32
    per = bench.algorithmic_bytes_eval(J, P, C) / (J * P * C)
    assert per == pytest.approx(4 + 4 / C + 128 / (P * C), rel=1e-12)
    assert bench.algorithmic_bytes_best(J, P, C, G, M) == 4.0 * J * P * C + 4.0 * J * P + 12.0 * J * G * C * M


def test_sort_launch_count_follows_the_bitonic_network():
    """Stages of a bitonic network over n keys with tiles of t keys: the stages up to t take one launch; stage k > t
    takes log2(k / t) launches with strides of a tile or more and one for the strides inside the tiles."""
    def brute(n, t=2048):
        t = min(n, t)
        launches, k = 1, 2
        while k <= n:
            if k > t:
                s = k // 2
                while s >= t:
                    launches += 1
                    s //= 2
                launches += 1
            k *= 2
        return launches
    for J in (1, 2, 64, 2048, 2049, 4096, 9000, 16384, 100000):
        n = 2
        while n < J:
            n *= 2
        assert bench.sort_launches(J) == brute(n)
    assert bench.sort_launches(16384) == 10 and bench.sort_launches(1500) == 1


def test_reference_arm_prints_one_json_line(capsys):
    import json
    import types
    args = types.SimpleNamespace(workload="tiny", jobs=None, nodes=None, ref_jobs=4, ref_threads=1, warmup=1, steps=2, gpus=1)
    os.environ.pop("RANK", None)
    bench.run_reference(args)
    line = json.loads(capsys.readouterr().out.strip())
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["cpu_baseline"]["cores"] == 1 and line["cpu_baseline"]["cores_per_stage"]["round"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["metric"] == bench.METRIC
    os.environ["RANK"] = "1"
    try:
        bench.run_reference(args)                            # other ranks print nothing and do no work
        assert capsys.readouterr().out == ""
    finally:
        os.environ.pop("RANK")
