"""rubick_greedy_round_noalloc against rubick_greedy_round.

The no-allocation entry point exists for hosts that may not allocate device memory while they
schedule (a daemon on a fixed memory budget next to jobs that fill the GPU, or a process whose
device memory belongs to a framework's allocator).  It keeps the per-job state of the round in a
fixed array inside the library instead of context scratch, and must decide exactly as the
ordinary entry point does: rounds are integer decisions, so the comparison is bit for bit.  Two
calls in a row (the second on fewer, different jobs) show that whatever the first call left in
the shared array does not leak into the second.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

from gpu_util import Gpu, assert_rounds_equal, has_cuda, unpack_round
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def both_rounds(gpu, jobs, n_nodes):
    """Curve tables from the library itself, then the round through both entry points."""
    t = gpu.torch
    J = len(jobs["P"])
    d_jobs, d_thr, d_feas = gpu.eval(jobs)
    d_cv, d_cp, d_cg = gpu.best(d_thr, d_feas, J)
    res = []
    for noalloc in (False, True):
        d_out = t.zeros(J * rb.ASSIGN_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
        d_node = t.zeros(n_nodes * rb.NODE_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
        call = gpu.ctx.greedy_round_noalloc if noalloc else gpu.ctx.greedy_round
        steps, capped = call(d_jobs, J, d_cv, d_cp, d_cg, d_feas, n_nodes, 1 << 30, d_out, d_node)
        res.append(unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE), rb.from_device(d_node, rb.NODE_DTYPE),
                                steps, capped, None))
    return res


def test_noalloc_round_matches_the_ordinary_round_twice_in_a_row():
    cfg = workloads.make("events", J=1500, n_nodes=128)
    gpu = Gpu(cfg)
    want, got = both_rounds(gpu, cfg["jobs"], 128)
    assert want["steps"] > 100 and (want["status"] == rb.RUNNING).sum() > 10
    assert_rounds_equal(got, want)
    # second call: other jobs, fewer of them, a smaller cluster; the array still holds call one's state
    sub = workloads.take(cfg["jobs"], np.arange(1499, 600, -3))
    want2, got2 = both_rounds(gpu, sub, 40)
    assert want2["steps"] > 10
    assert_rounds_equal(got2, want2)
    assert not np.array_equal(want2["g"], want["g"][:len(want2["g"])])


def test_noalloc_round_leaves_device_memory_as_it_found_it():
    """What the entry point is for: in a fresh context, with 9,000 jobs (a count at which the ordinary entry point
    has to grow its context's scratch with cudaMalloc), the call must not change the amount of free device memory
    as the driver reports it, while the ordinary call on a fresh context does."""
    cfg = workloads.make("throughput-stress", J=9000, n_nodes=48)
    J, N = 9000, 48
    gpu = Gpu(cfg)
    t = gpu.torch
    d_jobs, d_thr, d_feas = gpu.eval(cfg["jobs"])
    d_cv, d_cp, d_cg = gpu.best(d_thr, d_feas, J)
    d_out = t.zeros(J * rb.ASSIGN_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
    d_node = t.zeros(N * rb.NODE_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
    warm = Gpu(workloads.make("tiny"))                    # the library's kernels are loaded before anything is measured
    tiny_out = t.zeros(4 * rb.ASSIGN_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
    tj, tt, tf = warm.eval(warm.cfg["jobs"])
    tv, tp, tg = warm.best(tt, tf, 4)
    warm.ctx.greedy_round_noalloc(tj, 4, tv, tp, tg, tf, 1, 100, tiny_out)
    warm.ctx.greedy_round(tj, 4, tv, tp, tg, tf, 1, 100, tiny_out)
    t.cuda.synchronize()
    free0 = t.cuda.mem_get_info()[0]
    gpu.ctx.greedy_round_noalloc(d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, 1 << 30, d_out, d_node)
    t.cuda.synchronize()
    assert t.cuda.mem_get_info()[0] == free0
    gpu.ctx.greedy_round(d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, 1 << 30, d_out, d_node)
    t.cuda.synchronize()
    assert t.cuda.mem_get_info()[0] < free0               # the ordinary round allocated its scratch


def test_noalloc_round_covers_job_counts_beyond_shared_memory_and_rejects_too_many():
    # 9000 jobs: the ordinary entry point moves the job state to allocated scratch here
    cfg = workloads.make("throughput-stress", J=9000, n_nodes=48)
    gpu = Gpu(cfg)
    want, got = both_rounds(gpu, cfg["jobs"], 48)
    assert_rounds_equal(got, want)
    d = gpu.empty(64, gpu.torch.float32)
    with pytest.raises(rb.RubickError) as ei:
        gpu.ctx.greedy_round_noalloc(d, rb.NOALLOC_MAX_JOBS + 1, d, d, d, d, 48, 10, d, None)
    assert ei.value.code == rb.EINVAL and "RUBICK_NOALLOC_MAX_JOBS" in str(ei.value)
