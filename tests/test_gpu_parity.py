"""Parity of the CUDA path with the oracle, element by element, through the C ABI.

Tolerances:
  predicted throughput   1e-5 relative (single-precision kernel vs double-precision oracle)
  feasibility words      bit exact
  plan / allocation      bit exact when both sides see the same table; through the whole
                         single-precision path an index may differ only where the oracle's
                         value of the GPU's choice lies within 1e-6 relative of the oracle's best
"""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, assert_chain_parity, assert_rounds_equal, has_cuda, unpack_round
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]

THR_RTOL = 1e-5
TIE_RTOL = 1e-6


def oracle_tables(cfg, jobs=None, nthreads=8, prefix=True, environment=None):
    jobs = cfg["jobs"] if jobs is None else jobs
    plans, goff = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(jobs, plans, environment or cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    thr32 = thr.astype(np.float32)
    cv, cp, cg = oracle.best_plan(thr32, feas, plans, cfg["g_levels"], len(cfg["m_levels"]), prefix=prefix, nthreads=nthreads)
    return plans, thr, feas, cv.astype(np.float32), cp, cg


def check_thr(got, want):
    assert got.shape == want.shape
    zero = want == 0
    assert np.array_equal(got == 0, zero)
    rel = np.abs(got[~zero].astype(np.float64) - want[~zero]) / want[~zero]
    assert rel.max() <= THR_RTOL, rel.max()
    return rel.max()


def test_plan_enumerators_agree():
    for levels in ([1, 2, 3, 4, 5, 6, 7, 8], [1, 2, 4, 8, 16, 32, 64], [1 << i for i in range(9)]):
        a, aoff = rb.enumerate_plans(levels)
        b, boff = oracle.enumerate_plans(levels)
        assert np.array_equal(aoff, boff)
        got = np.stack([1 << a["log2d"].astype(np.int64), 1 << a["log2t"].astype(np.int64),
                        1 << a["log2p"].astype(np.int64), a["zero"], a["gc"], a["off"]], axis=1)
        assert np.array_equal(got, b[:, :6]) and not b[:, 6].any()


@pytest.mark.parametrize("name,J", [("tiny", None), ("paper-scale", None), ("cluster-512", 1024), ("cluster-512", 77)])
def test_candidate_table_and_mask(name, J):
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    Jn = len(cfg["jobs"]["P"])
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    plans, thr, feas, *_ = oracle_tables(cfg)
    assert np.array_equal(gpu.np_feas(d_feas, Jn), feas)
    worst = check_thr(gpu.np_thr(d_thr, Jn), thr)
    assert worst < THR_RTOL
    assert (feas != 0).any() and (feas == 0).any()


def test_strict_zero_dp_only_and_other_environments():
    cfg = workloads.make("paper-scale")
    for e in (env(strict_zero_dp_only=1), env(gpu_mem_bytes=24_000_000_000, B_inter=12.5e9, B_pcie=12e9),
              env(gpus_per_node=4, cpus_per_node=48, mem_per_node_bytes=256 * GIB), env(zero3_extra_volume=1)):
        cfg["env"] = e
        gpu = Gpu(cfg)
        _, d_thr, d_feas = gpu.eval(cfg["jobs"])
        plans, thr, feas, *_ = oracle_tables(cfg)
        assert np.array_equal(gpu.np_feas(d_feas, 64), feas)
        check_thr(gpu.np_thr(d_thr, 64), thr)
        gpu.assert_one_pass_curves_match(cfg["jobs"])


def test_hand_made_jobs_with_odd_shapes():
    # batch not a power of two, micro-batch cap not dividing the batch, few layers, odd hidden size
    jobs = stack_jobs(one_job(b=48, mu_cap=5, l=3, h=2052, P=3.3e9 + 1),
                      one_job(b=1, mu_cap=1, l=96, h=8192, s=4096, P=65e9, k_sync=1.0, k_off=1.0, k_swap=1.0),
                      one_job(b=96, mu_cap=7, l=12, h=768, s=512, P=125e6, k_sync=4.0, k_off=4.0, k_swap=4.0),
                      one_job(b=256, mu_cap=1, l=48, h=5120, s=2048, P=13e9 - 7, host_base_bytes=GIB + 12345))
    cfg = workloads.make("cluster-512", J=4)
    cfg["jobs"] = jobs
    gpu = Gpu(cfg)
    _, d_thr, d_feas = gpu.eval(jobs)
    plans, thr, feas, *_ = oracle_tables(cfg)
    assert np.array_equal(gpu.np_feas(d_feas, 4), feas)
    check_thr(gpu.np_thr(d_thr, 4), thr)


def test_everything_infeasible_and_single_memory_level():
    cfg = workloads.make("tiny")
    cfg["env"] = env(gpu_mem_bytes=1 << 20)               # nothing fits a 1 MiB GPU
    cfg["m_levels"] = cfg["m_levels"][:1]
    gpu = Gpu(cfg)
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    assert not feas.any() and np.array_equal(gpu.np_feas(d_feas, 4), feas)
    check_thr(gpu.np_thr(d_thr, 4), thr)                   # predictions do not depend on memory
    gpu.assert_one_pass_curves_match(cfg["jobs"])
    bv, bp, bg = gpu.best(d_thr, d_feas, 4)
    assert not bv.cpu().numpy().any() and (bp.cpu().numpy() == -1).all() and not bg.cpu().numpy().any()
    r = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 1)
    assert r["steps"] == 0 and not r["g"].any()


def test_zero_jobs():
    cfg = workloads.make("tiny")
    gpu = Gpu(cfg)
    assert gpu.ctx.eval_candidates(None, 0, None, None) == 0
    assert gpu.ctx.best_plan(None, None, 0, None, None, None) == 0
    steps, capped = gpu.ctx.schedule_round(None, 0, 1, 10, None)
    assert steps == 0 and not capped


@pytest.mark.parametrize("name,J", [("tiny", None), ("paper-scale", None), ("cluster-512", 96)])
@pytest.mark.parametrize("raw", [False, True])
def test_best_plan_on_the_oracle_table_is_bit_exact(name, J, raw):
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    t = gpu.torch
    Jn = len(cfg["jobs"]["P"])
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg, prefix=not raw)
    d_thr = t.from_numpy(thr.astype(np.float32).reshape(-1)).cuda()
    d_feas = t.from_numpy(feas.view(np.int32).reshape(-1)).cuda()
    bv, bp, bg = gpu.best(d_thr, d_feas, Jn, flags=rb.BEST_RAW if raw else 0)
    sh = gpu.shape4(Jn)
    assert np.array_equal(bv.cpu().numpy().reshape(sh), cv)
    assert np.array_equal(bp.cpu().numpy().reshape(sh), cp)
    assert np.array_equal(bg.cpu().numpy().reshape(sh), cg)


def test_best_plan_with_scattered_feasibility_levels():
    """Random thresholds per plan (not only the two values the memory rule produces) and random
    values with many exact ties."""
    cfg = workloads.make("paper-scale", J=16)
    gpu = Gpu(cfg)
    t = gpu.torch
    rng = np.random.default_rng(3)
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    J, nC, P, nM = 16, gpu.nC, gpu.P, gpu.nM
    thr = rng.integers(0, 6, (J, nC, P)).astype(np.float32)               # few distinct values: ties everywhere
    f = rng.integers(0, nM + 8, (J, P))
    feas = np.where(f >= nM, 0, (0xFFFFFFFF << f) & 0xFFFFFFFF).astype(np.uint32)
    cv, cp, cg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], nM, prefix=True, nthreads=8)
    bv, bp, bg = gpu.best(t.from_numpy(thr.reshape(-1)).cuda(), t.from_numpy(feas.view(np.int32).reshape(-1)).cuda(), J)
    sh = gpu.shape4(J)
    assert np.array_equal(bv.cpu().numpy().reshape(sh), cv.astype(np.float32))
    assert np.array_equal(bp.cpu().numpy().reshape(sh), cp)
    assert np.array_equal(bg.cpu().numpy().reshape(sh), cg)


@pytest.mark.parametrize("raw", [False, True])
def test_best_plan_with_two_class_and_scattered_masks_in_one_batch(raw):
    """Jobs whose masks have one first level per (GPU level, offload class) take the streaming
    kernel, the others the general one; both in one call, with tie-heavy values, classes without
    feasible plans, and either class lower than the other."""
    cfg = workloads.make("paper-scale", J=24)
    gpu = Gpu(cfg)
    t = gpu.torch
    rng = np.random.default_rng(7)
    plans, group_off = oracle.enumerate_plans(cfg["g_levels"])
    J, nC, P, nM, nG = 24, gpu.nC, gpu.P, gpu.nM, gpu.nG
    thr = rng.integers(0, 5, (J, nC, P)).astype(np.float32)
    thr[:, :, ::7] *= 0.5
    level_of = np.searchsorted(np.asarray(group_off[1:], dtype=np.int64), np.arange(P), side="right")
    odd = (np.arange(P) & 1).astype(np.int64)
    first = rng.integers(0, nM + 6, (J, nG, 2))                           # >= nM: the class has no feasible plan
    f = first[np.arange(J)[:, None], level_of[None, :], odd[None, :]]
    f = np.where(rng.uniform(size=(J, P)) < 0.4, nM, f)                   # plans that fit nowhere (GPU memory)
    scattered = np.arange(J) % 3 == 1
    f[scattered] = rng.integers(0, nM + 8, (int(scattered.sum()), P))
    f[5, :] = nM                                                          # a job with nothing feasible
    feas = np.where(f >= nM, 0, (0xFFFFFFFF << np.minimum(f, 31)) & 0xFFFFFFFF).astype(np.uint32)
    cv, cp, cg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], nM, prefix=not raw, nthreads=8)
    bv, bp, bg = gpu.best(t.from_numpy(thr.reshape(-1)).cuda(), t.from_numpy(feas.view(np.int32).reshape(-1)).cuda(), J,
                          flags=rb.BEST_RAW if raw else 0)
    sh = gpu.shape4(J)
    assert np.array_equal(bv.cpu().numpy().reshape(sh), cv.astype(np.float32))
    assert np.array_equal(bp.cpu().numpy().reshape(sh), cp)
    assert np.array_equal(bg.cpu().numpy().reshape(sh), cg)


@pytest.mark.parametrize("name,J", [("tiny", None), ("paper-scale", None), ("cluster-512", 203)])
@pytest.mark.parametrize("raw", [False, True])
def test_curves_in_one_pass_equal_table_then_best_plan(name, J, raw):
    """rubick_curves never writes the table; mask and curves must be bit-identical to the two-call path."""
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    t = gpu.torch
    Jn = len(cfg["jobs"]["P"])
    flags = rb.BEST_RAW if raw else 0
    d_jobs, d_thr, d_feas = gpu.eval(cfg["jobs"])
    bv, bp, bg = gpu.best(d_thr, d_feas, Jn, flags=flags)
    n = Jn * gpu.nG * gpu.nC * gpu.nM
    f2 = gpu.empty(Jn * gpu.P, t.int32)
    cv, cp, cg = gpu.empty(n, t.float32), gpu.empty(n, t.int32), gpu.empty(n, t.int32)
    gpu.ctx.curves(d_jobs, Jn, f2, cv, cp, cg, flags=flags)
    gpu.ctx.sync()
    assert t.equal(f2, d_feas)
    assert t.equal(cv.view(t.int32), bv.view(t.int32)) and t.equal(cp, bp) and t.equal(cg, bg)


def test_non_threshold_feasibility_word_is_reported():
    cfg = workloads.make("tiny")
    gpu = Gpu(cfg)
    t = gpu.torch
    thr = np.ones((4, gpu.nC, gpu.P), dtype=np.float32)
    feas = np.full((4, gpu.P), 0b101, dtype=np.uint32)
    n = 4 * gpu.nG * gpu.nC * gpu.nM
    bv, bp, bg = gpu.empty(n, t.float32), gpu.empty(n, t.int32), gpu.empty(n, t.int32)
    gpu.ctx.best_plan(t.from_numpy(thr.reshape(-1)).cuda(), t.from_numpy(feas.view(np.int32).reshape(-1)).cuda(), 4, bv, bp, bg)
    with pytest.raises(rb.RubickError) as ei:
        gpu.ctx.sync()
    assert ei.value.code == rb.ESTATE
    assert gpu.ctx.sync() == 0                                             # the flag is cleared once reported


@pytest.mark.parametrize("name,J", [("paper-scale", None), ("cluster-512", 512)])
def test_best_plan_through_the_single_precision_table(name, J):
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    Jn = len(cfg["jobs"]["P"])
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    bv, bp, bg = (x.cpu().numpy().reshape(gpu.shape4(Jn)) for x in gpu.best(d_thr, d_feas, Jn, flags=rb.BEST_RAW))
    plans, thr, feas, *_ = oracle_tables(cfg)
    ov, op, og = oracle.best_plan(thr, feas, plans, cfg["g_levels"], gpu.nM, prefix=False, nthreads=8)
    assert np.array_equal(bp >= 0, op >= 0) and np.array_equal(bg, og)
    has = op >= 0
    rel = np.abs(bv[has] - ov[has]) / ov[has]
    assert rel.max() <= THR_RTOL
    diff = has & (bp != op)
    # where the index differs, the GPU's plan must be a near tie under the oracle's own values
    jj, gg, cc, mm = np.nonzero(diff)
    alt = thr[jj, cc, bp[diff]]
    assert np.all(alt >= ov[diff] * (1 - TIE_RTOL))
    assert np.all((feas[jj, bp[diff]] >> mm) & 1)
    assert diff.mean() < 0.01


def random_states(cfg, cv, rng):
    J = cv.shape[0]
    nG, nC = cv.shape[1], cv.shape[2]
    gi = rng.integers(-1, nG, J)
    ci = rng.integers(0, nC, J)
    g = np.where(gi >= 0, cfg["g_levels"][np.maximum(gi, 0)], 0)
    c = np.where(gi >= 0, cfg["c_levels"][ci], 0)
    val = np.where(gi >= 0, cv[np.arange(J), np.maximum(gi, 0), ci, rng.integers(0, cv.shape[3], J)], 0).astype(np.float32)
    return g, c, val


@pytest.mark.parametrize("name,J", [("tiny", None), ("paper-scale", None), ("cluster-512", 300)])
def test_marginal_gain_is_bit_exact(name, J):
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    t = gpu.torch
    Jn = len(cfg["jobs"]["P"])
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    rng = np.random.default_rng(11)
    for _ in range(3):
        g, c, val = random_states(cfg, cv, rng)
        st = np.zeros(Jn, dtype=rb.ASSIGN_DTYPE)
        st["g"], st["c"], st["thr"] = g, c, val
        outs = [gpu.empty(Jn, t.float32), gpu.empty(Jn, t.float32), gpu.empty(Jn, t.int32), gpu.empty(Jn, t.int32)]
        gpu.ctx.marginal_gain(gpu.jobs_to_device(cfg["jobs"]), Jn, t.from_numpy(cv.reshape(-1)).cuda(), rb.to_device(st), *outs)
        gpu.ctx.sync()
        want = oracle.gain(cfg["jobs"], cv, cfg["g_levels"], cfg["c_levels"], g, c, val)
        for a, b in zip(outs, want):
            assert np.array_equal(a.cpu().numpy().view(np.uint32), b.view(np.uint32))
        assert (want[0] > 0).any() and (name == "tiny" or (want[1] > 0).any())


# (the last two: 4,096 and 8,192 sort keys, which a cluster of two and of four CTAs sorts in one launch)
ROUND_CASES = [("tiny", None, None), ("paper-scale", None, None), ("cluster-512", 96, 24), ("cluster-512", 700, 64),
               ("events", 1500, 128), ("events", 3000, 256), ("throughput-stress", 6000, 192)]


@pytest.mark.parametrize("name,J,N", ROUND_CASES)
def test_greedy_round_on_the_oracle_tables_is_bit_exact(name, J, N):
    cfg = workloads.make(name, J=J, n_nodes=N)
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 cfg["n_nodes"], want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"])
    assert_rounds_equal(got, want)
    assert want["steps"] > 0


@pytest.mark.parametrize("mem_gib,cpus", [(96, 40), (64, 96), (48, 96)])
def test_greedy_round_under_memory_pressure_and_small_nodes(mem_gib, cpus):
    """Host memory tight enough that commits are rejected or pick a lower memory level."""
    cfg = workloads.make("cluster-512", J=200, n_nodes=12)
    cfg["jobs"]["gmin_idx"][:] = -1
    cfg["jobs"]["cmin_idx"][:] = -1
    cfg["env"] = env(mem_per_node_bytes=mem_gib * GIB, cpus_per_node=cpus)
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 12, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 12)
    assert_rounds_equal(got, want)
    assert (want["log"] & 1 == 0).any()                    # some increment was rejected and frozen
    assert (want["n_nodes"] > 1).any()                     # and some job spans whole nodes


@pytest.mark.parametrize("mem_gib,share", [(48, 1.0), (64, 0.7), (160, 1.0)])
def test_guaranteed_jobs_when_nodes_run_out_of_host_memory(mem_gib, share):
    """Phase A under memory pressure: the node first fit finds has GPUs and cores left but no memory for any
    level, so the job stays pending; jobs with the same minimum levels that follow fare the same until another
    job is placed (the device round remembers such outcomes instead of trying again)."""
    rng = np.random.default_rng(77)
    J, N = 300, 6
    cfg = workloads.make("cluster-512", J=J, n_nodes=N)
    guar = rng.uniform(size=J) < share
    cfg["jobs"]["gmin_idx"] = np.where(guar, rng.integers(0, 3, J), -1)
    cfg["jobs"]["cmin_idx"] = np.where(guar, rng.integers(0, 3, J), -1)
    cfg["env"] = env(mem_per_node_bytes=mem_gib * GIB)
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 N, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, N)
    assert_rounds_equal(got, want)
    pending = want["status"] == rb.PENDING
    assert pending.any() and (want["status"] == rb.RUNNING).any()
    if mem_gib <= 64 and share == 1.0:
        assert (want["node"][:, 0] > 0).any()              # GPUs are left over: memory is what ran out


def test_greedy_round_step_cap():
    cfg = workloads.make("paper-scale")
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 8, max_steps=5, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 8, max_steps=5)
    assert want["capped"] and want["steps"] == 5
    assert_rounds_equal(got, want)


def test_greedy_round_with_many_jobs_uses_global_state():
    """More jobs than fit the shared-memory job state: the kernel keeps it in global scratch."""
    cfg = workloads.make("throughput-stress", J=9000, n_nodes=40)
    gpu = Gpu(cfg)
    # synthetic concave single-resource curves keep the oracle side fast at this job count
    rng = np.random.default_rng(2)
    J, nG, nC, nM = 9000, gpu.nG, gpu.nC, gpu.nM
    inc = np.sort(rng.uniform(0.1, 4.0, (J, nG)), axis=1)[:, ::-1]
    cv = np.broadcast_to(np.cumsum(inc, axis=1).astype(np.float32)[:, :, None, None], (J, nG, nC, nM)).copy()
    cp = np.zeros((J, nG, nC, nM), dtype=np.int32)
    for gi in range(nG):
        cp[:, gi] = gpu.group_off[gi]
    cg = np.broadcast_to(cfg["g_levels"].astype(np.int32)[None, :, None, None], (J, nG, nC, nM)).copy()
    feas = np.full((J, gpu.P), 0xFFFFFFFF, dtype=np.uint32)
    jobs = cfg["jobs"]
    jobs["gmin_idx"][:] = -1
    jobs["cmin_idx"][:] = -1
    want = oracle.schedule_round(jobs, cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], 40,
                                 want_log=True)
    got = gpu.round_on_tables(jobs, cv, cp, cg, feas, 40)
    assert_rounds_equal(got, want)


def run_full_path(gpu, cfg, host=False):
    t = gpu.torch
    J = len(cfg["jobs"]["P"])
    N = cfg["n_nodes"]
    if host:
        h_jobs = rb.pack_jobs(cfg["jobs"])
        h_out = np.zeros(J, dtype=rb.ASSIGN_DTYPE)
        h_node = np.zeros(N, dtype=rb.NODE_DTYPE)
        steps, capped = gpu.ctx.schedule_round_host(h_jobs, J, N, 1 << 30, h_out, h_node)
        return unpack_round(h_out, h_node, steps, capped, None)
    d_out = gpu.empty(J * rb.ASSIGN_DTYPE.itemsize, t.uint8)
    d_node = gpu.empty(N * rb.NODE_DTYPE.itemsize, t.uint8)
    steps, capped = gpu.ctx.schedule_round(gpu.jobs_to_device(cfg["jobs"]), J, N, 1 << 30, d_out, d_node)
    return unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE), rb.from_device(d_node, rb.NODE_DTYPE), steps, capped, None)


@pytest.mark.parametrize("name,J,N", [("tiny", None, None), ("paper-scale", None, None), ("cluster-512", 600, 48),
                                      ("cluster-512", 1024, 64), ("events", 800, 64), ("throughput-stress", 2000, 64)])
@pytest.mark.parametrize("host", [False, True])
def test_whole_path_round_against_the_oracle(name, J, N, host):
    """Candidate table -> curves -> round, all on the GPU in one call, against the oracle's own chain.  The two
    chains read tables that differ by single-precision rounding, which can change a decision only at a near tie:
    the step logs must be identical up to the first decision the oracle itself takes by a margin within that
    rounding, the allocations up to there equal, and without such a near tie the whole round equal."""
    cfg = workloads.make(name, J=J, n_nodes=N)
    gpu = Gpu(cfg)
    got = run_full_path(gpu, cfg, host=host)
    assert_chain_parity(gpu, cfg, cfg["n_nodes"], oracle_tables(cfg), got=got, tie_rtol=TIE_RTOL, thr_rtol=THR_RTOL)
    # whatever was decided is a consistent packing
    Gn = cfg["env"]["gpus_per_node"]
    assert got["g"].sum() + got["node"][:, 0].sum() == cfg["n_nodes"] * Gn
    assert (got["node"][:, :3] >= 0).all()


@pytest.mark.parametrize("seed", range(6))
def test_whole_path_entry_points_equal_curves_then_round_bit_for_bit(seed):
    """rubick_schedule_round and rubick_schedule_round_host build the tables in context scratch (and hand the round's
    preparation a packed copy of their top memory level); the outcome must be the one of rubick_curves followed by
    rubick_greedy_round on caller-owned tables, byte for byte."""
    rng = np.random.default_rng(12000 + seed)
    name = ["paper-scale", "cluster-512", "events", "throughput-stress", "tiny", "events"][seed]
    J = int(rng.integers(20, 3000)) if name != "tiny" else None
    N = int(rng.integers(3, 400))
    cfg = workloads.make(name, J=J, n_nodes=N)
    Jn = len(cfg["jobs"]["P"])
    gpu = Gpu(cfg)
    t = gpu.torch
    d_jobs = gpu.jobs_to_device(cfg["jobs"])
    n = Jn * gpu.nG * gpu.nC * gpu.nM
    d_feas = gpu.empty(Jn * gpu.P, t.int32)
    cv, cp, cg = gpu.empty(n, t.float32), gpu.empty(n, t.int32), gpu.empty(n, t.int32)
    gpu.ctx.curves(d_jobs, Jn, d_feas, cv, cp, cg)
    o1, n1 = t.zeros(Jn * rb.ASSIGN_DTYPE.itemsize, dtype=t.uint8, device="cuda:0"), t.zeros(N * rb.NODE_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
    o2, n2 = t.zeros_like(o1), t.zeros_like(n1)
    s1, _ = gpu.ctx.greedy_round(d_jobs, Jn, cv, cp, cg, d_feas, N, 1 << 30, o1, n1)
    s2, _ = gpu.ctx.schedule_round(d_jobs, Jn, N, 1 << 30, o2, n2)
    h_out, h_nodes = np.zeros(Jn, dtype=rb.ASSIGN_DTYPE), np.zeros(N, dtype=rb.NODE_DTYPE)
    s3, _ = gpu.ctx.schedule_round_host(np.ascontiguousarray(rb.pack_jobs(cfg["jobs"])), Jn, N, 1 << 30, h_out, h_nodes)
    assert s1 == s2 == s3 and s1 > 0
    assert t.equal(o1, o2) and t.equal(n1, n2)
    assert o1.cpu().numpy().tobytes() == h_out.tobytes() and n1.cpu().numpy().tobytes() == h_nodes.tobytes()


def test_whole_path_reuses_scratch_between_calls():
    cfg = workloads.make("paper-scale")
    gpu = Gpu(cfg)
    a = run_full_path(gpu, cfg)
    b = run_full_path(gpu, cfg)
    c = run_full_path(gpu, cfg, host=True)
    assert_rounds_equal(a, b)
    assert_rounds_equal(a, c)


def test_disabled_plans_are_never_chosen():
    cfg = workloads.make("paper-scale")
    plans, _ = rb.enumerate_plans(cfg["g_levels"])
    plans = plans.copy()
    plans["disabled"] = (plans["off"] == 1) | (plans["zero"] == 3)
    gpu = Gpu(cfg, plans=plans)
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    thr = gpu.np_thr(d_thr, 64)
    feas = gpu.np_feas(d_feas, 64)
    dis = plans["disabled"].astype(bool)
    assert not thr[:, :, dis].any() and not feas[:, dis].any()
    oplans, othr, ofeas, *_ = oracle_tables(cfg)
    assert np.array_equal(feas[:, ~dis], ofeas[:, ~dis])
    check_thr(thr[:, :, ~dis], othr[:, :, ~dis])
    gpu.assert_one_pass_curves_match(cfg["jobs"])


def test_argument_validation():
    cfg = workloads.make("tiny")
    gpu = Gpu(cfg)
    t = gpu.torch
    plans, _ = rb.enumerate_plans(cfg["g_levels"])
    with pytest.raises(rb.RubickError) as ei:
        gpu.ctx.set_space(plans[:-1], cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
    assert ei.value.code == rb.EINVAL
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_space(plans, cfg["g_levels"][::-1].copy(), cfg["c_levels"], cfg["m_levels"])
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_space(plans[::-1].copy(), cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
    with pytest.raises(rb.RubickError):
        gpu.ctx.eval_candidates(None, 3, None, None)
    d = gpu.empty(64, t.float32)
    with pytest.raises(rb.RubickError):
        gpu.ctx.schedule_round(d, 1, 0, 10, d)
    with pytest.raises(rb.RubickError):
        rb.Context(env(gpus_per_node=6))
    fresh = rb.Context(cfg["env"])
    with pytest.raises(rb.RubickError) as ei:
        fresh.eval_candidates(d, 1, d, d)
    assert ei.value.code == rb.ESTATE
    # the context stays usable after rejected calls
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    assert gpu.np_thr(d_thr, 4).max() > 0


@pytest.mark.parametrize("name,J,N", [("paper-scale", None, None), ("cluster-512", 500, 32)])
def test_greedy_round_with_tenant_quotas_is_bit_exact(name, J, N):
    cfg = workloads.make(name, J=J, n_nodes=N)
    Jn = len(cfg["jobs"]["P"])
    rng = np.random.default_rng(21)
    cfg["jobs"]["tenant"] = rng.integers(0, 5, Jn)
    cfg["jobs"]["gmin_idx"] = np.where(rng.uniform(size=Jn) < 0.6, rng.integers(0, 4, Jn), -1)
    cfg["jobs"]["cmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, rng.integers(0, 3, Jn), -1)
    quota = np.stack([rng.integers(4, 40, 5), rng.integers(16, 200, 5)], axis=1)
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 cfg["n_nodes"], want_log=True, quota=quota)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], quota=quota)
    assert_rounds_equal(got, want)
    free = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 cfg["n_nodes"])
    assert not np.array_equal(want["status"], free["status"])                # the quotas bite
    with pytest.raises(rb.RubickError):
        gpu.ctx.greedy_round(None, 0, None, None, None, None, 4, 10, None, quota=np.zeros((300, 2)))


@pytest.mark.parametrize("seed", range(16))
def test_greedy_round_on_random_instances_is_bit_exact(seed):
    """Random cluster shapes, job mixes and guarantees: the batched device round must replay the
    oracle's one-step-at-a-time round exactly, step log included."""
    rng = np.random.default_rng(1000 + seed)
    name = ["paper-scale", "cluster-512", "events"][seed % 3]
    J = int(rng.integers(40, 420))
    N = int(rng.integers(3, 40))
    cfg = workloads.make(name, J=J, n_nodes=N)
    gn = int(rng.choice([4, 8]))
    cfg["env"] = env(gpus_per_node=gn, cpus_per_node=int(rng.choice([32, 64, 96])),
                     mem_per_node_bytes=int(rng.choice([128, 256, 512, 1024])) * GIB)
    if gn == 4:
        cfg["g_levels"] = np.array([g for g in cfg["g_levels"] if g <= 4 or g % 4 == 0])
    share = float(rng.choice([0.0, 0.2, 0.6]))
    guar = rng.uniform(size=J) < share
    cfg["jobs"]["gmin_idx"] = np.where(guar, rng.integers(0, 4, J), -1)
    cfg["jobs"]["cmin_idx"] = np.where(guar, rng.integers(0, 4, J), -1)
    if seed % 4 == 0:
        cfg["jobs"]["w"] = np.ones(J)                     # raw aggregated throughput instead of normalised
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 N, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, N)
    assert_rounds_equal(got, want)


@pytest.mark.parametrize("seed", range(12))
def test_greedy_round_on_larger_random_instances_is_bit_exact(seed):
    """As above with up to 1,400 jobs on up to 300 nodes, so that a turn of the device round has many candidates to
    choose from: batches across two warps, chains of general commits, runs of failing class heads."""
    rng = np.random.default_rng(5000 + seed)
    name = ["paper-scale", "cluster-512", "events", "throughput-stress"][seed % 4]
    J = int(rng.integers(40, 1400))
    N = int(rng.integers(3, 300))
    cfg = workloads.make(name, J=J, n_nodes=N)
    gn = int(rng.choice([4, 8]))
    cfg["env"] = env(gpus_per_node=gn, cpus_per_node=int(rng.choice([32, 64, 96])),
                     mem_per_node_bytes=int(rng.choice([128, 256, 512, 1024])) * GIB)
    if gn == 4:
        cfg["g_levels"] = np.array([g for g in cfg["g_levels"] if g <= 4 or g % 4 == 0])
    share = float(rng.choice([0.0, 0.2, 0.6]))
    guar = rng.uniform(size=J) < share
    cfg["jobs"]["gmin_idx"] = np.where(guar, rng.integers(0, 4, J), -1)
    cfg["jobs"]["cmin_idx"] = np.where(guar, rng.integers(0, 4, J), -1)
    if seed % 5 == 0:
        cfg["jobs"]["w"] = np.ones(J)
    gpu = Gpu(cfg)
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 N, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, N)
    assert_rounds_equal(got, want)


def test_odd_grid_shapes_through_every_kernel():
    """Five core levels (an odd count: the arg-max handles them in pairs), seven memory levels, five GPU
    levels of which one is not a power of two, 4-GPU nodes: table, mask, curves, gains and round."""
    cfg = workloads.make("paper-scale", J=37, n_nodes=9)
    cfg["g_levels"] = np.array([1, 2, 4, 8, 12, 16])
    cfg["c_levels"] = np.array([2, 6, 10, 30, 50])
    cfg["m_levels"] = np.array([16, 48, 100, 200, 333, 512, 700]) * GIB
    cfg["env"] = env(gpus_per_node=4, cpus_per_node=50, mem_per_node_bytes=700 * GIB)
    cfg["jobs"]["gmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, 1, -1)
    cfg["jobs"]["cmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, 2, -1)
    gpu = Gpu(cfg)
    J = 37
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    assert len(plans) == 16 * (1 + 3 + 6 + 10 + 15) and np.array_equal(gpu.np_feas(d_feas, J), feas)
    check_thr(gpu.np_thr(d_thr, J), thr)
    t = gpu.torch
    d_thr32 = t.from_numpy(thr.astype(np.float32).reshape(-1)).cuda()
    for raw in (False, True):
        ov, op, og = oracle.best_plan(thr.astype(np.float32), feas, plans, cfg["g_levels"], gpu.nM, prefix=not raw, nthreads=4)
        bv, bp, bg = gpu.best(d_thr32, d_feas, J, flags=rb.BEST_RAW if raw else 0)
        sh = gpu.shape4(J)
        assert np.array_equal(bv.cpu().numpy().reshape(sh), ov.astype(np.float32))
        assert np.array_equal(bp.cpu().numpy().reshape(sh), op) and np.array_equal(bg.cpu().numpy().reshape(sh), og)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 9, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 9)
    assert_rounds_equal(got, want)
    assert want["steps"] > 5 and (want["n_nodes"] > 1).any()
    gpu.assert_one_pass_curves_match(cfg["jobs"])


def test_largest_supported_grid_and_cluster():
    """64 core levels, 32 memory levels, 4,096 nodes (the limits of the shared-memory state)."""
    cfg = workloads.make("paper-scale", J=48, n_nodes=4096)
    cfg["c_levels"] = np.arange(1, 65)
    cfg["env"] = env(cpus_per_node=64)
    gpu = Gpu(cfg)
    assert gpu.nC == 64 and gpu.nM == 32
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    plans, thr, feas, cv, cp, cg = oracle_tables(cfg)
    assert np.array_equal(gpu.np_feas(d_feas, 48), feas)
    check_thr(gpu.np_thr(d_thr, 48), thr)
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 4096, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 4096)
    assert_rounds_equal(got, want)
    gpu.assert_one_pass_curves_match(cfg["jobs"])
    with pytest.raises(rb.RubickError):
        gpu.ctx.greedy_round(None, 0, None, None, None, None, 4097, 10, None)
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_space(gpu.plans, cfg["g_levels"], np.arange(1, 66), cfg["m_levels"])


def test_outputs_stay_inside_their_buffers():
    """Every output buffer sits between two guard regions filled with a pattern; after the whole path has
    run on a ragged job count the guards must be untouched."""
    cfg = workloads.make("cluster-512", J=203, n_nodes=21)
    gpu = Gpu(cfg)
    t = gpu.torch
    J, N, G = 203, 21, 4096                                  # guard bytes on either side

    def guarded(nbytes):
        buf = t.full((nbytes + 2 * G,), 0xA5, dtype=t.uint8, device="cuda:0")
        return buf, buf[G:G + nbytes]

    d_jobs = gpu.jobs_to_device(cfg["jobs"])
    thr_b, thr = guarded(J * gpu.nC * gpu.P * 4)
    feas_b, feas = guarded(J * gpu.P * 4)
    n = J * gpu.nG * gpu.nC * gpu.nM
    cv_b, cv = guarded(n * 4); cp_b, cp = guarded(n * 4); cg_b, cg = guarded(n * 4)
    out_b, out = guarded(J * rb.ASSIGN_DTYPE.itemsize); node_b, node = guarded(N * rb.NODE_DTYPE.itemsize)
    log_b, log = guarded(4 * (J * (gpu.nG + gpu.nC + 2) + 1))
    gains = [guarded(J * 4) for _ in range(4)]
    req_out = [guarded(J * 4) for _ in range(3)]
    gpu.ctx.eval_candidates(d_jobs, J, thr, feas)
    gpu.ctx.best_plan(thr, feas, J, cv, cp, cg)
    state = t.zeros(J * rb.ASSIGN_DTYPE.itemsize, dtype=t.uint8, device="cuda:0")
    gpu.ctx.marginal_gain(d_jobs, J, cv, state, *[g[1] for g in gains])
    rec = np.zeros(J, dtype=rb.REQUEST_DTYPE)
    rec["g_idx"], rec["c_idx"], rec["m_idx"], rec["plan"] = 3, 5, 20, 170
    gpu.ctx.min_resources(thr, feas, cv, J, rb.to_device(rec), *[r[1] for r in req_out])
    steps, _ = gpu.ctx.greedy_round(d_jobs, J, cv, cp, cg, feas, N, J * (gpu.nG + gpu.nC + 2) + 1, out, node, log)
    gpu.ctx.greedy_round_noalloc(d_jobs, J, cv, cp, cg, feas, N, 1 << 30, out, node)
    # the incremental round from that allocation (with and without a step log), and model fitting
    out2_b, out2 = guarded(J * rb.ASSIGN_DTYPE.itemsize); node2_b, node2 = guarded(N * rb.NODE_DTYPE.itemsize)
    log2_b, log2 = guarded(4 * (2 * J * (gpu.nG + gpu.nC + 2) + 1))
    rc = np.zeros(J, dtype=rb.RECONF_DTYPE)
    rc["active"], rc["T"], rc["delta"] = (np.arange(J) % 5 != 0), 5000.0, 20.0
    d_rc = rb.to_device(rc)
    gpu.ctx.incremental_round(d_jobs, J, cv, cp, cg, feas, N, 2 * J * (gpu.nG + gpu.nC + 2) + 1, out2, node2, log2,
                              d_prev=out.clone(), d_prev_nodes=node.clone(), d_reconf=d_rc)
    gpu.ctx.incremental_round(d_jobs, J, cv, cp, cg, feas, N, 1 << 30, out2, node2, None,
                              d_prev=out.clone(), d_prev_nodes=node.clone(), d_reconf=d_rc)
    S = 5
    smp = np.zeros((J, S), dtype=rb.SAMPLE_DTYPE)
    smp["plan"], smp["cores"], smp["thr"] = np.arange(J * S).reshape(J, S) % 64, 8, 1.0
    th_b, th = guarded(J * 7 * 8); rm_b, rm = guarded(J * 2 * 8)
    gpu.ctx.fit_models(d_jobs, J, rb.to_device(smp), S, 3, th, rm)
    gpu.ctx.sync()
    assert steps > 0
    for whole in [thr_b, feas_b, cv_b, cp_b, cg_b, out_b, node_b, log_b, out2_b, node2_b, log2_b, th_b, rm_b] \
            + [g[0] for g in gains] + [r[0] for r in req_out]:
        assert bool((whole[:G] == 0xA5).all()) and bool((whole[-G:] == 0xA5).all())


def test_a_failed_scratch_allocation_leaves_the_context_usable():
    """A job count whose curve tables cannot be allocated (three tables of 69 GB each beside a 26 GB mask: the
    third one no longer fits the GPU) is refused with ENOMEM before anything is launched; none of the
    half-grown tables may survive into the next, ordinary call, which must give the usual result."""
    cfg = workloads.make("paper-scale")
    gpu = Gpu(cfg)
    t = gpu.torch
    want = run_full_path(gpu, cfg)
    d_jobs = gpu.jobs_to_device(cfg["jobs"])
    d_out = gpu.empty(64 * rb.ASSIGN_DTYPE.itemsize, t.uint8)
    for J in (2_500_000, 40_000_000):
        if J * gpu.nG * gpu.nC * gpu.nM * 12 + J * gpu.P * 4 < t.cuda.mem_get_info()[0]:
            continue                                          # a GPU with room for it all: nothing to refuse
        with pytest.raises(rb.RubickError) as ei:
            gpu.ctx.schedule_round(d_jobs, J, 8, 10, d_out)   # the job records are never read: allocation comes first
        assert ei.value.code == rb.ENOMEM
        again = run_full_path(gpu, cfg)
        assert_rounds_equal(again, want)
        again = run_full_path(gpu, cfg, host=True)
        assert_rounds_equal(again, want)
    gpu.ctx.close()
