"""Spread placement through the CUDA path against the oracle: predictions of the spread classes (1e-5 relative,
masks bit-exact, one-pass curves bit-identical to the two-kernel path), and the round that assembles jobs from
pieces (allocations, pieces, classes, node states, values and step log bit-exact on the same tables)."""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, assert_rounds_equal, has_cuda, unpack_round
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads
from test_gpu_parity import check_thr
from test_oracle_spread import class_tables, odd_sized_cluster

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def gpu_for(cfg):
    if cfg.get("any_degrees"):
        plans, _ = rb.enumerate_plans_wide(cfg["g_levels"])
        return Gpu(cfg, plans=plans)
    return Gpu(cfg)


@pytest.mark.parametrize("wide", [False, True])
def test_predictions_of_the_spread_classes(wide):
    cfg = odd_sized_cluster("paper-scale", 40, 4) if wide else workloads.make("paper-scale", J=40)
    gpu = gpu_for(cfg)
    plans, _ = oracle.enumerate_plans(cfg["g_levels"], any_degrees=wide)
    for a in (4, 2, 1, 0):
        gpu.ctx.set_placement(a)
        _, d_thr, d_feas = gpu.eval(cfg["jobs"])
        thr, feas = oracle.eval_candidates(cfg["jobs"], plans, dict(cfg["env"], spread_align=a), cfg["c_levels"], cfg["m_levels"], nthreads=8)
        assert np.array_equal(gpu.np_feas(d_feas, 40), feas)
        check_thr(gpu.np_thr(d_thr, 40), thr)
        if a:
            assert (thr > 0).any() and not thr[:, :, np.prod(plans[:, :3], axis=1) > 8].any()
        gpu.assert_one_pass_curves_match(cfg["jobs"])
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_placement(8)                               # a piece as large as a node is not spreading
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_placement(3)


def spread_round(gpu, jobs, packed, classes, n_nodes, max_steps=1 << 30):
    """rubick_greedy_round_spread on host-provided tables -> dict like the oracle's, with pieces and cls."""
    t = gpu.torch
    J = len(jobs["P"])
    dev = lambda a, dt: t.from_numpy(np.ascontiguousarray(a, dtype=dt).reshape(-1)).cuda()
    feas_dev = lambda f: t.from_numpy(np.ascontiguousarray(f, dtype=np.uint32).view(np.int32).reshape(-1)).cuda()
    cv, cp, cg, feas = packed
    d_tabs = (dev(cv, np.float32), dev(cp, np.int32), dev(cg, np.int32), feas_dev(feas))
    d_classes = [(a, dev(v, np.float32), dev(p, np.int32), dev(g, np.int32), feas_dev(f)) for a, v, p, g, f in classes]
    cap = int(min(max_steps, J * (gpu.nG + gpu.nC + 2) + 1))
    d_out = gpu.empty(max(J, 1) * rb.ASSIGN_DTYPE.itemsize, t.uint8)
    d_node = gpu.empty(n_nodes * rb.NODE_DTYPE.itemsize, t.uint8)
    d_log = gpu.empty(max(cap, 1), t.int32)
    d_pieces = gpu.empty(max(J, 1) * rb.MAX_PIECES, t.int32)
    d_cls = gpu.empty(max(J, 1), t.int32)
    steps, capped = gpu.ctx.greedy_round_spread(gpu.jobs_to_device(jobs), J, *d_tabs, d_classes, n_nodes, cap, d_out, d_pieces, d_cls,
                                                d_node, d_log)
    r = unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE)[:J], rb.from_device(d_node, rb.NODE_DTYPE), steps, capped,
                     d_log.cpu().numpy()[:steps])
    r["pieces"] = d_pieces.cpu().numpy().reshape(-1, rb.MAX_PIECES)[:J]
    r["cls"] = d_cls.cpu().numpy()[:J]
    return r


@pytest.mark.parametrize("name,J,N,aligns", [("paper-scale", 64, 6, (4, 2, 1)), ("cluster-512", 300, 14, (4, 2, 1)), ("events", 200, 12, (2,)),
                                             ("cluster-512", 150, 40, (1,)), ("paper-scale", 64, 3, (4, 2))])
def test_round_with_spread_classes_is_bit_exact(name, J, N, aligns):
    cfg = odd_sized_cluster(name, J, N)
    gpu = gpu_for(cfg)
    plans, feas, cv, cp, cg = class_tables(cfg, 0, nthreads=8)
    classes = []
    for a in aligns:
        _, fs, v, p_, g_ = class_tables(cfg, a, nthreads=8)
        classes.append((a, v, p_, g_, fs))
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], N,
                                 want_log=True, spread=classes)
    got = spread_round(gpu, cfg["jobs"], (cv, cp, cg, feas), classes, N)
    assert_rounds_equal(got, want)
    assert np.array_equal(got["cls"], want["cls"]) and np.array_equal(got["pieces"], want["pieces"])
    if N <= 14:
        assert (want["cls"] >= 0).any()
    # a step limit stops both at the same place
    k = max(1, want["steps"] // 2)
    want_k = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], N,
                                   want_log=True, spread=classes, max_steps=k)
    got_k = spread_round(gpu, cfg["jobs"], (cv, cp, cg, feas), classes, N, max_steps=k)
    assert_rounds_equal(got_k, want_k)
    assert np.array_equal(got_k["pieces"], want_k["pieces"])


def test_without_classes_it_is_the_plain_round():
    cfg = workloads.make("cluster-512", J=300, n_nodes=20)
    gpu = Gpu(cfg)
    plans, feas, cv, cp, cg = class_tables(cfg, 0, nthreads=8)
    got = spread_round(gpu, cfg["jobs"], (cv, cp, cg, feas), [], 20)
    plain = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, 20)
    assert_rounds_equal(got, plain)
    assert (got["cls"] < 0).all() and (got["pieces"] < 0).all()


def test_the_whole_chain_on_the_gpu_with_spread_classes():
    """Tables of every class from the library itself (rubick_set_placement + rubick_curves), then the round; the oracle
    replays the round on those tables."""
    cfg = odd_sized_cluster("cluster-512", 200, 10)
    gpu = gpu_for(cfg)
    t = gpu.torch
    J, N = 200, 10
    n = J * gpu.nG * gpu.nC * gpu.nM
    d_jobs = gpu.jobs_to_device(cfg["jobs"])
    tabs = {}
    for a in (0, 4, 2, 1):
        gpu.ctx.set_placement(a)
        d_feas = gpu.empty(J * gpu.P, t.int32)
        cv, cp, cg = gpu.empty(n, t.float32), gpu.empty(n, t.int32), gpu.empty(n, t.int32)
        gpu.ctx.curves(d_jobs, J, d_feas, cv, cp, cg)
        gpu.ctx.sync()
        tabs[a] = (cv, cp, cg, d_feas)
    gpu.ctx.set_placement(0)
    sh = gpu.shape4(J)
    host = {a: (x[0].cpu().numpy().reshape(sh), x[1].cpu().numpy().reshape(sh), x[2].cpu().numpy().reshape(sh), gpu.np_feas(x[3], J))
            for a, x in tabs.items()}
    classes = [(a,) + host[a] for a in (4, 2, 1)]
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], *host[0], cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], N, want_log=True, spread=classes)
    got = spread_round(gpu, cfg["jobs"], host[0], classes, N)
    assert_rounds_equal(got, want)
    assert np.array_equal(got["pieces"], want["pieces"]) and np.array_equal(got["cls"], want["cls"]) and (want["cls"] >= 0).any()


def test_hand_made_case_and_argument_checks():
    g_levels = np.array([1, 2, 4, 6, 8]); c_levels = np.array([4, 8]); m_levels = np.array([64, 128]) * GIB
    jobs = stack_jobs(one_job(gmin_idx=3, cmin_idx=0), one_job(gmin_idx=3, cmin_idx=0), one_job())
    cfg = dict(workloads.make("tiny"), g_levels=g_levels, c_levels=c_levels, m_levels=m_levels, jobs=jobs, any_degrees=True)
    gpu = gpu_for(cfg)
    J, nG, nC, nM, P = 3, 5, 2, 2, gpu.P
    val = np.array([[1.0, 2.0, 3.5, 5.0, 5.0], [1.0, 2.0, 3.5, 5.0, 5.0], [0.0, 0.0, 3.5, 3.5, 3.5]], dtype=np.float32)
    plan = np.array([[0, 1, 2, 3, 3], [0, 1, 2, 3, 3], [-1, -1, 2, 2, 2]], dtype=np.int32)
    used = np.array([[1, 2, 4, 6, 6], [1, 2, 4, 6, 6], [0, 0, 4, 4, 4]], dtype=np.int32)
    full = lambda x: np.broadcast_to(x[:, :, None, None], (J, nG, nC, nM)).copy()
    cv, cp, cg = full(val), full(plan), full(used)
    feas = np.full((J, P), 0b11, dtype=np.uint32)
    sv, sp_, sg = full(val * np.float32(0.75)), full(plan), full(used)
    sv[:, :2] = 0; sp_[:, :2] = -1; sg[:, :2] = 0
    got = spread_round(gpu, jobs, (cv, cp, cg, feas), [(2, sv, sp_, sg, feas)], 2)
    assert list(got["g"]) == [6, 6, 4] and list(got["cls"]) == [-1, -1, 0] and got["n_nodes"][2] == 2
    assert [int(x) for x in got["pieces"][2] if x >= 0] == [(0 << 8) | 2, (1 << 8) | 2]
    assert got["thr"][2] == np.float32(3.5 * 0.75)
    t = gpu.torch
    d = gpu.empty(64, t.float32)
    with pytest.raises(rb.RubickError):
        gpu.ctx.greedy_round_spread(d, 1, d, d, d, d, [(3, d, d, d, d)], 2, 10, d, d, d)          # 3 is not a power of two
    with pytest.raises(rb.RubickError):
        gpu.ctx.greedy_round_spread(d, 1, d, d, d, d, [(2, d, d, d, d)] * 5, 2, 10, d, d, d)      # too many classes
