"""The wider plan space (degrees of any size: the paper's 3-GPU tensor-parallel plan, 12- and 24-GPU jobs)
through the CUDA path, against the oracle on the same plans: throughput within 1e-5 relative, masks and
everything downstream bit-exact."""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, assert_chain_parity, assert_rounds_equal, has_cuda, unpack_round
from helpers import GIB, env
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads
from test_gpu_parity import check_thr

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def wide_config(J, levels, gpus_per_node, n_nodes, seed=6):
    cfg = workloads.make("paper-scale", J=J, n_nodes=n_nodes)
    rng = np.random.default_rng(seed)
    cfg["g_levels"] = np.asarray(levels)
    cfg["env"] = env(gpus_per_node=gpus_per_node)
    jobs = cfg["jobs"]
    # shapes that odd degrees divide: hidden sizes with a factor 3 or 5, batches with a factor 3
    jobs["h"] = rng.choice([768, 1536, 3072, 1280, 2560, 1920, 1024], J)
    jobs["b"] = rng.choice([48, 96, 24, 64, 30], J)
    jobs["l"] = rng.integers(12, 49, J)
    jobs["gmin_idx"] = np.where(rng.uniform(size=J) < 0.3, rng.integers(0, 3, J), -1)
    jobs["cmin_idx"] = np.where(jobs["gmin_idx"] >= 0, 0, -1)
    return cfg


def oracle_wide(cfg, nthreads=8, accumulation_levels=1):
    plans, goff = oracle.enumerate_plans(cfg["g_levels"], any_degrees=True, accumulation_levels=accumulation_levels)
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    cv, cp, cg = oracle.best_plan(thr.astype(np.float32), feas, plans, cfg["g_levels"], len(cfg["m_levels"]), prefix=True, nthreads=nthreads)
    return plans, goff, thr, feas, cv.astype(np.float32), cp, cg


def test_wide_enumerators_agree():
    for levels, n_acc in (([1, 2, 3, 4, 5, 6, 7, 8], 1), ([1, 2, 3, 4, 6, 8, 16, 24, 48], 3), ([1, 2, 4, 8, 16], 2)):
        got, goff = rb.enumerate_plans_wide(levels, accumulation_levels=n_acc)
        want, woff = oracle.enumerate_plans(levels, any_degrees=True, accumulation_levels=n_acc)
        assert np.array_equal(goff, woff) and len(got) == len(want)
        for col, name in enumerate(("d", "t", "p", "zero", "gc", "off", "accum")):
            assert np.array_equal(got[name].astype(np.int64), want[:, col])
        assert np.array_equal(got["g_level"], np.searchsorted(woff[1:], np.arange(len(want)), side="right"))


@pytest.mark.parametrize("levels,gn,N,n_acc", [([1, 2, 3, 4, 6, 8, 16, 24, 48], 8, 7, 1), ([1, 2, 3, 4, 8, 12, 24], 4, 9, 1),
                                               ([1, 2, 3, 4, 6, 8, 16], 8, 5, 3)])
def test_wide_plan_space_through_every_kernel(levels, gn, N, n_acc):
    J = 41
    cfg = wide_config(J, levels, gn, N)
    if n_acc > 1:
        cfg["env"]["gpu_mem_bytes"] = 24_000_000_000       # small GPUs: plans that only fit with smaller micro-batches
    plans, goff, thr, feas, cv, cp, cg = oracle_wide(cfg, accumulation_levels=n_acc)
    gpu_plans, _ = rb.enumerate_plans_wide(levels, accumulation_levels=n_acc)
    gpu = Gpu(cfg, plans=gpu_plans)
    assert gpu.P == len(plans)
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    assert np.array_equal(gpu.np_feas(d_feas, J), feas)
    check_thr(gpu.np_thr(d_thr, J), thr)
    odd = (plans[:, 0] % 3 == 0) | (plans[:, 1] % 3 == 0) | (plans[:, 2] % 3 == 0)
    assert (thr[:, 0, odd] > 0).any() and feas[:, odd].any()               # plans with a degree of 3, 6, 12 ... do run
    t = gpu.torch
    d_thr32 = t.from_numpy(thr.astype(np.float32).reshape(-1)).cuda()
    bv, bp, bg = gpu.best(d_thr32, d_feas, J)
    sh = gpu.shape4(J)
    assert np.array_equal(bv.cpu().numpy().reshape(sh), cv)
    assert np.array_equal(bp.cpu().numpy().reshape(sh), cp) and np.array_equal(bg.cpu().numpy().reshape(sh), cg)
    assert odd[cp[cp >= 0]].any()                                          # and win somewhere
    if n_acc > 1:
        assert (plans[cp[cp >= 0], 6] > 0).any()                           # plans with extra accumulation win where memory is short
    gpu.assert_one_pass_curves_match(cfg["jobs"])
    want = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 N, want_log=True)
    got = gpu.round_on_tables(cfg["jobs"], cv, cp, cg, feas, N)
    assert_rounds_equal(got, want)
    assert want["steps"] > 5
    # the whole path in one call on the library's own tables: the same round up to the first near tie of the two chains
    d_out = gpu.empty(J * rb.ASSIGN_DTYPE.itemsize, t.uint8)
    d_node = gpu.empty(N * rb.NODE_DTYPE.itemsize, t.uint8)
    steps, capped = gpu.ctx.schedule_round(gpu.jobs_to_device(cfg["jobs"]), J, N, 1 << 30, d_out, d_node)
    one_call = unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE), rb.from_device(d_node, rb.NODE_DTYPE), steps, capped, None)
    assert_chain_parity(gpu, cfg, N, (plans, thr, feas, cv, cp, cg), got=one_call)
    assert not capped


def test_wide_space_validation_and_limits():
    cfg = wide_config(8, [1, 2, 3, 4, 6, 8], 8, 2)
    plans, _ = rb.enumerate_plans_wide(cfg["g_levels"])
    gpu = Gpu(cfg, plans=plans)
    bad = plans.copy()
    bad["d"][0] = 2                                        # d * t * p no longer the level's GPU count
    with pytest.raises(rb.RubickError):
        gpu.ctx.set_space(bad, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
    with pytest.raises(rb.RubickError):                    # 12 GPUs on 8-GPU nodes is not a whole number of nodes
        gpu.ctx.set_space(*((lambda p: (p, [1, 2, 12], cfg["c_levels"], cfg["m_levels"]))(rb.enumerate_plans_wide([1, 2, 12])[0])))
    # the power-of-two format refuses other degrees; the wide format on power-of-two levels equals it
    t = gpu.torch
    p2, _ = rb.enumerate_plans([1, 2, 4, 8])
    w2, _ = rb.enumerate_plans_wide([1, 2, 4, 8])
    assert np.array_equal(1 << p2["log2d"].astype(np.int64), w2["d"]) and np.array_equal(1 << p2["log2t"].astype(np.int64), w2["t"])
    cfg2 = workloads.make("tiny")
    cfg2["g_levels"] = np.array([1, 2, 4, 8])
    a = Gpu(cfg2, plans=p2)
    b = Gpu(cfg2, plans=w2)
    _, thr_a, feas_a = a.eval(cfg2["jobs"])
    _, thr_b, feas_b = b.eval(cfg2["jobs"])
    assert t.equal(feas_a, feas_b)
    assert np.allclose(thr_a.cpu().numpy(), thr_b.cpu().numpy(), rtol=2e-6, atol=0)


def test_model_fitting_on_the_wide_plan_space():
    """Samples on plans with odd degrees and explicit accumulation; same decisions as the oracle's fit."""
    from test_gpu_fit import gpu_fit
    from test_oracle_fit import with_coefficients
    J, S = 24, 16
    cfg = wide_config(J, [1, 2, 3, 4, 6, 8], 8, 2)
    plans, goff, thr, feas, *_ = oracle_wide(cfg, accumulation_levels=2)
    picks = workloads.draw_fit_picks(5, J, S, len(cfg["c_levels"]))
    sp, sc, sy = workloads.fit_samples(cfg, plans, thr, feas, picks)
    assert ((plans[np.maximum(sp, 0), 1] == 3) & (sp >= 0)).any() and ((plans[np.maximum(sp, 0), 6] == 1) & (sp >= 0)).any()
    start = with_coefficients(cfg["jobs"], {k: np.float32(v) for k, v in workloads.FIT_NOMINAL.items()})
    want_theta, want_rmsle, margin = oracle.fit(start, plans, cfg["env"], sp, sc, sy, sweeps=10)
    gpu_plans, _ = rb.enumerate_plans_wide(cfg["g_levels"], accumulation_levels=2)
    gpu = Gpu(cfg, plans=gpu_plans)
    theta, rmsle = gpu_fit(gpu, start, sp, sc, sy, sweeps=10)
    assert np.allclose(rmsle, want_rmsle, rtol=1e-9, atol=1e-13)
    firm = margin > 1e-11
    assert firm.mean() > 0.8 and np.array_equal(theta[firm], want_theta[firm])
    assert np.all(rmsle[:, 1] <= rmsle[:, 0]) and np.median(rmsle[:, 1]) < 0.5 * np.median(rmsle[:, 0])
