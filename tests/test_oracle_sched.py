"""Pins of the oracle's marginal gains and greedy round (paper Section 5.2, Algorithm 1).

The paper calls its policy a heuristic for an NP-hard packing problem and claims no
optimality, so exhaustive search gives an upper bound in general and equality only where
mathematics guarantees it (separable concave gains in one resource)."""
import numpy as np
import pytest

import oracle
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import workloads


def tables(cfg, nthreads=4):
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    cv, cp, cg = oracle.best_plan(thr.astype(np.float32), feas, plans, cfg["g_levels"], len(cfg["m_levels"]),
                                  prefix=True, nthreads=nthreads)
    return plans, feas, cv.astype(np.float32), cp, cg


def run_round(cfg, tb, **kw):
    plans, feas, cv, cp, cg = tb
    return oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                 cfg["m_levels"], cfg["n_nodes"], **kw)


def check_invariants(cfg, tb, r):
    """Whatever the policy decided must be a consistent packing of the cluster."""
    plans, feas, cv, cp, cg = tb
    e = cfg["env"]
    Gn, Cn, Mn = e["gpus_per_node"], e["cpus_per_node"], e["mem_per_node_bytes"]
    N = cfg["n_nodes"]
    used = np.zeros((N, 3), dtype=np.int64)
    J = len(r["g"])
    for j in range(J):
        if r["status"][j] != 1:
            assert r["g"][j] == 0 and r["plan"][j] == -1 and r["thr"][j] == 0
            continue
        g, c, m, k, n0, pl = (int(r[x][j]) for x in ("g", "c", "m_bytes", "n_nodes", "first_node", "plan"))
        assert g in cfg["g_levels"] and c in cfg["c_levels"] and m in cfg["m_levels"]
        assert int(np.prod(plans[pl, :3])) == g
        gi = list(cfg["g_levels"]).index(g)
        ci = list(cfg["c_levels"]).index(c)
        f = int(r["m_level"][j])
        assert m == cfg["m_levels"][f] and (feas[j, pl] >> f) & 1 and (f == 0 or not (feas[j, pl] >> (f - 1)) & 1)
        # the value is the curve's, read at some host-memory level at or above the plan's need
        assert r["thr"][j] in cv[j, gi, ci, f:]
        if k == 1:
            assert g <= Gn
            used[n0] += (g, c, m)
        else:
            assert g == k * Gn
            own = np.nonzero(r["node"][:, 3] == j)[0]
            assert len(own) == k and own[0] == n0
            used[own] += (Gn, -(-c // k), -(-m // k))
    assert np.all(used <= np.array([Gn, Cn, Mn]))
    assert np.array_equal(r["node"][:, 0], Gn - used[:, 0])
    assert np.array_equal(r["node"][:, 1], Cn - used[:, 1])
    assert np.array_equal(r["node"][:, 2], Mn - used[:, 2])


def test_tiny_round_is_a_valid_packing_and_below_the_optimum(tiny):
    tb = tables(tiny)
    r = run_round(tiny, tb, want_log=True)
    check_invariants(tiny, tb, r)
    plans, feas, cv, cp, cg = tb
    best = oracle.bruteforce(tiny["jobs"], tiny["env"], cv, cp, cg, feas, tiny["g_levels"], tiny["c_levels"], tiny["m_levels"])
    w = tiny["jobs"]["w"].astype(np.float32)
    total = float((w * r["thr"]).astype(np.float64).sum())
    assert 0 < total <= best * (1 + 1e-6)
    assert total >= 0.9 * best               # reported gap on this instance is small
    assert r["g"].sum() == 8                 # all GPUs of the node are handed out


@pytest.mark.parametrize("seed", range(6))
def test_random_small_instances_never_beat_the_optimum(seed):
    cfg = workloads.make("tiny")
    rng = np.random.Generator(np.random.PCG64(100 + seed))
    cfg["jobs"] = workloads.draw_jobs(rng, 3 + seed % 2, [1, 2, 3, 4, 5, 6, 7, 8], 4, pmax=13e9)
    cfg["env"]["mem_per_node_bytes"] = 384 * GIB
    tb = tables(cfg)
    r = run_round(cfg, tb)
    check_invariants(cfg, tb, r)
    plans, feas, cv, cp, cg = tb
    best = oracle.bruteforce(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
    w = cfg["jobs"]["w"].astype(np.float32)
    assert float((w * r["thr"]).astype(np.float64).sum()) <= best * (1 + 1e-6)


def concave_instance(seed, J=4, G=8):
    """Curves that are strictly increasing and strictly concave in the GPU count alone."""
    rng = np.random.default_rng(seed)
    inc = np.sort(rng.uniform(0.1, 4.0, (J, G)), axis=1)[:, ::-1]        # decreasing increments
    cv = np.cumsum(inc, axis=1).astype(np.float32)[:, :, None, None]
    cp = np.zeros((J, G, 1, 1), dtype=np.int32)
    cg = np.broadcast_to(np.arange(1, G + 1, dtype=np.int32)[None, :, None, None], (J, G, 1, 1)).copy()
    feas = np.ones((J, 1), dtype=np.uint32)
    jobs = stack_jobs(*[one_job(host_base_bytes=0) for _ in range(J)])
    return jobs, cv, cp, cg, feas


@pytest.mark.parametrize("seed", range(8))
def test_greedy_is_optimal_for_separable_concave_gains(seed):
    jobs, cv, cp, cg, feas = concave_instance(seed)
    gl, cl, ml = np.arange(1, 9), np.array([4]), np.array([GIB])
    r = oracle.schedule_round(jobs, env(), cv, cp, cg, feas, gl, cl, ml, 1, want_log=True)
    best = oracle.bruteforce(jobs, env(), cv, cp, cg, feas, gl, cl, ml)
    assert r["g"].sum() == 8 and r["steps"] == 8
    assert float(r["thr"].astype(np.float64).sum()) == pytest.approx(best, rel=1e-6)
    # every step took the largest remaining increment
    inc = np.diff(np.concatenate([np.zeros((4, 1), np.float32), cv[:, :, 0, 0]], axis=1), axis=1)
    taken = sorted(inc.ravel(), reverse=True)[:8]
    assert float(r["thr"].sum()) == pytest.approx(float(np.sum(taken)), rel=1e-5)


def test_ties_go_to_the_lowest_job_index_and_gpu_before_cpu():
    cfg = workloads.make("tiny")
    same = workloads.take(cfg["jobs"], [0, 0, 0])
    same["gmin_idx"] = np.array([-1, -1, -1])
    same["cmin_idx"] = np.array([-1, -1, -1])
    cfg["jobs"] = same
    tb = tables(cfg)
    r = run_round(cfg, tb, want_log=True)
    log = r["log"]
    assert (log[0] >> 2) == 0 and (log[1] >> 2) == 1 and (log[2] >> 2) == 2
    types = (log >> 1) & 1
    first_cpu = np.argmax(types) if types.any() else len(types)
    assert not types[:first_cpu].any() and types[first_cpu:].all()      # all GPU steps come first here


def test_gains_by_hand():
    # one job, curve over g levels (1, 2, 4, 8) and c levels (4, 8); w = 0.5
    cv = np.zeros((1, 4, 2, 1), dtype=np.float32)
    cv[0, :, 0, 0] = [10, 10, 16, 40]
    cv[0, :, 1, 0] = [12, 12, 20, 48]
    jobs = one_job(w=0.5)
    gl, cl = [1, 2, 4, 8], [4, 8]
    gg, gc, ng, nc = oracle.gain(jobs, cv, gl, cl, [0], [0], [0.0])
    assert (ng[0], nc[0]) == (0, -1) and gg[0] == np.float32(0.5 * 10 / 1) and gc[0] == 0
    gg, gc, ng, nc = oracle.gain(jobs, cv, gl, cl, [1], [4], [10.0])
    # the flat level 2 is skipped: next improving level is 4 GPUs: (0.5*16 - 0.5*10) / (4 - 1)
    assert ng[0] == 2 and gg[0] == np.float32((8.0 - 5.0) / 3.0)
    assert nc[0] == 1 and gc[0] == np.float32((6.0 - 5.0) / 4.0)
    gg, gc, ng, nc = oracle.gain(jobs, cv, gl, cl, [8], [8], [48.0])
    assert (ng[0], nc[0]) == (-1, -1) and gg[0] == 0 and gc[0] == 0


def test_guaranteed_minimum_is_placed_first_or_left_pending():
    cfg = workloads.make("tiny")
    jobs = workloads.take(cfg["jobs"], [0, 1, 2, 3])
    jobs["gmin_idx"] = np.array([-1, -1, -1, 7])          # job 3 is guaranteed all 8 GPUs
    jobs["cmin_idx"] = np.array([-1, -1, -1, 1])
    cfg["jobs"] = jobs
    tb = tables(cfg)
    r = run_round(cfg, tb)
    check_invariants(cfg, tb, r)
    assert r["status"][3] == 1 and r["g"][3] == 8 and r["c"][3] >= 8
    assert np.all(r["status"][:3] == 0)
    # two such jobs cannot both be served: the second stays pending and takes nothing less
    jobs["gmin_idx"] = np.array([7, -1, -1, 7])
    jobs["cmin_idx"] = np.array([0, -1, -1, 0])
    r = run_round(cfg, tables(cfg))
    assert r["status"][0] == 1 and r["status"][3] == 2 and r["g"][3] == 0


def test_step_cap_is_reported(tiny):
    tb = tables(tiny)
    full = run_round(tiny, tb)
    assert not full["capped"] and full["steps"] >= 2
    r = run_round(tiny, tb, max_steps=1)
    assert r["capped"] and r["steps"] == 1
    check_invariants(tiny, tb, r)


def test_multi_node_round_is_a_valid_packing():
    cfg = workloads.make("cluster-512", J=96, n_nodes=24)
    tb = tables(cfg, nthreads=8)
    r = run_round(cfg, tb)
    check_invariants(cfg, tb, r)
    assert (r["n_nodes"] > 1).any()                      # some job spans whole nodes
    assert r["g"].sum() <= 24 * 8
    assert (r["c"] > cfg["c_levels"][0]).any()           # cores were handed to an offloading job


def test_slope_aware_split_beats_the_equal_split():
    """Section 7.2 micro-benchmark, qualitatively: on two jobs sharing one node, allocating by
    slope yields at least the total normalised throughput of splitting the GPUs evenly."""
    wins = 0
    for seed in range(20):
        cfg = workloads.make("tiny")
        rng = np.random.Generator(np.random.PCG64(500 + seed))
        cfg["jobs"] = workloads.draw_jobs(rng, 2, list(range(1, 9)), 4, pmax=3e9, guaranteed_share=0.0)
        plans, feas, cv, cp, cg = tb = tables(cfg)
        r = run_round(cfg, tb)
        w = cfg["jobs"]["w"].astype(np.float32)
        greedy = float((w * r["thr"]).sum())
        ci = [list(cfg["c_levels"]).index(max(int(c), 4)) if r["status"][j] == 1 else 0 for j, c in enumerate(r["c"])]
        equal = float(sum(w[j] * cv[j, 3, ci[j], -1] for j in range(2)))     # 4 GPUs each
        wins += greedy >= equal * (1 - 1e-6)
    assert wins >= 18


def test_tenant_quotas_limit_the_privileged_jobs():
    """Section 5.1 / 5.2: a guaranteed job is placed first only while its minimum demand fits what is
    left of its tenant's quota; the quota is used up by the minimum demand of the jobs placed."""
    cfg = workloads.make("paper-scale")
    J = 64
    jobs = cfg["jobs"]
    jobs["gmin_idx"] = np.full(J, 1)                 # every job is guaranteed 2 GPUs ...
    jobs["cmin_idx"] = np.full(J, 0)                 # ... and 4 cores
    jobs["tenant"] = np.arange(J) % 2
    tb = tables(cfg)
    plans, feas, cv, cp, cg = tb
    kw = dict(want_log=True)
    free = run_round(cfg, tb, **kw)
    quota = np.array([[6, 12], [64, 4]])             # tenant 0: 6 GPUs; tenant 1: cores for one job only
    lim = oracle.schedule_round(jobs, cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                cfg["n_nodes"], quota=quota, **kw)
    check_invariants(cfg, tb, lim)
    placed = lim["status"] == 1
    t = jobs["tenant"]
    # Phase A placed at most what the quotas allow, in job order; nobody beyond the quota runs at all
    assert placed[t == 0].sum() <= 3 and placed[t == 1].sum() <= 1
    first0 = np.nonzero((t == 0) & (cv[:, 1, 0, -1] > 0))[0][:3]
    assert placed[first0].all()
    assert (lim["status"][~placed] == 2).all() and placed.sum() < (free["status"] == 1).sum()
    # without quotas the same call places more jobs; a generous quota changes nothing
    big = oracle.schedule_round(jobs, cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                cfg["n_nodes"], quota=np.array([[10**6, 10**6]] * 2), **kw)
    for k in ("g", "c", "plan", "status", "first_node"):
        assert np.array_equal(big[k], free[k])


# ---------------------------------------------------------------- single- against double-precision decisions
def double_tables(cfg, nthreads=4):
    """The oracle's chain without any rounding to single precision."""
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    cv, cp, cg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], len(cfg["m_levels"]), prefix=True, nthreads=nthreads)
    return plans, feas, cv, cp, cg


def test_candidate_dump_reproduces_every_decision_of_a_round(paper_scale):
    """The dump of what every job offered is the arbiter of the near-tie checks below: replaying the rule on it
    must give the logged decision at every step of a round, and nothing after the last one."""
    import near_tie
    cfg = paper_scale
    tb = tables(cfg)
    full = run_round(cfg, tb, want_log=True)
    assert full["steps"] > 20
    for k in range(full["steps"] + 1):
        r = run_round(cfg, tb, max_steps=k, want_log=True, want_candidates=True)
        assert r["steps"] == k and np.array_equal(r["log"], full["log"][:k])
        pick = near_tie.oracle_pick(r["cand"])
        assert pick == (near_tie.decode(full["log"][k])[:2] if k < full["steps"] else None)
        c = r["cand"]
        has = c["next"] >= 0
        # the gain is the weighted rise per unit, to single-precision rounding
        w = np.asarray(cfg["jobs"]["w"])[:, None]
        rise = (w * (c["v_next"] - c["v_cur"]))[has] / c["units"][has]
        assert np.allclose(c["gain"][has], rise, rtol=0, atol=float((1e-6 * w * (c["v_next"] + c["v_cur"]))[has].max()))


@pytest.mark.parametrize("name,J,N", [("tiny", None, None), ("paper-scale", None, None), ("cluster-512", 1024, 64),
                                      ("events", 800, 64), ("throughput-stress", 2000, 64)])
def test_single_precision_decisions_part_from_double_only_at_a_near_tie(name, J, N):
    """The round decides in single precision on the curve table rounded to single precision (so that a GPU
    kernel can follow it bit for bit); the method itself is stated in real numbers.  Deciding in double
    precision on the unrounded table must give the same step log up to the first decision whose margin is
    within the single-precision rounding of its gains; without such a near tie, the same round altogether."""
    import near_tie
    cfg = workloads.make(name, J=J, n_nodes=N)
    plans, feas, cv, cp, cg = double_tables(cfg, nthreads=8)
    args = (cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], cfg["n_nodes"])
    single = oracle.schedule_round(*args, want_log=True)
    double = oracle.schedule_round(*args, want_log=True, double_decisions=True)
    found = near_tie.assert_divergence_is_a_near_tie(
        lambda k: oracle.schedule_round(*args, max_steps=k, want_log=True, double_decisions=True, want_candidates=True),
        double["log"], single["log"], cfg["jobs"]["w"], tol=2.0 ** -24)
    if found is None:
        for key in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "node"):
            assert np.array_equal(single[key], double[key]), key
        assert np.allclose(single["thr"], double["thr"], rtol=2.0 ** -23, atol=0)
    w = np.asarray(cfg["jobs"]["w"], dtype=np.float64)
    assert float((w * single["thr"]).sum()) == pytest.approx(float((w * double["thr"]).sum()), rel=1e-4)


def test_near_tie_check_refuses_a_planted_mistake():
    """The check must not pass whatever it is given: a second chain that reads a table off by a tenth of a percent
    for some jobs (a planted mistake, far outside rounding) parts from the oracle at a decision with a clear margin."""
    import near_tie
    cfg = workloads.make("cluster-512", J=600, n_nodes=48)
    plans, feas, cv, cp, cg = double_tables(cfg, nthreads=8)
    args = lambda table: (cfg["jobs"], cfg["env"], table, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], cfg["n_nodes"])
    good = oracle.schedule_round(*args(cv), want_log=True, double_decisions=True)
    rng = np.random.default_rng(11)
    refused = 0
    for trial in range(6):
        bad_table = cv * (1.0 + 1e-3 * rng.uniform(-1.0, 1.0, (cv.shape[0], 1, 1, 1)))
        bad = oracle.schedule_round(*args(bad_table), want_log=True, double_decisions=True)
        if near_tie.first_difference(good["log"], bad["log"]) is None:
            continue
        try:
            near_tie.assert_divergence_is_a_near_tie(
                lambda k: oracle.schedule_round(*args(cv), max_steps=k, want_log=True, double_decisions=True, want_candidates=True),
                good["log"], bad["log"], cfg["jobs"]["w"], tol=2.0 ** -24)
        except AssertionError:
            refused += 1
    assert refused >= 5
