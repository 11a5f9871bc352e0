"""Pins of the oracle's incremental round: Algorithm 1 with its shrink step, started from the
previous allocation, and the reconfiguration gate (paper Section 5.2).

The paper gives no worked example and calls the policy a heuristic, so the pins are reductions
to the grow-only round, fixed points, the exhaustive optimum on separable concave instances
(where an exchange argument proves that slope-ordered exchanges reach it), hand-made exchanges
and the invariants the text states (minimum demand kept, gate respected, preemption only of
best-effort jobs)."""
import numpy as np
import pytest

import oracle
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import workloads
from test_oracle_sched import check_invariants, concave_instance, tables


def incr(cfg, tb, prev, **kw):
    plans, feas, cv, cp, cg = tb
    return oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                             cfg["m_levels"], cfg["n_nodes"], prev, **kw)


def same_allocation(a, b):
    return all(np.array_equal(a[k], b[k]) for k in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "m_level")) \
        and np.array_equal(a["thr"], b["thr"]) and np.array_equal(a["node"], b["node"])


def test_from_an_empty_cluster_with_room_for_everyone_it_is_the_grow_only_round():
    """No exchange can happen when every increment fits free resources: same steps, same result."""
    cfg = workloads.make("paper-scale", J=24, n_nodes=64)
    tb = tables(cfg)
    plans, feas, cv, cp, cg = tb
    grow = oracle.schedule_round(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"],
                                 cfg["n_nodes"], want_log=True)
    r = incr(cfg, tb, None, want_log=True)
    assert same_allocation(r, grow)
    # every free-resource step of the grow-only log appears in order; the rest are failed exchanges
    free_steps = r["log"][((r["log"] >> 2) & 1) == 0]
    assert np.array_equal(((free_steps >> 3) << 2) | (free_steps & 3), grow["log"])
    assert not (r["log"][((r["log"] >> 2) & 1) == 1] & 1).any()


def test_a_fully_pinned_cluster_is_a_fixed_point(paper_scale):
    cfg = paper_scale
    tb = tables(cfg)
    first = incr(cfg, tb, None)
    check_invariants(cfg, tb, first)
    J = len(first["g"])
    again = incr(cfg, tb, first, T=np.zeros(J), want_log=True)          # T = 0: nobody passes the gate
    assert same_allocation(again, first)
    # queued jobs may still try (and fail) to get in; nothing that runs is touched
    assert not (again["log"] & 1).any()


def test_the_gate_counts_the_contemplated_reconfiguration():
    """(T - (N + 1) delta) / T > 0.97: with T = 100 s and delta = 1 s a job that has been
    reconfigured once passes (0.98) and one reconfigured twice does not (0.97 is not above 0.97)."""
    jobs, cv, cp, cg, feas = concave_instance(3, J=2)
    gl, cl, ml = np.arange(1, 9), np.array([4]), np.array([GIB])
    e = env(cpus_per_node=16)
    cfg = dict(jobs=jobs, env=e, g_levels=gl, c_levels=cl, m_levels=ml, n_nodes=1)
    tb = (None, feas, cv, cp, cg)
    start = incr(cfg, tb, None, max_steps=2)                            # one GPU each, six left free
    assert list(start["g"]) == [1, 1]
    T, d = np.array([100.0, 100.0]), np.array([1.0, 1.0])
    r = incr(cfg, tb, start, T=T, delta=d, nrec=np.array([1, 2]))
    assert r["g"][0] == 7 and r["g"][1] == 1                            # job 1 is pinned, job 0 takes the rest
    r = incr(cfg, tb, start, T=T, delta=d, nrec=np.array([2, 1]))
    assert r["g"][0] == 1 and r["g"][1] == 7
    r = incr(cfg, tb, start, T=np.array([0.0, 100.0]), delta=np.zeros(2), nrec=np.zeros(2))
    assert r["g"][0] == 1 and r["g"][1] == 7                            # T = 0: nothing trained yet, pinned


@pytest.mark.parametrize("seed", range(8))
def test_exchanges_reach_the_optimum_on_separable_concave_instances(seed):
    """One node, strictly concave curves in the GPU count, every GPU count valid.  Whatever the
    previous split, moving one GPU at a time from the lowest loss to the highest gain while the gain
    exceeds the loss ends in the optimum of the separable concave problem (exchange argument)."""
    jobs, cv, cp, cg, feas = concave_instance(seed)
    gl, cl, ml = np.arange(1, 9), np.array([4]), np.array([GIB])
    e = env(cpus_per_node=64)
    cfg = dict(jobs=jobs, env=e, g_levels=gl, c_levels=cl, m_levels=ml, n_nodes=1)
    tb = (None, feas, cv, cp, cg)
    best = oracle.bruteforce(jobs, e, cv, cp, cg, feas, gl, cl, ml)
    rng = np.random.default_rng(seed)
    # a deliberately bad previous allocation: the whole node to one random job
    J = 4
    hog = int(rng.integers(0, J))
    prev = dict(g=np.zeros(J, np.int64), c=np.zeros(J, np.int64), m_bytes=np.zeros(J, np.int64), plan=np.full(J, -1),
                first_node=np.full(J, -1), n_nodes=np.zeros(J, np.int64), status=np.zeros(J, np.int64),
                m_level=np.full(J, -1), thr=np.zeros(J, np.float32), node=np.array([[0, 60, 0, -1]]))
    prev["g"][hog], prev["c"][hog], prev["m_bytes"][hog], prev["plan"][hog] = 8, 4, GIB, 0
    prev["first_node"][hog], prev["n_nodes"][hog], prev["status"][hog], prev["m_level"][hog] = 0, 1, 1, 0
    prev["thr"][hog] = cv[hog, 7, 0, 0]
    r = incr(cfg, tb, prev, want_log=True)
    assert r["g"].sum() == 8
    assert float(r["thr"].astype(np.float64).sum()) == pytest.approx(best, rel=1e-6)
    assert ((r["log"] >> 2) & 1).all()                                   # nothing was free: every step an exchange


def test_hand_made_exchange_steps():
    """Two jobs on one 8-GPU node, curve values by hand.  Job 0 runs on all 8 GPUs (value 16, its
    next lower valid count is 4 with value 12: loss slope 1 per GPU).  Job 1 is queued; its first
    level is 2 GPUs with value 6 (gain 3 per GPU), then 4 GPUs with value 8 (gain 1 per GPU)."""
    cv = np.zeros((2, 4, 1, 1), dtype=np.float32)
    cg = np.zeros((2, 4, 1, 1), dtype=np.int32)
    cp = np.full((2, 4, 1, 1), -1, dtype=np.int32)
    gl, cl, ml = np.array([1, 2, 4, 8]), np.array([4]), np.array([GIB])
    # job 0: valid at 2 (value 7), 4 (12), 8 (16); the curve is flat below its first valid count
    cv[0, :, 0, 0] = [0, 7, 12, 16]; cg[0, :, 0, 0] = [0, 2, 4, 8]; cp[0, 1:, 0, 0] = 0
    cv[1, :, 0, 0] = [0, 6, 8, 8]; cg[1, :, 0, 0] = [0, 2, 4, 4]; cp[1, 1:, 0, 0] = 0
    feas = np.ones((2, 1), dtype=np.uint32)
    jobs = stack_jobs(one_job(host_base_bytes=0), one_job(host_base_bytes=0))
    e = env(cpus_per_node=8)
    cfg = dict(jobs=jobs, env=e, g_levels=gl, c_levels=cl, m_levels=ml, n_nodes=1)
    tb = (None, feas, cv, cp, cg)
    prev = dict(g=np.array([8, 0]), c=np.array([4, 0]), m_bytes=np.array([GIB, 0]), plan=np.array([0, -1]),
                first_node=np.array([0, -1]), n_nodes=np.array([1, 0]), status=np.array([1, 0]), m_level=np.array([0, -1]),
                thr=np.array([16, 0], np.float32), node=np.array([[0, 4, 0, -1]]))
    r = incr(cfg, tb, prev, want_log=True)
    # step 1: job 1 asks for 2 GPUs at gain 3 > loss 1: job 0 drops to 4 GPUs (frees 4), job 1 gets 2.
    # step 2: job 1 asks for 4 GPUs at gain (8 - 6) / 2 = 1; two GPUs are free: a plain increment.
    # job 0 was shrunk in this round and does not grow back.
    assert list(r["g"]) == [4, 4] and list(r["thr"]) == [12, 8]
    assert list(r["log"]) == [(1 << 3) | (1 << 2) | 1, (1 << 3) | 1]
    # with a loss above the gain nothing moves: make job 0's step down cost 3.5 per GPU
    cv2 = cv.copy(); cv2[0, :, 0, 0] = [0, 1, 2, 16]
    prev2 = dict(prev)
    r = incr(cfg, (None, feas, cv2, cp, cg), prev2, want_log=True)
    assert list(r["g"]) == [8, 0] and list(r["log"]) == [(1 << 3) | (1 << 2)]
    # a guaranteed queued job is placed at its minimum even at a loss (2 GPUs; job 0 drops to 4)
    jobs_g = stack_jobs(one_job(host_base_bytes=0), one_job(host_base_bytes=0, gmin_idx=1, cmin_idx=0))
    r = oracle.schedule_round_incremental(jobs_g, e, cv2, cp, cg, feas, gl, cl, ml, 1, prev2, want_log=True)
    assert r["status"][1] == 1 and r["g"][1] >= 2 and r["g"][0] == 4
    # a best-effort job without a lower valid count is preempted for it; a guaranteed one is not
    cv3 = cv2.copy(); cg3 = cg.copy(); cp3 = cp.copy()
    cv3[0, :, 0, 0] = [0, 0, 0, 16]; cg3[0, :, 0, 0] = [0, 0, 0, 8]; cp3[0, :3, 0, 0] = -1
    r = oracle.schedule_round_incremental(jobs_g, e, cv3, cp3, cg3, feas, gl, cl, ml, 1, prev2)
    assert r["status"][0] == 0 and r["g"][0] == 0 and r["status"][1] == 1
    jobs_gg = stack_jobs(one_job(host_base_bytes=0, gmin_idx=3, cmin_idx=0), one_job(host_base_bytes=0, gmin_idx=1, cmin_idx=0))
    r = oracle.schedule_round_incremental(jobs_gg, e, cv3, cp3, cg3, feas, gl, cl, ml, 1, prev2)
    assert r["status"][0] == 1 and r["g"][0] == 8 and r["status"][1] == 2


def random_events(cfg, tb, rounds, rng):
    """A sequence of incremental rounds with arrivals, completions and gate inputs; yields each round's
    inputs and result."""
    J = len(cfg["jobs"]["P"])
    active = np.zeros(J, dtype=np.int32)
    prev = None
    T = np.zeros(J, dtype=np.float32)
    nrec = np.zeros(J, dtype=np.int32)
    delta = rng.uniform(5.0, 60.0, J).astype(np.float32)
    for rnd in range(rounds):
        arrive = rng.uniform(size=J) < (0.1 if rnd == 0 else 0.25)        # few jobs first: they grow large, later arrivals reclaim
        leave = (rng.uniform(size=J) < 0.15) & (active == 1)
        active = np.where(leave, 0, np.where(arrive, 1, active)).astype(np.int32)
        if prev is not None:
            prev = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in prev.items()}
            gone = (active == 0) | leave
            prev["status"] = np.where(gone, 0, prev["status"])
            T = np.where(prev["status"] == 1, T + rng.uniform(100.0, 5000.0, J), 0).astype(np.float32)
            nrec = np.where(prev["status"] == 1, nrec, 0).astype(np.int32)
        r = incr(cfg, tb, prev, active=active, T=T, delta=delta, nrec=nrec, want_log=True)
        yield dict(prev=prev, active=active.copy(), T=T.copy(), delta=delta, nrec=nrec.copy()), r
        if prev is not None:
            was = prev["status"] == 1
            changed = was & (r["status"] == 1) & ((r["g"] != prev["g"]) | (r["c"] != prev["c"]) | (r["plan"] != prev["plan"]))
            nrec = nrec + changed.astype(np.int32)
        prev = r


def event_config(seed, name="paper-scale", J=40, n_nodes=3):
    cfg = workloads.make(name, J=J, n_nodes=n_nodes)
    rng = np.random.default_rng(40 + seed)
    cfg["jobs"]["gmin_idx"] = np.where(rng.uniform(size=J) < 0.4, rng.integers(0, 3, J), -1)
    cfg["jobs"]["cmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, rng.integers(0, 2, J), -1)
    return cfg, rng


def test_event_sequences_keep_the_stated_invariants():
    exchanges = 0
    for seed in range(4):
        exchanges += run_event_sequence(seed)
    assert exchanges >= 5                                # the sequences do exercise the exchange step


def run_event_sequence(seed):
    cfg, rng = event_config(seed)
    tb = tables(cfg)
    plans, feas, cv, cp, cg = tb
    gl, cl = list(cfg["g_levels"]), list(cfg["c_levels"])
    exchanges = preemptions = 0
    for inp, r in random_events(cfg, tb, 8, rng):
        assert r["steps"] is not None and not r["capped"]
        check_invariants(cfg, tb, r)
        assert not r["g"][inp["active"] == 0].any()
        prev = inp["prev"]
        exchanges += int((((r["log"] >> 2) & 1) & (r["log"] & 1)).sum())
        if prev is None:
            continue
        was = prev["status"] == 1
        t = inp["T"]
        gate = (t > 0) & ((t - (inp["nrec"] + 1).astype(np.float32) * inp["delta"]) / np.where(t > 0, t, 1) > np.float32(0.97))
        for j in np.nonzero(was)[0]:
            if not gate[j]:                              # pinned: carried over untouched
                assert all(r[k][j] == prev[k][j] for k in ("g", "c", "m_bytes", "plan", "first_node", "status"))
                continue
            gmin, cmin = int(cfg["jobs"]["gmin_idx"][j]), max(int(cfg["jobs"]["cmin_idx"][j]), 0)
            if gmin >= 0 and cp[j, gmin, cmin, -1] >= 0:
                # a guaranteed job that ran keeps at least its minimum demand (it is never preempted)
                assert r["status"][j] == 1
                assert r["g"][j] >= min(int(cg[j, gmin, cmin, -1]), int(prev["g"][j]))
                assert r["c"][j] >= min(cl[cmin], int(prev["c"][j]))
            elif r["status"][j] != 1:
                preemptions += 1
                assert gmin < 0 or cp[j, gmin, cmin, -1] < 0
    return exchanges


def test_inconsistent_previous_state_is_refused(tiny):
    tb = tables(tiny)
    first = incr(tiny, tb, None)
    bad = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in first.items()}
    j = int(np.nonzero(first["status"] == 1)[0][0])
    bad["g"][j] = 3 if 3 not in tiny["g_levels"] else 1000            # not a GPU level of the grid
    assert incr(tiny, tb, bad)["steps"] is None
    bad = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in first.items()}
    bad["c"][:] = np.where(first["status"] == 1, 32, 0)                # more cores than the node has
    bad["status"][:] = first["status"]
    if (first["status"] == 1).sum() * 32 > tiny["env"]["cpus_per_node"]:
        assert incr(tiny, tb, bad)["steps"] is None


def preemption_frees_cores_case():
    """One node with 8 GPUs and 8 cores, all held by best-effort job 0, which runs on 8 GPUs only (value 8
    with 8 cores, 2 with 4).  Queued job 1 wants 2 GPUs and 4 cores for a value of 6: 3 per GPU, 1.5 per core."""
    cv = np.zeros((2, 4, 2, 1), dtype=np.float32)
    cg = np.zeros((2, 4, 2, 1), dtype=np.int32)
    cp = np.full((2, 4, 2, 1), -1, dtype=np.int32)
    gl, cl, ml = np.array([1, 2, 4, 8]), np.array([4, 8]), np.array([GIB])
    cv[0, 3, :, 0] = [2, 8]; cg[0, 3, :, 0] = 8; cp[0, 3, :, 0] = 0
    cv[1, 1:, :, 0] = 6; cg[1, 1:, :, 0] = 2; cp[1, 1:, :, 0] = 0
    feas = np.ones((2, 1), dtype=np.uint32)
    jobs = stack_jobs(one_job(host_base_bytes=0), one_job(host_base_bytes=0))
    cfg = dict(jobs=jobs, env=env(cpus_per_node=8), g_levels=gl, c_levels=cl, m_levels=ml, n_nodes=1)
    prev = dict(g=np.array([8, 0]), c=np.array([8, 0]), m_bytes=np.array([GIB, 0]), plan=np.array([0, -1]),
                first_node=np.array([0, -1]), n_nodes=np.array([1, 0]), status=np.array([1, 0]), m_level=np.array([0, -1]),
                thr=np.array([8, 0], np.float32), node=np.array([[0, 0, 0, -1]]))
    return cfg, (None, feas, cv, cp, cg), prev


def test_a_preemption_in_the_gpu_phase_frees_the_cores_the_newcomer_needs():
    """Job 0's cores cost 1.5 each, not below the newcomer's 1.5 per core, so cores alone could not be taken;
    but its GPUs cost 1 each against a gain of 3, it has no smaller GPU count, so it is preempted, and its
    cores come free with it."""
    cfg, tb, prev = preemption_frees_cores_case()
    r = incr(cfg, tb, prev, want_log=True)
    assert list(r["status"]) == [0, 1] and list(r["g"]) == [0, 2] and list(r["c"]) == [0, 4]
    assert r["log"][0] == (1 << 3) | (1 << 2) | 1
