"""Pins of spread placement in the oracle (paper Section 4.1: groups whose GPUs sit on several nodes talk at the
inter-node bandwidth; Section 5.2 / Algorithm 1: a job's placement is a list of per-node allocations found node by
node, and the plan is chosen for the placement found).

The paper fixes neither the piece size nor the rank layout of a job that sits on several nodes in part; the
reading here (pieces of `a` GPUs, tensor-parallel groups inside a piece, data-parallel groups inside a piece only
when d * t divides it, pipeline traffic across nodes) is this project's: "parity unpinned by the paper", pinned by
hand numbers of the bandwidth classes, by the reduction to the packed round and by packing invariants."""
import numpy as np
import pytest

import oracle
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import workloads


def spread_env(a, **kw):
    return env(spread_align=a, **kw)


def test_which_plans_may_be_spread():
    job = one_job(b=64, h=2048, l=24)
    ok = lambda plan, a: oracle.terms(job, 0, spread_env(a), plan, 8)["valid"] == 1.0
    assert ok((4, 1, 1, 0, 0, 0), 2) and ok((2, 2, 1, 0, 0, 0), 2) and ok((1, 2, 2, 0, 0, 0), 2)
    assert not ok((1, 4, 1, 0, 0, 0), 2)                # a tensor-parallel group of 4 would straddle pieces of 2
    assert ok((2, 4, 1, 0, 0, 0), 4) and not ok((1, 8, 1, 0, 0, 0), 4)
    assert not ok((2, 1, 1, 0, 0, 0), 2)                # 2 GPUs in pieces of 2 is one piece: nothing to spread
    assert not ok((4, 1, 1, 0, 0, 0), 4) and not ok((2, 1, 1, 0, 0, 0), 4)
    assert not ok((3, 1, 1, 0, 0, 0), 2)                # 3 GPUs are not a whole number of pieces of 2
    assert not ok((16, 1, 1, 0, 0, 0), 2)               # more than a node: whole nodes, never spread
    assert ok((8, 1, 1, 0, 0, 0), 1) and ok((2, 1, 4, 0, 0, 0), 1) and not ok((4, 2, 1, 0, 0, 0), 1)


def test_bandwidth_classes_of_a_spread_job_by_hand():
    """e = 2 bytes, P = 1e9: V_dp of d = 4 is 2 * 1e9 * 2 * 3 / 4 = 3e9 bytes: 7.5 ms at 400 GB/s inside a node,
    30 ms at 100 GB/s between nodes."""
    job = one_job()
    packed = oracle.terms(job, 0, env(), (4, 1, 1, 0, 0, 0), 8)
    spread = oracle.terms(job, 0, spread_env(2), (4, 1, 1, 0, 0, 0), 8)
    assert packed["T_dp"] == pytest.approx(7.5e-3, rel=1e-12) and spread["T_dp"] == pytest.approx(3e-2, rel=1e-12)
    assert spread["V_dp"] == packed["V_dp"] and spread["T_fwd"] == packed["T_fwd"]
    # d * t = 2 divides the piece: the data-parallel ring stays inside it, only the pipeline crosses nodes
    packed = oracle.terms(job, 0, env(), (2, 1, 2, 0, 0, 0), 8)
    spread = oracle.terms(job, 0, spread_env(2), (2, 1, 2, 0, 0, 0), 8)
    assert spread["T_dp"] == packed["T_dp"] and spread["T_pp"] == pytest.approx(4 * packed["T_pp"], rel=1e-12)
    # tensor parallelism never leaves a piece
    packed = oracle.terms(job, 0, env(), (1, 2, 2, 0, 0, 0), 8)
    spread = oracle.terms(job, 0, spread_env(2), (1, 2, 2, 0, 0, 0), 8)
    assert spread["T_tp"] == packed["T_tp"] and spread["T_pp"] == pytest.approx(4 * packed["T_pp"], rel=1e-12)
    # with equal bandwidths inside and between nodes spreading costs nothing
    flat = dict(B_intra=100e9, B_inter=100e9)
    assert oracle.terms(job, 0, env(**flat), (4, 1, 1, 0, 0, 0), 8)["thr"] == oracle.terms(job, 0, spread_env(2, **flat), (4, 1, 1, 0, 0, 0), 8)["thr"]


def test_spreading_never_predicts_more_than_packing(paper_scale):
    cfg = paper_scale
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    packed, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=4)
    for a in (1, 2, 4):
        e = dict(cfg["env"], spread_align=a)
        thr, fs = oracle.eval_candidates(cfg["jobs"], plans, e, cfg["c_levels"], cfg["m_levels"], nthreads=4)
        on = thr > 0
        assert on.any() and np.all(packed[on] > 0)
        assert np.all(thr[on] < packed[on])              # some group always leaves its piece
        g = plans[:, 0] * plans[:, 1] * plans[:, 2]
        may = (g <= 8) & (g > a) & (g % a == 0) & (a % plans[:, 1] == 0)
        assert not thr[:, :, ~may].any() and not fs[:, ~may].any()
        assert np.array_equal(fs[:, may] != 0, (feas[:, may] != 0) & (thr[:, 0, may] > 0))      # memory needs are those of the packed job


def odd_sized_cluster(name, J, N, seed=3):
    """GPU levels that are not all powers of two (jobs of 3, 5 or 6 GPUs leave nodes partly free in ways powers of
    two never do) with plans of any degrees, and job shapes such degrees divide."""
    cfg = workloads.make(name, J=J, n_nodes=N)
    rng = np.random.default_rng(seed)
    cfg["g_levels"] = np.array([1, 2, 3, 4, 5, 6, 8, 16])
    cfg["jobs"]["h"] = rng.choice([768, 1536, 3072, 1280, 2560, 1920, 1024], J)
    cfg["jobs"]["b"] = rng.choice([48, 96, 24, 64, 30, 120], J)
    cfg["jobs"]["gmin_idx"] = np.where(rng.uniform(size=J) < 0.3, rng.integers(0, 6, J), -1)
    cfg["jobs"]["cmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, 0, -1)
    cfg["any_degrees"] = True
    return cfg


def class_tables(cfg, a, nthreads=4):
    plans, _ = oracle.enumerate_plans(cfg["g_levels"], any_degrees=bool(cfg.get("any_degrees", False)))
    e = dict(cfg["env"], spread_align=a)
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, e, cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    cv, cp, cg = oracle.best_plan(thr.astype(np.float32), feas, plans, cfg["g_levels"], len(cfg["m_levels"]), prefix=True, nthreads=nthreads)
    return plans, feas, cv.astype(np.float32), cp, cg


def packing_holds(cfg, r, aligns, n_nodes):
    """Every node's free amounts are what the assignments (whole jobs, whole-node sets and pieces) leave."""
    e = cfg["env"]
    Gn, Cn, Mn = e["gpus_per_node"], e["cpus_per_node"], e["mem_per_node_bytes"]
    used = np.zeros((n_nodes, 3), dtype=np.int64)
    for j in np.nonzero(r["status"] == 1)[0]:
        g, c, m, k, n0 = (int(r[x][j]) for x in ("g", "c", "m_bytes", "n_nodes", "first_node"))
        if r["cls"][j] >= 0:
            a = aligns[r["cls"][j]]
            pcs = [(int(x) >> 8, int(x) & 255) for x in r["pieces"][j] if x >= 0]
            assert len(pcs) == k >= 2 and sum(q for _, q in pcs) == g <= Gn and all(q % a == 0 for _, q in pcs)
            assert [n for n, _ in pcs] == sorted(n for n, _ in pcs) and pcs[0][0] == n0
            cpp, mpp = -(-c * a // g), -(-m * a // g)
            for n, q in pcs:
                used[n] += (q, q // a * cpp, q // a * mpp)
        elif k == 1:
            used[n0] += (g, c, m)
        else:
            own = np.nonzero(r["node"][:, 3] == j)[0]
            assert len(own) == k
            used[own] += (Gn, -(-c // k), -(-m // k))
    assert np.all(used <= np.array([Gn, Cn, Mn]))
    assert np.array_equal(r["node"][:, 0], Gn - used[:, 0]) and np.array_equal(r["node"][:, 1], Cn - used[:, 1])
    assert np.array_equal(r["node"][:, 2], Mn - used[:, 2])


@pytest.mark.parametrize("name,J,N", [("paper-scale", 64, 6), ("cluster-512", 300, 14), ("events", 200, 12)])
def test_round_with_spread_classes_packs_consistently_and_uses_them(name, J, N):
    cfg = odd_sized_cluster(name, J, N)
    plans, feas, cv, cp, cg = class_tables(cfg, 0)
    aligns = [4, 2, 1]
    spread = []
    for a in aligns:
        _, fs, v, p_, g_ = class_tables(cfg, a)
        spread.append((a, v, p_, g_, fs))
    args = (cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], N)
    plain = oracle.schedule_round(*args, want_log=True)
    r = oracle.schedule_round(*args, want_log=True, spread=spread)
    packing_holds(cfg, r, aligns, N)
    sp = r["cls"] >= 0
    assert sp.sum() >= 1                                       # a crowded cluster: some job is assembled from pieces
    # a spread job runs a plan of its class: tensor-parallel groups inside a piece, the class's own prediction
    for j in np.nonzero(sp)[0]:
        a = aligns[r["cls"][j]]
        assert a % plans[r["plan"][j], 1] == 0
        gi = list(cfg["g_levels"]).index(r["g"][j]); ci = list(cfg["c_levels"]).index(r["c"][j])
        assert r["thr"][j] in spread[r["cls"][j]][1][j, gi, ci, int(r["m_level"][j]):]
    # the packed round leaves guaranteed jobs waiting or GPUs idle where pieces serve them
    assert (r["status"] == 1).sum() >= (plain["status"] == 1).sum() or r["node"][:, 0].sum() <= plain["node"][:, 0].sum()


def test_without_need_the_spread_round_is_the_packed_round(paper_scale):
    """Room for everybody on whole nodes: no job is ever assembled from pieces, and nothing else changes."""
    cfg = dict(paper_scale, n_nodes=600)
    plans, feas, cv, cp, cg = class_tables(cfg, 0)
    spread = [(a,) + tuple(class_tables(cfg, a)[i] for i in (2, 3, 4, 1)) for a in (4, 2, 1)]
    args = (cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], 600)
    plain = oracle.schedule_round(*args, want_log=True)
    r = oracle.schedule_round(*args, want_log=True, spread=spread)
    assert not (r["cls"] >= 0).any() and (plain["node"][:, 0] == 8).any()        # empty nodes are left over
    for key in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "node", "log"):
        assert np.array_equal(plain[key], r[key]), key


def test_a_job_assembled_from_two_half_free_nodes_by_hand():
    """Two nodes of 8 GPUs.  Jobs 0 and 1 are guaranteed 6 GPUs each and gain nothing beyond (one node each, 2 GPUs
    left on either).  Job 2, best effort, needs at least 4 GPUs to run at all; no node has 4 free.  Without spread
    classes it stays in the queue; with pieces of 2 it gets 2 + 2 on nodes 0 and 1, at the spread table's value,
    with cores and memory shared out evenly."""
    g_levels = np.array([1, 2, 4, 6, 8]); c_levels = np.array([4, 8]); m_levels = np.array([64, 128]) * GIB
    jobs = stack_jobs(one_job(gmin_idx=3, cmin_idx=0), one_job(gmin_idx=3, cmin_idx=0), one_job())
    J, nG, nC, nM, P = 3, 5, 2, 2, 8
    # curves (running maximum over GPUs, flat in cores and memory) with the plan and the GPU count they really use
    val = np.array([[1.0, 2.0, 3.5, 5.0, 5.0], [1.0, 2.0, 3.5, 5.0, 5.0], [0.0, 0.0, 3.5, 3.5, 3.5]], dtype=np.float32)
    plan = np.array([[0, 1, 2, 3, 3], [0, 1, 2, 3, 3], [-1, -1, 2, 2, 2]], dtype=np.int32)
    used = np.array([[1, 2, 4, 6, 6], [1, 2, 4, 6, 6], [0, 0, 4, 4, 4]], dtype=np.int32)
    full = lambda x: np.broadcast_to(x[:, :, None, None], (J, nG, nC, nM)).copy()
    cv, cp, cg = full(val), full(plan), full(used)
    feas = np.full((J, P), 0b11, dtype=np.uint32)
    # spread predictions for pieces of 2: three quarters of the packed value, for 4 GPUs and more
    sv, sp_, sg = full(val * np.float32(0.75)), full(plan), full(used)
    sv[:, :2] = 0; sp_[:, :2] = -1; sg[:, :2] = 0
    args = (jobs, env(), cv, cp, cg, feas, g_levels, c_levels, m_levels, 2)
    plain = oracle.schedule_round(*args, want_log=True)
    assert list(plain["g"]) == [6, 6, 0] and list(plain["first_node"]) == [0, 1, -1] and plain["steps"] == 0
    r = oracle.schedule_round(*args, want_log=True, spread=[(2, sv, sp_, sg, feas)])
    assert list(r["g"]) == [6, 6, 4] and list(r["cls"]) == [-1, -1, 0] and r["n_nodes"][2] == 2 and r["first_node"][2] == 0
    assert [int(x) for x in r["pieces"][2] if x >= 0] == [(0 << 8) | 2, (1 << 8) | 2]
    assert r["thr"][2] == np.float32(3.5 * 0.75) and r["plan"][2] == 2 and list(r["log"]) == [(2 << 2) | 1]
    # 4 cores in two pieces: 2 a piece; 64 GiB in two pieces: 32 GiB a piece; the guaranteed jobs hold 6 GPUs, 4 cores, 64 GiB each
    assert list(r["node"][:, 0]) == [0, 0] and list(r["node"][:, 1]) == [96 - 4 - 2, 96 - 4 - 2]
    assert list(r["node"][:, 2]) == [1024 * GIB - 64 * GIB - 32 * GIB] * 2
    # pieces of 4 cannot be found (2 free GPUs a node): the job stays in the queue
    none = oracle.schedule_round(*args, want_log=True, spread=[(4, sv, sp_, sg, feas)])
    assert list(none["g"]) == [6, 6, 0] and (none["cls"] < 0).all()
