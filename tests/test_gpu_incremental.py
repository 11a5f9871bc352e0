"""rubick_incremental_round against the oracle's incremental round: same previous state, same tables,
bit-exact allocations, node states and step logs (integer and single-precision work only)."""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, assert_rounds_equal, has_cuda, incremental_on_tables
from helpers import GIB, env, one_job, stack_jobs
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads
from test_oracle_incremental import event_config, preemption_frees_cores_case, random_events
from test_oracle_sched import concave_instance, tables

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def both(gpu, cfg, tb, prev, **kw):
    plans, feas, cv, cp, cg = tb
    want = oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                             cfg["m_levels"], cfg["n_nodes"], prev, want_log=True, **kw)
    got = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], prev, **kw)
    return want, got


@pytest.mark.parametrize("seed", range(4))
def test_event_sequences_are_bit_exact(seed):
    """Arrivals, completions, pinned jobs, guaranteed minima, exchanges and preemptions over eight rounds;
    every round starts from the oracle's previous result on both sides."""
    cfg, rng = event_config(seed)
    tb = tables(cfg)
    gpu = Gpu(cfg)
    plans, feas, cv, cp, cg = tb
    exchanges = 0
    for inp, want in random_events(cfg, tb, 8, rng):
        got = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], inp["prev"], active=inp["active"],
                                    T=inp["T"], delta=inp["delta"], nrec=inp["nrec"])
        assert_rounds_equal(got, want)
        bulk = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], inp["prev"], active=inp["active"],
                                     T=inp["T"], delta=inp["delta"], nrec=inp["nrec"], want_log=False)
        assert_rounds_equal(bulk, want)                  # no log: hopeless candidates frozen in bulk, same result and count
        exchanges += int((((want["log"] >> 2) & 1) & (want["log"] & 1)).sum())
    if seed >= 2:
        assert exchanges > 0


@pytest.mark.parametrize("name,J,N,rounds", [("cluster-512", 320, 20, 6), ("paper-scale", 64, 2, 10)])
def test_larger_event_sequences_with_quotas_are_bit_exact(name, J, N, rounds):
    cfg, rng = event_config(11, name=name, J=J, n_nodes=N)
    cfg["jobs"]["tenant"] = rng.integers(0, 3, J)
    quota = np.array([[N * 3, N * 40], [N * 2, N * 30], [N, N * 10]])
    tb = tables(cfg, nthreads=8)
    gpu = Gpu(cfg)
    plans, feas, cv, cp, cg = tb
    active = np.zeros(J, dtype=np.int32)
    prev = None
    T = np.zeros(J, dtype=np.float32)
    nrec = rng.integers(0, 2, J).astype(np.int32)
    delta = rng.uniform(5.0, 60.0, J).astype(np.float32)
    seen_exchange = seen_pending = False
    for rnd in range(rounds):
        arrive = rng.uniform(size=J) < (0.08 if rnd == 0 else 0.2)
        leave = (rng.uniform(size=J) < 0.1) & (active == 1)
        active = np.where(leave, 0, np.where(arrive, 1, active)).astype(np.int32)
        if prev is not None:
            T = np.where((prev["status"] == 1) & (active == 1), T + rng.uniform(100.0, 5000.0, J), 0).astype(np.float32)
        kw = dict(active=active, T=T, delta=delta, nrec=nrec, quota=quota)
        want = oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                                 cfg["m_levels"], N, prev, want_log=True, **kw)
        got = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, N, prev, **kw)
        assert want["steps"] is not None
        assert_rounds_equal(got, want)
        assert_rounds_equal(incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, N, prev, want_log=False, **kw), want)
        seen_exchange |= bool((((want["log"] >> 2) & 1) & (want["log"] & 1)).any())
        seen_pending |= bool((want["status"] == 2).any())
        prev = want
    assert seen_exchange


def test_small_nodes_and_few_levels_are_bit_exact():
    """4-GPU nodes, three core levels, two memory levels: other list lengths, more preemptions."""
    cfg = workloads.make("paper-scale", J=48, n_nodes=5)
    cfg["env"] = env(gpus_per_node=4, cpus_per_node=24, mem_per_node_bytes=256 * GIB)
    cfg["g_levels"] = np.array([1, 2, 4, 8, 16])
    cfg["c_levels"] = np.array([2, 6, 12])
    cfg["m_levels"] = np.array([64, 192]) * GIB
    rng = np.random.default_rng(77)
    cfg["jobs"]["gmin_idx"] = np.where(rng.uniform(size=48) < 0.3, rng.integers(0, 2, 48), -1)
    cfg["jobs"]["cmin_idx"] = np.where(cfg["jobs"]["gmin_idx"] >= 0, 0, -1)
    tb = tables(cfg, nthreads=8)
    gpu = Gpu(cfg)
    plans, feas, cv, cp, cg = tb
    prev = None
    active = np.zeros(48, dtype=np.int32)
    for rnd in range(8):
        active = np.where(rng.uniform(size=48) < 0.12, 0, np.where(rng.uniform(size=48) < 0.3, 1, active)).astype(np.int32)
        T = rng.uniform(0.0, 3000.0, 48).astype(np.float32)
        kw = dict(active=active, T=T, delta=np.full(48, 20.0, np.float32), nrec=rng.integers(0, 3, 48))
        want = oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                                 cfg["m_levels"], 5, prev, want_log=True, **kw)
        got = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, 5, prev, **kw)
        assert_rounds_equal(got, want)
        assert_rounds_equal(incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, 5, prev, want_log=False, **kw), want)
        for cap in (3, 7, 15):                           # the step cap falls inside a run of bulk-frozen candidates
            kc = dict(kw, max_steps=cap)
            wc = oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                                   cfg["m_levels"], 5, prev, want_log=True, **kc)
            gc_ = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, 5, prev, want_log=False, **kc)
            assert gc_["steps"] == wc["steps"] and gc_["capped"] == wc["capped"]
            if not wc["capped"]:
                assert_rounds_equal(gc_, wc)
        prev = want


def test_from_an_empty_cluster_and_with_quotas():
    cfg = workloads.make("paper-scale")
    J = 64
    jobs = cfg["jobs"]
    jobs["gmin_idx"] = np.where(np.arange(J) % 3 == 0, 1, -1)
    jobs["cmin_idx"] = np.where(np.arange(J) % 3 == 0, 0, -1)
    jobs["tenant"] = np.arange(J) % 2
    tb = tables(cfg)
    gpu = Gpu(cfg)
    want, got = both(gpu, cfg, tb, None)
    assert_rounds_equal(got, want)
    quota = np.array([[6, 12], [64, 8]])
    want_q, got_q = both(gpu, cfg, tb, None, quota=quota)
    assert_rounds_equal(got_q, want_q)
    assert (want_q["status"] == 2).any()
    # second round on the first one's result: queued guaranteed jobs push in by exchange once the quota is lifted
    want2, got2 = both(gpu, cfg, tb, want_q)
    assert_rounds_equal(got2, want2)


@pytest.mark.parametrize("seed", range(4))
def test_concave_exchanges_are_bit_exact(seed):
    jobs, cv, cp, cg, feas = concave_instance(seed)
    gl, cl, ml = np.arange(1, 9), np.array([4]), np.array([GIB])
    cfg = dict(jobs=jobs, env=env(cpus_per_node=64), g_levels=gl, c_levels=cl, m_levels=ml, n_nodes=1)
    plans, _ = rb.enumerate_plans(gl)
    gpu = Gpu(cfg, plans=plans)
    J = 4
    hog = seed % J
    prev = dict(g=np.zeros(J, np.int64), c=np.zeros(J, np.int64), m_bytes=np.zeros(J, np.int64), plan=np.full(J, -1),
                first_node=np.full(J, -1), n_nodes=np.zeros(J, np.int64), status=np.zeros(J, np.int64),
                m_level=np.full(J, -1), thr=np.zeros(J, np.float32), node=np.array([[0, 60, 0, -1]]))
    prev["g"][hog], prev["c"][hog], prev["m_bytes"][hog], prev["plan"][hog] = 8, 4, GIB, 0
    prev["first_node"][hog], prev["n_nodes"][hog], prev["status"][hog], prev["m_level"][hog] = 0, 1, 1, 0
    prev["thr"][hog] = cv[hog, 7, 0, 0]
    feas_full = np.zeros((J, gpu.P), dtype=np.uint32)
    feas_full[:, 0] = 1
    tb = (None, feas_full, cv, cp, cg)
    want, got = both(gpu, cfg, tb, prev)
    assert_rounds_equal(got, want)
    assert ((want["log"] >> 2) & 1).all() and (want["log"] & 1).any()


def test_multi_node_jobs_are_carried_over_and_never_shrunk():
    cfg = workloads.make("cluster-512", J=96, n_nodes=24)
    tb = tables(cfg, nthreads=8)
    gpu = Gpu(cfg)
    want, got = both(gpu, cfg, tb, None)
    assert_rounds_equal(got, want)
    assert (want["n_nodes"] > 1).any()
    J = 96
    rng = np.random.default_rng(5)
    active = (rng.uniform(size=J) < 0.8).astype(np.int32)
    prev = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in want.items()}
    prev["status"] = np.where(active == 1, prev["status"], 0)
    T = rng.uniform(0.0, 4000.0, J).astype(np.float32)
    delta = rng.uniform(5.0, 60.0, J).astype(np.float32)
    want2, got2 = both(gpu, cfg, tb, prev, active=active, T=T, delta=delta, nrec=rng.integers(0, 3, J))
    assert_rounds_equal(got2, want2)
    multi = (prev["n_nodes"] > 1) & (prev["status"] == 1)
    assert (want2["g"][multi] >= prev["g"][multi]).all()


def test_inconsistent_previous_state_is_refused():
    cfg = workloads.make("tiny")
    tb = tables(cfg)
    gpu = Gpu(cfg)
    want, got = both(gpu, cfg, tb, None)
    assert_rounds_equal(got, want)
    bad = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in want.items()}
    j = int(np.nonzero(want["status"] == 1)[0][0])
    bad["g"][j] = 1000
    plans, feas, cv, cp, cg = tb
    assert oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                             cfg["m_levels"], cfg["n_nodes"], bad)["steps"] is None
    with pytest.raises(rb.RubickError) as ei:
        incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], bad)
    assert ei.value.code == rb.ESTATE
    # the context stays usable
    again = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas, cfg["n_nodes"], want)
    want2 = oracle.schedule_round_incremental(cfg["jobs"], cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                              cfg["m_levels"], cfg["n_nodes"], want, want_log=True)
    assert_rounds_equal(again, want2)


def test_step_cap_and_argument_validation():
    cfg = workloads.make("paper-scale", J=32, n_nodes=2)
    tb = tables(cfg)
    gpu = Gpu(cfg)
    want, got = both(gpu, cfg, tb, None, max_steps=5)
    assert want["capped"] and got["capped"]
    assert_rounds_equal(got, want)
    t = gpu.torch
    d = gpu.empty(64, t.uint8)
    cl, _ = rb.make_cluster(2)
    import ctypes as C
    steps = C.c_int32(0)
    rc = rb.lib().rubick_incremental_round(gpu.ctx._h, rb._ptr(d), 1, rb._ptr(d), rb._ptr(d), rb._ptr(d), rb._ptr(d), C.byref(cl),
                                           rb._ptr(d), None, None, C.c_float(0.97), 10, rb._ptr(d), None, None, C.byref(steps))
    assert rc == rb.EINVAL                       # previous assignments without the previous node states


def test_events_with_state_kept_in_the_context_match_the_oracle():
    """rubick_incremental_event_host: slots, previous allocation and cached tables live in the context;
    only changed slots are uploaded and re-evaluated.  The oracle replays every event on the tables the
    library itself computes for the slots' current jobs."""
    cfg, rng = event_config(5, J=48, n_nodes=3)
    pool = workloads.make("paper-scale", J=200)["jobs"]               # jobs that arrive into the 48 slots
    gpu = Gpu(cfg)
    J, N = 48, 3
    slot_jobs = {k: np.asarray(v).copy() for k, v in cfg["jobs"].items()}
    records = rb.pack_jobs(slot_jobs)
    h_out = np.zeros(J, dtype=rb.ASSIGN_DTYPE)
    h_nodes = np.zeros(N, dtype=rb.NODE_DTYPE)
    reconf = np.zeros(J, dtype=rb.RECONF_DTYPE)
    reconf["delta"] = rng.uniform(5.0, 40.0, J)
    prev = None
    next_pool = 0
    for rnd in range(8):
        changed = []
        for s in range(J):
            if reconf["active"][s] and rng.uniform() < 0.12:
                reconf["active"][s] = 0                                   # finished
            elif not reconf["active"][s] and rng.uniform() < 0.25:
                for k in slot_jobs:                                       # a new job takes the slot
                    if k in pool:
                        slot_jobs[k][s] = pool[k][next_pool]
                slot_jobs["gmin_idx"][s] = int(rng.integers(0, 3)) if rng.uniform() < 0.4 else -1
                slot_jobs["cmin_idx"][s] = 0 if slot_jobs["gmin_idx"][s] >= 0 else -1
                next_pool += 1
                reconf["active"][s] = 1
                reconf["T"][s] = 0
                reconf["n_reconf"][s] = 0
                changed.append(s)
        records = rb.pack_jobs(slot_jobs)
        if prev is not None:
            running = (prev["status"] == 1) & (reconf["active"] == 1)
            reconf["T"] = np.where(running, reconf["T"] + rng.uniform(100.0, 4000.0, J), 0).astype(np.float32)
        steps, capped = gpu.ctx.incremental_event_host(records, J, N, h_out, changed=None if rnd == 0 else changed,
                                                       h_reconf=reconf, h_node_out=h_nodes)
        # the oracle on the library's own tables of the current slot jobs
        d_jobs, d_thr, d_feas = gpu.eval(slot_jobs)
        bv, bp, bg = gpu.best(d_thr, d_feas, J)
        sh = gpu.shape4(J)
        cv, cp, cg = bv.cpu().numpy().reshape(sh), bp.cpu().numpy().reshape(sh), bg.cpu().numpy().reshape(sh)
        feas = gpu.np_feas(d_feas, J)
        want = oracle.schedule_round_incremental(slot_jobs, cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                                                 cfg["m_levels"], N, prev, active=reconf["active"], T=reconf["T"],
                                                 delta=reconf["delta"], nrec=reconf["n_reconf"])
        assert want["steps"] == steps and not capped
        for k in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "m_level"):
            assert np.array_equal(h_out[k].astype(np.int64), want[k]), (rnd, k)
        assert np.array_equal(h_out["thr"].view(np.uint32), want["thr"].view(np.uint32))
        assert np.array_equal(np.stack([h_nodes["free_g"], h_nodes["free_c"], h_nodes["free_m"], h_nodes["owner"]], axis=1).astype(np.int64), want["node"])
        if prev is not None:
            was = (prev["status"] == 1) & (reconf["active"] == 1)
            moved = was & (want["status"] == 1) & ((want["g"] != prev["g"]) | (want["c"] != prev["c"]) | (want["plan"] != prev["plan"]))
            reconf["n_reconf"] += moved.astype(np.int32)
        prev = want


def test_degenerate_sizes():
    """No jobs, no active slot, one node, and the largest cluster the node state supports."""
    cfg = workloads.make("tiny")
    tb = tables(cfg)
    plans, feas, cv, cp, cg = tb
    gpu = Gpu(cfg)
    J = len(cfg["jobs"]["P"])
    none = np.zeros(J, dtype=np.int32)
    want, got = both(gpu, cfg, tb, None, active=none)
    assert_rounds_equal(got, want)
    assert want["steps"] == 0 and not want["g"].any()
    t = gpu.torch
    d_out = gpu.empty(64, t.uint8)
    steps, capped = gpu.ctx.incremental_round(None, 0, None, None, None, None, 3, 10, d_out)
    assert steps == 0 and not capped
    big = dict(cfg, n_nodes=4096)
    want, got = both(gpu, big, tb, None)
    assert_rounds_equal(got, want)
    again_w, again_g = both(gpu, big, tb, want, T=np.full(J, 1e6), delta=np.zeros(J), nrec=np.zeros(J))
    assert_rounds_equal(again_g, again_w)


def test_cores_freed_by_a_preemption_are_seen_with_and_without_a_step_log():
    cfg, tb, prev = preemption_frees_cores_case()
    plans, feas, cv, cp, cg = tb
    gpu_plans, _ = rb.enumerate_plans(cfg["g_levels"])
    gpu = Gpu(cfg, plans=gpu_plans)
    feas_full = np.zeros((2, gpu.P), dtype=np.uint32)
    feas_full[:, 0] = 1
    tb = (None, feas_full, cv, cp, cg)
    want, got = both(gpu, cfg, tb, prev)
    assert_rounds_equal(got, want)
    assert list(want["status"]) == [0, 1]
    bulk = incremental_on_tables(gpu, cfg["jobs"], cv, cp, cg, feas_full, 1, prev, want_log=False)
    assert_rounds_equal(bulk, want)
