"""Glue for the GPU parity tests: builds a context for a workload and moves arrays across."""
import numpy as np

from paper_2408_08586_b200 import binding as rb


def has_cuda():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


class Gpu:
    """A context with the workload's plan space installed, plus typed device-buffer helpers."""

    def __init__(self, cfg, env=None, plans=None):
        import torch
        self.torch = torch
        self.cfg = cfg
        self.ctx = rb.Context(env or cfg["env"], device=0)
        if plans is None:
            plans, self.group_off = rb.enumerate_plans(cfg["g_levels"])
        self.plans = plans
        self.ctx.set_space(plans, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
        self.P, self.nG, self.nC, self.nM = len(plans), len(cfg["g_levels"]), len(cfg["c_levels"]), len(cfg["m_levels"])

    def empty(self, n, dtype):
        return self.torch.empty(int(n), dtype=dtype, device="cuda:0")

    def jobs_to_device(self, jobs):
        return rb.to_device(rb.pack_jobs(jobs))

    def eval(self, jobs):
        t = self.torch
        J = len(jobs["P"])
        d_jobs = self.jobs_to_device(jobs)
        d_thr = self.empty(J * self.nC * self.P, t.float32)
        d_feas = self.empty(J * self.P, t.int32)
        self.ctx.eval_candidates(d_jobs, J, d_thr, d_feas)
        self.ctx.sync()
        return d_jobs, d_thr, d_feas

    def best(self, d_thr, d_feas, J, flags=0):
        t = self.torch
        n = J * self.nG * self.nC * self.nM
        bv, bp, bg = self.empty(n, t.float32), self.empty(n, t.int32), self.empty(n, t.int32)
        self.ctx.best_plan(d_thr, d_feas, J, bv, bp, bg, flags=flags)
        self.ctx.sync()
        return bv, bp, bg

    def assert_one_pass_curves_match(self, jobs):
        """rubick_curves against rubick_eval_candidates + rubick_best_plan on the same jobs: bit-identical."""
        t = self.torch
        J = len(jobs["P"])
        d_jobs, d_thr, d_feas = self.eval(jobs)
        n = J * self.nG * self.nC * self.nM
        for flags in (0, rb.BEST_RAW):
            bv, bp, bg = self.best(d_thr, d_feas, J, flags=flags)
            f2 = self.empty(J * self.P, t.int32)
            cv, cp, cg = self.empty(n, t.float32), self.empty(n, t.int32), self.empty(n, t.int32)
            self.ctx.curves(d_jobs, J, f2, cv, cp, cg, flags=flags)
            self.ctx.sync()
            assert t.equal(f2, d_feas)
            assert t.equal(cv.view(t.int32), bv.view(t.int32)) and t.equal(cp, bp) and t.equal(cg, bg)

    def shape4(self, J):
        return (J, self.nG, self.nC, self.nM)

    def np_thr(self, d_thr, J):
        return d_thr.cpu().numpy().reshape(J, self.nC, self.P)

    def np_feas(self, d_feas, J):
        return d_feas.cpu().numpy().view(np.uint32).reshape(J, self.P)

    def round_on_tables(self, jobs, cv, cp, cg, feas, n_nodes, max_steps=1 << 30, want_log=True, quota=None):
        """rubick_greedy_round on host-provided tables -> dict like the oracle's."""
        t = self.torch
        J = len(jobs["P"])
        d_jobs = self.jobs_to_device(jobs)
        d_cv = t.from_numpy(np.ascontiguousarray(cv, dtype=np.float32).reshape(-1)).cuda()
        d_cp = t.from_numpy(np.ascontiguousarray(cp, dtype=np.int32).reshape(-1)).cuda()
        d_cg = t.from_numpy(np.ascontiguousarray(cg, dtype=np.int32).reshape(-1)).cuda()
        d_feas = t.from_numpy(np.ascontiguousarray(feas, dtype=np.uint32).view(np.int32).reshape(-1)).cuda()
        cap = int(min(max_steps, J * (self.nG + self.nC + 2) + 1))
        d_out = self.empty(max(J, 1) * rb.ASSIGN_DTYPE.itemsize, t.uint8)
        d_node = self.empty(n_nodes * rb.NODE_DTYPE.itemsize, t.uint8)
        d_log = self.empty(max(cap, 1), t.int32) if want_log else None
        steps, capped = self.ctx.greedy_round(d_jobs, J, d_cv, d_cp, d_cg, d_feas, n_nodes, cap, d_out, d_node, d_log, quota=quota)
        return unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE)[:J], rb.from_device(d_node, rb.NODE_DTYPE), steps, capped,
                            d_log.cpu().numpy()[:steps] if want_log else None)


def pack_prev(prev, J, n_nodes):
    """The dict a round returned -> (ASSIGN_DTYPE records, NODE_DTYPE records)."""
    a = np.zeros(max(J, 1), dtype=rb.ASSIGN_DTYPE)
    for k in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "m_level", "thr"):
        a[k][:J] = np.asarray(prev[k])
    nd = np.zeros(n_nodes, dtype=rb.NODE_DTYPE)
    node = np.asarray(prev["node"])
    nd["free_g"], nd["free_c"], nd["free_m"], nd["owner"] = node[:, 0], node[:, 1], node[:, 2], node[:, 3]
    return a, nd


def incremental_on_tables(gpu, jobs, cv, cp, cg, feas, n_nodes, prev, active=None, T=None, delta=None, nrec=None,
                          theta=0.97, max_steps=1 << 30, quota=None, want_log=True):
    """rubick_incremental_round on host-provided tables and previous state -> dict like the oracle's.
    Without a step log the library sorts out hopeless exchange candidates in bulk (another code path,
    same allocation and step count)."""
    t = gpu.torch
    J = len(jobs["P"])
    d_jobs = gpu.jobs_to_device(jobs)
    d_cv = t.from_numpy(np.ascontiguousarray(cv, dtype=np.float32).reshape(-1)).cuda()
    d_cp = t.from_numpy(np.ascontiguousarray(cp, dtype=np.int32).reshape(-1)).cuda()
    d_cg = t.from_numpy(np.ascontiguousarray(cg, dtype=np.int32).reshape(-1)).cuda()
    d_feas = t.from_numpy(np.ascontiguousarray(feas, dtype=np.uint32).view(np.int32).reshape(-1)).cuda()
    cap = int(min(max_steps, 2 * J * (gpu.nG + gpu.nC + 2) + 1))
    d_out = gpu.empty(max(J, 1) * rb.ASSIGN_DTYPE.itemsize, t.uint8)
    d_node = gpu.empty(n_nodes * rb.NODE_DTYPE.itemsize, t.uint8)
    d_log = gpu.empty(max(cap, 1), t.int32) if want_log else None
    d_prev = d_prev_nodes = d_reconf = None
    if prev is not None:
        a, nd = pack_prev(prev, J, n_nodes)
        d_prev, d_prev_nodes = rb.to_device(a), rb.to_device(nd)
    if not (active is None and T is None and delta is None and nrec is None):
        rc = np.zeros(max(J, 1), dtype=rb.RECONF_DTYPE)
        rc["active"][:J] = 1 if active is None else np.asarray(active)
        rc["T"][:J] = 1e9 if T is None else np.asarray(T, dtype=np.float32)
        rc["delta"][:J] = 0 if delta is None else np.asarray(delta, dtype=np.float32)
        rc["n_reconf"][:J] = 0 if nrec is None else np.asarray(nrec)
        d_reconf = rb.to_device(rc)
    steps, capped = gpu.ctx.incremental_round(d_jobs, J, d_cv, d_cp, d_cg, d_feas, n_nodes, cap, d_out, d_node, d_log,
                                              d_prev=d_prev, d_prev_nodes=d_prev_nodes, d_reconf=d_reconf, theta=theta, quota=quota)
    return unpack_round(rb.from_device(d_out, rb.ASSIGN_DTYPE)[:J], rb.from_device(d_node, rb.NODE_DTYPE), steps, capped,
                        d_log.cpu().numpy()[:steps] if want_log else None)


def unpack_round(out, node, steps, capped, log):
    return dict(g=out["g"].astype(np.int64), c=out["c"].astype(np.int64), m_bytes=out["m_bytes"].astype(np.int64),
                plan=out["plan"].astype(np.int64), first_node=out["first_node"].astype(np.int64),
                n_nodes=out["n_nodes"].astype(np.int64), status=out["status"].astype(np.int64),
                m_level=out["m_level"].astype(np.int64), thr=out["thr"].copy(),
                node=np.stack([node["free_g"], node["free_c"], node["free_m"], node["owner"]], axis=1).astype(np.int64),
                steps=steps, capped=capped, log=log)


def assert_rounds_equal(a, b):
    for k in ("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "m_level", "node"):
        assert np.array_equal(a[k], b[k]), k
    assert np.array_equal(a["thr"].view(np.uint32), b["thr"].view(np.uint32))
    assert a["steps"] == b["steps"] and a["capped"] == b["capped"]
    if a["log"] is not None and b["log"] is not None:
        assert np.array_equal(a["log"], b["log"])


def assert_chain_parity(gpu, cfg, n_nodes, oracle_chain, got=None, tie_rtol=1e-6, thr_rtol=1e-5):
    """The library's whole chain (its own single-precision table -> curves -> round) against the oracle's chain
    (double-precision table rounded once -> curves -> round).  The two tables differ by rounding, so:
      - masks are equal, curve values agree to thr_rtol, and the largest relative difference seen is `tol`;
      - the step logs are identical up to the first decision that the oracle takes by a margin within what
        `tol` can move (near_tie.assert_divergence_is_a_near_tie); up to there both sides hold the same GPUs
        and cores on the same nodes, and plans differ only where the oracle rates the library's plan within
        tie_rtol of its own;
      - without such a near tie the two rounds are the same round.
    oracle_chain = (plans, thr float64 [J, C, P], feas, cv float32, cp, cg) from the oracle; got (optional): the
    result of the one-call path (rubick_schedule_round*), which must equal the logged round bit for bit.
    Returns the description of the near tie, or None."""
    import near_tie
    import oracle
    jobs = cfg["jobs"]
    J = len(jobs["P"])
    plans, thr, feas, cv, cp, cg = oracle_chain
    d_jobs, d_thr, d_feas = gpu.eval(jobs)
    bv, bp, bg = gpu.best(d_thr, d_feas, J)
    sh = gpu.shape4(J)
    gcv, gcp, gcg = bv.cpu().numpy().reshape(sh), bp.cpu().numpy().reshape(sh), bg.cpu().numpy().reshape(sh)
    gfeas = gpu.np_feas(d_feas, J)
    assert np.array_equal(gfeas, feas)
    has = cv > 0
    assert np.array_equal(gcv > 0, has)
    tol = float((np.abs(gcv[has].astype(np.float64) - cv[has]) / cv[has]).max()) if has.any() else 0.0
    assert tol <= thr_rtol, tol
    logged = gpu.round_on_tables(jobs, gcv, gcp, gcg, gfeas, n_nodes)
    if got is not None:
        assert_rounds_equal(got, logged)
    args = (jobs, cfg["env"], cv, cp, cg, feas, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"], n_nodes)
    want = oracle.schedule_round(*args, want_log=True)
    found = near_tie.assert_divergence_is_a_near_tie(
        lambda k: oracle.schedule_round(*args, max_steps=k, want_log=True, want_candidates=True), want["log"], logged["log"],
        jobs["w"], tol, lambda j, gi, ci, mi: gcp[j, gi, ci, mi] != cp[j, gi, ci, mi] or gcg[j, gi, ci, mi] != cg[j, gi, ci, mi])
    if found is not None:
        k = near_tie.first_difference(want["log"], logged["log"])
        want = oracle.schedule_round(*args, max_steps=k, want_log=True)
        logged = gpu.round_on_tables(jobs, gcv, gcp, gcg, gfeas, n_nodes, max_steps=k)
        assert np.array_equal(want["log"], logged["log"])
    for key in ("g", "c", "status", "first_node", "n_nodes"):
        assert np.array_equal(want[key], logged[key]), key
    assert np.array_equal(want["node"][:, [0, 1, 3]], logged["node"][:, [0, 1, 3]])
    run = want["status"] == rb.RUNNING
    assert np.allclose(logged["thr"][run], want["thr"][run], rtol=thr_rtol, atol=0)
    other = np.nonzero(want["plan"] != logged["plan"])[0]
    if len(other):
        # another plan only where the oracle rates it as good as its own choice
        ci = np.searchsorted(cfg["c_levels"], want["c"][other])
        assert np.all(thr[other, ci, logged["plan"][other]] >= want["thr"][other].astype(np.float64) * (1 - tie_rtol - 2.0 ** -23))
        assert len(other) <= max(2, J // 50)
    same = want["plan"] == logged["plan"]
    assert np.array_equal(want["m_bytes"][same], logged["m_bytes"][same])
    if not len(other):
        assert np.array_equal(want["node"], logged["node"])
    return found


def jobs_from_records(rec):
    """JOB_DTYPE records -> the dict of per-job arrays the generators produce (exact: every field is a double,
    an integer or a single-precision value)."""
    return {k: np.asarray(rec[k], dtype=np.float64 if rec.dtype[k].kind == "f" else np.int64)
            for k in rec.dtype.names if k not in ("flags", "pad")}


def curves_of(gpu, records):
    """The library's own mask and curve tables of the given job records (rubick_curves, the kernel the
    scheduling entry points use) -> (cv [J, G, C, M] float32, cp, cg int32, feas [J, P] uint32)."""
    t = gpu.torch
    J = len(records)
    n = J * gpu.nG * gpu.nC * gpu.nM
    d_jobs = rb.to_device(records)
    d_feas = gpu.empty(J * gpu.P, t.int32)
    cv, cp, cg = gpu.empty(n, t.float32), gpu.empty(n, t.int32), gpu.empty(n, t.int32)
    gpu.ctx.curves(d_jobs, J, d_feas, cv, cp, cg)
    gpu.ctx.sync()
    sh = gpu.shape4(J)
    return cv.cpu().numpy().reshape(sh), cp.cpu().numpy().reshape(sh), cg.cpu().numpy().reshape(sh), gpu.np_feas(d_feas, J)
