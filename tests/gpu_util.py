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
