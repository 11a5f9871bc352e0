"""Small helpers shared by the tests (no arithmetic of the method lives here)."""
import numpy as np

from paper_2408_08586_b200 import workloads

GIB = workloads.GIB


def one_job(**kw):
    """A single hand-specified job as the dict-of-arrays the generators produce."""
    base = dict(P=1e9, l=24, h=2048, s=1024, b=16, mu_cap=4, alpha_act=34, tau=0.01,
                k_bwd=2.0, k_sync=2.0, k_opt=1e-11, k_opt_off=2e-8, k_off=2.0, k_swap=2.0,
                k_const=0.05, w=1.0, gmin_idx=-1, cmin_idx=-1, host_base_bytes=4 * GIB)
    base.update(kw)
    return {k: np.asarray([v]) for k, v in base.items()}


def env(**kw):
    e = dict(workloads.ENV)
    e.update(kw)
    return e


def stack_jobs(*jobs):
    return {k: np.concatenate([np.asarray(j[k]) for j in jobs]) for k in jobs[0]}


def requests_for(cfg, group_off, guaranteed_share=0.5):
    """[J, 4] int64 requests (g level, c level, m level, original plan; plan -1 = best effort) from
    the generator's draws; the plan is picked by rank inside the plans of the requested GPU level."""
    J = len(cfg["jobs"]["P"])
    rq = workloads.draw_requests(cfg["seed"], J, [int(g) for g in cfg["g_levels"]], len(cfg["c_levels"]),
                                 len(cfg["m_levels"]), guaranteed_share)
    off = np.asarray(group_off, dtype=np.int64)
    size = off[rq["g_idx"] + 1] - off[rq["g_idx"]]
    plan = np.where(rq["plan_rank"] >= 0, off[rq["g_idx"]] + np.floor(np.maximum(rq["plan_rank"], 0) * size).astype(np.int64), -1)
    return np.stack([rq["g_idx"], rq["c_idx"], rq["m_idx"], plan], axis=1).astype(np.int64)


fit_samples = workloads.fit_samples
