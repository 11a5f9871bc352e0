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


def fit_samples(cfg, plans, thr, feas, picks, g_max=8, noisy=True):
    """Measured samples for model fitting from a candidate table `thr` [J, C, P] (whoever computed it):
    plans the job can run on at most g_max GPUs, the first third of the slots among offloading plans.
    -> (plan [J, S] int32, cores [J, S] int64, throughput [J, S] float64); unused slots have plan -1."""
    plans = np.asarray(plans)
    J, S = picks["rank"].shape
    g = plans[:, 0].astype(np.int64) * plans[:, 1] * plans[:, 2]
    sp = np.full((J, S), -1, dtype=np.int32)
    sc = np.zeros((J, S), dtype=np.int64)
    sy = np.zeros((J, S), dtype=np.float64)
    cl = np.asarray(cfg["c_levels"])
    for j in range(J):
        ok = (thr[j, 0] > 0) & (feas[j] != 0) & (g <= g_max)
        off = np.nonzero(ok & (plans[:, 5] == 1))[0]
        non = np.nonzero(ok & (plans[:, 5] == 0))[0]
        for i in range(S):
            pool = off if (i < S // 3 and len(off)) else non
            if len(pool) == 0:
                continue
            pl = int(pool[min(int(picks["rank"][j, i] * len(pool)), len(pool) - 1)])
            ci = int(picks["c_idx"][j, i])
            sp[j, i], sc[j, i] = pl, cl[ci]
            sy[j, i] = thr[j, ci, pl] * (picks["noise"][j, i] if noisy else 1.0)
    return sp, sc, sy
