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
