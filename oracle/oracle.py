"""ctypes front end of the C oracle (``rubick_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Builds ``liboracle.so`` beside the source with gcc on first use
and marshals numpy arrays into the oracle's own plain layouts (jobs as rows of doubles,
plans as rows of seven int32, environment as a row of doubles).  Nothing here touches the
CUDA library.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rubick_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")

JOB_FIELDS = ["P", "l", "h", "s", "b", "mu_cap", "alpha_act", "tau", "k_bwd", "k_sync", "k_opt",
              "k_opt_off", "k_off", "k_swap", "k_const", "w", "gmin_idx", "cmin_idx", "host_base_bytes", "tenant"]
ENV_FIELDS = ["B_intra", "B_inter", "B_pcie", "gpu_mem_bytes", "gpus_per_node", "cpus_per_node",
              "mem_per_node_bytes", "bytes_per_elem", "strict_zero_dp_only", "zero3_extra_volume", "spread_align"]
TERM_FIELDS = ["valid", "mu", "m", "a", "T_fwd", "T_bwd", "V_dp", "V_tp", "V_pp", "T_dp", "T_tp",
               "T_pp", "T_cc", "T_opt", "T_off", "T_oo", "T_iter", "thr"]
MEM_FIELDS = ["params", "grads", "opt", "act", "gpu_total", "gpu_ok", "host_need", "nodes"]

_lib = None


def build(force=False):
    """Compile the oracle with gcc (-O2, no fast-math, no FMA contraction, OpenMP over jobs)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _plans(plans):
    """Plans as the C side reads them: rows of (d, t, p, ZeRO stage, gc, off, micro-batch halvings); a
    six-column input (no explicit accumulation) gets a zero seventh column."""
    a = np.atleast_2d(np.asarray(plans, dtype=np.int32))
    if a.shape[1] == 6:
        a = np.concatenate([a, np.zeros((a.shape[0], 1), dtype=np.int32)], axis=1)
    assert a.shape[1] == 7
    return np.ascontiguousarray(a)


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_SO)
        L.oracle_overlap.restype = C.c_double
        L.oracle_overlap.argtypes = [C.c_double, C.c_double, C.c_double]
        L.oracle_bruteforce.restype = C.c_double
        L.oracle_feas_word.restype = C.c_uint32
        L.oracle_enumerate_plans.restype = C.c_int
        L.oracle_round.restype = C.c_int
        _lib = L
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def job_rows(jobs):
    """dict of per-job arrays (keys = JOB_FIELDS) -> [J, len(JOB_FIELDS)] float64 rows."""
    J = len(np.atleast_1d(jobs["P"]))
    rows = np.zeros((J, len(JOB_FIELDS)), dtype=np.float64)
    for i, k in enumerate(JOB_FIELDS):
        if k == "tenant" and k not in jobs:
            continue                                   # single tenant
        rows[:, i] = np.asarray(jobs[k], dtype=np.float64)
    return rows


def env_row(env):
    return _f64([float(env.get(k, 0.0)) for k in ENV_FIELDS])


def overlap(k, x, y):
    return lib().oracle_overlap(float(k), float(x), float(y))


def terms(jobs, j, env, plan, c):
    """All model terms (TERM_FIELDS) of job j under plan = (d, t, p, z, gc, off) with c cores."""
    rows = job_rows(jobs)
    out = np.zeros(len(TERM_FIELDS))
    pl = _plans(plan).reshape(-1)
    lib().oracle_terms(_p(rows[j], C.c_double), _p(env_row(env), C.c_double), _p(pl, C.c_int32),
                       C.c_double(float(c)), _p(out, C.c_double))
    return dict(zip(TERM_FIELDS, out.tolist()))


def memory(jobs, j, env, plan):
    rows = job_rows(jobs)
    out = np.zeros(len(MEM_FIELDS), dtype=np.int64)
    pl = _plans(plan).reshape(-1)
    lib().oracle_memory(_p(rows[j], C.c_double), _p(env_row(env), C.c_double), _p(pl, C.c_int32),
                        _p(out, C.c_int64))
    return dict(zip(MEM_FIELDS, out.tolist()))


def feas_word(jobs, j, env, plan, m_levels):
    rows = job_rows(jobs)
    ml = _i64(m_levels)
    return int(lib().oracle_feas_word(_p(rows[j], C.c_double), _p(env_row(env), C.c_double),
                                      _p(_plans(plan).reshape(-1), C.c_int32), _p(ml, C.c_int64), C.c_int(len(ml))))


def enumerate_plans(g_levels, any_degrees=False, accumulation_levels=1):
    """-> (plans [P, 7] int32 = d, t, p, z, gc, off, micro-batch halvings; group_off [nG + 1] int32).
    any_degrees: every factorisation of every GPU level instead of power-of-two degrees on power-of-two
    levels; accumulation_levels > 1 (with any_degrees): the explicit accumulation axis, 0 .. levels - 1
    halvings of the micro-batch."""
    gl = _i64(g_levels)
    off = np.zeros(len(gl) + 1, dtype=np.int32)
    dummy = np.zeros((1, 7), dtype=np.int32)
    if any_degrees:
        f = lib().oracle_enumerate_plans_any
        n = f(_p(gl, C.c_int64), C.c_int(len(gl)), C.c_int(accumulation_levels), _p(dummy, C.c_int32), C.c_int(0), _p(off, C.c_int32))
        plans = np.zeros((max(n, 1), 7), dtype=np.int32)
        f(_p(gl, C.c_int64), C.c_int(len(gl)), C.c_int(accumulation_levels), _p(plans, C.c_int32), C.c_int(n), _p(off, C.c_int32))
        return plans[:n], off
    assert accumulation_levels == 1
    n = lib().oracle_enumerate_plans(_p(gl, C.c_int64), C.c_int(len(gl)), _p(dummy, C.c_int32), C.c_int(0),
                                     _p(off, C.c_int32))
    plans = np.zeros((max(n, 1), 7), dtype=np.int32)
    lib().oracle_enumerate_plans(_p(gl, C.c_int64), C.c_int(len(gl)), _p(plans, C.c_int32), C.c_int(n),
                                 _p(off, C.c_int32))
    return plans[:n], off


def eval_candidates(jobs, plans, env, c_levels, m_levels, nthreads=1):
    """-> (thr [J, C, P] float64, feas [J, P] uint32)."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    plans = _plans(plans)
    Pn = plans.shape[0]
    cl, ml = _i64(c_levels), _i64(m_levels)
    thr = np.zeros((J, len(cl), Pn), dtype=np.float64)
    feas = np.zeros((J, Pn), dtype=np.uint32)
    lib().oracle_eval(_p(rows, C.c_double), C.c_int(J), _p(plans, C.c_int32), C.c_int(Pn),
                      _p(env_row(env), C.c_double), _p(cl, C.c_int64), C.c_int(len(cl)),
                      _p(ml, C.c_int64), C.c_int(len(ml)), _p(thr, C.c_double), _p(feas, C.c_uint32),
                      C.c_int(nthreads))
    return thr, feas


def best_plan(thr, feas, plans, g_levels, nM, prefix=True, nthreads=1):
    """thr [J, C, P] (any float dtype; compared in float64), feas [J, P] ->
    (best_val [J, G, C, M] float64, best_plan int32, best_g int32)."""
    thr = _f64(thr)
    feas = np.ascontiguousarray(feas, dtype=np.uint32)
    J, nC, Pn = thr.shape
    plans = _plans(plans)
    gl = _i64(g_levels)
    nG = len(gl)
    bv = np.zeros((J, nG, nC, nM), dtype=np.float64)
    bp = np.zeros((J, nG, nC, nM), dtype=np.int32)
    bg = np.zeros((J, nG, nC, nM), dtype=np.int32)
    lib().oracle_best_plan(_p(thr, C.c_double), _p(feas, C.c_uint32), C.c_int(J), _p(plans, C.c_int32),
                           C.c_int(Pn), _p(gl, C.c_int64), C.c_int(nG), C.c_int(nC), C.c_int(nM),
                           C.c_int(1 if prefix else 0), _p(bv, C.c_double), _p(bp, C.c_int32),
                           _p(bg, C.c_int32), C.c_int(nthreads))
    return bv, bp, bg


def gain(jobs, curve_val, g_levels, c_levels, state_g, state_c, state_val):
    """Marginal gains for a given per-job state -> (gain_gpu, gain_cpu, next_g, next_c)."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    cv = np.ascontiguousarray(curve_val, dtype=np.float32)
    gl, cl = _i64(g_levels), _i64(c_levels)
    nM = cv.shape[3]
    sg, sc = _i64(state_g), _i64(state_c)
    sv = np.ascontiguousarray(state_val, dtype=np.float32)
    gg = np.zeros(J, dtype=np.float32)
    gc = np.zeros(J, dtype=np.float32)
    ng = np.zeros(J, dtype=np.int32)
    nc = np.zeros(J, dtype=np.int32)
    lib().oracle_gain(_p(rows, C.c_double), C.c_int(J), _p(cv, C.c_float), _p(gl, C.c_int64), C.c_int(len(gl)),
                      _p(cl, C.c_int64), C.c_int(len(cl)), C.c_int(nM), _p(sg, C.c_int64), _p(sc, C.c_int64),
                      _p(sv, C.c_float), _p(gg, C.c_float), _p(gc, C.c_float), _p(ng, C.c_int32),
                      _p(nc, C.c_int32))
    return gg, gc, ng, nc


CAND_FIELDS = ("gain", "next", "placeable", "v_cur", "v_next", "units", "shut", "m_commit", "v_commit", "g_commit", "gi", "ci")


MAX_PIECES = 32


def schedule_round(jobs, env, curve_val, curve_plan, curve_g, feas, g_levels, c_levels, m_levels,
                   n_nodes, max_steps=1 << 30, want_log=False, quota=None, double_decisions=False, want_candidates=False,
                   spread=None):
    """One greedy round.  Default: decisions in single precision on the curve table rounded to single
    precision.  double_decisions: every decision in double precision on curve_val as given (float64).
    spread: None, or a list of (align, curve_val, curve_plan, curve_g, feas) -- the tables of spread placement classes
    (pieces of `align` GPUs on several nodes), widest pieces first; the result then carries `pieces` [J, 32]
    (node << 8 | GPUs, -1 = unused) and `cls` [J] (-1 = packed).
    want_candidates: also `cand`, a dict of [J, 2] arrays (CAND_FIELDS; axis 1 = GPU / CPU increment) with
    what every job offered for the decision the round stopped at (the step `max_steps` cut off, or the
    last look that found nothing to do).

    -> dict(g, c, m_bytes, plan, first_node, n_nodes, status, m_level, thr, node (N x 4:
    free g, free c, free m, owner), steps, capped, log[, cand])."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    cv = np.ascontiguousarray(curve_val, dtype=np.float32)
    cv64 = _f64(curve_val) if double_decisions else None
    cp, cg = _i32(curve_plan), _i32(curve_g)
    feas = np.ascontiguousarray(feas, dtype=np.uint32)
    Pn = feas.shape[1] if feas.ndim == 2 else 0
    gl, cl, ml = _i64(g_levels), _i64(c_levels), _i64(m_levels)
    out_i = np.zeros((max(J, 1), 8), dtype=np.int64)
    out_v = np.zeros(max(J, 1), dtype=np.float32)
    out_v64 = np.zeros(max(J, 1), dtype=np.float64)
    node = np.zeros((n_nodes, 4), dtype=np.int64)
    cap = int(min(max_steps, J * (len(gl) + len(cl) + 2) + 1))
    log = np.zeros(max(cap, 1), dtype=np.int32)
    cand = np.zeros((max(J, 1), 2, len(CAND_FIELDS)), dtype=np.float64)
    qt = None if quota is None else _i64(quota).reshape(-1, 2)      # per tenant: GPUs, cores
    nK = 0 if not spread else len(spread)
    keep = []
    if nK:
        al = _i64([int(x[0]) for x in spread])
        tabs = [(np.ascontiguousarray(x[1], dtype=np.float32), _i32(x[2]), _i32(x[3]), np.ascontiguousarray(x[4], dtype=np.uint32)) for x in spread]
        keep = [al, tabs]
        ptr = lambda i, t: (C.POINTER(t) * nK)(*[_p(tb[i], t) for tb in tabs])
        k_val, k_plan, k_g, k_feas = ptr(0, C.c_float), ptr(1, C.c_int32), ptr(2, C.c_int32), ptr(3, C.c_uint32)
        al_p = _p(al, C.c_int64)
    else:
        k_val = k_plan = k_g = k_feas = al_p = None
    pieces = np.full((max(J, 1), MAX_PIECES), -1, dtype=np.int32)
    cls = np.full(max(J, 1), -1, dtype=np.int32)
    r = lib().oracle_round(_p(rows, C.c_double), C.c_int(J), _p(env_row(env), C.c_double), _p(cv, C.c_float),
                           _p(cp, C.c_int32), _p(cg, C.c_int32), _p(feas, C.c_uint32), C.c_int(Pn),
                           _p(gl, C.c_int64), C.c_int(len(gl)), _p(cl, C.c_int64), C.c_int(len(cl)),
                           _p(ml, C.c_int64), C.c_int(len(ml)), C.c_int(n_nodes), C.c_int(cap),
                           _p(qt, C.c_int64) if qt is not None else None, C.c_int(0 if qt is None else len(qt)),
                           _p(out_i, C.c_int64), _p(out_v, C.c_float), _p(node, C.c_int64),
                           _p(log, C.c_int32) if want_log else None,
                           _p(cv64, C.c_double) if cv64 is not None else None, _p(out_v64, C.c_double),
                           _p(cand, C.c_double) if want_candidates else None,
                           C.c_int(nK), al_p, k_val, k_plan, k_g, k_feas, _p(pieces, C.c_int32), _p(cls, C.c_int32))
    del keep
    capped = r < 0
    steps = -r - 1 if capped else r
    out_i = out_i[:J]
    res = dict(g=out_i[:, 0].copy(), c=out_i[:, 1].copy(), m_bytes=out_i[:, 2].copy(),
               plan=out_i[:, 3].copy(), first_node=out_i[:, 4].copy(), n_nodes=out_i[:, 5].copy(),
               status=out_i[:, 6].copy(), m_level=out_i[:, 7].copy(),
               thr=out_v64[:J].copy() if double_decisions else out_v[:J].copy(), node=node,
               steps=steps, capped=capped, log=log[:steps].copy() if want_log else None)
    if want_candidates:
        res["cand"] = {k: cand[:J, :, i].copy() for i, k in enumerate(CAND_FIELDS)}
    if nK:
        res["pieces"], res["cls"] = pieces[:J].copy(), cls[:J].copy()
    return res


def schedule_round_incremental(jobs, env, curve_val, curve_plan, curve_g, feas, g_levels, c_levels, m_levels,
                               n_nodes, prev, active=None, T=None, delta=None, nrec=None, theta=0.97,
                               max_steps=1 << 30, want_log=False, quota=None):
    """One incremental round (shrink / exchange step and reconfiguration gate) from `prev`, the dict a
    previous round returned (None: an empty cluster).  active [J] marks used job slots; T, delta
    (seconds) and nrec feed the gate.  -> dict like schedule_round; steps is None when `prev` does
    not fit the grid or the cluster."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    cv = np.ascontiguousarray(curve_val, dtype=np.float32)
    cp, cg = _i32(curve_plan), _i32(curve_g)
    feas = np.ascontiguousarray(feas, dtype=np.uint32)
    Pn = feas.shape[1] if feas.ndim == 2 else 0
    gl, cl, ml = _i64(g_levels), _i64(c_levels), _i64(m_levels)
    prev_i = np.zeros((max(J, 1), 8), dtype=np.int64)
    prev_v = np.zeros(max(J, 1), dtype=np.float32)
    prev_owner = np.full(n_nodes, -1, dtype=np.int32)
    if prev is not None:
        for col, key in enumerate(("g", "c", "m_bytes", "plan", "first_node", "n_nodes", "status", "m_level")):
            prev_i[:J, col] = np.asarray(prev[key], dtype=np.int64)
        prev_v[:J] = np.asarray(prev["thr"], dtype=np.float32)
        prev_owner[:] = np.asarray(prev["node"], dtype=np.int64)[:, 3].astype(np.int32)
    act = np.ones(max(J, 1), dtype=np.int32) if active is None else np.ascontiguousarray(active, dtype=np.int32)
    Tt = np.full(max(J, 1), 1e9, dtype=np.float32) if T is None else np.ascontiguousarray(T, dtype=np.float32)
    dl = np.zeros(max(J, 1), dtype=np.float32) if delta is None else np.ascontiguousarray(delta, dtype=np.float32)
    nr = np.zeros(max(J, 1), dtype=np.int32) if nrec is None else np.ascontiguousarray(nrec, dtype=np.int32)
    out_i = np.zeros((max(J, 1), 8), dtype=np.int64)
    out_v = np.zeros(max(J, 1), dtype=np.float32)
    node = np.zeros((n_nodes, 4), dtype=np.int64)
    cap = int(min(max_steps, 2 * J * (len(gl) + len(cl) + 2) + 1))
    log = np.zeros(max(cap, 1), dtype=np.int32)
    qt = None if quota is None else _i64(quota).reshape(-1, 2)
    f = lib().oracle_round_incremental
    f.restype = C.c_int
    r = f(_p(rows, C.c_double), C.c_int(J), _p(env_row(env), C.c_double), _p(cv, C.c_float),
          _p(cp, C.c_int32), _p(cg, C.c_int32), _p(feas, C.c_uint32), C.c_int(Pn),
          _p(gl, C.c_int64), C.c_int(len(gl)), _p(cl, C.c_int64), C.c_int(len(cl)),
          _p(ml, C.c_int64), C.c_int(len(ml)), C.c_int(n_nodes), C.c_int(cap),
          _p(qt, C.c_int64) if qt is not None else None, C.c_int(0 if qt is None else len(qt)),
          _p(prev_i, C.c_int64), _p(prev_v, C.c_float), _p(prev_owner, C.c_int32), _p(act, C.c_int32),
          _p(Tt, C.c_float), _p(dl, C.c_float), _p(nr, C.c_int32), C.c_float(theta),
          _p(out_i, C.c_int64), _p(out_v, C.c_float), _p(node, C.c_int64),
          _p(log, C.c_int32) if want_log else None)
    if r == -2 ** 31:
        return dict(steps=None)
    capped = r < 0
    steps = -r - 1 if capped else r
    out_i = out_i[:J]
    return dict(g=out_i[:, 0].copy(), c=out_i[:, 1].copy(), m_bytes=out_i[:, 2].copy(),
                plan=out_i[:, 3].copy(), first_node=out_i[:, 4].copy(), n_nodes=out_i[:, 5].copy(),
                status=out_i[:, 6].copy(), m_level=out_i[:, 7].copy(), thr=out_v[:J].copy(), node=node,
                steps=steps, capped=capped, log=log[:steps].copy() if want_log else None)


FIT_NAMES = ("k_bwd", "k_sync", "k_opt", "k_opt_off", "k_off", "k_swap", "k_const")


def fit(jobs, plans, env, sample_plan, sample_c, sample_thr, sweeps=14):
    """Section 4.3 model fitting by RMSLE.  sample_plan [J, S] plan indices (-1: unused slot), sample_c
    [J, S] cores, sample_thr [J, S] measured throughput; the start is the coefficients in `jobs`.
    -> (theta [J, 7] in FIT_NAMES order, rmsle [J, 2] before / after, margin [J])."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    plans = _plans(plans)
    spn = np.ascontiguousarray(sample_plan, dtype=np.int32).reshape(J, -1)
    S = spn.shape[1]
    scs = _i64(sample_c).reshape(J, S)
    sth = _f64(sample_thr).reshape(J, S)
    theta = np.zeros((J, 7), dtype=np.float64)
    rmsle = np.zeros((J, 2), dtype=np.float64)
    margin = np.zeros(J, dtype=np.float64)
    f = lib().oracle_fit
    f.restype = None
    f(_p(rows, C.c_double), C.c_int(J), _p(env_row(env), C.c_double), _p(plans, C.c_int32), C.c_int(plans.shape[0]),
      _p(spn, C.c_int32), _p(scs, C.c_int64), _p(sth, C.c_double), C.c_int(S), C.c_int(sweeps),
      _p(theta, C.c_double), _p(rmsle, C.c_double), _p(margin, C.c_double))
    return theta, rmsle, margin


def bruteforce(jobs, env, curve_val, curve_plan, curve_g, feas, g_levels, c_levels, m_levels):
    """Best total weighted throughput over all single-node assignments (tiny instances)."""
    rows = job_rows(jobs)
    J = rows.shape[0]
    cv = np.ascontiguousarray(curve_val, dtype=np.float32)
    cp, cg = _i32(curve_plan), _i32(curve_g)
    feas = np.ascontiguousarray(feas, dtype=np.uint32)
    gl, cl, ml = _i64(g_levels), _i64(c_levels), _i64(m_levels)
    return float(lib().oracle_bruteforce(_p(rows, C.c_double), C.c_int(J), _p(env_row(env), C.c_double),
                                         _p(cv, C.c_float), _p(cp, C.c_int32), _p(cg, C.c_int32),
                                         _p(feas, C.c_uint32), C.c_int(feas.shape[1]), _p(gl, C.c_int64),
                                         C.c_int(len(gl)), _p(cl, C.c_int64), C.c_int(len(cl)),
                                         _p(ml, C.c_int64), C.c_int(len(ml))))


def min_resources(thr, feas, curve_val, plans, g_levels, req):
    """Minimum demand of guaranteed jobs.  req [J, 4] = requested g level, c level, m level, plan
    (plan < 0: best effort) -> (gmin_idx, cmin_idx int32, baseline float64)."""
    thr = _f64(thr)
    feas = np.ascontiguousarray(feas, dtype=np.uint32)
    cv = _f64(curve_val)
    J, nC, Pn = thr.shape
    nG, nM = cv.shape[1], cv.shape[3]
    plans = _plans(plans)
    gl = _i64(g_levels)
    rq = _i64(req).reshape(J, 4)
    gm = np.zeros(J, dtype=np.int32)
    cm = np.zeros(J, dtype=np.int32)
    base = np.zeros(J, dtype=np.float64)
    lib().oracle_min_resources(_p(thr, C.c_double), _p(feas, C.c_uint32), _p(cv, C.c_double), C.c_int(J),
                               _p(plans, C.c_int32), C.c_int(Pn), _p(gl, C.c_int64), C.c_int(nG), C.c_int(nC),
                               C.c_int(nM), _p(rq, C.c_int64), _p(gm, C.c_int32), _p(cm, C.c_int32),
                               _p(base, C.c_double))
    return gm, cm, base
