"""Pins of the oracle's plan enumeration, best-plan search and sensitivity curve
(paper Section 3 plan families, Section 5.2 curves)."""
import os

import numpy as np
import pytest

import oracle
from test_oracle_memory import facts


def tri(k):
    return (k + 1) * (k + 2) // 2


@pytest.mark.parametrize("gmax,key", [(8, "triples_up_to_8_gpus"), (64, "triples_up_to_64_gpus"),
                                      (256, "triples_up_to_256_gpus")])
def test_plan_counts(gmax, key):
    levels = [1 << i for i in range(gmax.bit_length())]
    plans, off = oracle.enumerate_plans(levels)
    assert len(plans) == 16 * int(facts()[key])
    assert list(np.diff(off)) == [16 * tri(k) for k in range(len(levels))]


def test_plans_are_exactly_the_power_of_two_factorisations():
    levels = list(range(1, 9))
    plans, off = oracle.enumerate_plans(levels)
    want = set()
    for g in (1, 2, 4, 8):
        for d in (1, 2, 4, 8):
            for t in (1, 2, 4, 8):
                for p in (1, 2, 4, 8):
                    if d * t * p == g:
                        for z in range(4):
                            for gc in range(2):
                                for o in range(2):
                                    want.add((d, t, p, z, gc, o))
    got = [tuple(int(x) for x in r[:6]) for r in plans]
    assert len(got) == len(set(got)) == 320 and set(got) == want and not plans[:, 6].any()
    # groups: level index i holds the plans using g_levels[i] GPUs; other levels are empty
    for i, g in enumerate(levels):
        grp = plans[off[i]:off[i + 1]]
        if g & (g - 1):
            assert len(grp) == 0
        else:
            assert np.all(grp[:, 0] * grp[:, 1] * grp[:, 2] == g)


def test_plan_order_resolves_ties_toward_simpler_plans():
    plans, _ = oracle.enumerate_plans([1, 2, 4, 8])
    keys = [(int(r[0] * r[1] * r[2]), int(r[1]), int(r[2]), int(r[3]), int(r[4]), int(r[5])) for r in plans]
    assert keys == sorted(keys)            # g, then TP, then PP, then ZeRO stage, GC, offload


def numpy_best(thr, feas, plans, g_levels, nM):
    J, nC, P = thr.shape
    g_of = plans[:, 0] * plans[:, 1] * plans[:, 2]
    bv = np.zeros((J, len(g_levels), nC, nM))
    bp = -np.ones((J, len(g_levels), nC, nM), dtype=np.int64)
    for gi, g in enumerate(g_levels):
        sel = np.nonzero(g_of == g)[0]
        if len(sel) == 0:
            continue
        for mi in range(nM):
            ok = ((feas[:, sel] >> mi) & 1).astype(bool)                 # [J, n]
            v = np.where(ok[:, None, :], thr[:, :, sel], 0.0)           # [J, C, n]
            a = v.argmax(axis=2)                                         # first maximum
            mx = np.take_along_axis(v, a[:, :, None], 2)[:, :, 0]
            bv[:, gi, :, mi] = mx
            bp[:, gi, :, mi] = np.where(mx > 0, sel[a], -1)
    return bv, bp


def test_best_plan_matches_a_masked_argmax(paper_scale):
    cfg = paper_scale
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=4)
    nM = len(cfg["m_levels"])
    bv, bp, bg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], nM, prefix=False, nthreads=4)
    wv, wp = numpy_best(thr, feas, plans, cfg["g_levels"], nM)
    assert np.array_equal(bv, wv) and np.array_equal(bp, wp)
    assert np.array_equal(bg, np.where(bp >= 0, cfg["g_levels"][None, :, None, None], 0))
    # exact ties exist (ZeRO stages 1 and 2 predict the same time) and go to the lower index
    tie = thr[:, :, 4::16] == thr[:, :, 8::16]
    assert tie.any()


def test_curve_is_the_running_maximum_over_gpu_levels(tiny):
    cfg = tiny
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"])
    nM = len(cfg["m_levels"])
    bv, bp, bg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], nM, prefix=False)
    cv, cp, cg = oracle.best_plan(thr, feas, plans, cfg["g_levels"], nM, prefix=True)
    assert np.array_equal(cv, np.maximum.accumulate(bv, axis=1))
    # invalid GPU counts (3, 5, 6, 7) have zero throughput; the curve stays flat across them
    for gi in (2, 4, 5, 6):
        assert np.all(bv[:, gi] == 0) and np.all(bp[:, gi] == -1)
        assert np.array_equal(cv[:, gi], cv[:, gi - 1]) and np.array_equal(cg[:, gi], cg[:, gi - 1])
    # the carried plan really yields the carried value with the carried GPU count
    J, nG, nC, _ = cv.shape
    for j in range(J):
        for gi in range(nG):
            for ci in range(nC):
                for mi in range(nM):
                    p = cp[j, gi, ci, mi]
                    if p < 0:
                        assert cv[j, gi, ci, mi] == 0
                        continue
                    assert thr[j, ci, p] == cv[j, gi, ci, mi]
                    assert int(np.prod(plans[p, :3])) == cg[j, gi, ci, mi] <= cfg["g_levels"][gi]
                    assert (feas[j, p] >> mi) & 1


def test_best_is_monotone_in_host_memory_and_cores(paper_scale):
    cfg = paper_scale
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=4)
    bv, _, _ = oracle.best_plan(thr, feas, plans, cfg["g_levels"], len(cfg["m_levels"]), prefix=False, nthreads=4)
    assert np.all(np.diff(bv, axis=3) >= 0)          # more host memory never hurts
    assert np.all(np.diff(bv, axis=2) >= 0)          # more cores never hurt
    assert (np.diff(bv, axis=2) > 0).any()           # and help where offload is the best plan


def ordered_factorisations(g):
    """Number of ordered triples (d, t, p) with d * t * p = g: multiplicative, C(a + 2, 2) per prime power."""
    n, out, q = g, 1, 2
    while n > 1:
        a = 0
        while n % q == 0:
            n //= q
            a += 1
        out *= (a + 1) * (a + 2) // 2
        q += 1
    return out


def test_any_degree_plan_space():
    """The wider plan space (Section 7.2 uses a 3-GPU tensor-parallel plan, Table 2 GPU counts such as 12 and
    24): every ordered factorisation of every GPU level, same canonical order; on power-of-two levels it is
    the power-of-two list."""
    levels = [1, 2, 3, 4, 6, 8, 12, 16, 24, 36]
    plans, off = oracle.enumerate_plans(levels, any_degrees=True)
    assert len(plans) == off[-1] == 16 * sum(ordered_factorisations(g) for g in levels)
    for i, g in enumerate(levels):
        grp = plans[off[i]:off[i + 1]]
        assert len(grp) == 16 * ordered_factorisations(g)
        assert np.all(grp[:, 0].astype(np.int64) * grp[:, 1] * grp[:, 2] == g)
        triples = grp[::16, :3]
        keys = [(int(t), int(p)) for d, t, p in triples]
        assert keys == sorted(keys) and len(set(keys)) == len(keys)          # TP ascending, then PP ascending, no repeats
        tail = grp[:16, 3:6]
        assert [tuple(r) for r in tail] == [(z, gc, o) for z in range(4) for gc in range(2) for o in range(2)]
    pow2 = [1, 2, 4, 8, 16, 64]
    a, oa = oracle.enumerate_plans(pow2, any_degrees=True)
    b, ob = oracle.enumerate_plans(pow2)
    assert np.array_equal(a, b) and np.array_equal(oa, ob)
    # the 3-GPU tensor-parallel plan exists and is valid for a job whose hidden size divides by 3
    p3 = plans[off[2]:off[3]]
    assert any((r[:3] == [1, 3, 1]).all() for r in p3)


def test_explicit_accumulation_axis():
    """Table 1 lists the accumulation steps among a plan's parameters; the axis halves the micro-batch 0, 1, 2
    ... times below the largest one a replica may run.  Pinned by the closed forms: the micro-batch halves, the
    number of passes doubles, so the compute of an iteration (a forwards of mu samples each) is unchanged
    without pipelining, the pipeline bubble shrinks with more micro-batches, the activation memory halves,
    and a micro-batch below one sample does not exist."""
    from helpers import env, one_job
    levels = [1, 2, 3, 4, 6, 8]
    base, boff = oracle.enumerate_plans(levels, any_degrees=True)
    plans, off = oracle.enumerate_plans(levels, any_degrees=True, accumulation_levels=3)
    assert len(plans) == 3 * len(base) and np.array_equal(off, 3 * boff)
    keys = [(int(r[0] * r[1] * r[2]), int(r[1]), int(r[2]), int(r[6]), int(r[3]), int(r[4]), int(r[5])) for r in plans]
    assert keys == sorted(keys)            # g, TP, PP, accumulation, ZeRO stage, GC, offload
    assert np.array_equal(plans[plans[:, 6] == 0][:, :6], base[:, :6])
    job = one_job(b=64, mu_cap=8, l=24, h=1536)
    e = env()
    t0 = oracle.terms(job, 0, e, (4, 1, 1, 0, 0, 0, 0), 8)          # r = 16, mu = 8, a = 2
    t1 = oracle.terms(job, 0, e, (4, 1, 1, 0, 0, 0, 1), 8)          # mu = 4, a = 4
    t2 = oracle.terms(job, 0, e, (4, 1, 1, 0, 0, 0, 3), 8)          # mu = 1, a = 16
    assert (t0["mu"], t0["a"], t1["mu"], t1["a"], t2["mu"], t2["a"]) == (8, 2, 4, 4, 1, 16)
    assert t1["T_fwd"] == pytest.approx(t0["T_fwd"] / 2, rel=1e-15) and t0["a"] * t0["T_fwd"] == pytest.approx(t1["a"] * t1["T_fwd"], rel=1e-15)
    # only the overlapped last backward changes: T_cc differs by f(T_bwd, T_dp) evaluated at the smaller backward
    k = float(job["k_sync"][0])
    for tm in (t0, t1, t2):
        want = tm["a"] * tm["T_fwd"] + (tm["a"] - 1) * tm["T_bwd"] + oracle.overlap(k, tm["T_bwd"], tm["T_dp"]) + tm["T_tp"] + tm["T_pp"]
        assert tm["T_cc"] == pytest.approx(want, rel=1e-15)
    assert oracle.terms(job, 0, e, (4, 1, 1, 0, 0, 0, 4), 8)["valid"] == 0          # 8 >> 4 = 0 samples
    # pipelining: m micro-batches, bubble (m + p - 1) / m of the ideal time, smaller with more micro-batches
    p0 = oracle.terms(job, 0, e, (1, 1, 4, 0, 0, 0, 0), 8)          # r = 64, mu = 8, m = 8
    p1 = oracle.terms(job, 0, e, (1, 1, 4, 0, 0, 0, 2), 8)          # mu = 2, m = 32
    assert (p0["m"], p1["m"]) == (8, 32)
    assert p1["T_fwd"] / p0["T_fwd"] == pytest.approx((32 + 3) / 32 / ((8 + 3) / 8), rel=1e-12)
    # activations: with checkpointing off they scale with the micro-batch
    m0 = oracle.memory(job, 0, e, (4, 1, 1, 0, 0, 0, 0))
    m1 = oracle.memory(job, 0, e, (4, 1, 1, 0, 0, 0, 1))
    assert m1["act"] * 2 == m0["act"] and m1["params"] == m0["params"] and m1["opt"] == m0["opt"]
