"""Parity of rubick_min_resources with the oracle (paper Section 5.2: minimum demand of guaranteed
jobs).  Level indices are integer decisions: bit exact on the same table; through the
single-precision chain they may differ only where the oracle's curve is within 1e-6 of the
guaranteed performance."""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, has_cuda
from helpers import requests_for
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def run_gpu(gpu, d_thr, d_feas, d_cv, req):
    t = gpu.torch
    J = len(req)
    rec = np.zeros(J, dtype=rb.REQUEST_DTYPE)
    rec["g_idx"], rec["c_idx"], rec["m_idx"], rec["plan"] = req[:, 0], req[:, 1], req[:, 2], req[:, 3]
    gm, cm, base = gpu.empty(J, t.int32), gpu.empty(J, t.int32), gpu.empty(J, t.float32)
    gpu.ctx.min_resources(d_thr, d_feas, d_cv, J, rb.to_device(rec), gm, cm, base)
    gpu.ctx.sync()
    return gm.cpu().numpy(), cm.cpu().numpy(), base.cpu().numpy()


@pytest.mark.parametrize("name,J", [("tiny", None), ("paper-scale", None), ("cluster-512", 700)])
def test_on_the_oracle_tables_it_is_bit_exact(name, J):
    cfg = workloads.make(name, J=J)
    gpu = Gpu(cfg)
    t = gpu.torch
    Jn = len(cfg["jobs"]["P"])
    plans, goff = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=8)
    thr32 = thr.astype(np.float32)
    cv, _, _ = oracle.best_plan(thr32, feas, plans, cfg["g_levels"], gpu.nM, prefix=True, nthreads=8)
    req = requests_for(cfg, goff, guaranteed_share=0.7)
    req[0] = [99, 0, 0, 5]                                         # off the grid: no guarantee can be stated
    want = oracle.min_resources(thr32, feas, cv, plans, cfg["g_levels"], req)
    got = run_gpu(gpu, t.from_numpy(thr32.reshape(-1)).cuda(), t.from_numpy(feas.view(np.int32).reshape(-1)).cuda(),
                  t.from_numpy(cv.astype(np.float32).reshape(-1)).cuda(), req)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    assert np.array_equal(got[2], want[2].astype(np.float32))
    assert got[0][0] == -1 and (got[0][1:] >= 0).any() and (got[0] == -1).sum() > 1


def test_through_the_single_precision_chain():
    cfg = workloads.make("cluster-512", J=800)
    gpu = Gpu(cfg)
    J = 800
    _, d_thr, d_feas = gpu.eval(cfg["jobs"])
    d_cv, _, _ = gpu.best(d_thr, d_feas, J)
    plans, goff = oracle.enumerate_plans(cfg["g_levels"])
    req = requests_for(cfg, goff, guaranteed_share=0.7)
    gm, cm, base = run_gpu(gpu, d_thr, d_feas, d_cv, req)
    thr, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=8)
    cv, _, _ = oracle.best_plan(thr, feas, plans, cfg["g_levels"], gpu.nM, prefix=True, nthreads=8)
    wg, wc, wb = oracle.min_resources(thr, feas, cv, plans, cfg["g_levels"], req)
    nz = wb > 0
    assert np.array_equal(base > 0, nz) and np.allclose(base[nz], wb[nz], rtol=1e-5, atol=0)
    same = (gm == wg) & (cm == wc)
    # a different answer is legitimate only at a near tie between a curve value and the guarantee
    for j in np.nonzero(~same)[0]:
        m = req[j, 2]
        a, b = cv[j, gm[j], cm[j], m], cv[j, wg[j], wc[j], m]
        assert min(abs(a - wb[j]), abs(b - wb[j])) <= 1e-5 * wb[j]
    assert same.mean() > 0.98
