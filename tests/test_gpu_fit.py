"""rubick_fit_models against the oracle's fit: same samples, same start.  Candidate values are built from
correctly rounded operations, so the two searches take identical decisions unless a comparison sits within
rounding of its threshold (the oracle reports the closest one per model): parameters must then be
bit-identical, and the error reached must agree to 1e-9 relative everywhere."""
import numpy as np
import pytest

import oracle
from gpu_util import Gpu, has_cuda
from helpers import fit_samples
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import workloads
from test_oracle_fit import NAMES, problem, with_coefficients

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not has_cuda(), reason="needs a CUDA device")]


def gpu_fit(gpu, jobs, sp, sc, sy, sweeps=14):
    t = gpu.torch
    J, S = sp.shape
    smp = np.zeros((J, S), dtype=rb.SAMPLE_DTYPE)
    smp["plan"], smp["cores"], smp["thr"] = sp, sc, sy
    d_jobs = gpu.jobs_to_device(jobs)
    d_smp = rb.to_device(smp)
    d_theta = gpu.empty(J * 7, t.float64)
    d_rmsle = gpu.empty(J * 2, t.float64)
    gpu.ctx.fit_models(d_jobs, J, d_smp, S, sweeps, d_theta, d_rmsle)
    gpu.ctx.sync()
    return d_theta.cpu().numpy().reshape(J, 7), d_rmsle.cpu().numpy().reshape(J, 2)


@pytest.mark.parametrize("name,J,S,noisy,sweeps", [("paper-scale", 64, 16, True, 14), ("paper-scale", 37, 9, False, 10),
                                                   ("cluster-512", 96, 24, True, 14)])
def test_fit_matches_the_oracle(name, J, S, noisy, sweeps):
    cfg, plans, sp, sc, sy = problem(J=J, S=S, seed=7, noisy=noisy, name=name)
    # the job record holds single-precision coefficients: start both sides from the same rounded values
    start = with_coefficients(cfg["jobs"], {k: np.float32(v) for k, v in workloads.FIT_NOMINAL.items()})
    want_theta, want_rmsle, margin = oracle.fit(start, plans, cfg["env"], sp, sc, sy, sweeps=sweeps)
    gpu = Gpu(cfg)
    theta, rmsle = gpu_fit(gpu, start, sp, sc, sy, sweeps=sweeps)
    assert np.allclose(rmsle, want_rmsle, rtol=1e-9, atol=1e-13)
    firm = margin > 1e-11                            # every decision of these fits is clear of rounding
    assert firm.mean() > 0.8
    assert np.array_equal(theta[firm], want_theta[firm])
    assert (theta == want_theta).all(axis=1).mean() > 0.95
    assert np.allclose(theta, want_theta, rtol=0.5)  # a flipped decision still lands next door
    assert np.all(rmsle[:, 1] <= rmsle[:, 0])


def test_fit_edge_cases():
    cfg, plans, sp, sc, sy = problem(J=12, S=8, seed=2, noisy=True)
    start = with_coefficients(cfg["jobs"], {k: np.float32(v) for k, v in workloads.FIT_NOMINAL.items()})
    gpu = Gpu(cfg)
    # no samples at all, samples with plans off the list, zero sweeps: the start comes back
    none = np.full_like(sp, -1)
    theta, rmsle = gpu_fit(gpu, start, none, sc, sy)
    want = np.stack([np.asarray(start[k], dtype=np.float32).astype(np.float64) for k in NAMES], axis=1)
    assert np.array_equal(theta, want) and not rmsle.any()
    theta, rmsle = gpu_fit(gpu, start, sp, sc, sy, sweeps=0)
    assert np.array_equal(theta, want) and np.array_equal(rmsle[:, 0], rmsle[:, 1])
    # starts outside the bounds are clamped on both sides
    wild = with_coefficients(start, dict(k_sync=np.float32(0.3), k_const=np.float32(50.0), k_opt=np.float32(0.0)))
    want_theta, want_rmsle, margin = oracle.fit(wild, plans, cfg["env"], sp, sc, sy, sweeps=6)
    theta, rmsle = gpu_fit(gpu, wild, sp, sc, sy, sweeps=6)
    assert np.allclose(rmsle, want_rmsle, rtol=1e-9, atol=1e-13)
    firm = margin > 1e-11
    assert np.array_equal(theta[firm], want_theta[firm])
    # argument validation
    t = gpu.torch
    d = gpu.empty(1024, t.float64)
    with pytest.raises(rb.RubickError):
        gpu.ctx.fit_models(d, 1, d, 0, 4, d, d)
    with pytest.raises(rb.RubickError):
        gpu.ctx.fit_models(d, 1, d, 4, 100, d, d)
    assert gpu.ctx.fit_models(None, 0, None, 4, 4, None, None) == 0
