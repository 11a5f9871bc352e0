"""Pins of the oracle's performance model (paper Section 4) against what the paper and
plain mathematics fix: limits and closed forms of the overlap function, message counts of
a simulated ring all-reduce and a simulated pipeline, hand-worked numbers, the two
special cases the paper writes out for T_cc, homogeneity and monotonicity."""
import itertools
import math

import numpy as np
import pytest

import oracle
from helpers import env, one_job


# ---------------------------------------------------------------- overlap (Section 4.3)
def test_overlap_k1_is_sum():
    for x, y in [(0.3, 0.7), (5.0, 1e-3), (2.0, 2.0)]:
        assert oracle.overlap(1.0, x, y) == pytest.approx(x + y, rel=1e-14)


def test_overlap_large_k_tends_to_max():
    for x, y in [(0.3, 0.7), (5.0, 1e-3), (2.0, 2.5)]:
        assert oracle.overlap(200.0, x, y) == pytest.approx(max(x, y), rel=5e-3)
        assert oracle.overlap(2000.0, 0.3, 0.7) == pytest.approx(0.7, rel=1e-6)


def test_overlap_closed_forms():
    assert oracle.overlap(2.0, 3.0, 4.0) == pytest.approx(5.0, rel=1e-14)       # 3-4-5 triangle
    assert oracle.overlap(3.0, 1.0, 1.0) == pytest.approx(2.0 ** (1 / 3), rel=1e-14)
    assert oracle.overlap(4.0, 2.0, 2.0) == pytest.approx(2.0 * 2.0 ** 0.25, rel=1e-14)


def test_overlap_bounds_symmetry_monotone():
    rng = np.random.default_rng(0)
    for _ in range(200):
        x, y = rng.uniform(1e-4, 10, 2)
        k = rng.uniform(1.0, 6.0)
        f = oracle.overlap(k, x, y)
        assert max(x, y) * (1 - 1e-12) <= f <= (x + y) * (1 + 1e-12)
        assert f == pytest.approx(oracle.overlap(k, y, x), rel=1e-14)
        assert oracle.overlap(k, x * 1.1, y) > f and oracle.overlap(k, x, y * 1.1) > f
        assert oracle.overlap(k + 0.5, x, y) < f                                  # power mean order
        lam = rng.uniform(0.1, 10)
        assert oracle.overlap(k, lam * x, lam * y) == pytest.approx(lam * f, rel=1e-13)


def test_overlap_zero_stage():
    assert oracle.overlap(2.5, 0.0, 0.37) == 0.37
    assert oracle.overlap(2.5, 0.37, 0.0) == 0.37


# ---------------------------------------------------------------- communication volumes
def ring_allreduce_bytes_per_rank(n, size):
    """Simulate a ring all-reduce of `size` bytes over n ranks chunk by chunk and count what
    one rank sends: n-1 reduce-scatter steps then n-1 all-gather steps of size/n each."""
    sent = [0.0] * n
    chunk = size / n
    for _phase in range(2):
        for _step in range(n - 1):
            for r in range(n):
                sent[r] += chunk
    assert len(set(sent)) == 1
    return sent[0]


@pytest.mark.parametrize("d,t,p", [(2, 1, 1), (4, 2, 2), (8, 1, 4), (16, 4, 1), (64, 1, 1)])
def test_v_dp_is_ring_allreduce_of_the_shard(d, t, p):
    job = one_job(P=3e9, b=64, l=32)
    tm = oracle.terms(job, 0, env(), (d, t, p, 0, 0, 0), 8)
    assert tm["valid"] == 1
    shard_bytes = 2 * 3e9 / (t * p)                       # fp16 gradients of one TP x PP shard
    assert tm["V_dp"] == pytest.approx(ring_allreduce_bytes_per_rank(d, shard_bytes), rel=1e-12)


def test_v_dp_hand_number():
    # P = 1e9 parameters in fp16 = 2e9 bytes; d=4, t=2, p=2:  2e9 * 2*3 / 16 = 7.5e8
    tm = oracle.terms(one_job(P=1e9), 0, env(), (4, 2, 2, 0, 0, 0), 8)
    assert tm["V_dp"] == pytest.approx(7.5e8, rel=1e-14)
    assert tm["T_dp"] == pytest.approx(7.5e8 / 400e9, rel=1e-14)     # d*t = 8 fits one node
    tm = oracle.terms(one_job(P=1e9), 0, env(), (8, 2, 1, 0, 0, 0), 8)
    # d*t = 16 > 8 GPUs per node: the gradient ring crosses nodes
    assert tm["T_dp"] == pytest.approx(2e9 * 2 * 7 / 16 / 100e9, rel=1e-14)


@pytest.mark.parametrize("d,t", [(1, 2), (2, 4), (4, 8)])
def test_v_tp_is_four_allreduces_per_layer(d, t):
    b, s, h, l = 32, 1024, 2048, 24
    job = one_job(b=b, s=s, h=h, l=l)
    tm = oracle.terms(job, 0, env(), (d, t, 1, 0, 0, 0), 8)
    per_allreduce = ring_allreduce_bytes_per_rank(t, 2.0 * (b / d) * s * h)
    assert tm["V_tp"] == pytest.approx(4 * l * per_allreduce, rel=1e-12)
    assert tm["T_tp"] == pytest.approx(tm["V_tp"] / 400e9, rel=1e-14)


def test_v_pp_hand_number():
    # 2 * p * b*s*h / (d*t) elements, fp16: p=4, b=16, s=1024, h=2048, d=2, t=1
    tm = oracle.terms(one_job(), 0, env(), (2, 1, 4, 0, 0, 0), 8)
    assert tm["V_pp"] == pytest.approx(2 * 2 * 4 * 16 * 1024 * 2048 / 2, rel=1e-14)
    assert tm["T_pp"] == pytest.approx(tm["V_pp"] / 400e9, rel=1e-14)
    tm = oracle.terms(one_job(), 0, env(), (2, 1, 8, 0, 0, 0), 8)              # 16 GPUs: two nodes
    assert tm["T_pp"] == pytest.approx(tm["V_pp"] / 100e9, rel=1e-14)


def test_degree_one_sends_nothing():
    tm = oracle.terms(one_job(), 0, env(), (1, 1, 1, 3, 0, 0), 8)
    assert tm["V_dp"] == 0 and tm["V_tp"] == 0 and tm["V_pp"] == 0
    tm = oracle.terms(one_job(), 0, env(), (4, 1, 1, 0, 0, 0), 8)
    assert tm["V_dp"] > 0 and tm["V_tp"] == 0 and tm["V_pp"] == 0
    tm = oracle.terms(one_job(), 0, env(), (1, 4, 1, 0, 0, 0), 8)
    assert tm["V_dp"] == 0 and tm["V_tp"] > 0 and tm["V_pp"] == 0
    tm = oracle.terms(one_job(), 0, env(), (1, 1, 4, 0, 0, 0), 8)
    assert tm["V_dp"] == 0 and tm["V_tp"] == 0 and tm["V_pp"] > 0


def test_every_zero_stage_moves_the_ring_volume_of_section_4_1():
    """Section 4.1 gives V_dp = P 2(d-1)/(d t p) and applies it to the whole ZeRO series: with e = 2 bytes,
    P = 1e9, d = 4 that is 2 * 1e9 * 2 * 3 / 4 = 3e9 bytes for every stage.  The factor 1.5 for stage 3
    (parameter gathers) is an option of the environment, outside the paper and off by default."""
    for z in range(4):
        assert oracle.terms(one_job(), 0, env(), (4, 1, 1, z, 0, 0), 8)["V_dp"] == 3e9
    assert oracle.terms(one_job(), 0, env(), (2, 2, 1, 3, 0, 0), 8)["V_dp"] == 1e9        # 2 * 1e9 * 2 * 1 / (2 * 2)
    on = env(zero3_extra_volume=1)
    assert oracle.terms(one_job(), 0, on, (4, 1, 1, 3, 0, 0), 8)["V_dp"] == 4.5e9
    assert oracle.terms(one_job(), 0, on, (4, 1, 1, 2, 0, 0), 8)["V_dp"] == 3e9


# ---------------------------------------------------------------- pipeline forward time
def pipeline_forward_finish(p, m, slot):
    """Event simulation of m micro-batches flowing forward through p stages, each taking
    `slot` seconds: stage s starts micro-batch i when stage s-1 finished it and stage s
    finished micro-batch i-1."""
    done = [[0.0] * m for _ in range(p)]
    for s_ in range(p):
        for i in range(m):
            ready = max(done[s_ - 1][i] if s_ else 0.0, done[s_][i - 1] if i else 0.0)
            done[s_][i] = ready + slot
    return done[p - 1][m - 1]


@pytest.mark.parametrize("p,b,mu_cap,d", [(2, 16, 4, 1), (4, 32, 2, 2), (8, 64, 1, 1), (4, 16, 8, 4)])
def test_t_fwd_pipeline_bubble(p, b, mu_cap, d):
    tau = 0.02
    job = one_job(b=b, mu_cap=mu_cap, tau=tau, l=32)
    tm = oracle.terms(job, 0, env(), (d, 1, p, 0, 0, 0), 8)
    mu = min(b // d, mu_cap)
    m = (b // d) // mu
    assert tm["mu"] == mu and tm["m"] == m and tm["a"] == 1
    slot = tau * mu / p                                     # one stage = 1/p of the layers
    assert tm["T_fwd"] == pytest.approx(pipeline_forward_finish(p, m, slot), rel=1e-12)


def test_t_fwd_scales_with_batch_and_tensor_shard():
    base = oracle.terms(one_job(b=16, mu_cap=16), 0, env(), (1, 1, 1, 0, 0, 0), 8)["T_fwd"]
    assert base == pytest.approx(0.01 * 16, rel=1e-14)
    assert oracle.terms(one_job(b=16, mu_cap=16), 0, env(), (2, 1, 1, 0, 0, 0), 8)["T_fwd"] == pytest.approx(base / 2)
    assert oracle.terms(one_job(b=16, mu_cap=16), 0, env(), (1, 4, 1, 0, 0, 0), 8)["T_fwd"] == pytest.approx(base / 4)


def test_gradient_accumulation_steps():
    tm = oracle.terms(one_job(b=64, mu_cap=2), 0, env(), (4, 1, 1, 0, 0, 0), 8)
    assert (tm["mu"], tm["m"], tm["a"]) == (2, 1, 8)
    tm = oracle.terms(one_job(b=64, mu_cap=2), 0, env(), (4, 1, 2, 0, 0, 0), 8)
    assert (tm["mu"], tm["m"], tm["a"]) == (2, 8, 1)


def test_t_bwd_and_checkpointing():
    t0 = oracle.terms(one_job(k_bwd=1.75), 0, env(), (2, 2, 1, 0, 0, 0), 8)
    t1 = oracle.terms(one_job(k_bwd=1.75), 0, env(), (2, 2, 1, 0, 1, 0), 8)
    assert t0["T_bwd"] == pytest.approx(1.75 * t0["T_fwd"], rel=1e-14)
    assert t1["T_bwd"] == pytest.approx(t0["T_bwd"] + t0["T_fwd"], rel=1e-14)   # one more forward


# ---------------------------------------------------------------- combination: T_cc, T_oo, Eq. 1
def literal_3d(job, e, d, t, p, gc):
    """The 3D-parallel case exactly as the paper writes it (no accumulation):
    T_cc = T_fwd + f(T_bwd, T_dp) + T_tp + T_pp; T_opt = k_opt P / (t p); T_iter = T_cc + T_opt + k_const."""
    g = {k: float(v[0]) for k, v in job.items()}
    mu = min(g["b"] / d, g["mu_cap"])
    m = g["b"] / d / mu
    t_fwd = g["tau"] * mu / t / p * ((m + p - 1) if p > 1 else 1)
    t_bwd = g["k_bwd"] * t_fwd + (t_fwd if gc else 0)
    v_dp = 2 * g["P"] * 2 * (d - 1) / (d * t * p) if d > 1 else 0
    v_tp = 2 * 8 * (t - 1) * g["b"] * g["s"] * g["h"] * g["l"] / (d * t) if t > 1 else 0
    v_pp = 2 * 2 * p * g["b"] * g["s"] * g["h"] / (d * t) if p > 1 else 0
    b_dp = e["B_intra"] if d * t <= 8 else e["B_inter"]
    b_pp = e["B_intra"] if d * t * p <= 8 else e["B_inter"]
    ks = g["k_sync"]
    x, y = t_bwd, v_dp / b_dp
    f = (x ** ks + y ** ks) ** (1 / ks) if y > 0 else x
    t_cc = t_fwd + f + v_tp / e["B_intra"] + v_pp / b_pp
    return g["b"] / (t_cc + g["k_opt"] * g["P"] / (t * p) + g["k_const"])


def literal_dp_ga(job, e, d, zero, off, gc, c):
    """The data-parallel family with gradient accumulation as the paper writes it:
    T_cc = a T_fwd + (a-1) T_bwd + f(T_bwd, T_dp); T_opt = k_opt P / d under ZeRO-DP, k_opt P
    otherwise; under ZeRO-Offload T_oo = f_off(T_dp, T_off) + f_swap(k_opt_off P/(d c), T_off)."""
    g = {k: float(v[0]) for k, v in job.items()}
    mu = min(g["b"] / d, g["mu_cap"])
    a = g["b"] / d / mu
    t_fwd = g["tau"] * mu
    t_bwd = g["k_bwd"] * t_fwd + (t_fwd if gc else 0)
    t_dp = (2 * g["P"] * 2 * (d - 1) / d if d > 1 else 0) / (e["B_intra"] if d <= 8 else e["B_inter"])

    def f(k, x, y):
        if x == 0:
            return y
        if y == 0:
            return x
        return (x ** k + y ** k) ** (1 / k)
    t_cc = a * t_fwd + (a - 1) * t_bwd + f(g["k_sync"], t_bwd, t_dp)
    if off:
        t_off = 2 * g["P"] / (d * e["B_pcie"])
        t_oo = f(g["k_off"], t_dp, t_off) + f(g["k_swap"], g["k_opt_off"] * g["P"] / (d * c), t_off)
    else:
        t_oo = g["k_opt"] * g["P"] / (d if zero else 1)
    return g["b"] / (t_cc + t_oo + g["k_const"])


def test_unified_tcc_reduces_to_the_3d_case():
    e = env()
    job = one_job(P=6e9, b=64, mu_cap=64, l=32, h=4096, k_sync=1.7)     # mu_cap = b: never accumulates
    for d, t, p in itertools.product([1, 2, 4, 8], [1, 2, 4, 8], [1, 2, 4]):
        for gc in (0, 1):
            tm = oracle.terms(job, 0, e, (d, t, p, 0, gc, 0), 8)
            assert tm["valid"] == 1 and (tm["a"] == 1)
            assert tm["thr"] == pytest.approx(literal_3d(job, e, d, t, p, gc), rel=1e-12)


def test_unified_tcc_reduces_to_the_accumulation_case():
    e = env()
    job = one_job(P=1.3e9, b=128, mu_cap=2, k_sync=2.6, k_off=1.4, k_swap=3.1)
    for d in (1, 2, 4, 8, 16, 32):
        for z, off, gc in [(0, 0, 0), (0, 0, 1), (2, 0, 0), (2, 1, 0), (2, 1, 1), (1, 0, 0)]:
            for c in (4, 16, 64):
                tm = oracle.terms(job, 0, e, (d, 1, 1, z, gc, off), c)
                assert tm["valid"] == 1 and tm["a"] == 128 // d // 2
                assert tm["thr"] == pytest.approx(literal_dp_ga(job, e, d, z >= 1, off, gc, c), rel=1e-12)


def test_single_gpu_closed_form():
    # one GPU, no communication: T_iter = (1 + k_bwd) tau b + k_opt P + k_const
    #   = 3 * 0.01 * 16 + 1e-11 * 1e9 + 0.05 = 0.54 s  ->  16 / 0.54 samples per second
    tm = oracle.terms(one_job(), 0, env(), (1, 1, 1, 0, 0, 0), 4)
    assert tm["T_iter"] == pytest.approx(0.54, rel=1e-13)
    assert tm["thr"] == pytest.approx(16 / 0.54, rel=1e-13)


def test_iteration_time_is_the_sum_of_its_parts_when_nothing_overlaps():
    # k = 1 everywhere: every overlap is a plain sum, so Eq. 1 is additive in all terms
    job = one_job(P=2e9, b=64, mu_cap=2, k_sync=1.0, k_off=1.0, k_swap=1.0, l=32)
    tm = oracle.terms(job, 0, env(), (4, 2, 2, 2, 1, 1), 12)
    a = tm["a"]
    parts = (a * tm["T_fwd"] + a * tm["T_bwd"] + tm["T_dp"] + tm["T_tp"] + tm["T_pp"]
             + tm["T_dp"] + tm["T_off"] + tm["T_opt"] + tm["T_off"] + 0.05)
    assert tm["T_iter"] == pytest.approx(parts, rel=1e-13)
    assert tm["thr"] == pytest.approx(64 / tm["T_iter"], rel=1e-14)


def test_optimizer_time_cases():
    P = 2e9
    base = dict(P=P, k_opt=3e-11, k_opt_off=5e-8)
    assert oracle.terms(one_job(**base), 0, env(), (2, 2, 2, 0, 0, 0), 8)["T_opt"] == pytest.approx(3e-11 * P / 4)
    assert oracle.terms(one_job(**base), 0, env(), (8, 1, 1, 2, 0, 0), 8)["T_opt"] == pytest.approx(3e-11 * P / 8)
    t = oracle.terms(one_job(**base), 0, env(), (4, 1, 1, 2, 0, 1), 24)
    assert t["T_opt"] == pytest.approx(5e-8 * P / (4 * 24))
    assert t["T_off"] == pytest.approx(2 * P / (4 * 25e9))


def test_homogeneity_in_time_units():
    """Measuring time in another unit (all time coefficients x lam, bandwidths / lam) scales
    the predicted throughput by 1 / lam: catches a term with the wrong units."""
    lam = 3.7
    job = one_job(P=5e9, b=64, mu_cap=2, l=40, h=4096)
    job2 = {k: v.copy() for k, v in job.items()}
    for k in ("tau", "k_opt", "k_opt_off", "k_const"):
        job2[k] = job2[k] * lam
    e2 = env(B_intra=400e9 / lam, B_inter=100e9 / lam, B_pcie=25e9 / lam)
    for plan in [(4, 2, 2, 0, 0, 0), (8, 1, 1, 2, 1, 1), (2, 4, 4, 3, 1, 0), (16, 1, 2, 2, 0, 1)]:
        a = oracle.terms(job, 0, env(), plan, 16)["thr"]
        b = oracle.terms(job2, 0, e2, plan, 16)["thr"]
        assert a > 0 and b == pytest.approx(a / lam, rel=1e-12)


def test_cpu_cores_matter_only_under_offload():
    job = one_job(P=7e9, b=32, mu_cap=1, l=32, h=4096, s=2048)
    cs = [4, 8, 16, 32, 64, 96]
    for plan in [(1, 1, 1, 0, 0, 0), (4, 2, 1, 2, 1, 0), (2, 1, 4, 3, 0, 0)]:
        v = [oracle.terms(job, 0, env(), plan, c)["thr"] for c in cs]
        assert len(set(v)) == 1
    for plan in [(1, 1, 1, 2, 0, 1), (4, 1, 1, 3, 1, 1), (2, 2, 2, 2, 0, 1)]:
        v = [oracle.terms(job, 0, env(), plan, c)["thr"] for c in cs]
        assert all(b > a for a, b in zip(v, v[1:]))
        # doubling the cores helps by at most 2x (the paper measured 1.7x on LLaMA-2-7B, Section 7.2)
        assert all(1.0 < b / a < 2.0 for a, b in zip(v[:-2], v[1:-1]))


def test_structural_validity():
    e = env()
    assert oracle.terms(one_job(), 0, e, (1, 16, 1, 0, 0, 0), 8)["valid"] == 0      # TP beyond a node
    assert oracle.terms(one_job(l=4), 0, e, (1, 1, 8, 0, 0, 0), 8)["valid"] == 0    # more stages than layers
    assert oracle.terms(one_job(b=16), 0, e, (32, 1, 1, 0, 0, 0), 8)["valid"] == 0  # replicas > batch
    assert oracle.terms(one_job(), 0, e, (2, 1, 1, 0, 0, 1), 8)["valid"] == 0       # offload needs ZeRO-2/3
    assert oracle.terms(one_job(), 0, e, (2, 1, 1, 1, 0, 1), 8)["valid"] == 0
    assert oracle.terms(one_job(), 0, e, (2, 1, 1, 2, 0, 1), 8)["valid"] == 1
    assert oracle.terms(one_job(h=2052), 0, e, (1, 8, 1, 0, 0, 0), 8)["valid"] == 0      # 2052 % 8 != 0
    strict = env(strict_zero_dp_only=1)
    assert oracle.terms(one_job(), 0, strict, (2, 2, 1, 2, 0, 0), 8)["valid"] == 0
    assert oracle.terms(one_job(), 0, strict, (2, 2, 1, 0, 0, 0), 8)["valid"] == 1
    assert oracle.terms(one_job(), 0, strict, (4, 1, 1, 2, 0, 1), 8)["valid"] == 1


def test_table_matches_terms(tiny):
    plans, _ = oracle.enumerate_plans(tiny["g_levels"])
    thr, feas = oracle.eval_candidates(tiny["jobs"], plans, tiny["env"], tiny["c_levels"], tiny["m_levels"])
    rng = np.random.default_rng(1)
    for _ in range(200):
        j, ci, pi = rng.integers(4), rng.integers(4), rng.integers(len(plans))
        tm = oracle.terms(tiny["jobs"], j, tiny["env"], plans[pi], tiny["c_levels"][ci])
        assert thr[j, ci, pi] == (tm["thr"] if tm["valid"] else 0.0)
        assert int(feas[j, pi]) == oracle.feas_word(tiny["jobs"], j, tiny["env"], plans[pi], tiny["m_levels"])
    assert math.isfinite(thr.max()) and thr.min() >= 0
