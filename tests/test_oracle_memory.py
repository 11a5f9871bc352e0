"""Pins of the oracle's memory-feasibility rule.

The paper prints no memory formula (it relies on the training frameworks' estimators), so
the rule is this project's reading and is "unpinned by the paper" beyond the qualitative
facts below; they are listed with their sources in tests/golden/paper_facts.txt.  The rule
is additionally recomputed here with Python integers, term by term, from its description."""
import os

import numpy as np
import pytest

import oracle
from helpers import GIB, env, one_job
from paper_2408_08586_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")


def facts():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def all_single_gpu_plans():
    return [(1, 1, 1, z, gc, off) for z in range(4) for gc in range(2) for off in range(2)]


def test_7b_on_one_80gb_gpu_only_offload_is_feasible():
    f = facts()
    job = one_job(P=f["llama2_7b_params"], l=32, h=4096, s=2048, b=32, mu_cap=1)
    e = env(gpu_mem_bytes=int(f["a800_gpu_bytes"]))
    levels = [1024 * GIB]
    ok = {pl: oracle.feas_word(job, 0, e, pl, levels) for pl in all_single_gpu_plans()}
    assert any(ok[pl] for pl in ok if pl[5] == 1)                  # ZeRO-Offload runs
    assert not any(ok[pl] for pl in ok if pl[5] == 0)              # nothing else does
    # switching to offload raises the host-memory demand (Section 7.2)
    need_off = oracle.memory(job, 0, e, (1, 1, 1, 2, 0, 1))["host_need"]
    need_no = oracle.memory(job, 0, e, (1, 1, 1, 0, 0, 0))["host_need"]
    assert need_off > need_no


def test_offload_of_a_1_2b_model_fails_with_10gb_of_host_memory():
    f = facts()
    job = one_job(P=f["t5_params"], l=24, h=2048, s=512, b=16, mu_cap=4, host_base_bytes=0)
    word = oracle.feas_word(job, 0, env(), (1, 1, 1, 2, 1, 1), [int(f["t5_failing_host_bytes"]), 64 * GIB])
    assert word == 0b10                                           # fails at 10 GB, runs with more


def py_rule(job, e, plan, m_levels):
    """The rule again with Python integers: model states 2 + 2 + 12 bytes per shard parameter
    with ZeRO stage 1 / 2 / 3 spreading optimizer / gradients / parameters over the replicas,
    offload moving gradients and optimizer to the host (14 bytes per parameter there),
    activations per layer alpha*s*mu*h/t (2*s*mu*h kept + one layer live under checkpointing)
    for the layers of one stage and the micro-batches in flight."""
    d, t, p, z, gc, off = plan[:6]
    ga = plan[6] if len(plan) > 6 else 0              # explicit accumulation: the micro-batch halved ga times
    g = {k: int(v[0]) for k, v in job.items() if k not in ("tau", "k_bwd", "k_sync", "k_opt", "k_opt_off",
                                                            "k_off", "k_swap", "k_const", "w")}
    cd = lambda a, b: -(-a // b)
    Gn = e["gpus_per_node"]
    if t > Gn or p > g["l"] or d > g["b"] or g["b"] % d or (off and z < 2) or g["h"] % t:
        return 0
    r = g["b"] // d
    mu = min(r, g["mu_cap"]) >> ga
    if mu < 1:
        return 0
    n = cd(r, mu)
    m = n if p > 1 else 1
    psi = cd(g["P"], t * p)
    states = 2 * cd(psi, d if z == 3 else 1)
    if not off:
        states += 2 * cd(psi, d if z >= 2 else 1) + 12 * cd(psi, d if z >= 1 else 1)
    A = cd(g["alpha_act"] * g["s"] * mu * g["h"], t)
    q = min(m, p) if p > 1 else 1
    L = cd(g["l"], p)
    act = L * q * 2 * g["s"] * mu * g["h"] + A if gc else L * q * A
    if states + act > e["gpu_mem_bytes"]:
        return 0
    gpus = d * t * p
    need = gpus * g["host_base_bytes"] + (14 * g["P"] if off else 0)
    nodes = 1 if gpus <= Gn else gpus // Gn
    word = 0
    for i, lv in enumerate(m_levels):
        if need <= lv and cd(need, nodes) <= e["mem_per_node_bytes"]:
            word |= 1 << i
    return word


def test_rule_recomputed_with_python_integers(paper_scale):
    cfg = paper_scale
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    _, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"][:1], cfg["m_levels"])
    rng = np.random.default_rng(5)
    from paper_2408_08586_b200 import workloads
    n_set = 0
    for _ in range(3000):
        j, pi = int(rng.integers(64)), int(rng.integers(len(plans)))
        job = workloads.take(cfg["jobs"], slice(j, j + 1))
        want = py_rule(job, cfg["env"], tuple(int(x) for x in plans[pi]), [int(x) for x in cfg["m_levels"]])
        assert int(feas[j, pi]) == want
        n_set += want != 0
    assert 300 < n_set < 2700                                       # both outcomes are exercised


def test_words_are_thresholds_and_memory_only_helps(paper_scale):
    cfg = paper_scale
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    _, feas = oracle.eval_candidates(cfg["jobs"], plans, cfg["env"], cfg["c_levels"][:1], cfg["m_levels"])
    nM = len(cfg["m_levels"])
    full = (1 << nM) - 1
    w = feas.astype(np.uint64)
    lowest = w & (~w + np.uint64(1))                               # lowest set bit
    # feasible at a level => feasible at every larger one
    assert np.all((w == 0) | (w == (np.uint64(full) & ~(lowest - np.uint64(1)))))


def test_feasibility_exactly_at_the_gpu_memory_bound():
    job = one_job(P=2e9, l=24, h=2048, s=1024, b=16, mu_cap=4)
    plan = (2, 2, 1, 1, 0, 0)
    total = oracle.memory(job, 0, env(), plan)["gpu_total"]
    lv = [1024 * GIB]
    assert oracle.feas_word(job, 0, env(gpu_mem_bytes=total), plan, lv) == 1
    assert oracle.feas_word(job, 0, env(gpu_mem_bytes=total - 1), plan, lv) == 0
    need = oracle.memory(job, 0, env(), plan)["host_need"]
    assert oracle.feas_word(job, 0, env(), plan, [need - 1, need, need + 1]) == 0b110


def test_memory_terms_by_hand():
    # P = 1e9, t*p = 4 -> shard 2.5e8 parameters; d = 4
    job = one_job(P=1e9, l=24, h=2048, s=1024, b=16, mu_cap=4, alpha_act=34)
    m0 = oracle.memory(job, 0, env(), (4, 2, 2, 0, 0, 0))
    assert (m0["params"], m0["grads"], m0["opt"]) == (5 * 10**8, 5 * 10**8, 3 * 10**9)
    m1 = oracle.memory(job, 0, env(), (4, 2, 2, 1, 0, 0))
    assert (m1["params"], m1["grads"], m1["opt"]) == (5 * 10**8, 5 * 10**8, 75 * 10**7)
    m2 = oracle.memory(job, 0, env(), (4, 2, 2, 2, 0, 0))
    assert (m2["params"], m2["grads"], m2["opt"]) == (5 * 10**8, 125 * 10**6, 75 * 10**7)
    m3 = oracle.memory(job, 0, env(), (4, 2, 2, 3, 0, 0))
    assert (m3["params"], m3["grads"], m3["opt"]) == (125 * 10**6, 125 * 10**6, 75 * 10**7)
    mo = oracle.memory(job, 0, env(), (4, 2, 2, 2, 0, 1))
    assert (mo["params"], mo["grads"], mo["opt"]) == (5 * 10**8, 0, 0)
    assert mo["host_need"] == 16 * 4 * GIB + 14 * 10**9 and mo["nodes"] == 2
    # activations: r = 4, mu = 4, m = 1 -> q = min(1, 2) = 1; 12 layers per stage;
    # per layer 34 * 1024 * 4 * 2048 / 2 bytes
    A = 34 * 1024 * 4 * 2048 // 2
    assert m0["act"] == 12 * A
    mg = oracle.memory(job, 0, env(), (4, 2, 2, 0, 1, 0))
    assert mg["act"] == 12 * 2 * 1024 * 4 * 2048 + A


def test_micro_batches_in_flight_and_layers_per_stage_by_hand():
    """A pipelined plan with more micro-batches than stages: b = 64, d = 2 -> 32 samples per replica in
    micro-batches of 2 -> m = 16 > p = 4, so 4 micro-batches are in flight (the smaller of the two);
    26 layers over 4 stages -> 7 on the fullest stage (rounded up).  t = 2.
    Per layer and micro-batch 34 * 1024 * 2 * 2048 / 2 = 71,303,168 bytes."""
    job = one_job(P=1e9, l=26, h=2048, s=1024, b=64, mu_cap=2, alpha_act=34)
    plain = oracle.memory(job, 0, env(), (2, 2, 4, 0, 0, 0))
    assert plain["act"] == 1_996_488_704                      # 7 layers * 4 in flight * 71,303,168
    ckpt = oracle.memory(job, 0, env(), (2, 2, 4, 0, 1, 0))
    assert ckpt["act"] == 306_184_192                         # 28 * (2 * 1024 * 2 * 2048) + one live layer
    # fewer micro-batches than stages: b = 8, d = 2, micro-batch 2 -> m = 2 < p = 4 -> 2 in flight
    few = oracle.memory(one_job(P=1e9, l=26, h=2048, s=1024, b=8, mu_cap=2, alpha_act=34), 0, env(), (2, 2, 4, 0, 0, 0))
    assert few["act"] == 998_244_352                          # 7 * 2 * 71,303,168
    tm = oracle.terms(job, 0, env(), (2, 2, 4, 0, 0, 0), 8)
    assert (tm["mu"], tm["m"], tm["a"]) == (2, 16, 1)


def test_per_node_share_of_host_memory_on_a_multi_node_plan_by_hand():
    """32 GPUs = 4 whole nodes, ZeRO-Offload: host need = 32 * 4 GiB + 14 * (1e11 + 1) = 1,537,438,953,486
    bytes, a quarter of it per node = 384,359,738,371.5 -> 384,359,738,372 (rounded up).  The plan runs at a
    memory level that covers the total only if a node also holds its share."""
    job = one_job(P=100_000_000_001, l=24, h=2048, s=1024, b=16, mu_cap=1)
    plan = (4, 8, 1, 2, 0, 1)
    levels = [1400 * GIB, 1500 * GIB]                         # below / above the total need
    mem = oracle.memory(job, 0, env(), plan)
    assert mem["host_need"] == 1_537_438_953_486 and mem["nodes"] == 4 and mem["gpu_ok"] == 1
    assert oracle.feas_word(job, 0, env(mem_per_node_bytes=384_359_738_372), plan, levels) == 0b10
    assert oracle.feas_word(job, 0, env(mem_per_node_bytes=384_359_738_371), plan, levels) == 0
    # on one node (8 GPUs) the whole need sits on that node
    one = oracle.memory(job, 0, env(), (1, 8, 1, 2, 0, 1))
    assert one["host_need"] == 8 * 4 * GIB + 1_400_000_000_014 and one["nodes"] == 1
    assert oracle.feas_word(job, 0, env(mem_per_node_bytes=one["host_need"] - 1), (1, 8, 1, 2, 0, 1), [2048 * GIB]) == 0


def test_rule_on_the_wider_plan_space_with_python_integers(paper_scale):
    """Degrees of any size and the explicit accumulation axis: the same independent recomputation."""
    cfg = dict(paper_scale)
    cfg["g_levels"] = np.array([1, 2, 3, 4, 6, 8, 16, 24])
    jobs = {k: np.asarray(v).copy() for k, v in cfg["jobs"].items()}
    rng = np.random.default_rng(9)
    jobs["h"] = rng.choice([768, 1536, 3072, 1920], 64)
    jobs["b"] = rng.choice([48, 96, 24, 64], 64)
    plans, _ = oracle.enumerate_plans(cfg["g_levels"], any_degrees=True, accumulation_levels=3)
    assert len(plans) % 48 == 0 and set(plans[:, 6]) == {0, 1, 2}
    _, feas = oracle.eval_candidates(jobs, plans, cfg["env"], cfg["c_levels"][:1], cfg["m_levels"])
    seen_ga = 0
    for _ in range(4000):
        j, pi = int(rng.integers(64)), int(rng.integers(len(plans)))
        job = workloads.take(jobs, [j])
        want = py_rule(job, cfg["env"], tuple(int(x) for x in plans[pi]), [int(x) for x in cfg["m_levels"]])
        assert int(feas[j, pi]) == want, (j, pi, plans[pi])
        seen_ga += int(want != 0 and plans[pi, 6] > 0)
    assert seen_ga > 50
    # more accumulation never makes a plan that fits stop fitting in GPU memory, and lets some plans fit that did not
    base = feas[:, plans[:, 6] == 0] != 0
    more = feas[:, plans[:, 6] == 2] != 0
    can_halve_twice = np.zeros_like(base)
    for j in range(64):
        r = jobs["b"][j] // np.maximum(plans[plans[:, 6] == 0, 0], 1)
        can_halve_twice[j] = np.minimum(r, jobs["mu_cap"][j]) >= 4
    assert not (base & ~more & can_halve_twice).any()
    assert (more & ~base).any()
