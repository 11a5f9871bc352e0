"""Seeded synthetic workloads shaped like the paper's evaluation (Section 7).

This module only draws numbers.  It holds none of the scheduler's arithmetic and is the one
piece of code that both the CUDA library's tests and the CPU checker read their inputs from.

Shapes follow the paper's setting: transformer jobs between 125 M and 13 B / 70 B parameters
(Table 2 spans 86 M - 30 B), nodes of 8 GPUs (80 GB each) with 96 cores, 400 GB/s inside and
100 GB/s between nodes (Section 7).  The paper prints no fitted coefficients and its job
trace is not public in numeric form, so coefficients are a nominal constant times a
uniform factor in [0.5, 2] and arrivals are Poisson with log-normal lengths.

Every floating-point job coefficient is rounded to single precision here, so that a
double-precision consumer and a single-precision consumer start from identical values.
"""
import numpy as np

GIB = 1 << 30

# nominal coefficient values (constants of this generator; the paper gives none)
NOMINAL = dict(k_bwd=2.0, k_sync=2.0, k_opt=1e-11, k_opt_off=2e-8, k_off=2.0, k_swap=2.0, k_const=0.05)
PEAK_FLOPS_PER_SAMPLE_DIVISOR = 1.25e14      # tau nominal = 2 * P * s / 1.25e14 seconds per sample
ALPHA_ACT = 34                               # activation bytes per token x hidden per layer
HOST_BASE = 4 * GIB                          # host bytes per training process

ENV = dict(B_intra=400e9, B_inter=100e9, B_pcie=25e9, gpu_mem_bytes=80_000_000_000,
           gpus_per_node=8, cpus_per_node=96, mem_per_node_bytes=1024 * GIB, bytes_per_elem=2,
           strict_zero_dp_only=0, zero3_extra_volume=0)

CONFIGS = {
    # name: (seed, jobs, nodes, g levels, c levels, m levels [GiB], largest parameter count)
    "tiny": dict(seed=0, J=4, N=1, g=list(range(1, 9)), c=[4, 8, 16, 32], m=[64, 128, 256], pmax=13e9),
    "paper-scale": dict(seed=1, J=64, N=8, g=[1, 2, 4, 8, 16, 32, 64], c=list(range(4, 97, 4)),
                        m=list(range(32, 1025, 32)), pmax=13e9),
    "cluster-512": dict(seed=2, J=1024, N=64, g=[1 << i for i in range(9)], c=list(range(4, 97, 4)),
                        m=list(range(32, 1025, 32)), pmax=70e9),
    "throughput-stress": dict(seed=3, J=16384, N=512, g=[1 << i for i in range(9)], c=list(range(4, 97, 4)),
                              m=list(range(32, 1025, 32)), pmax=70e9),
    "events": dict(seed=4, J=4096, N=512, g=[1 << i for i in range(9)], c=list(range(4, 97, 4)),
                   m=list(range(32, 1025, 32)), pmax=70e9),
}


def _f32(x):
    return np.asarray(x, dtype=np.float32).astype(np.float64)


def draw_jobs(rng, J, g_levels, n_c_levels, pmax=13e9, pmin=125e6, guaranteed_share=0.25):
    """Per-job model inputs as a dict of length-J arrays, drawn field by field in a fixed order."""
    P = np.floor(np.exp(rng.uniform(np.log(pmin), np.log(pmax), J)))
    l = rng.integers(12, 49, J)
    h = 128 * rng.integers(768 // 128, 5120 // 128 + 1, J)
    b = rng.choice([16, 32, 64, 128], J)
    s = rng.choice([512, 1024, 2048], J)
    mu_cap = rng.choice([1, 2, 4, 8], J)
    tau = _f32(2.0 * P * s / PEAK_FLOPS_PER_SAMPLE_DIVISOR * rng.uniform(0.5, 2.0, J))
    jobs = dict(P=P, l=l, h=h, s=s, b=b, mu_cap=mu_cap, alpha_act=np.full(J, ALPHA_ACT), tau=tau)
    for k in ("k_bwd", "k_sync", "k_opt", "k_opt_off", "k_off", "k_swap", "k_const"):
        jobs[k] = _f32(NOMINAL[k] * rng.uniform(0.5, 2.0, J))
    # weight: seconds of one-GPU compute per sample, so that weighted throughput reads as a
    # speed-up over a one-GPU run and jobs of different sizes compare (Section 7.2 normalises
    # each job's throughput before adding them up)
    jobs["w"] = _f32(3.0 * tau)
    # a share of the jobs is "guaranteed" with a small minimum demand, the rest best effort
    pow2_idx = [i for i, g in enumerate(g_levels) if g & (g - 1) == 0][:4]
    guaranteed = rng.uniform(0.0, 1.0, J) < guaranteed_share
    gpick = rng.choice(pow2_idx, J)
    cpick = rng.integers(0, min(3, n_c_levels), J)
    jobs["gmin_idx"] = np.where(guaranteed, gpick, -1)
    jobs["cmin_idx"] = np.where(guaranteed, cpick, -1)
    jobs["host_base_bytes"] = np.full(J, HOST_BASE)
    return jobs


def draw_requests(seed, J, g_levels, n_c_levels, n_m_levels, guaranteed_share=0.5):
    """What users asked for (Section 5.1: a requested amount of resources and an original plan):
    level indices of GPUs / cores / host memory and `plan_rank` in [0, 1), the position of the
    original plan among the plans of the requested GPU level (-1 marks a best-effort job).  Drawn
    from a generator of its own so that the job fields above keep their values."""
    rng = np.random.Generator(np.random.PCG64(seed + 2000))
    pow2_idx = np.asarray([i for i, g in enumerate(g_levels) if g & (g - 1) == 0])
    g_idx = rng.choice(pow2_idx, J)
    c_idx = rng.integers(0, n_c_levels, J)
    m_idx = rng.integers(n_m_levels // 2, n_m_levels, J)
    rank = rng.uniform(0.0, 1.0, J)
    guaranteed = rng.uniform(0.0, 1.0, J) < guaranteed_share
    return dict(g_idx=g_idx, c_idx=c_idx, m_idx=m_idx, plan_rank=np.where(guaranteed, rank, -1.0))


def make(name, J=None, n_nodes=None, seed=None):
    """Build a named configuration; J / n_nodes override the size and seed the configuration's seed (same recipe)."""
    cfg = CONFIGS[name]
    seed = cfg["seed"] if seed is None else seed
    rng = np.random.Generator(np.random.PCG64(seed))
    J = cfg["J"] if J is None else J
    jobs = draw_jobs(rng, J, cfg["g"], len(cfg["c"]), pmax=cfg["pmax"])
    return dict(name=name, seed=seed, jobs=jobs, env=dict(ENV),
                g_levels=np.asarray(cfg["g"], dtype=np.int64),
                c_levels=np.asarray(cfg["c"], dtype=np.int64),
                m_levels=np.asarray(cfg["m"], dtype=np.int64) * GIB,
                n_nodes=cfg["N"] if n_nodes is None else n_nodes)


def take(jobs, idx):
    """Sub-select jobs (dict of arrays) by index array / slice."""
    return {k: np.asarray(v)[idx] for k, v in jobs.items()}


def reconf_cost(jobs, fixed_s=20.0, bytes_per_param=14.0, storage_bytes_per_s=5e9):
    """Checkpoint-resume seconds of each job (the delta of the reconfiguration gate, Section 5.2): a
    fixed restart time plus the optimizer and model states written and read back once over the
    checkpoint storage.  Generator constants; the paper prints no value."""
    P = np.asarray(jobs["P"], dtype=np.float64)
    return (fixed_s + 2.0 * bytes_per_param * P / storage_bytes_per_s).astype(np.float32)


FIT_NOMINAL = dict(k_bwd=2.0, k_sync=2.0, k_opt=1e-11, k_opt_off=2e-8, k_off=2.0, k_swap=2.0, k_const=0.05)


def draw_fit_picks(seed, J, S, n_c_levels, noise_sigma=0.03):
    """Random draws from which the tests and the benchmark build the measured samples of Section 4.3 for J
    model types: per sample slot a rank in [0, 1) used to pick a plan among those the job can run (the
    first third of the slots among offloading plans, as the paper asks for), a core-level index and a
    log-normal measurement-noise factor.  No model arithmetic here: the throughputs come from whoever
    uses the picks."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return dict(rank=rng.uniform(0.0, 1.0, (J, S)), c_idx=rng.integers(0, n_c_levels, (J, S)),
                noise=np.exp(rng.normal(0.0, noise_sigma, (J, S))))


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


def draw_events(seed, n_jobs, mean_interarrival_s=30.0, median_len_s=7200.0, sigma=1.5):
    """Arrival times (Poisson process) and nominal lengths (log-normal) for an event-driven run."""
    rng = np.random.Generator(np.random.PCG64(seed + 1000))
    arrivals = np.cumsum(rng.exponential(mean_interarrival_s, n_jobs))
    lengths = np.exp(rng.normal(np.log(median_len_s), sigma, n_jobs))
    return arrivals, lengths
