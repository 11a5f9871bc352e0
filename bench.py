#!/usr/bin/env python
"""Benchmark of the Rubick scheduler hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole path over one synthetic batch of jobs: candidate table +
feasibility mask, best plans and sensitivity curves, marginal gains, and one greedy scheduling
round, each through the C ABI with inputs resident in HBM.  Rank 0 prints one JSON line.  With
N > 1 (torchrun) every rank runs the path on its own independent batch (another tenant's
cluster: same recipe, another seed); there is no data-path collective, times are the maximum
over ranks, and `value` is the job total.

`--impl reference` times the CPU checker (oracle/) as it stands on a bounded sample of the same
workload; it is a deliberately slow program and serves as a reported baseline only.
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2408_08586_b200 import workloads  # noqa: E402

METRIC = "candidate_evals_per_sec"
UNIT = "stored candidate evaluations/s (job x plan x cpu-level; host-memory levels resolved by mask bits)"
UNIT_E2E = "candidate evaluations/s (job x plan x cpu-level; evaluated inside the one-pass curves kernel, not stored)"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one eval_candidates launch from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum)
# on `jobs` jobs; valid only for the kernel source it was taken on (sha1 of k_eval.cu), otherwise reported as
# null.  The capture lies BELOW the algorithmic bytes by a constant (57 MB at 2,048 jobs, 58 MB at 4,096): the last
# lines written are still dirty in the 126 MB L2 when the kernel ends.  A full launch is therefore reported as its
# algorithmic bytes less that residue.
NCU_EVAL_TRAFFIC = {"k_eval_sha1": "d2990fdbd7a2c785469d255f508032ccc14a673b", "jobs": 4096, "dram_bytes": 1022851840 + 645888}


# Single-precision and transcendental-unit instructions of the evaluation code per (job, plan quad), counted from
# eval_quad in k_eval.cu (power-of-two instance): what does not depend on the core count (forward / backward,
# three communication times, two overlaps with the gradient ring, two divisions into throughputs, their reciprocals
# of exponents), the offload prelude (transfer time, one overlap, two reciprocals) and, per core level, a quarter of a
# swap overlap plus one reciprocal-multiply.  A division counts as 1 transcendental + 7 single-precision instructions,
# an overlap f^k as 5 + 5.
def eval_quad_ops(C):
    fp32 = 68 + 24 + 3.5 * C
    xu = 13 + 7 + 2.25 * C
    return fp32, xu


def shard_seed_offset(rank):
    """Each rank schedules an independent cluster drawn from the same recipe."""
    return 100 * rank


def _reduce(x, world, op_name):
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def reduce_max_ms(ms, world):
    """Max over ranks of a per-rank time (the job is as slow as its slowest rank)."""
    return _reduce(ms, world, "MAX")


def reduce_sum(x, world):
    return _reduce(x, world, "SUM")


def make_workload(name, rank=0, J=None, n_nodes=None):
    return workloads.make(name, J=J, n_nodes=n_nodes, seed=workloads.CONFIGS[name]["seed"] + shard_seed_offset(rank))


def sort_launches(J, tile=2048):
    """Launches of the round's key sort: tiles of 2,048 keys are sorted in shared memory; every later stage of the
    bitonic network takes one launch per stride of a tile or more and one for the strides inside the tiles."""
    n = 2
    while n < J:
        n <<= 1
    t = min(n, tile)
    launches, k = 1, 2 * t
    while k <= n:
        launches += (k // 2).bit_length() - t.bit_length() + 1 + 1
        k <<= 1
    return launches


def algorithmic_bytes_eval(J, P, C):
    """Bytes one eval_candidates launch must move: 4 per stored candidate (the table), 4 per
    (job, plan) (the mask word), 128 per job (its record)."""
    return 4.0 * J * P * C + 4.0 * J * P + 128.0 * J


def algorithmic_bytes_best(J, P, C, G, M):
    """best_plan: reads the table and the mask once, writes value + plan + g per (j, g, c, m)."""
    return 4.0 * J * P * C + 4.0 * J * P + 12.0 * J * G * C * M


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "of measured (MEASURED_PEAKS.json hbm_gbs: copy, read + write bytes)"
    except Exception:
        return FALLBACK_HBM_GBS, "of fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_sample(cfg, J_sample, n_nodes, nthreads):
    """One pass of the checker over the first J_sample jobs: table, curves, round -> (seconds, P, seconds per stage).
    The table and the curves run on `nthreads` threads (OpenMP over jobs); the round is sequential by nature and
    always runs on one."""
    import oracle
    jobs = workloads.take(cfg["jobs"], slice(0, J_sample))
    t0 = time.perf_counter()
    plans, _ = oracle.enumerate_plans(cfg["g_levels"])
    thr, feas = oracle.eval_candidates(jobs, plans, cfg["env"], cfg["c_levels"], cfg["m_levels"], nthreads=nthreads)
    t1 = time.perf_counter()
    cv, cp, cg = oracle.best_plan(thr.astype(np.float32), feas, plans, cfg["g_levels"], len(cfg["m_levels"]), nthreads=nthreads)
    t2 = time.perf_counter()
    oracle.schedule_round(jobs, cfg["env"], cv.astype(np.float32), cp, cg, feas, cfg["g_levels"], cfg["c_levels"],
                          cfg["m_levels"], n_nodes)
    t3 = time.perf_counter()
    return t3 - t0, len(plans), {"table": t1 - t0, "curves": t2 - t1, "round": t3 - t2}


def baseline_record(cfg, J_s, nodes_s, threads, J_full):
    dt, P, stages = oracle_sample(cfg, J_s, nodes_s, threads)
    C = len(cfg["c_levels"])
    return {"value": J_s * P * C / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "cores_per_stage": {"table": threads, "curves": threads, "round": 1},
            "stages_s": {k: round(v, 3) for k, v in stages.items()},
            "sample": f"first {J_s} of {J_full} jobs on {nodes_s} nodes, one pass: table + curves + greedy round ({dt:.1f} s); "
                      "the round's cost grows faster than the job count, so the figure depends on the sample size"}


def run_reference(args):
    """The CPU checker as the reference arm: rank 0 only, a bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg = make_workload(args.workload, J=args.jobs, n_nodes=args.nodes)
    J_full = len(cfg["jobs"]["P"])
    threads = max(1, args.ref_threads)                    # single thread unless asked otherwise: the primary baseline
    J_s = min(J_full, args.ref_jobs if args.ref_jobs else (96 if threads == 1 else 1024))
    nodes = max(1, cfg["n_nodes"] * J_s // J_full)
    for _ in range(args.warmup):
        oracle_sample(cfg, min(J_s, 16), nodes, threads)
    t = 0.0
    P = 0
    stages = {"table": 0.0, "curves": 0.0, "round": 0.0}
    for _ in range(args.steps):
        dt, P, st = oracle_sample(cfg, J_s, nodes, threads)
        t += dt
        for k in stages:
            stages[k] += st[k]
    C = len(cfg["c_levels"])
    value = J_s * P * C * args.steps / t
    sample = (f"first {J_s} of {J_full} jobs on {nodes} nodes per step: table + curves + greedy round; the round's cost grows "
              "faster than the job count, so the figure depends on the sample size")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "jobs": J_s, "plans": P, "cpu_levels": C, "nodes": nodes},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "cores_per_stage": {"table": threads, "curves": threads, "round": 1},
                             "stages_s_per_step": {k: round(v / args.steps, 4) for k, v in stages.items()}},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_strong(args, cfg, rank, world, local, dev):
    """One problem on all GPUs (paper Section 5.2: the curves of different jobs are independent and "can be computed
    in parallel"): rank r builds mask and curves of its contiguous job tile with rubick_curves, one all-gather per
    table brings every tile into every rank's HBM, and every rank runs the same greedy round on the full tables
    (a round needs a global arg-max per step, so it is replicated, not sharded).  All ranks must reach the same
    allocation; that is checked after the timed region."""
    import torch
    import torch.distributed as dist
    from paper_2408_08586_b200 import binding as rb
    from paper_2408_08586_b200 import sharding
    jobs, N = cfg["jobs"], cfg["n_nodes"]
    J = len(jobs["P"])
    plans, _ = rb.enumerate_plans(cfg["g_levels"])
    P, G, C, M = len(plans), len(cfg["g_levels"]), len(cfg["c_levels"]), len(cfg["m_levels"])
    stream = torch.cuda.Stream(device=dev)
    ctx = rb.Context(cfg["env"], device=local, stream=stream.cuda_stream)
    ctx.set_space(plans, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])
    d_jobs = rb.to_device(rb.pack_jobs(jobs), dev)
    rows = sharding.table_rows(P, G, C, M)
    cap = sharding.tile_capacity(J, world)
    start, count = sharding.job_tile(J, world, rank)
    tile = {k: torch.zeros(cap * n, dtype=dt, device=dev) for k, (n, dt) in rows.items()}
    full = {k: torch.empty(J * n, dtype=dt, device=dev) for k, (n, dt) in rows.items()}
    d_out = torch.empty(J * rb.ASSIGN_DTYPE.itemsize + N * rb.NODE_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    d_assign, d_node = d_out[: J * rb.ASSIGN_DTYPE.itemsize], d_out[J * rb.ASSIGN_DTYPE.itemsize:]
    compute = sharding.curves_tile_fn(ctx, d_jobs, rb.JOB_DTYPE.itemsize)
    steps_taken = [0]

    def step():
        with torch.cuda.stream(stream):
            if count:
                compute(start, count, tile)
            for k, (n, _) in rows.items():
                sharding.gather_tiles(tile[k], J, world, n, full[k])
            steps_taken[0], _ = ctx.greedy_round(d_jobs, J, full["cv"], full["cp"], full["cg"], full["feas"], N, 1 << 30, d_assign, d_node)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    barrier()
    launches_before = rb.kernel_launches()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        step()
    b.record(stream)
    barrier()
    gpu_launches = rb.kernel_launches() - launches_before
    clocks = sampler.stop() if sampler else None
    ms_per_step = reduce_max_ms(a.elapsed_time(b), world) / args.steps
    agree = sharding.assignments_agree(d_out, world)
    if not agree:
        raise SystemExit("the ranks reached different allocations from the same tables")
    if rank == 0:
        gathered = sum(J * n * torch.empty(0, dtype=dt).element_size() for n, dt in rows.values())
        line = {"metric": METRIC, "value": float(J) * P * C / (ms_per_step * 1e-3), "unit": UNIT_E2E, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": args.workload, "jobs": J, "jobs_per_gpu_tile": cap, "plans": P, "gpu_levels": G, "cpu_levels": C,
                           "mem_levels": M, "nodes": N,
                           "step": "rubick_curves on this rank's job tile + all-gather of mask and curve tables + greedy_round (replicated)",
                           "l2": "the tables gathered per step are %.2f GB, larger than the 126 MB L2" % (gathered / 1e9)},
                "clocks": clocks, "gpu_launches": int(gpu_launches), "all_gather_bytes_per_rank": int(gathered),
                "ranks_agree": True, "round": {"steps": int(steps_taken[0])},
                "roofline": None, "cpu_baseline": None, "e2e": None}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="throughput-stress", choices=list(workloads.CONFIGS))
    ap.add_argument("--jobs", type=int, default=None, help="override the job count (small captures)")
    ap.add_argument("--nodes", type=int, default=None)
    ap.add_argument("--ref-jobs", type=int, default=0, help="jobs per step of the CPU arm (0: 96 on one thread, 1024 on several)")
    ap.add_argument("--ref-threads", type=int, default=1, help="threads of the CPU arm's table and curve stages (the round always runs on one)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-probes", action="store_true", help="skip the machine probes and the curves-kernel roofline")
    ap.add_argument("--events", type=int, default=1000, help="scheduling events of the event-driven run (0 = skip)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: one independent problem per GPU; strong: ONE problem, curves built in job tiles across the GPUs, "
                         "all-gathered, the round replicated")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_2408_08586_b200 import binding as rb
    from paper_2408_08586_b200 import build as rbuild

    rank = int(os.environ.get("RANK", "0"))
    if not os.path.exists(rb.LIB_PATH) and int(os.environ.get("LOCAL_RANK", "0")) == 0:
        rbuild.build()                      # the library is built in-tree; compile it if this checkout has not been built yet
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg = make_workload(args.workload, rank=0 if args.scaling == "strong" else rank, J=args.jobs, n_nodes=args.nodes)
    if args.scaling == "strong":
        return run_strong(args, cfg, rank, world, local, dev)
    jobs, N = cfg["jobs"], cfg["n_nodes"]
    J = len(jobs["P"])
    plans, _ = rb.enumerate_plans(cfg["g_levels"])
    P, G, C, M = len(plans), len(cfg["g_levels"]), len(cfg["c_levels"]), len(cfg["m_levels"])
    stream = torch.cuda.Stream(device=dev)
    ctx = rb.Context(cfg["env"], device=local, stream=stream.cuda_stream)
    ctx.set_space(plans, cfg["g_levels"], cfg["c_levels"], cfg["m_levels"])

    # device buffers (inputs resident in HBM before the timed region)
    h_jobs = rb.pack_jobs(jobs)
    d_jobs = rb.to_device(h_jobs, dev)
    d_thr = torch.empty(J * C * P, dtype=torch.float32, device=dev)
    d_feas = torch.empty(J * P, dtype=torch.int32, device=dev)
    ncurve = J * G * C * M
    d_cv = torch.empty(ncurve, dtype=torch.float32, device=dev)
    d_cp = torch.empty(ncurve, dtype=torch.int32, device=dev)
    d_cg = torch.empty(ncurve, dtype=torch.int32, device=dev)
    d_state = torch.zeros(J * rb.ASSIGN_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    d_gain = [torch.empty(J, dtype=torch.float32, device=dev) for _ in range(2)]
    d_next = [torch.empty(J, dtype=torch.int32, device=dev) for _ in range(2)]
    d_out = torch.empty(J * rb.ASSIGN_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    d_node = torch.empty(N * rb.NODE_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    max_steps = 1 << 30
    round_steps = [0]
    torch.cuda.synchronize()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    def step(marks=None):
        m = [ev()] if marks is not None else None
        ctx.eval_candidates(d_jobs, J, d_thr, d_feas)
        if m: m.append(ev())
        ctx.best_plan(d_thr, d_feas, J, d_cv, d_cp, d_cg)
        if m: m.append(ev())
        ctx.marginal_gain(d_jobs, J, d_cv, d_state, d_gain[0], d_gain[1], d_next[0], d_next[1])
        if m: m.append(ev())
        round_steps[0], _ = ctx.greedy_round(d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, max_steps, d_out, d_node)
        if m:
            m.append(ev())
            marks.append(m)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None       # nvidia-smi needs a moment to start: launch it before the warm-up
    for _ in range(args.warmup):
        step()
    barrier()
    marks = []
    launches_before = rb.kernel_launches()
    t_start = ev()
    for _ in range(args.steps):
        step(marks)
    t_end = ev()
    barrier()
    gpu_launches = rb.kernel_launches() - launches_before        # counted by the library at every launch site
    clocks = sampler.stop() if sampler else None
    total_ms = reduce_max_ms(t_start.elapsed_time(t_end), world)
    stage_ms = np.array([[m[i].elapsed_time(m[i + 1]) for i in range(4)] for m in marks]).mean(axis=0)
    evals_all = reduce_sum(float(J) * P * C, world)
    ms_per_step = total_ms / args.steps
    value = evals_all / (ms_per_step * 1e-3)

    # end to end through the host-buffer entry point: pinned job records in, assignments out
    e2e = None
    if not args.no_e2e:
        hp_jobs = torch.from_numpy(h_jobs.view(np.uint8).reshape(-1).copy()).pin_memory()
        hp_out = torch.empty(J * rb.ASSIGN_DTYPE.itemsize, dtype=torch.uint8).pin_memory()
        hp_node = torch.empty(N * rb.NODE_DTYPE.itemsize, dtype=torch.uint8).pin_memory()
        for _ in range(max(1, min(args.warmup, 3))):
            ctx.schedule_round_host(hp_jobs, J, N, max_steps, hp_out, hp_node)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            ctx.schedule_round_host(hp_jobs, J, N, max_steps, hp_out, hp_node)
        torch.cuda.synchronize()
        e2e_ms = reduce_max_ms(1e3 * (time.perf_counter() - t0) / args.steps, world)
        e2e = {"value": evals_all / (e2e_ms * 1e-3), "unit": UNIT_E2E, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(J * rb.JOB_DTYPE.itemsize),
               "d2h_bytes_per_step": int(J * rb.ASSIGN_DTYPE.itemsize + N * rb.NODE_DTYPE.itemsize),
               "call": "rubick_schedule_round_host: pinned job records in, assignments and node states out"}

    # the one-pass curves kernel (what the scheduling entry points run) on the same jobs, and the machine probes its
    # roofline is quoted against: write-only and read-only streams, FP32 and transcendental-unit rates (rank 0 only)
    curves_roofline = None
    probes = None
    if rank == 0 and not args.no_probes:
        for _ in range(2):
            ctx.curves(d_jobs, J, d_feas, d_cv, d_cp, d_cg)
        reps = max(3, min(args.steps, 20))
        cs = ClockSampler(local)
        time.sleep(0.3)
        a = ev()
        for _ in range(reps):
            ctx.curves(d_jobs, J, d_feas, d_cv, d_cp, d_cg)
        b = ev()
        torch.cuda.synchronize()
        curves_ms = a.elapsed_time(b) / reps
        curves_clk = cs.stop()

        def timed_probe(kind, buf, iters, reps_):
            ctx.probe(kind, buf, iters)                            # warm-up launch
            s = ClockSampler(local)
            time.sleep(0.3)
            a_ = ev()
            work = 0.0
            for _ in range(reps_):
                work += ctx.probe(kind, buf, iters)
            b_ = ev()
            torch.cuda.synchronize()
            clk = s.stop()
            return work / (a_.elapsed_time(b_) * 1e-3), clk["sm_mhz"]

        wr, _ = timed_probe(rb.PROBE_WRITE, d_thr, 1, 20)
        rd, _ = timed_probe(rb.PROBE_READ, d_thr, 1, 20)
        fma, fma_mhz = timed_probe(rb.PROBE_FMA, d_thr, 1 << 17, 8)
        xu, xu_mhz = timed_probe(rb.PROBE_XU, d_thr, 1 << 15, 8)
        probes = {"write_only_gbs": wr / 1e9, "read_only_gbs": rd / 1e9, "fp32_fma_per_s": fma, "fp32_sm_mhz": fma_mhz,
                  "xu_ops_per_s": xu, "xu_sm_mhz": xu_mhz,
                  "what": "rubick_probe micro-kernels timed with CUDA events: float4 streaming stores / loads over the 4 GB table buffer, "
                          "register-resident FMA chains, lg2/ex2/rcp chains; SM clock = median of nvidia-smi samples during the probe"}
        fp_q, xu_q = eval_quad_ops(C)
        quads = float(J) * (P // 4)
        run_mhz = curves_clk["sm_mhz"]
        scale = (lambda probe_mhz: (run_mhz / probe_mhz) if run_mhz and probe_mhz else 1.0)
        out_bytes = 4.0 * J * P + 12.0 * J * G * C * M + 128.0 * J
        floors = {"xu": quads * xu_q / (xu * scale(xu_mhz)), "fp32": quads * fp_q / (fma * scale(fma_mhz)), "hbm_write": out_bytes / wr}
        bound = max(floors, key=floors.get)
        curves_roofline = {"kernel": "curves_kernel", "ms_per_launch": curves_ms, "sm_mhz": run_mhz,
                           "bound": {"xu": "alu", "fp32": "alu", "hbm_write": "hbm"}[bound], "binding_floor": bound,
                           "floors_ms": {k: 1e3 * v for k, v in floors.items()},
                           "frac": floors[bound] / (curves_ms * 1e-3),
                           "fp32_instr_per_evaluation": fp_q / (4.0 * C), "xu_instr_per_evaluation": xu_q / (4.0 * C),
                           "bytes_written_per_launch": out_bytes,
                           "evaluations_per_sec": float(J) * P * C / (curves_ms * 1e-3),
                           "what": "time the busiest unit would need at its probed rate (transcendental unit, FP32 pipe at the clock of this run, "
                                   "or the write stream of mask + curves) over the measured time; the kernel itself is bound by instruction issue "
                                   "(integer feasibility arithmetic, selects and reductions), see profiles/"}

    # minimum demand of guaranteed jobs on the same tables (first widening row; rank 0 only)
    minres_ms = None
    if rank == 0:
        _, goff = rb.enumerate_plans(cfg["g_levels"])
        rq = workloads.draw_requests(cfg["seed"], J, [int(g) for g in cfg["g_levels"]], C, M, 0.5)
        size = goff[rq["g_idx"] + 1] - goff[rq["g_idx"]]
        rec = np.zeros(J, dtype=rb.REQUEST_DTYPE)
        rec["g_idx"], rec["c_idx"], rec["m_idx"] = rq["g_idx"], rq["c_idx"], rq["m_idx"]
        rec["plan"] = np.where(rq["plan_rank"] >= 0, goff[rq["g_idx"]] + np.floor(np.maximum(rq["plan_rank"], 0) * size), -1)
        d_req = rb.to_device(rec, dev)
        d_gm, d_cm = torch.empty(J, dtype=torch.int32, device=dev), torch.empty(J, dtype=torch.int32, device=dev)
        d_bl = torch.empty(J, dtype=torch.float32, device=dev)
        ctx.min_resources(d_thr, d_feas, d_cv, J, d_req, d_gm, d_cm, d_bl)
        a = ev()
        for _ in range(10):
            ctx.min_resources(d_thr, d_feas, d_cv, J, d_req, d_gm, d_cm, d_bl)
        b = ev()
        torch.cuda.synchronize()
        minres_ms = a.elapsed_time(b) / 10

    # model fitting (Section 4.3) for the first model types of the batch: samples read off the candidate
    # table this run just computed, with measurement noise; start from the generator's nominal coefficients
    fit = None
    if rank == 0 and J > 0:
        Jf, S, sweeps = min(J, 1024), 16, 14
        picks = workloads.draw_fit_picks(cfg["seed"], Jf, S, C)
        thr_h = d_thr[: Jf * C * P].cpu().numpy().reshape(Jf, C, P)
        feas_h = d_feas[: Jf * P].cpu().numpy().view(np.uint32).reshape(Jf, P)
        pl6 = np.stack([1 << plans["log2d"].astype(np.int64), 1 << plans["log2t"].astype(np.int64), 1 << plans["log2p"].astype(np.int64),
                        plans["zero"], plans["gc"], plans["off"]], axis=1)
        sp_, sc_, sy_ = workloads.fit_samples(cfg, pl6, thr_h, feas_h, picks)
        smp = np.zeros((Jf, S), dtype=rb.SAMPLE_DTYPE)
        smp["plan"], smp["cores"], smp["thr"] = sp_, sc_, sy_
        fj = workloads.take(jobs, slice(0, Jf))
        for k_, v_ in workloads.FIT_NOMINAL.items():
            fj[k_] = np.full(Jf, v_)
        d_fj, d_smp = rb.to_device(rb.pack_jobs(fj), dev), rb.to_device(smp, dev)
        d_theta = torch.empty(Jf * 7, dtype=torch.float64, device=dev)
        d_rm = torch.empty(Jf * 2, dtype=torch.float64, device=dev)
        ctx.fit_models(d_fj, Jf, d_smp, S, sweeps, d_theta, d_rm)
        ctx.sync()
        a = ev()
        for _ in range(3):
            ctx.fit_models(d_fj, Jf, d_smp, S, sweeps, d_theta, d_rm)
        b = ev()
        torch.cuda.synchronize()
        rm = d_rm.cpu().numpy().reshape(Jf, 2)
        fit_ms = a.elapsed_time(b) / 3
        fit = {"model_types": Jf, "samples_per_model": S, "sweeps": sweeps, "ms": fit_ms, "fits_per_sec": Jf / (fit_ms * 1e-3),
               "rmsle_before_median": float(np.median(rm[:, 0])), "rmsle_after_median": float(np.median(rm[:, 1])),
               "what": "rubick_fit_models: 7 coefficients per model type by RMSLE over noisy samples (sigma 0.03) of this run's candidate table"}

    # event-driven run: every arrival / completion re-plans all active jobs (rank 0 only)
    events = None
    if args.events > 0 and rank == 0:
        from paper_2408_08586_b200 import events as ev_mod
        ecfg = make_workload("events")
        ectx = rb.Context(ecfg["env"], device=local, stream=stream.cuda_stream)
        eplans, _ = rb.enumerate_plans(ecfg["g_levels"])
        ectx.set_space(eplans, ecfg["g_levels"], ecfg["c_levels"], ecfg["m_levels"])
        ev_mod.run_events(ectx, ecfg, n_events=5)                                    # warm-up: scratch allocation
        r = ev_mod.run_events(ectx, ecfg, n_events=args.events)
        events = {"events": int(len(r["latency_ms"])), "nodes": int(ecfg["n_nodes"]),
                  "active_jobs_min": int(r["active"].min()), "active_jobs_max": int(r["active"].max()),
                  "round_latency_ms_p50": float(np.percentile(r["latency_ms"], 50)),
                  "round_latency_ms_p99": float(np.percentile(r["latency_ms"], 99)),
                  "steps_per_round_mean": float(r["steps"].mean()),
                  "what": "rubick_schedule_round_host per event: host job records in, table + curves + round on the GPU, assignments out"}
        # the same stream through the incremental round (previous allocation and tables kept on the device)
        ev_mod.run_events_incremental(ectx, ecfg, n_events=5)
        ri = ev_mod.run_events_incremental(ectx, ecfg, n_events=args.events)
        inc_lat = ri["latency_ms"][1:] if len(ri["latency_ms"]) > 1 else ri["latency_ms"]      # event 0 builds every table
        events["incremental"] = {
            "events": int(len(ri["latency_ms"])), "slots": 4096,
            "first_event_ms": float(ri["latency_ms"][0]),
            "round_latency_ms_p50": float(np.percentile(inc_lat, 50)),
            "round_latency_ms_p99": float(np.percentile(inc_lat, 99)),
            "steps_per_round_mean": float(ri["steps"][1:].mean()) if len(ri["steps"]) > 1 else float(ri["steps"].mean()),
            "reconfigured_per_round_mean": float(ri["reconfigured"][1:].mean()) if len(ri["reconfigured"]) > 1 else 0.0,
            "what": "rubick_incremental_event_host per event: changed slot and gate inputs in, tables of that slot + incremental round "
                    "(shrink / exchange step, reconfiguration gate at 0.97) on the GPU, assignments out"}
        ectx.close()

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peak, peak_src = measured_hbm_peak()
    eval_gbs = algorithmic_bytes_eval(J, P, C) / (stage_ms[0] * 1e-3) / 1e9
    best_gbs = algorithmic_bytes_best(J, P, C, G, M) / (stage_ms[1] * 1e-3) / 1e9
    sha = hashlib.sha1(open(os.path.join(ROOT, "paper_2408_08586_b200", "csrc", "k_eval.cu"), "rb").read()).hexdigest()
    traffic = None
    if NCU_EVAL_TRAFFIC["k_eval_sha1"] == sha and J >= NCU_EVAL_TRAFFIC["jobs"]:
        residue = algorithmic_bytes_eval(NCU_EVAL_TRAFFIC["jobs"], P, C) - NCU_EVAL_TRAFFIC["dram_bytes"]
        traffic = algorithmic_bytes_eval(J, P, C) - residue

    # the checker as it stands on this machine's host cores: one thread (the primary figure), then all cores for the
    # two stages that have a parallel loop (the round is sequential and stays on one)
    cpu_baseline = None
    if not args.no_cpu_baseline:
        J1 = min(J, 512)                                        # about twelve seconds on one core
        cpu_baseline = baseline_record(cfg, J1, max(1, N * J1 // J), 1, J)
        threads = os.cpu_count() or 1
        J2 = min(J, 4096)                                       # a few seconds on all cores
        cpu_baseline["threaded"] = baseline_record(cfg, J2, max(1, N * J2 // J), threads, J)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": args.workload, "jobs_per_gpu": J, "plans": P, "gpu_levels": G, "cpu_levels": C,
                   "mem_levels": M, "nodes": N,
                   "l2": "the table written per step is %.2f GB, larger than the 126 MB L2" % (4e-9 * J * P * C),
                   "step": "eval_candidates + best_plan + marginal_gain + greedy_round"},
        "clocks": clocks,
        "e2e": e2e,
        # per step: eval, best_plan + its general-mask kernel, gain, prepare, keys, the sort's launches, round
        "gpu_launches": int(gpu_launches),
        "roofline": {"kernel": "eval_candidates_kernel", "bound": "hbm", "achieved": eval_gbs, "peak": peak, "unit": "GB/s",
                     "frac": eval_gbs / peak, "traffic": traffic, "peak_source": peak_src,
                     "bytes_per_candidate": algorithmic_bytes_eval(J, P, C) / (float(J) * P * C),
                     "ms_per_launch": float(stage_ms[0]),
                     "frac_of_write_only_probe": (eval_gbs / probes["write_only_gbs"]) if probes else None,
                     "frac_of_8000_gbs_spec": eval_gbs / 8000.0,
                     "traffic_source": (f"ncu capture on {NCU_EVAL_TRAFFIC['jobs']} jobs: {NCU_EVAL_TRAFFIC['dram_bytes']} bytes against "
                                        f"{int(algorithmic_bytes_eval(NCU_EVAL_TRAFFIC['jobs'], P, C))} algorithmic (the last lines written are still dirty "
                                        "in L2 when the kernel ends; no re-reads); a full launch = its algorithmic bytes less that residue"
                                        if traffic else "null: no capture of this kernel source or a smaller workload than the capture")},
        "cpu_baseline": cpu_baseline,
        "stages_ms": {"eval_candidates": float(stage_ms[0]), "best_plan": float(stage_ms[1]),
                      "marginal_gain": float(stage_ms[2]), "greedy_round": float(stage_ms[3])},
        "eval_kernel_candidates_per_sec": float(J) * P * C / (stage_ms[0] * 1e-3),
        "logical_candidates_per_sec": value * M,
        "best_plan_roofline": {"bound": "hbm", "achieved": best_gbs, "peak": peak, "unit": "GB/s", "frac": best_gbs / peak,
                               "frac_of_read_only_probe": (best_gbs / probes["read_only_gbs"]) if probes else None},
        "curves_roofline": curves_roofline,
        "probes": probes,
        "events": events,
        "min_resources_ms": minres_ms,
        "fit": fit,
        "round": {"steps": int(round_steps[0]), "latency_ms": float(stage_ms[3]),
                  "us_per_step": float(1e3 * stage_ms[3] / max(1, round_steps[0]))},
    }
    print(json.dumps(line))
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
