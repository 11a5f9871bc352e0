"""Event-driven harness: every job arrival or completion triggers one full scheduling round.

Host-side glue only (the paper's Section 7.4 uses a simulator for the same purpose): it keeps
the set of active jobs, calls ``rubick_schedule_round_host`` on them at every event, advances each
job by the throughput the round predicted for it, and records the latency of every round.  A job
of nominal length L (seconds at the speed of one GPU) progresses at rate w * thr, the weighted
throughput the scheduler itself maximises, so that rounds with better allocations finish jobs
sooner.  Arrivals are Poisson and lengths log-normal (``workloads.draw_events``).
"""
import time

import numpy as np

from . import binding as rb
from . import workloads


def run_events(ctx, cfg, n_events=1000, warm_jobs=1500, max_steps=1 << 30, sync=None):
    """Replays n_events scheduling events.  -> dict(latency_ms [n_events], active [n_events], steps [n_events]).

    cfg: a workload dict whose jobs are the pool arrivals are drawn from, in order; the first
    `warm_jobs` of them are already in the system at time 0 so that rounds start at a realistic size.
    """
    jobs = cfg["jobs"]
    pool = len(jobs["P"])
    arrivals, lengths = workloads.draw_events(cfg["seed"], pool)
    warm = min(warm_jobs, pool)
    arrivals = np.concatenate([np.zeros(warm), arrivals[: pool - warm] if pool > warm else []])
    remaining = lengths.copy()
    records = rb.pack_jobs(jobs)
    N = cfg["n_nodes"]
    w = np.asarray(jobs["w"], dtype=np.float64)

    active = list(range(warm))
    next_arrival = warm
    now = 0.0
    h_out = np.zeros(pool, dtype=rb.ASSIGN_DTYPE)
    lat, act, stp = [], [], []
    for _ in range(n_events):
        if not active and next_arrival >= pool:
            break
        idx = np.asarray(active, dtype=np.int64)
        h_jobs = np.ascontiguousarray(records[idx])
        t0 = time.perf_counter()
        steps, _ = ctx.schedule_round_host(h_jobs, len(idx), N, max_steps, h_out[: len(idx)])
        if sync is not None:
            sync()
        lat.append(1e3 * (time.perf_counter() - t0))
        act.append(len(idx))
        stp.append(steps)
        # advance to the next event: the earliest completion or the next arrival
        rate = w[idx] * h_out["thr"][: len(idx)].astype(np.float64)
        with np.errstate(divide="ignore", invalid="ignore"):
            eta = np.where(rate > 0, remaining[idx] / rate, np.inf)
        t_done = now + (eta.min() if len(eta) else np.inf)
        t_arr = arrivals[next_arrival] if next_arrival < pool else np.inf
        t_next = min(t_done, t_arr)
        if not np.isfinite(t_next):
            break
        remaining[idx] -= rate * (t_next - now)
        now = t_next
        if t_arr <= t_done:
            active.append(next_arrival)
            next_arrival += 1
        finished = set(idx[remaining[idx] <= 1e-9 * lengths[idx]].tolist())
        if t_done <= t_arr and not finished:
            finished = {int(idx[int(np.argmin(eta))])}
        if finished:
            active = [j for j in active if j not in finished]
    return dict(latency_ms=np.asarray(lat), active=np.asarray(act), steps=np.asarray(stp))
