"""Event-driven harness: every job arrival or completion triggers one scheduling round, either a full
re-plan of all active jobs (``run_events``) or the incremental round that starts from the previous
allocation (``run_events_incremental``).

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


def run_events(ctx, cfg, n_events=1000, warm_jobs=1500, max_steps=1 << 30, sync=None, on_round=None):
    """Replays n_events scheduling events.  -> dict(latency_ms [n_events], active [n_events], steps [n_events]).

    cfg: a workload dict whose jobs are the pool arrivals are drawn from, in order; the first
    `warm_jobs` of them are already in the system at time 0 so that rounds start at a realistic size.
    on_round(event, pool_indices, h_jobs, h_out, h_nodes, steps), if given, sees every round's inputs and results
    (outside the timed part); the node states are only fetched when it is given.
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
    h_nodes = np.zeros(N, dtype=rb.NODE_DTYPE) if on_round is not None else None
    lat, act, stp = [], [], []
    for ev in range(n_events):
        if not active and next_arrival >= pool:
            break
        idx = np.asarray(active, dtype=np.int64)
        h_jobs = np.ascontiguousarray(records[idx])
        t0 = time.perf_counter()
        steps, _ = ctx.schedule_round_host(h_jobs, len(idx), N, max_steps, h_out[: len(idx)], h_nodes)
        if sync is not None:
            sync()
        lat.append(1e3 * (time.perf_counter() - t0))
        act.append(len(idx))
        stp.append(steps)
        if on_round is not None:
            on_round(ev, idx, h_jobs, h_out[: len(idx)], h_nodes, steps)
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


def run_events_incremental(ctx, cfg, n_events=1000, warm_jobs=1500, slots=4096, theta=0.97, max_steps=1 << 30, on_round=None):
    """The same event stream through ``rubick_incremental_event_host``: jobs live in `slots` fixed slots,
    the previous allocation and the curve tables stay on the device, and an event uploads only the slot
    that changed.  A job's checkpoint-resume cost is ``workloads.reconf_cost``; its trained time T and
    reconfiguration count feed the gate of Section 5.2.  on_round(event, slot_job, h_jobs, reconf, changed, h_out,
    h_nodes, steps), if given, sees every round's inputs and results (outside the timed part).
    -> dict(latency_ms, active, steps, reconfigured [n_events])."""
    jobs = cfg["jobs"]
    pool = len(jobs["P"])
    arrivals, lengths = workloads.draw_events(cfg["seed"], pool)
    warm = min(warm_jobs, pool, slots)
    arrivals = np.concatenate([np.zeros(warm), arrivals[: pool - warm] if pool > warm else []])
    remaining = lengths.copy()
    records = rb.pack_jobs(jobs)
    N = cfg["n_nodes"]
    w = np.asarray(jobs["w"], dtype=np.float64)
    cost = workloads.reconf_cost(jobs)

    slot_job = np.full(slots, -1, dtype=np.int64)          # pool index of the job in each slot
    slot_job[:warm] = np.arange(warm)
    free = list(range(slots - 1, warm - 1, -1))
    h_jobs = np.zeros(slots, dtype=rb.JOB_DTYPE)
    h_jobs[:warm] = records[:warm]
    reconf = np.zeros(slots, dtype=rb.RECONF_DTYPE)
    reconf["active"][:warm] = 1
    reconf["delta"][:warm] = cost[:warm]
    h_out = np.zeros(slots, dtype=rb.ASSIGN_DTYPE)
    prev = np.zeros(slots, dtype=rb.ASSIGN_DTYPE)
    next_arrival = warm
    now = 0.0
    changed = None                                          # first event: everything is new
    h_nodes = np.zeros(N, dtype=rb.NODE_DTYPE) if on_round is not None else None
    lat, act, stp, rec = [], [], [], []
    for ev in range(n_events):
        live = np.nonzero(slot_job >= 0)[0]
        if len(live) == 0 and next_arrival >= pool:
            break
        t0 = time.perf_counter()
        steps, _ = ctx.incremental_event_host(h_jobs, slots, N, h_out, changed=changed, h_reconf=reconf, theta=theta,
                                              restart=changed is None, max_steps=max_steps, h_node_out=h_nodes)
        lat.append(1e3 * (time.perf_counter() - t0))
        act.append(len(live))
        stp.append(steps)
        if on_round is not None:
            on_round(ev, slot_job, h_jobs, reconf, changed, h_out, h_nodes, steps)
        was = (prev["status"] == rb.RUNNING) & (slot_job >= 0)
        moved = was & (h_out["status"] == rb.RUNNING) & ((h_out["g"] != prev["g"]) | (h_out["c"] != prev["c"]) | (h_out["plan"] != prev["plan"]))
        reconf["n_reconf"] += moved.astype(np.int32)
        rec.append(int(moved.sum()))
        prev[:] = h_out
        # advance to the next event
        idx = slot_job[live]
        rate = w[idx] * h_out["thr"][live].astype(np.float64)
        with np.errstate(divide="ignore", invalid="ignore"):
            eta = np.where(rate > 0, remaining[idx] / rate, np.inf)
        t_done = now + (eta.min() if len(eta) else np.inf)
        t_arr = arrivals[next_arrival] if next_arrival < pool and free else np.inf
        t_next = min(t_done, t_arr)
        if not np.isfinite(t_next):
            break
        dt = t_next - now
        remaining[idx] -= rate * dt
        reconf["T"][live] = np.where(h_out["status"][live] == rb.RUNNING, reconf["T"][live] + dt, 0.0)
        now = t_next
        changed = []
        if t_arr <= t_done:
            s = free.pop()
            slot_job[s] = next_arrival
            h_jobs[s] = records[next_arrival]
            reconf[s] = (0.0, cost[next_arrival], 0, 1)
            changed.append(s)
            next_arrival += 1
        done = live[remaining[idx] <= 1e-9 * lengths[idx]]
        if t_done <= t_arr and len(done) == 0:
            done = live[[int(np.argmin(eta))]]
        for s in done:
            slot_job[s] = -1
            reconf["active"][s] = 0
            free.append(int(s))
    return dict(latency_ms=np.asarray(lat), active=np.asarray(act), steps=np.asarray(stp), reconfigured=np.asarray(rec))
