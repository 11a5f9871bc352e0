"""Job-sharded curve construction across the GPUs of one node.

The resource-sensitivity curves of different jobs are independent of each other (paper Section 5.2: they
"can be computed in parallel ... and then cached"), so the one part of the path that shards is the
evaluation + best-plan step: rank r builds the mask and the curve tables of one contiguous tile of jobs with
``rubick_curves``, one all-gather brings every tile into every rank's own HBM, and every rank then runs the
same greedy round on the full tables.  The round needs a global arg-max at every step, so it is replicated,
not sharded; since it is deterministic, all ranks reach the same allocation, which ``assignments_agree``
checks.

Only plumbing lives here: tile bounds, padded buffers for ``torch.distributed.all_gather_into_tensor`` (NCCL
on GPUs, gloo in the CPU tests) and the copy of each tile to its place.  Remote data always lands in local
memory through the collective; no kernel of the library reads another GPU's memory.
"""
import numpy as np


def job_tile(J, world, rank):
    """Contiguous tile of rank `rank` when J jobs are split over `world` ranks: the first J % world ranks hold
    one job more.  -> (first job, number of jobs)."""
    base, extra = divmod(int(J), int(world))
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def tile_capacity(J, world):
    """Jobs in the largest tile (every rank's send buffer is padded to it: the collective wants equal sizes)."""
    return -(-int(J) // int(world))


def gather_tiles(local, J, world, row_elems, out, group=None):
    """All-gathers per-job rows.  `local`: this rank's tile, a 1-D tensor of tile_capacity(J, world) * row_elems
    elements whose first count * row_elems are meaningful; `out`: 1-D tensor of J * row_elems elements that
    receives all tiles in job order.  Uses one all_gather_into_tensor plus, when the tiles are uneven, one copy
    per rank to close the gaps the padding left."""
    import torch
    import torch.distributed as dist
    cap = tile_capacity(J, world)
    assert local.numel() == cap * row_elems and out.numel() == J * row_elems
    if world == 1:
        out.copy_(local[: J * row_elems])
        return out
    if J % world == 0:
        dist.all_gather_into_tensor(out, local, group=group)        # tiles are already back to back
        return out
    staged = torch.empty(world * cap * row_elems, dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(staged, local, group=group)
    for r in range(world):
        start, count = job_tile(J, world, r)
        out[start * row_elems:(start + count) * row_elems].copy_(staged[r * cap * row_elems: (r * cap + count) * row_elems])
    return out


def sharded_tables(compute_tile, J, world, rank, rows, device, group=None):
    """Builds the full per-job tables on every rank from per-rank tiles.

    compute_tile(start, count, bufs): fills, for jobs [start, start + count), the first count rows of each
    buffer in `bufs` (a dict name -> 1-D tensor of tile_capacity * row_elems elements).
    rows: dict name -> (row_elems, torch dtype).  -> dict name -> 1-D tensor of J * row_elems elements."""
    import torch
    cap = tile_capacity(J, world)
    start, count = job_tile(J, world, rank)
    bufs = {k: torch.zeros(cap * n, dtype=dt, device=device) for k, (n, dt) in rows.items()}
    if count:
        compute_tile(start, count, bufs)
    full = {k: torch.empty(J * n, dtype=dt, device=device) for k, (n, dt) in rows.items()}
    for k, (n, _) in rows.items():
        gather_tiles(bufs[k], J, world, n, full[k], group=group)
    return full


def assignments_agree(out_bytes, world, group=None):
    """True when every rank holds the same bytes in `out_bytes` (a uint8 tensor: the round's assignments and
    node states).  One all-reduce of the element-wise maximum and one of the minimum: equal exactly when all
    ranks agree."""
    import torch
    import torch.distributed as dist
    if world == 1:
        return True
    hi = out_bytes.to(torch.int32)
    lo = hi.clone()
    dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
    return bool(torch.equal(hi, lo))


def curves_tile_fn(ctx, d_jobs, rb_job_itemsize):
    """compute_tile for sharded_tables that runs rubick_curves on this rank's tile of the resident job records
    (`d_jobs`: uint8 tensor of all J records)."""
    def compute(start, count, bufs):
        jobs = d_jobs[start * rb_job_itemsize:(start + count) * rb_job_itemsize]
        ctx.curves(jobs, count, bufs["feas"], bufs["cv"], bufs["cp"], bufs["cg"])
    return compute


def table_rows(P, G, C, M):
    """Row sizes and dtypes of the four per-job tables a round reads."""
    import torch
    return {"feas": (P, torch.int32), "cv": (G * C * M, torch.float32), "cp": (G * C * M, torch.int32),
            "cg": (G * C * M, torch.int32)}


def tiles_cover(J, world):
    """All tiles as (start, count); used by the tests: they must partition range(J) in order."""
    return np.asarray([job_tile(J, world, r) for r in range(world)], dtype=np.int64)
