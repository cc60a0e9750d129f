"""Multi-GPU layout: replications are independent, so they are sharded across ranks.

Rank k of W simulates global replications [offset_k, offset_k + count_k); random streams are keyed by the
global replication index, so results do not depend on W.  There is no data-path collective; the only
exchange is the gather of per-replication statistics at the end (rank order = replication order, so the
fp64 totals are summed in a fixed order).
"""
from __future__ import annotations

import numpy as np


def shard(R: int, world: int, rank: int) -> tuple[int, int]:
    """(count, offset) of the contiguous block of replications owned by `rank`; counts differ by at most 1."""
    if not (0 <= rank < world) or R < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(R, world)
    count = base + (1 if rank < extra else 0)
    offset = rank * base + min(rank, extra)
    return count, offset


def gather_stats(local: dict, group=None) -> dict:
    """All-gather per-replication statistics (dict of arrays whose first axis is the local replication)
    into arrays over all replications, in global replication order.  Works with any torch.distributed
    backend; keys starting with '_' are dropped."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = {}
    for k in sorted(local):
        if k.startswith("_"):
            continue
        parts = [None] * world
        dist.all_gather_object(parts, np.ascontiguousarray(local[k]), group=group)
        out[k] = np.concatenate(parts, axis=0)
    return out


def totals(stats: dict) -> dict:
    """Sums over replications taken in replication order (integers exactly, fp64 in a fixed order)."""
    out = {}
    for k, v in stats.items():
        if v.dtype.kind == "f":
            acc = np.zeros(v.shape[1:], np.float64)
            for r in range(v.shape[0]):
                acc = acc + v[r]
            out[k] = acc
        else:
            out[k] = v.sum(axis=0, dtype=np.uint64)
    return out


def combine_totals(mine: dict, my_ms: float, group=None) -> dict:
    """End-of-run exchange of a sharded run: every rank contributes its own totals (a dict of numbers) and its device
    time.  Integers are summed exactly, floats are added in rank order (a fixed order), and the time is the maximum over
    ranks ("max_ms").  With one process (no process group) the input comes back unchanged.  This is the only exchange of
    the multi-GPU layout: the simulation itself never communicates."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return dict(mine, max_ms=float(my_ms))
    world = dist.get_world_size(group)
    parts = [None] * world
    dist.all_gather_object(parts, (dict(mine), float(my_ms)), group=group)
    out = {}
    for k in mine:
        vals = [p[0][k] for p in parts]
        if all(isinstance(v, (int, np.integer)) for v in vals):
            out[k] = int(sum(int(v) for v in vals))
        else:
            acc = 0.0
            for v in vals:
                acc = acc + float(v)
            out[k] = acc
    out["max_ms"] = max(p[1] for p in parts)
    return out
