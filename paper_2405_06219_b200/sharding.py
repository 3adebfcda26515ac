"""Multi-GPU layout of the decode path: one process per GPU, no data-path collective.

(sequence, KV head) units are independent, so each rank owns whole sequences and runs the
single-GPU path on them.  The only exchanges are control-plane reductions of timings and token
counts (max over ranks, sum over ranks), which work on any torch.distributed backend.
"""
from __future__ import annotations

import dataclasses


def rank_workload(w, rank: int, world: int):
    """Weak scaling: every rank gets a workload of the same shape with its own random streams."""
    assert 0 <= rank < world
    return dataclasses.replace(w, seed=w.seed + 1000 * rank) if rank else w


def split_sequences(batch: int, rank: int, world: int) -> range:
    """Strong-scaling helper: the contiguous block of sequence indices rank owns out of ``batch``."""
    base, extra = divmod(batch, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def reduce_job(elapsed_ms: float, units: float, device=None):
    """(max over ranks of elapsed_ms, sum over ranks of units); identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(elapsed_ms), float(units)
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def _reduce(values, op_name: str, device=None):
    """Element-wise reduction of a list of floats over the ranks; identity without a process group."""
    import torch
    import torch.distributed as dist
    vals = [float(x) for x in values]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return vals
    t = torch.tensor(vals, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return [float(x) for x in t.tolist()]


def reduce_max_list(values, device=None):
    """Per-pass timings: every entry becomes the slowest rank's."""
    return _reduce(values, "MAX", device)


def reduce_max(value: float, device=None) -> float:
    return _reduce([value], "MAX", device)[0]


def reduce_sum(value: float, device=None) -> float:
    """Units of work: the whole job's."""
    return _reduce([value], "SUM", device)[0]
