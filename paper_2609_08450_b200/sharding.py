"""Row sharding for multi-GPU runs.

Rows are selected independently, so a batch is split across ranks by rows with no
data-path collective: each rank runs the single-GPU library on its slice and keeps its
outputs.  Only timings are reduced (max over ranks).
"""
import numpy as np


def partition_rows(row_lengths, world_size):
    """Contiguous row ranges [(begin, end)] per rank, balanced by total valid length."""
    lengths = np.clip(np.asarray(row_lengths, dtype=np.int64), 0, None)
    M = len(lengths)
    total = int(lengths.sum())
    bounds = [0]
    prefix = np.concatenate([[0], np.cumsum(lengths)])
    for r in range(1, world_size):
        target = total * r / world_size
        cut = int(np.searchsorted(prefix, target, side="left"))
        cut = min(max(cut, bounds[-1]), M)
        bounds.append(cut)
    bounds.append(M)
    return [(bounds[i], bounds[i + 1]) for i in range(world_size)]


def max_over_ranks(value, device=None):
    """Max of a scalar over all ranks (identity without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, device=None):
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
