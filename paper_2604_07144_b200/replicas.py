"""Multi-GPU plumbing: the serving iteration has no exchange step (every
sequence, and every kv head, is independent), so N GPUs run N independent
replicas -- one process per GPU, each with its own pool and its own batch --
and nothing of the data path crosses GPUs.  What is shared is only the
measurement: a barrier around the timed region, the maximum of the per-rank
times and the sum of the per-rank work.  ``torch.distributed`` carries those
scalars (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Optional, Tuple


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch replica ``rank`` serves (replicas draw different batches)."""
    return int(base_seed) + 1000 * int(rank)


def barrier(device=None) -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def _reduce(value: float, op, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=op)
    return float(t.item())


def reduce_max(value: float, device=None) -> float:
    import torch.distributed as dist
    return _reduce(value, dist.ReduceOp.MAX, device)


def reduce_sum(value: float, device=None) -> float:
    import torch.distributed as dist
    return _reduce(value, dist.ReduceOp.SUM, device)


def whole_job_throughput(units_this_rank: float, ms_this_rank: float, device=None) -> Tuple[float, float, float]:
    """(total units of all ranks, max time over ranks in ms, units per second of the whole job)."""
    total = reduce_sum(units_this_rank, device)
    ms = reduce_max(ms_this_rank, device)
    return total, ms, total / (ms * 1e-3)
