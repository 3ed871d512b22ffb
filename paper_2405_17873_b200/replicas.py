"""Multi-GPU form of the layer sweep: independent replicas, one process per GPU.

The path has no exchange step (every image batch runs the whole sweep on its own GPU with
its own copy of the packed weights), so the only collective is the bookkeeping of a
measurement: a barrier around the timed region and the maximum over ranks of the device
times.  The functions work with any ``torch.distributed`` backend (NCCL on GPUs, gloo in
the CPU tests).
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world() > 1:
        dist.barrier()


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum over all ranks of a short list of floats (device times)."""
    if world() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank: float, ms_max: float) -> float:
    """Units per second of the whole job: every rank processed ``units_per_rank`` in the
    slowest rank's time (weak scaling)."""
    return world() * units_per_rank / (ms_max * 1e-3)
