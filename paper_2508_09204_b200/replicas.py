"""Multi-GPU plumbing of the routed layer: replicas only.

Samples are independent and every expert is replicated on every GPU, so N ranks run N shards of samples with no
data-path collective (the paper's method has no exchange step between samples: each sample is run by exactly one
expert, Section 3.1).  ``torch.distributed`` is used for the barrier and for the max over ranks of the timed
region only.  Works with any backend (``nccl`` on GPUs, ``gloo`` in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_seed(base_seed: int, rank: int) -> int:
    """Seed of rank's own shard of samples (activations and routing differ per rank; weights do not)."""
    return int(base_seed) + 1000 * int(rank)


def max_over_ranks(value: float, device: torch.device) -> float:
    """Max of a per-rank scalar (e.g. elapsed milliseconds) over all ranks; identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def whole_job_value(units_per_rank: int, world_size: int, ms_per_step: float) -> float:
    """Aggregate throughput of all ranks: every rank processes ``units_per_rank`` per step (weak scaling)."""
    return world_size * units_per_rank / (ms_per_step * 1e-3)
