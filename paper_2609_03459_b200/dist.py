"""Multi-GPU plumbing for batch-sharded replicas (one process per GPU, torch.distributed).

The TT-cores are small, so every rank holds all of them and its own shard of the batch.  The forward
needs no collective.  A training step has exactly one exchange: the sum of the core gradients over ranks
(one all-reduce of the flat gradient buffer), after which every rank applies the same SGD update.
These helpers contain no arithmetic of the method and work with any backend (NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch drawn by `rank` (rank 0 keeps the base seed, so N = 1 reproduces the single-GPU run)."""
    return base_seed if rank == 0 else base_seed + 7919 * rank


def allreduce_core_grads(flat_grads: torch.Tensor) -> torch.Tensor:
    """In-place sum over ranks of the flat core-gradient buffer (no-op for a single process)."""
    if world() > 1:
        dist.all_reduce(flat_grads, op=dist.ReduceOp.SUM)
    return flat_grads


def max_over_ranks(value: float, device=None) -> float:
    """Largest value over ranks (used for device-timed durations)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
