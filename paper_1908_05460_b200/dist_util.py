"""Rank plumbing for multi-GPU runs: one process per GPU, torch.distributed for the rendezvous.

The filter-gradient path shards over the batch with no exchange step (each rank owns its images and
produces its own dW), so the only collective the benchmark needs is the MAX of the per-rank step
times.  The functions work with any backend (nccl on GPUs, gloo in CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest `value` over all ranks (the value itself without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_batch(n: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [begin, end) range of a batch of n images owned by `rank` (strong-scaling split);
    ranks differ by at most one image."""
    base, extra = divmod(n, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def us_per_layer(ms_per_step: float, layer_passes: int, world: int) -> float:
    """Benchmark value: microseconds per layer pass, aggregated over `world` ranks that each ran
    `layer_passes` passes per step (weak scaling)."""
    return ms_per_step * 1e3 / (layer_passes * world)
