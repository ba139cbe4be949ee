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


# ---- data-parallel filter gradient (the paper's outlook, Section 5: schedules over machine, layer and batch) ----
# Each rank owns the images [shard_batch(n, rank, world)) of a batch and computes the filter gradient of its
# images; the gradients of a layer set then meet in ONE sum all-reduce of a flat fp32 bucket.  The exact path and
# the top-1 / top-k methods are sums over images, so the reduced result is the full-batch gradient (up to
# rounding order).  The zero gradient needs no exchange, and the random gradient is a function of (seed, element)
# alone: every rank draws the same values, so it must NOT be summed.

def needs_allreduce(method: int) -> bool:
    """Whether the per-rank dW of `method` (gaconv_method_t) are partial sums over the rank's images."""
    return method in (-1, 2, 3)          # exact, top-1, top-k; not zero (0) or random (1)


def allreduce_dw_bucket(dws, methods, group=None):
    """Sum-all-reduce the filter gradients of a layer set in one bucket.  `dws`: list of fp32 tensors (one per
    layer, any shape, on the backend's device); `methods`: the gaconv_method_t each layer used in this step.
    Layers whose method needs no exchange are left untouched.  Returns the number of bytes reduced."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return 0
    part = [t for t, m in zip(dws, methods) if needs_allreduce(m)]
    if not part:
        return 0
    flat = torch.cat([t.reshape(-1) for t in part])
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    off = 0
    for t in part:
        t.copy_(flat[off:off + t.numel()].view_as(t))
        off += t.numel()
    return flat.numel() * 4
