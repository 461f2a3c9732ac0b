"""Host-side helpers for running the forward as data-parallel replicas.

The quantized forward needs no exchange step: every token row is independent given the
weights, so N GPUs each run the unchanged single-GPU library on a contiguous slice of the
token batch (weights replicated) and the concatenated output equals the 1-GPU output byte
for byte.  These helpers hold only the bookkeeping (which rows a rank owns, how ranks agree
on a timing); they launch nothing.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def token_shard(num_tokens: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous [begin, end) slice of a batch of num_tokens rows owned by `rank`; the first
    num_tokens % world_size ranks get one extra row.  Slices tile the batch exactly."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, extra = divmod(num_tokens, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The maximum of a per-rank scalar (e.g. a device-measured duration) over the default
    process group; the value itself when no group is initialised."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
