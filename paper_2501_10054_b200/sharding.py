"""Token sharding over ranks.  The FFN acts on every token independently, so several GPUs split a batch
by tokens: every rank holds a full copy of the layer state, takes a contiguous slice of the tokens and
keeps its slice of the output; there is no exchange step on the data path.  Only timing (the slowest
rank decides) and counters cross ranks, through torch.distributed."""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def token_shard(n_tokens: int, world: int, rank: int) -> Tuple[int, int]:
    """(first token, token count) of `rank`: contiguous slices, sizes differing by at most one, the
    larger ones first."""
    if world <= 0 or not (0 <= rank < world) or n_tokens < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_tokens, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def max_over_ranks(value: float, device="cpu") -> float:
    """The largest `value` of all ranks (a step is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
