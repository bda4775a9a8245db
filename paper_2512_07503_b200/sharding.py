"""Host-side helpers for running the step on several GPUs.

Sequences are independent until the caller's scheduler looks at the accept lengths, so the step shards
over the batch axis with no exchange of data: every rank owns a contiguous slice of the sequences and the
Philox counter's sequence word carries the GLOBAL sequence index (`seq_base`), which makes a sharded run
reproduce the unsharded one bit for bit.  The only cross-rank operations are the barrier and the
max-over-ranks reduction of a measured time.
"""
from __future__ import annotations

from typing import Tuple


def shard_range(n_sequences: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the sequences owned by `rank`: contiguous, sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or n_sequences < 0:
        raise ValueError("need world >= 1, 0 <= rank < world, n_sequences >= 0")
    base, extra = divmod(n_sequences, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
