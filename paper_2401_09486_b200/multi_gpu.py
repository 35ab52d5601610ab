"""Plumbing for running the hot path on several GPUs of one node.

Every (batch, head) pair is independent in all three calls, so several GPUs
simply take different (batch, head) shards: there is no collective on the data
path.  What is shared is bookkeeping: which slice a rank owns, rank-dependent
seeds for synthetic inputs, and timing as the maximum over ranks.  These helpers
use torch.distributed only (NCCL on GPUs, gloo in the CPU tests).
"""

from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def shard_range(n_items: int, rank: int, world: int) -> range:
    """Contiguous, balanced slice of `n_items` (e.g. B*H pairs) owned by `rank`:
    the first n_items % world ranks get one extra item."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def rank_seed(base: int, rank: int, stream: int = 0) -> int:
    """Distinct seed per (rank, stream) so that ranks do not generate identical tensors."""
    return int(base) + 10 * int(rank) + int(stream)


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(units_per_rank: float, world: int, max_ms: float) -> float:
    """Whole-job throughput in units per second when every rank processes
    `units_per_rank` units (weak scaling) and the slowest rank took `max_ms`."""
    return world * units_per_rank / (max_ms * 1e-3)
