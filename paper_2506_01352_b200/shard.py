"""Host-side rank logic for running the codec on several GPUs (one process per GPU).

The path needs no collective: tiles are independent and the only coupled unit is the ranking group (one
sample, Sec. 3.2), so ranks work on disjoint tensors or on disjoint runs of whole samples, and each rank's
packed buffer is self-contained.  What is shared is bookkeeping: which data a rank takes, and the timing
reduction (the slowest rank decides).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_microbatches(rank: int, n_sets: int) -> list[int]:
    """Micro-batch indices of the boundary tensors rank `rank` encodes and decodes (disjoint over ranks)."""
    return [rank * n_sets + i for i in range(n_sets)]


def shard_samples(tokens: int, group_tokens: int, world: int, rank: int) -> tuple[int, int]:
    """(first token, token count) of rank `rank` when one [tokens x hidden] tensor is split over `world` ranks
    on ranking-group boundaries; the first `n_groups % world` ranks get one group more."""
    g = group_tokens or tokens
    if tokens % g:
        raise ValueError("group_tokens must divide tokens")
    n_groups = tokens // g
    base, extra = divmod(n_groups, world)
    mine = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first * g, mine * g


def max_over_ranks(ms: float, device: torch.device | str = "cpu") -> float:
    """The timing every rank reports: the maximum over the ranks (a no-op without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(bytes_per_rank: int, world: int, steps: int, ms: float) -> float:
    """GB/s over all ranks: every rank moved `bytes_per_rank` per step (weak scaling), `ms` is max-over-ranks."""
    return bytes_per_rank * world * steps / (ms * 1e-3) / 1e9
