"""Host-side logic of multi-GPU runs.

The MoE layer is token-parallel: a token's output depends on no other token.  So N GPUs run N
replicas of the layer (each with the full weights) on disjoint slices of the batch and no
collective touches the data path.  What the ranks do share is bookkeeping: who takes which tokens,
and the timing of a run (the slowest rank decides).
"""
from __future__ import annotations

from typing import Optional, Tuple


def shard_tokens(n_tokens: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice (start, count) of a batch of n_tokens for this rank; the first
    n_tokens % world ranks take one token more.  Slices are disjoint and cover the batch."""
    assert 0 <= rank < world and n_tokens >= 0
    base, extra = divmod(n_tokens, world)
    count = base + (1 if rank < extra else 0)
    start = rank * base + min(rank, extra)
    return start, count


def aggregate(local_ms: float, local_units: float, dist=None, device: Optional[str] = None
              ) -> Tuple[float, float]:
    """(max over ranks of the elapsed milliseconds, sum over ranks of the units processed).
    ``dist`` is an initialised torch.distributed module, or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    import torch
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def job_throughput(local_ms: float, local_units: float, dist=None, device: Optional[str] = None) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    ms, units = aggregate(local_ms, local_units, dist, device)
    return units / (ms * 1e-3)
