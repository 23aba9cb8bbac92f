"""Multi-GPU plumbing of the CSAT forward: none of the method's arithmetic lives here.

Every (batch, head) pair of the forward is independent, and the measurement matrix Phi_h is a pure
function of (seed, h), so a job is split over the batch axis with no exchange on the data path: each
rank builds its own context from the same seed and runs its slice.  Only timings are reduced.
"""
from __future__ import annotations


def shard_range(total: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous slice [start, start + count) of `total` items owned by `rank` of `world`.
    The first total % world ranks get one extra item; slices are disjoint and cover range(total)."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError(f"bad shard request: total={total} world={world} rank={rank}")
    base, extra = divmod(total, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
