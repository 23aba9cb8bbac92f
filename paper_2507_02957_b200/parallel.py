"""Multi-GPU plumbing of the CSAT forward: none of the method's arithmetic lives here.

Every (batch, head) pair of the forward is independent, and the measurement matrix Phi_h is a pure
function of (seed, h), so a job is split over the batch axis with no exchange on the data path: each
rank builds its own context from the same seed and runs its slice.  Only timings are reduced.

Where one (batch, head) pair's sequence does not fit one GPU, the token axis is sharded instead
(`sharded_forward`): the compression K~ = Phi K is a sum over tokens, so every rank compresses its own token
shard, the float32 partial sums are exchanged once (an all-gather that lands in each rank's own memory) and added
in rank order on every rank, and each rank then attends for its own queries.  That is the one exchange step of the
path.
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


def token_shard_range(n: int, world: int, rank: int, align: int = 64) -> tuple[int, int]:
    """Contiguous token shard [start, start + count) of rank `rank`: shards start at multiples of `align` (so that
    every load of the compression kernel stays aligned), are disjoint and cover range(n).  With fewer than
    world * align tokens the last ranks get none."""
    if n < 0 or align < 1:
        raise ValueError(f"bad token shard request: n={n} align={align}")
    units = (n + align - 1) // align
    u0, cnt = shard_range(units, world, rank)
    start = min(n, u0 * align)
    return start, min(n, (u0 + cnt) * align) - start


def all_gather_stacked(t, group=None):
    """[world, *t.shape]: every rank's tensor in rank order, in this rank's own memory (NCCL or gloo)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return t.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(t.shape), dtype=t.dtype, device=t.device)
    dist.all_gather(list(out.unbind(0)), t.contiguous(), group=group)
    return out


def sharded_forward(Q_local, K_shard, V_shard, n0: int, *, compress_partial, reduce_partials, attend, zeros_partial,
                    all_gather=all_gather_stacked):
    """Token-sharded forward of one rank.  The four callables are the library's steps (or stand-ins with the same
    meaning): compress_partial(K_shard, V_shard, n0) -> float32 partial sums of K~|V~; zeros_partial() -> the same
    shape filled with zeros (a rank without tokens); reduce_partials(stacked) adds the ranks' partials in rank
    order into the workspace; attend(Q_local) -> this rank's output rows.  Returns attend's result."""
    partial = compress_partial(K_shard, V_shard, n0) if K_shard.shape[-2] > 0 else zeros_partial()
    stacked = all_gather(partial)              # lands in this rank's own memory before any kernel reads it
    reduce_partials(stacked)
    return attend(Q_local)


def csat_sharded_forward(ctx, Q_local, K_shard, V_shard, n0: int, group=None):
    """sharded_forward on a binding.Csat context (created with the full sequence length n, the same seed on every
    rank and n_q = the number of local queries)."""
    import torch
    return sharded_forward(
        Q_local, K_shard, V_shard, n0,
        compress_partial=ctx.compress_partial,
        zeros_partial=lambda: torch.zeros(ctx.B, ctx.H, ctx.m, 2 * ctx.d, dtype=torch.float32, device=Q_local.device),
        reduce_partials=ctx.reduce_partials, attend=ctx.attend,
        all_gather=lambda t: all_gather_stacked(t, group))
