"""Sharding over more than one GPU: by tokens (the default) or by experts.

Tokens are routed independently, so the path shards over tokens with no collective on the data path: every rank
holds R1 and R2, routes a contiguous range of token rows and writes its own slice of the ids and gates.  The only
quantity that spans ranks is the per-expert count vector; a caller that wants global counts sums the M int32
values once (``allreduce_counts``).  The benchmark's multi-GPU mode gives every rank its own batch and needs no
collective at all.

When the router itself is too large for one GPU, or a layer's experts already live sharded, the EXPERT dimension
can be split instead: every rank routes all tokens over its own columns of R2 (``expert_range``), then the ranks
all-gather their k best (id, logit) pairs per token and their log-sum-exp (``gather_shard_reports``: ``k`` pairs per
token and rank cross the links, nothing of size M) and each merges them with ``more_merge_shards``.
"""
from __future__ import annotations


def token_range(T: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced split of ``T`` token rows: ranks ``< T % world`` get one extra row."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(T, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_counts(counts, group=None):
    """Sum per-rank expert counts in place over the process group (NCCL on GPUs, gloo on CPU tensors)."""
    import torch.distributed as dist
    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    return counts


def expert_range(M: int, rank: int, world: int, multiple: int = 8) -> tuple[int, int]:
    """Contiguous split of ``M`` experts into ``world`` ranges whose boundaries are multiples of ``multiple`` (the
    tensor-core path wants shard widths that are multiples of 8); the last range takes the remainder."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    if multiple < 1:
        raise ValueError("multiple must be positive")
    units = M // multiple
    base, extra = divmod(units, world)
    lo = (rank * base + min(rank, extra)) * multiple
    hi = ((rank + 1) * base + min(rank + 1, extra)) * multiple
    if rank == world - 1:
        hi = M
    return lo, hi


def gather_shard_reports(idx, topval, lse, group=None):
    """All-gather the per-rank reports of an expert-sharded router.

    ``idx``/``topval`` are this rank's ``[T, k]`` tensors (ids local to the shard, logits), ``lse`` its ``[T]``
    log-sum-exp or None.  Returns ``(idx [S, T, k], topval [S, T, k], lse [S, T] or None)`` on every rank, stacked by
    rank, ready for ``more_merge_shards`` together with the ranks' first expert ids as ``shard_base``.  All ranks
    must report the same k (a shard with fewer experts pads with id -1 / logit -inf)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    all_idx = torch.empty((world,) + tuple(idx.shape), dtype=idx.dtype, device=idx.device)
    all_val = torch.empty((world,) + tuple(topval.shape), dtype=topval.dtype, device=topval.device)
    # (list form: the gloo backend used by the CPU tests has no all_gather_into_tensor)
    dist.all_gather(list(all_idx.unbind(0)), idx.contiguous(), group=group)
    dist.all_gather(list(all_val.unbind(0)), topval.contiguous(), group=group)
    all_lse = None
    if lse is not None:
        all_lse = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype, device=lse.device)
        dist.all_gather(list(all_lse.unbind(0)), lse.contiguous(), group=group)
    return all_idx, all_val, all_lse
