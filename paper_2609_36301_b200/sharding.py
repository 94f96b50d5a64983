"""Token sharding for more than one GPU.

Tokens are routed independently, so the path shards over tokens with no collective on the data path: every rank
holds R1 and R2, routes a contiguous range of token rows and writes its own slice of the ids and gates.  The only
quantity that spans ranks is the per-expert count vector; a caller that wants global counts sums the M int32
values once (``allreduce_counts``).  The benchmark's multi-GPU mode gives every rank its own batch and needs no
collective at all.
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
