"""Data-parallel plumbing: which tokens a rank owns and how the weight gradients are combined.

The Monarch multiply is independent per token, so ranks split the token batch and run the whole
path on their shard with no data-path exchange; only the weight gradients dL, dR (sums over
tokens) are all-reduced, exactly as in ordinary data-parallel training.  This module holds host
logic only (no arithmetic of the method) and works with any torch.distributed backend.
"""
from __future__ import annotations


def shard_tokens(tokens: int, world: int, rank: int, granule: int = 64):
    """Contiguous token range [start, start+count) of `rank`.

    Whole granules (the kernels' 64-token tiles) are dealt out as evenly as possible, earlier ranks
    taking the extra ones; the ragged remainder goes to the last rank that owns any tokens.  The
    ranges of all ranks tile [0, tokens) in order without gaps or overlap.
    """
    if tokens < 0 or world < 1 or not 0 <= rank < world or granule < 1:
        raise ValueError("bad sharding arguments")
    full, tail = divmod(tokens, granule)
    base, extra = divmod(full, world)
    counts = [(base + (1 if r < extra else 0)) * granule for r in range(world)]
    owner = max((r for r in range(world) if counts[r] > 0), default=0)
    counts[owner] += tail
    start = sum(counts[:rank])
    return start, counts[rank]


def pack_grads(dL, dR):
    """One flat float32 buffer holding (dL, dR), so that a single all-reduce carries both."""
    import torch
    return torch.cat([dL.reshape(-1), dR.reshape(-1)])


def allreduce_grads(dL, dR, group=None):
    """Sum dL and dR over the ranks of `group`, in place, with one collective."""
    import torch.distributed as dist
    flat = pack_grads(dL, dR)
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    k = dL.numel()
    dL.copy_(flat[:k].view_as(dL))
    dR.copy_(flat[k:].view_as(dR))
    return dL, dR
