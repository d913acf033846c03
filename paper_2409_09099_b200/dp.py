"""Data parallelism over tokens: the only way the S-STE linear path shards.

Every rank holds the full dense weight (beta and the projection depend on W only, so they are
identical everywhere) and a contiguous shard of the tokens.  Forward, MVUE and grad_X are local;
grad_W = MVUE(grad_Z^T) X is a sum over tokens, so the per-rank partial grad_W is all-reduced
(the one exchange step of the path).  The MVUE counter is the global group index: a rank passes
the number of tokens that precede its shard, so the draws do not depend on the number of ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def token_shard(total_tokens: int, rank: int, world: int, multiple: int = 128):
    """(first token, token count) of `rank`'s contiguous shard; every shard is a multiple of `multiple`."""
    assert total_tokens % (multiple * world) == 0, "tokens must split into equal multiples of 128 per rank"
    per = total_tokens // world
    return rank * per, per


def allreduce_grad_w(tensors, group=None):
    """Sum the per-rank partial weight gradients in place (NCCL on GPUs, gloo on CPU); returns the handles."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return []
    return [dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group, async_op=True) for t in tensors]
