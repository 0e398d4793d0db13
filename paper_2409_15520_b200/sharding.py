"""One ZO step spread over several GPUs, one process per GPU.

The 2q replicas of a step are independent forward passes (Algorithm 1: query i has its own seed
and its own pair of losses), so rank k runs a contiguous block of queries, the ranks exchange the
2q loss scalars, and every rank regenerates all z_i and applies the same update to its own copy of
the trainable B tensors.  Nothing else crosses between GPUs.  Host logic only: the forward, the
projected gradients and the update run in the CUDA library.
"""
from __future__ import annotations


def query_shard(q: int, world_size: int, rank: int) -> tuple[int, int]:
    """(first query, number of queries) of `rank`: contiguous blocks, the first q % world_size
    ranks take one query more (a rank beyond q gets an empty block)."""
    if q < 1 or world_size < 1 or not 0 <= rank < world_size:
        raise ValueError("need q >= 1 and 0 <= rank < world_size")
    base, extra = divmod(q, world_size)
    begin = rank * base + min(rank, extra)
    return begin, base + (1 if rank < extra else 0)


def exchange_losses(buf, q: int, group=None):
    """Completes the loss array: every rank holds its own queries' losses and zeros elsewhere, so
    a sum over ranks is exact (one non-zero contributor per entry) and also covers uneven shards.
    `buf` is a float64 tensor (device tensor under NCCL, CPU tensor under gloo), reduced in place
    over its first 2q entries."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(buf[:2 * q], op=dist.ReduceOp.SUM, group=group)
    return buf


def exchange_step(buf, group=None):
    """The exchange of a sharded step in one collective: the whole loss array of the library, i.e.
    the 2 * max_q losses (zero outside each rank's block, also beyond 2q) and the fault slot at the
    end, summed over ranks.  Afterwards every rank holds all losses and knows whether ANY rank saw a
    device-side fault, so zo_apply_update skips the update everywhere or nowhere."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
    return buf


def sharded_step(est, prob, E, S, seed, q, eps, lr, rank=None, world_size=None, group=None,
                 tokens=None, labels=None):
    """One step of Algorithm 1 with the q queries spread over the ranks of `group`.  Every rank
    passes the same batch, seed, q, eps and lr and holds identical B tensors before and after.
    The collective runs on the current stream, which must be the estimator's.  The query shard is
    switched off again before returning, so a later plain `est.step` is a whole step."""
    import torch.distributed as dist
    if world_size is None:
        world_size = dist.get_world_size(group) if dist.is_initialized() else 1
    if rank is None:
        rank = dist.get_rank(group) if dist.is_initialized() else 0
    if world_size > q:
        raise ValueError("more ranks than queries: every rank needs at least one query of the step")
    begin, count = query_shard(q, world_size, rank)
    est.set_query_shard(begin, count)
    try:
        est.step(prob, E, S, seed, q, eps, 0.0, tokens=tokens, labels=labels)
    finally:
        est.set_query_shard(0, 0)
    exchange_step(est.loss_buffer(), group)
    est.apply_update(prob, seed, q, eps, lr)
