"""Batch sharding over GPUs (one process per GPU, torch.distributed).

Every (batch entry, head) of graph self-attention is independent given the graph, so a
batch is split over ranks with no exchange in the forward.  In the backward the relation
embedding table is shared by the whole batch (arXiv 1911.04070, Sec. 3.4), so its
gradient is the sum of the ranks' partial gradients: one all-reduce.
"""
from __future__ import annotations

import torch.distributed as dist


def batch_shard(global_batch: int, rank: int, world: int):
    """[start, stop) of the batch entries rank `rank` owns; sizes differ by at most one."""
    if not (0 <= rank < world) or global_batch < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(global_batch, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_d_rel(d_rel):
    """Sum the relation-embedding gradient over all ranks in place (no-op without a process group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(d_rel, op=dist.ReduceOp.SUM)
    return d_rel
