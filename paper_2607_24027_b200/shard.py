"""Splitting one attention call over several GPUs.

Every (batch, head) pair of the operator is independent -- routing, thresholds and the online softmax
never look across heads -- so a call shards by heads with no exchange step: rank r runs the same
kernels on its own contiguous range of (batch, head) pairs and writes its own slice of the output.
Nothing here touches a GPU; the bench and the tests share it.
"""
from __future__ import annotations


def head_partition(total_heads: int, world_size: int, rank: int) -> slice:
    """Contiguous range of flattened (batch, head) indices owned by `rank`.

    The first ``total_heads % world_size`` ranks get one head more; ranks beyond the head count get an
    empty range.  The ranges of all ranks are disjoint and cover ``range(total_heads)`` in rank order.
    """
    if total_heads < 0 or world_size <= 0 or not 0 <= rank < world_size:
        raise ValueError("bad partition request")
    base, extra = divmod(total_heads, world_size)
    start = rank * base + min(rank, extra)
    return slice(start, start + base + (1 if rank < extra else 0))
