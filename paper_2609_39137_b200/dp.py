"""Data-parallel glue: tokens are sharded across ranks, the router weights and
the controller state are replicated, and the only exchange is the sum of the
per-expert load counts before the controller update (Algorithm 1 line 4:
counts are summed over microbatches and the data-parallel group).  Integer
sums make the controller update bit-identical on every rank.

The exchange is one all-reduce(SUM) of L*E int32 (3 KB per layer): plain
torch.distributed; there is no compute step to fuse it with.
"""
from __future__ import annotations


def allreduce_loads(router, dist, group=None):
    """Replace this rank's load accumulators by the sum over all ranks.

    `router` needs loads_peek() -> int32 tensor [L][E] and loads_add(tensor);
    `dist` is torch.distributed (any backend that handles the tensor's device).
    """
    own = router.loads_peek()
    total = own.clone()
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    router.loads_add(total - own)
    return total
