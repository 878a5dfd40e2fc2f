"""Data-parallel glue: tokens are sharded across ranks, the router weights and
the controller state are replicated, and the only exchange is the sum of the
per-expert load counts between routing and the controller update (Algorithm 1
line 4 takes n_i over all microbatches and all data-parallel ranks of the
iteration).  Integer sums make the controller update bit-identical on every
rank.

The exchange is one in-place all-reduce(SUM) of L*E int32 (3 KB per layer) on
the accumulator buffer itself: one collective per step, enqueued on the stream
the kernels run on (plain torch.distributed -- NCCL on GPUs; there is no
compute step to fuse a 3 KB exchange with).
"""
from __future__ import annotations


def allreduce_loads(router, dist, group=None):
    """Replace this rank's load accumulators by the sum over all ranks.

    `router.loads_view()` must return an int32 tensor [L][E] that ALIASES the
    accumulators (binding.Router does, through moe_loads_buffer); the reduction
    happens in place, so nothing is copied, cloned or added afterwards.
    Objects without such a view (only loads_peek() / loads_add()) are served by
    the three-step form.  `dist` is torch.distributed with a backend that
    handles the tensor's device.
    """
    view = getattr(router, "loads_view", None)
    if view is not None:
        acc = view()
        dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
        return acc
    own = router.loads_peek()
    total = own.clone()
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    router.loads_add(total - own)
    return total
