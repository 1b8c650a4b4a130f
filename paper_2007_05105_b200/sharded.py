"""Column-sharded AdaScale step over several GPUs: one process per GPU, one 16-byte exchange.

The paper's setting is S workers whose gradients are combined synchronously (Sec. 2); its
estimator needs only two global numbers per iteration, sum_i ||g_i - gbar||^2 and ||gbar||^2
(App. B.3), and both are sums over coordinates.  So when the parameters are split by columns
- rank q holds all S rows of columns [q P / N, (q + 1) P / N), their parameters and momentum -
the only exchange is an all-reduce of that pair:

    adascale_reduce_sums   (this rank's mean gradient and its pair, on the device)
    all-reduce (sum) of the 2 float64 values over the ranks  (NCCL; gloo on CPU in tests)
    adascale_apply_sums    (scalar part on the completed sums, then this rank's update)

Every rank runs the scalar part on the identical two numbers and so reaches the identical r_t,
eta_t and tau.  No kernel reads another GPU's memory.  This module only sequences those three
calls; it holds none of the method's arithmetic.
"""
from __future__ import annotations


def split_columns(numels, rank, world, align=64):
    """Pieces of the tensor list that make up rank's share of the concatenated columns.

    The P columns of the concatenated tensors are cut into `world` contiguous ranges whose
    boundaries are multiples of `align` (the last range takes the remainder).  Returns a list of
    (tensor index, first element, length) for the pieces of `rank`, in order; lengths are > 0.
    """
    numels = [int(n) for n in numels]
    P = sum(numels)
    per = -(-P // world)
    per = -(-per // align) * align
    lo, hi = min(P, rank * per), min(P, (rank + 1) * per)
    pieces, start = [], 0
    for k, n in enumerate(numels):
        a, b = max(lo, start), min(hi, start + n)
        if b > a:
            pieces.append((k, a - start, b - a))
        start += n
    return pieces


class ShardedAdaScale:
    """One rank of a column-sharded run.

    ctx     an object with reduce_sums(grads, sums, stream) and apply_sums(sums, sched, params,
            momentum, stream): a binding.AdaScale over this rank's columns
    sums    a float64 tensor of 2 elements on the device the context works on
    group   torch.distributed process group (None = the default group); with one rank and no
            initialised process group the exchange is skipped
    """

    def __init__(self, ctx, sums, group=None):
        self.ctx = ctx
        self.sums = sums
        self.group = group

    def exchange(self):
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized():
            dist.all_reduce(self.sums, op=dist.ReduceOp.SUM, group=self.group)

    def step(self, grads, params, momentum, sched, stream=None):
        self.ctx.reduce_sums(grads, self.sums, stream)
        self.exchange()      # ordered after reduce_sums and before apply_sums on the current stream
        self.ctx.apply_sums(self.sums, sched, params, momentum, stream)
