"""Row-sharded epoch: one minibatch step over the rows of several devices.

The paper's SGD runs on one device.  Its step shards by rows with a single exchange: the gradient of a
minibatch (paper Eq. (double), symmetrised) is a sum over the minibatch's rows, so every rank forms the sum over
the rows it holds, the ranks add their n-float shares (one all-reduce per step), and every rank then applies
Q4 and the update (paper "End-to-end Quantization", Eq. (proxupdate)) to its own replica of x.  Q3 and Q4 draw
from counters keyed by (seed, epoch, step, coordinate), not by rank, so the replicas stay identical.

Partition: batch t holds the global rows [t B, min(m, (t+1) B)); rank r of W holds the rows
[t B + r B/W, min(t B + (r+1) B/W, end of the batch)) of it (B divisible by W).  Locally the rank's rows lie in
that order, so its local batch t (of size B/W) is its share of the global batch t; only the last batch can be
ragged, and a rank may hold nothing of it.

This module holds the partition and the step loop; the arithmetic of a step is the library's
(zipml_sgd_epoch for the share of the gradient, zipml_sgd_apply_gradient for Q4 and the update).
"""
from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence


@dataclass
class ShardPlan:
    m: int
    batch: int
    rank: int
    world: int

    def __post_init__(self):
        if self.world < 1 or not (0 <= self.rank < self.world):
            raise ValueError("rank/world out of range")
        if self.batch <= 0 or self.batch % self.world != 0:
            raise ValueError("the minibatch size must be a positive multiple of the number of ranks")
        if self.m <= 0:
            raise ValueError("no rows")

    @property
    def steps(self) -> int:
        return (self.m + self.batch - 1) // self.batch

    @property
    def local_batch(self) -> int:
        return self.batch // self.world

    def batch_rows(self, t: int) -> int:
        """Rows of the whole batch t."""
        return min(self.m, (t + 1) * self.batch) - t * self.batch

    def span(self, t: int):
        """Global rows [start, stop) of batch t that this rank holds (start == stop: none)."""
        end = min(self.m, (t + 1) * self.batch)
        start = min(end, t * self.batch + self.rank * self.local_batch)
        stop = min(end, t * self.batch + (self.rank + 1) * self.local_batch)
        return start, stop

    def count(self, t: int) -> int:
        start, stop = self.span(t)
        return stop - start

    def weight(self, t: int) -> float:
        """This rank's share of batch t: a mean over the rank's rows times this is its part of the batch's mean."""
        return self.count(t) / self.batch_rows(t)

    def row_spans(self) -> List[tuple]:
        """The rank's global rows as [start, stop) spans in local order."""
        return [s for s in (self.span(t) for t in range(self.steps)) if s[1] > s[0]]

    @property
    def local_rows(self) -> int:
        return sum(b - a for a, b in self.row_spans())

    @property
    def local_steps(self) -> int:
        return (self.local_rows + self.local_batch - 1) // self.local_batch if self.local_rows else 0


def run_steps(plan: ShardPlan, share: Callable, all_reduce: Callable, apply: Callable,
              order: Optional[Sequence[int]] = None, first_step: int = 0, num_steps: Optional[int] = None) -> None:
    """The step loop.  share(pos, t, weight) -> the rank's weighted share of the gradient of batch t at position
    pos (weight * the mean over its rows; zeros if it holds none); all_reduce(v) adds the ranks' vectors in place;
    apply(v, pos) is Q4 and the update on the rank's replica of x."""
    T = plan.steps
    stop = T if num_steps is None else first_step + num_steps
    if first_step < 0 or stop > T:
        raise ValueError("steps out of range")
    if order is not None and (len(order) != T or any(o < 0 or o >= T for o in order)):
        raise ValueError("batch order must hold one valid batch index per step")
    for pos in range(first_step, stop):
        t = int(order[pos]) if order is not None else pos
        v = share(pos, t, plan.weight(t))
        all_reduce(v)
        apply(v, pos)


def take_rows(plan: ShardPlan, rows):
    """The rank's rows of a row-indexed tensor or array (planes, labels, samples), in local order."""
    import torch
    spans = plan.row_spans()
    if isinstance(rows, torch.Tensor):
        return torch.cat([rows[a:b] for a, b in spans]).contiguous()
    import numpy as np
    return np.ascontiguousarray(np.concatenate([rows[a:b] for a, b in spans]))


class ShardedEpoch:
    """A rank's side of a row-sharded epoch.  data_local / b_local: the rank's rows in local order (see take_rows);
    x: the rank's replica of the model (device tensor, updated in place)."""

    def __init__(self, ctx, plan: ShardPlan, data_local, b_local, x, lr, batch_order=None, model_bits=0, grad_bits=0,
                 seed=0, epoch=0, reg=0, reg_param=0.0, engine=0):
        import torch
        self.ctx, self.plan, self.data, self.b, self.x, self.lr = ctx, plan, data_local, b_local, x, lr
        self.model_bits, self.grad_bits, self.seed, self.epoch = model_bits, grad_bits, seed, epoch
        self.reg, self.reg_param, self.engine = reg, reg_param, engine
        self.n = x.numel()
        self.g2 = torch.empty(2 * self.n, dtype=torch.float32, device=x.device)
        self.order = None if batch_order is None else [int(o) for o in batch_order]
        T_local = plan.local_steps
        # positions whose batch this rank does not hold are never executed; their entries only have to be valid
        self.order_local = None if self.order is None or not T_local else [min(o, T_local - 1) for o in self.order][:T_local]

    def share(self, pos, t, weight):
        """weight * the mean over the rank's rows of batch t of the symmetrised gradient, at the model (or its Q3
        image for position pos) as it stands; zeros if the rank holds none of the batch."""
        import torch
        if self.plan.count(t) == 0:
            return torch.zeros(self.n, dtype=torch.float32, device=self.x.device)
        kw = dict(model_bits=self.model_bits, grad_bits=0, seed=self.seed, epoch=self.epoch, num_steps=1, engine=self.engine,
                  first_step=pos, grad_out=self.g2)
        if self.order_local is not None:
            # the library keys Q3 by the position: the step runs at position pos of a local order that names t there
            if pos >= len(self.order_local):
                raise ValueError("under a batch order a rank that holds fewer batches than the epoch has steps cannot "
                                 "take a position beyond its own count")
            lo = list(self.order_local)
            lo[pos] = t
            kw["batch_order"] = lo
        self.ctx.zipml_sgd_epoch(self.data, self.b, self.x, self.plan.local_batch, 0.0, **kw)   # lr = 0: x stays
        return self.g2[:self.n] * weight

    def apply(self, v, pos):
        """Q4 and the update on this rank's replica."""
        self.ctx.zipml_sgd_apply_gradient(self.x, v.contiguous(), pos, self.lr, grad_bits=self.grad_bits, seed=self.seed,
                                          epoch=self.epoch, reg=self.reg, reg_param=self.reg_param)

    def run(self, group=None, first_step=0, num_steps=None, all_reduce=None):
        """The epoch (or a range of its steps).  The ranks meet in one all-reduce of n floats per step
        (torch.distributed on `group`; `all_reduce(v)` replaces it, e.g. for ranks emulated in one process)."""
        import torch.distributed as dist

        def reduce(v):
            if all_reduce is not None:
                all_reduce(v)
            elif dist.is_available() and dist.is_initialized() and self.plan.world > 1:
                dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)

        run_steps(self.plan, self.share, reduce, self.apply, order=self.order, first_step=first_step, num_steps=num_steps)
