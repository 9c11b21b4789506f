"""Data-parallel phase-2 training (paper Section V-B).

After the first epoch every device holds the full set of adapter parameters and the cached
activations of its share of the samples; the devices then train the adapters in a data-parallel
manner.  Here: one process per GPU, each with its own trainer over its shard of the cache.  A
global minibatch is the union of the ranks' local minibatches (equal sizes), every rank computes the
gradient of its local mean loss, the gradients are averaged across ranks with one all-reduce per
step, and every rank applies the identical AdamW update, so the replicas stay bit-identical.

The class only orchestrates: the local trainer does all arithmetic.  A local trainer provides
    train_step(ids) -> loss      gradients of the local mean loss left in grad_buffer()
    grad_buffer() -> tensor      the flat gradient vector, reduced IN PLACE
    param_buffer() -> tensor     the flat parameter vector (broadcast from rank 0 at start)
    params_changed()             called after the broadcast wrote into param_buffer()
    adam_step(hp)
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


class PacLocalTrainer:
    """Adapter around a PacContext: exposes its device buffers for in-place collectives."""

    def __init__(self, ctx):
        self.ctx = ctx
        self._params, self._grads = ctx.device_buffers()

    def train_step(self, ids) -> float:
        return self.ctx.train_step(ids, want_loss=True)

    def grad_buffer(self) -> torch.Tensor:
        return self._grads

    def param_buffer(self) -> torch.Tensor:
        return self._params

    def params_changed(self):
        self.ctx.params_changed()

    def adam_step(self, hp):
        self.ctx.adam_step(hp)


class DataParallel:
    def __init__(self, local, group: Optional[dist.ProcessGroup] = None, broadcast_params: bool = True):
        self.local, self.group = local, group
        self.world = dist.get_world_size(group)
        if broadcast_params and self.world > 1:
            # the paper's redistribution step: every device receives the complete adapter parameters
            dist.broadcast(local.param_buffer(), src=dist.get_global_rank(group, 0) if group is not None else 0, group=group)
            local.params_changed()

    def train_step(self, local_ids) -> float:
        """One step on this rank's share of the global minibatch; returns the global mean loss."""
        loss = self.local.train_step(local_ids)
        if self.world > 1:
            g = self.local.grad_buffer()
            dist.all_reduce(g, op=dist.ReduceOp.SUM, group=self.group)
            g.div_(self.world)                       # mean of the ranks' local-mean gradients
            t = torch.tensor([loss], dtype=torch.float64, device=g.device)
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)
            loss = float(t.item()) / self.world
        return loss

    def adam_step(self, hp):
        self.local.adam_step(hp)


def shard_ids(global_ids, rank: int, world: int):
    """Rank `rank`'s contiguous share of a global minibatch (its length must divide evenly)."""
    n = len(global_ids)
    if n % world != 0:
        raise ValueError("global minibatch does not divide evenly across ranks")
    per = n // world
    return list(global_ids[rank * per:(rank + 1) * per])
