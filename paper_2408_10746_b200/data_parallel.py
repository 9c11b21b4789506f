"""Data-parallel phase-2 training (paper Section V-B).

After the first epoch every device holds the full set of adapter parameters and the cached
activations of its share of the samples; the devices then train the adapters in a data-parallel
manner.  Here: one process per GPU, each with its own trainer over its shard of the cache.  A
global minibatch is the union of the ranks' local minibatches (equal sizes), every rank computes the
gradient of its local mean loss, the gradient buffers are summed across ranks with one all-reduce per
step, and every rank applies the identical AdamW update, so the replicas stay bit-identical.

Nothing in a step waits on the host.  The local step is enqueued without a loss read-back (the loss
goes to a slot of a device buffer), the all-reduce is enqueued on the same stream order (NCCL runs it
on its own stream between two events), the 1/world that turns the sum into the mean is a factor the
optimizer KERNEL applies while it reads the gradient (`set_grad_scale`), and the losses of an epoch
are reduced and read once, in `epoch_losses()`.  The class only orchestrates: the local trainer does
all arithmetic.  A local trainer provides

    train_step(ids, loss_slot)   enqueue forward + backward; local mean loss -> loss_slot (1-element tensor)
    grad_buffer() -> tensor      the flat gradient vector, reduced IN PLACE
    param_buffer() -> tensor     the flat parameter vector (broadcast from rank 0 at start)
    params_changed()             called after the broadcast wrote into param_buffer()
    set_grad_scale(s)            factor the optimizer applies to every gradient it reads
    adam_step(hp)
    new_loss_buffer(n) -> tensor n float32 slots on the trainer's device
    stream_context()             context manager under which collectives must be issued
"""
from __future__ import annotations

import contextlib
from typing import Optional

import torch
import torch.distributed as dist


class PacLocalTrainer:
    """Adapter around a PacContext: exposes its device buffers for in-place collectives.  `stream` is
    the torch stream whose handle the context was created on; collectives are issued under it, so that
    they are ordered behind the step's kernels and ahead of the optimizer's.  With None the context must
    have been created on the stream that is torch's current one whenever the orchestrator runs."""

    def __init__(self, ctx, stream: Optional["torch.cuda.Stream"] = None):
        self.ctx, self.stream = ctx, stream
        self._params, self._grads = ctx.device_buffers()

    def train_step(self, ids, loss_slot: torch.Tensor) -> None:
        self.ctx.train_step_dev_loss(ids, loss_slot.data_ptr())

    def grad_buffer(self) -> torch.Tensor:
        return self._grads

    def param_buffer(self) -> torch.Tensor:
        return self._params

    def params_changed(self):
        self.ctx.params_changed()

    def set_grad_scale(self, scale: float):
        self.ctx.set_grad_scale(scale)

    def adam_step(self, hp):
        self.ctx.adam_step(hp)

    def new_loss_buffer(self, n: int) -> torch.Tensor:
        return torch.zeros(n, dtype=torch.float32, device=self._grads.device)

    def stream_context(self):
        return torch.cuda.stream(self.stream) if self.stream is not None else contextlib.nullcontext()


class DataParallel:
    def __init__(self, local, group: Optional[dist.ProcessGroup] = None, broadcast_params: bool = True,
                 loss_slots: int = 4096):
        self.local, self.group = local, group
        self.world = dist.get_world_size(group)
        self.comm = f"all-reduce (sum) of the flat fp32 adapter gradient per step, {dist.get_backend(group)}"
        with local.stream_context():
            if broadcast_params and self.world > 1:
                # the paper's redistribution step: every device receives the complete adapter parameters
                dist.broadcast(local.param_buffer(), src=dist.get_global_rank(group, 0) if group is not None else 0, group=group)
                local.params_changed()
        local.set_grad_scale(1.0 / self.world)      # sum over ranks -> mean, applied inside the optimizer kernel
        self.losses = local.new_loss_buffer(loss_slots)
        self.n = 0

    def train_step(self, local_ids) -> None:
        """Enqueues one step on this rank's share of the global minibatch and the gradient exchange
        behind it.  Returns nothing: the loss stays on the device until epoch_losses()."""
        if self.n >= self.losses.numel():
            raise RuntimeError("loss buffer full: call epoch_losses() (at least once per loss_slots steps)")
        self.local.train_step(local_ids, self.losses[self.n:self.n + 1])
        self.n += 1
        if self.world > 1:
            with self.local.stream_context():
                dist.all_reduce(self.local.grad_buffer(), op=dist.ReduceOp.SUM, group=self.group)

    def adam_step(self, hp):
        self.local.adam_step(hp)

    def epoch_losses(self):
        """Global mean loss of every step since the last call: one collective and one host read."""
        with self.local.stream_context():
            t = self.losses[:self.n].clone()
            if self.world > 1:
                dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)
            out = t.cpu().numpy() / self.world
        self.n = 0
        return out


def shard_ids(global_ids, rank: int, world: int):
    """Rank `rank`'s contiguous share of a global minibatch (its length must divide evenly)."""
    n = len(global_ids)
    if n % world != 0:
        raise ValueError("global minibatch does not divide evenly across ranks")
    per = n // world
    return list(global_ids[rank * per:(rank + 1) * per])
