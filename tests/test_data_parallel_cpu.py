"""Data-parallel orchestration on CPU: two gloo ranks, each driving the oracle on its half of the
global minibatch, must reproduce the single-process oracle on the whole minibatch (the gradient of
a mean over the batch is the mean of the shard gradients) and keep the replicas identical."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import pac_inputs as pi  # noqa: E402
from oracle import pac_oracle as po  # noqa: E402

SPEC = pi.CacheSpec("dp_cpu", N=16, L=3, S=6, d=24, dtype="f32", r=8, n_out=3, B=8)
STEPS = 2


class OracleLocal:
    """The oracle behind the local-trainer interface (float64 so that the comparison is tight)."""

    def __init__(self, flat):
        cache = pi.cache_full(SPEC, 0).double().numpy()
        labels = pi.labels(SPEC, 0).numpy().astype(np.int64)
        self.tr = po.Trainer(cache, labels, po.unflatten(flat.astype(np.float64), SPEC.L, SPEC.d, SPEC.r, SPEC.n_out))
        self._p = torch.from_numpy(po.flatten(self.tr.P))
        self._g = torch.zeros_like(self._p)

    def train_step(self, ids, loss_slot):
        loss = self.tr.train_step(ids)
        self._g.copy_(torch.from_numpy(po.flatten(self.tr.grads)))
        loss_slot.fill_(loss)

    def set_grad_scale(self, scale):
        self.scale = scale

    def new_loss_buffer(self, n):
        return torch.zeros(n, dtype=torch.float64)

    def stream_context(self):
        import contextlib
        return contextlib.nullcontext()

    def grad_buffer(self):
        return self._g

    def param_buffer(self):
        return self._p

    def params_changed(self):
        self.tr.P = po.unflatten(self._p.numpy().copy(), SPEC.L, SPEC.d, SPEC.r, SPEC.n_out)

    def adam_step(self, hp):
        # the factor a device-side optimizer applies while reading the (summed) gradient buffer
        self.tr.grads = po.unflatten(self._g.numpy().copy() * self.scale, SPEC.L, SPEC.d, SPEC.r, SPEC.n_out)
        self.tr.hp = hp
        self.tr.adam_step()
        self._p.copy_(torch.from_numpy(po.flatten(self.tr.P)))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2408_10746_b200.data_parallel import DataParallel, shard_ids
    # rank 1 starts from different parameters: the broadcast must overwrite them
    flat = pi.random_params(SPEC, 3 if rank == 0 else 9)
    dp = DataParallel(OracleLocal(flat))
    perm = pi.epoch_permutation(SPEC.N, 2)
    for s in range(STEPS):
        gids = perm[s * SPEC.B:(s + 1) * SPEC.B].tolist()
        assert dp.train_step(shard_ids(gids, rank, world)) is None
        dp.adam_step(po.AdamW())
    losses = dp.epoch_losses().tolist()
    out[rank] = (losses, dp.local.param_buffer().numpy().copy())
    dist.destroy_process_group()


class RecordingLocal:
    """A local trainer that computes nothing and records what the orchestrator asks of it."""

    def __init__(self, n, rank):
        self.log, self.rank = [], rank
        self._p = torch.full((n,), float(rank + 1))
        self._g = torch.zeros(n)

    def train_step(self, ids, loss_slot):
        self.log.append(("train_step", tuple(ids)))
        self._g.fill_(float(self.rank + 1))           # rank-dependent "gradient"
        loss_slot.fill_(10.0 * (self.rank + 1) + len(self.log))

    def grad_buffer(self):
        return self._g

    def param_buffer(self):
        return self._p

    def params_changed(self):
        self.log.append(("params_changed",))

    def set_grad_scale(self, scale):
        self.log.append(("set_grad_scale", scale))

    def adam_step(self, hp):
        self.log.append(("adam_step", self._g[:1].clone()))   # what the optimizer would read (kept as a tensor)

    def new_loss_buffer(self, n):
        return torch.zeros(n)

    def stream_context(self):
        import contextlib
        return contextlib.nullcontext()


def _recording_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2408_10746_b200.data_parallel import DataParallel
    local = RecordingLocal(5, rank)
    dp = DataParallel(local)
    # from here on a step must not read anything back to the host: count every route a tensor has
    reads = []
    patched = {}
    for name in ("item", "tolist", "cpu", "numpy", "__float__", "__int__", "__bool__"):
        orig = getattr(torch.Tensor, name)
        patched[name] = orig

        def spy(self, *a, _orig=orig, _name=name, **k):
            reads.append(_name)
            return _orig(self, *a, **k)
        setattr(torch.Tensor, name, spy)
    try:
        for s in range(3):
            assert dp.train_step([s, s + 1]) is None
            dp.adam_step(None)
        reads_in_steps = list(reads)
    finally:
        for name, orig in patched.items():
            setattr(torch.Tensor, name, orig)
    losses = dp.epoch_losses().tolist()
    log = [(e[0], float(e[1][0])) if e[0] == "adam_step" else e for e in local.log]
    out[rank] = (log, reads_in_steps, losses, local.param_buffer().tolist())
    dist.destroy_process_group()


def test_orchestration_order_and_no_host_read_per_step():
    """Two ranks with recording trainers: parameters are broadcast once, the 1/world factor is handed
    to the optimizer (not applied in Python), every step is train_step -> all-reduce -> adam_step with
    the SUM of the ranks' gradients in the buffer, and no tensor is read back to the host until the
    losses of the epoch are asked for."""
    world, port = 2, 31000 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_recording_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        log, reads_in_steps, losses, params = out[rank]
        assert reads_in_steps == []
        assert params == [1.0] * 5                              # rank 0's parameters everywhere
        assert log[0] == ("params_changed",) and log[1] == ("set_grad_scale", 0.5)
        steps = log[2:]
        assert [e[0] for e in steps] == ["train_step", "adam_step"] * 3
        assert all(e == ("adam_step", 3.0) for e in steps[1::2])          # 1 + 2: the sum, unscaled
        assert [e[1] for e in steps[0::2]] == [(0, 1), (1, 2), (2, 3)]
        # mean over ranks of the per-rank losses 10*(rank+1) + k
        assert np.allclose(losses, [15.0 + k for k in (3, 5, 7)])


def test_two_ranks_match_single_process_oracle():
    world, port = 2, 29000 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    # single process on the whole minibatch
    cache = pi.cache_full(SPEC, 0).double().numpy()
    labels = pi.labels(SPEC, 0).numpy().astype(np.int64)
    tr = po.Trainer(cache, labels, po.unflatten(pi.random_params(SPEC, 3).astype(np.float64), SPEC.L, SPEC.d, SPEC.r, SPEC.n_out))
    perm = pi.epoch_permutation(SPEC.N, 2)
    ref_losses = []
    for s in range(STEPS):
        ref_losses.append(tr.train_step(perm[s * SPEC.B:(s + 1) * SPEC.B].tolist()))
        tr.adam_step()
    ref = po.flatten(tr.P)
    for rank in range(world):
        losses, params = out[rank]
        np.testing.assert_allclose(losses, ref_losses, rtol=1e-12)
        np.testing.assert_allclose(params, ref, rtol=1e-9, atol=1e-12)
    assert np.array_equal(out[0][1], out[1][1])             # replicas stay identical


def test_shard_ids():
    from paper_2408_10746_b200.data_parallel import shard_ids
    assert shard_ids(list(range(8)), 1, 2) == [4, 5, 6, 7]
    import pytest
    with pytest.raises(ValueError):
        shard_ids(list(range(7)), 0, 2)
