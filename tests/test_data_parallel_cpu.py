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

    def train_step(self, ids):
        loss = self.tr.train_step(ids)
        self._g.copy_(torch.from_numpy(po.flatten(self.tr.grads)))
        return loss

    def grad_buffer(self):
        return self._g

    def param_buffer(self):
        return self._p

    def params_changed(self):
        self.tr.P = po.unflatten(self._p.numpy().copy(), SPEC.L, SPEC.d, SPEC.r, SPEC.n_out)

    def adam_step(self, hp):
        self.tr.grads = po.unflatten(self._g.numpy().copy(), SPEC.L, SPEC.d, SPEC.r, SPEC.n_out)
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
    losses = []
    for s in range(STEPS):
        gids = perm[s * SPEC.B:(s + 1) * SPEC.B].tolist()
        losses.append(dp.train_step(shard_ids(gids, rank, world)))
        dp.adam_step(po.AdamW())
    out[rank] = (losses, dp.local.param_buffer().numpy().copy())
    dist.destroy_process_group()


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
