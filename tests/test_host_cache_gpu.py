"""A cache kept in host memory and reloaded per minibatch gives the same bits as the same cache
resident on the device: gather, evaluation, single steps, the asynchronous step, whole epochs
(where the reload of one step overlaps the kernels of the step before) and the LM head."""
import numpy as np
import pytest
import torch

import pac_inputs as pi
from oracle import pac_oracle as po
from tests.common import rel_l2

pytestmark = pytest.mark.gpu

TINY = pi.CONFIGS["tiny_fp32"].scaled(N=64, name="tiny_host")
TC = pi.CacheSpec("tc_host", N=48, L=12, S=128, d=768, dtype="bf16", r=64, n_out=3, B=8)
RAGGED = pi.CacheSpec("ragged_host", N=24, L=3, S=19, d=104, dtype="bf16", r=12, n_out=3, B=5)
LM = pi.CacheSpec("lm_host", N=12, L=3, S=24, d=128, dtype="bf16", r=16, n_out=1000, B=4, head="lm")


def make_pair(spec, pinned=True):
    """(context on a device-resident cache, context on the same cache in host memory)."""
    import paper_2408_10746_b200 as pac
    cache = pi.cache_full(spec, 0, "cuda")
    labels = pi.labels(spec, 0, "cuda")
    lm = pi.lm_head(spec, 0, "cuda") if spec.head == "lm" else None
    h_cache, h_labels = cache.cpu(), labels.cpu()
    if pinned:
        h_cache, h_labels = h_cache.pin_memory(), h_labels.pin_memory()
    out = []
    for host in (False, True):
        ctx = pac.PacContext(0)
        if host:
            ctx.cache_register_host(h_cache, h_labels)
        else:
            ctx.cache_register(cache, labels)
        ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B,
                         head=pac.PAC_HEAD_FROZEN_LM if spec.head == "lm" else pac.PAC_HEAD_MEANPOOL_CLS, lm_head=lm)
        ctx.set_params(pi.random_params(spec, 3))
        out.append(ctx)
    return out[0], out[1], cache


@pytest.mark.parametrize("spec", [TINY, TC, RAGGED, LM], ids=lambda s: s.name)
def test_host_cache_steps_match_device_cache(spec):
    import paper_2408_10746_b200 as pac
    dev, host, cache = make_pair(spec)
    hp = pac.AdamW()
    perm = np.concatenate([pi.epoch_permutation(spec.N, 2, epoch=e) for e in range(3)])
    B = spec.B
    # gather: bit-exact copies of the host slabs, boundary ids included
    ids = [spec.N - 1, 0] + perm[:B - 2].tolist()
    want = torch.empty((spec.L, B, spec.S, spec.d), dtype=cache.dtype, device="cuda")
    got = torch.empty_like(want)
    dev.gather(ids, want); host.gather(ids, got)
    dev.sync(); host.sync()
    assert torch.equal(want, got)
    assert torch.equal(got[:, 0], cache[spec.N - 1])
    # evaluation
    n_out = spec.n_out
    shape = (B, n_out) if spec.head == "cls" else (B, spec.S, n_out)
    la = torch.empty(shape, dtype=torch.float32, device="cuda"); lb = torch.empty_like(la)
    dev.eval_logits(ids, la); host.eval_logits(ids, lb)
    dev.sync(); host.sync()
    assert torch.equal(la, lb)
    # the staged path against the oracle directly (not only against the resident path): logits, then the
    # loss and every gradient block of the first step; fp32 caches at 1e-4, bf16 caches at the tensor
    # path's bounds
    flat = pi.random_params(spec, 3)
    C = spec.n_out if spec.head == "cls" else None
    P = po.unflatten(flat, spec.L, spec.d, spec.r, C)
    H = pi.cache_samples(spec, 0, ids, "cpu").float().numpy()
    W_lm = pi.lm_head(spec, 0, "cpu").float().numpy() if spec.head == "lm" else None
    tight = spec.dtype == "f32"
    assert rel_l2(lb.cpu().numpy(), po.eval_logits(P, H, 0, W_lm)) < (1e-4 if tight else 3e-3)
    labels_np = pi.labels(spec, 0, "cpu").numpy().astype(np.int64)
    # steps, partial batch included
    for i in range(5):
        step_ids = perm[i * B:(i + 1) * B] if i != 2 else perm[i * B:i * B + max(1, B // 2)]
        l1, l2 = dev.train_step(step_ids), host.train_step(step_ids)
        assert l1 == l2
        assert np.array_equal(dev.get_grads(), host.get_grads())
        if i == 0:
            Hs = pi.cache_samples(spec, 0, step_ids.tolist(), "cpu").float().numpy()
            lab = labels_np[step_ids]
            ref_loss, ref_g, _ = (po.loss_and_grads_cls(P, Hs, lab) if spec.head == "cls"
                                  else po.loss_and_grads_lm(P, Hs, lab, W_lm))
            assert abs(l2 - ref_loss) <= (1e-4 if tight else 2e-2) * abs(ref_loss)
            assert rel_l2(host.get_grads(), po.flatten(ref_g)) < (1e-4 if tight else 1e-2)
        dev.adam_step(hp); host.adam_step(hp)
    assert np.array_equal(dev.get_params(), host.get_params())


@pytest.mark.parametrize("spec", [TC, TINY], ids=lambda s: s.name)
def test_host_cache_epoch_and_async_steps(spec):
    import paper_2408_10746_b200 as pac
    dev, host, _ = make_pair(spec)
    hp = pac.AdamW()
    B = spec.B
    n_steps = 2 * (spec.N // B)                       # many more steps than staging slots
    perm = np.concatenate([pi.epoch_permutation(spec.N, 2, epoch=e) for e in range(2)])[:n_steps * B]
    la = dev.train_epoch(perm, B, hp)
    lb = host.train_epoch(perm, B, hp)
    assert np.array_equal(la, lb)
    assert np.array_equal(dev.get_params(), host.get_params())
    losses = torch.zeros(n_steps, dtype=torch.float32).pin_memory()
    for i in range(n_steps):
        host.train_step_async(perm[i * B:(i + 1) * B], hp, losses.data_ptr() + 4 * i)
    host.sync()
    lc = dev.train_epoch(perm, B, hp)
    assert np.array_equal(losses.numpy(), lc)
    assert np.array_equal(dev.get_params(), host.get_params())


def test_host_cache_pageable_memory_and_errors():
    import paper_2408_10746_b200 as pac
    spec = RAGGED
    dev, host, _ = make_pair(spec, pinned=False)
    hp = pac.AdamW()
    perm = pi.epoch_permutation(spec.N, 2)[:4 * spec.B]
    assert np.array_equal(dev.train_epoch(perm, spec.B, hp), host.train_epoch(perm, spec.B, hp))
    assert np.array_equal(dev.get_params(), host.get_params())
    before = host.get_params()
    with pytest.raises(pac.PacError) as e:
        host.train_step([0, spec.N])
    assert e.value.status_name == "PAC_ERR_SAMPLE_ID_RANGE"
    with pytest.raises(pac.PacError) as e:
        host.train_epoch_dev(torch.zeros(spec.B, dtype=torch.int32, device="cuda"), spec.B, hp, None)
    assert e.value.status_name == "PAC_ERR_UNSUPPORTED"
    host.sync()
    assert np.array_equal(host.get_params(), before)
