"""Transformer-body adapters (paper Section IV-A: the side network as a lightweight version of the
backbone transformer; Section VI-A: all widths 1/rho of the backbone's) on the plain fp32 CUDA
kernels against the oracle: loss, every gradient block, evaluation, and a 10-step AdamW trajectory."""
import numpy as np
import pytest
import torch

import pac_inputs as pi
from oracle import pac_oracle as po
from oracle import tbody_oracle as tb
from tests.common import rel_l2

pytestmark = pytest.mark.gpu

SPECS = [
    (pi.CacheSpec("tb_f32", N=16, L=3, S=12, d=40, dtype="f32", r=16, n_out=3, B=4), 4, 32),
    (pi.CacheSpec("tb_ragged_bf16", N=12, L=2, S=19, d=72, dtype="bf16", r=12, n_out=2, B=3), 3, 20),   # odd sizes, bf16 cache
    (pi.CacheSpec("tb_one_token", N=8, L=2, S=1, d=32, dtype="f32", r=8, n_out=4, B=5), 1, 8),
]


def random_flat(spec, f, seed):
    rng = np.random.default_rng(seed)
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    P = po.unflatten(pi.random_params(spec, seed), L, d, r, C)
    T = tb.BodyParams(g1=1 + rng.normal(0, 0.1, (L, r)), b1=rng.normal(0, 0.1, (L, r)),
                      Wq=rng.normal(0, r ** -0.5, (L, r, r)), Wk=rng.normal(0, r ** -0.5, (L, r, r)),
                      Wv=rng.normal(0, r ** -0.5, (L, r, r)), Wo=rng.normal(0, r ** -0.5, (L, r, r)),
                      g2=1 + rng.normal(0, 0.1, (L, r)), b2=rng.normal(0, 0.1, (L, r)),
                      W1=rng.normal(0, r ** -0.5, (L, r, f)), c1=rng.normal(0, 0.1, (L, f)),
                      W2=rng.normal(0, f ** -0.5, (L, f, r)), c2=rng.normal(0, 0.1, (L, r)))
    return tb.flatten(P, T).astype(np.float32)


def make_ctx(spec, heads, f):
    import paper_2408_10746_b200 as pac
    cache = pi.cache_full(spec, 0, "cuda")
    labels = pi.labels(spec, 0, "cuda")
    ctx = pac.PacContext(0)
    ctx.cache_register(cache, labels)
    ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B, body=1, n_heads=heads, ffn_width=f)
    return ctx


def block_names(spec, f):
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    out = [("W_down", L * d * r), ("lam", L), ("W_up", r * d), ("W_head", d * C), ("b_head", C)]
    for l in range(L):
        out += [(f"{n}[{l}]", int(np.prod(s))) for n, s in tb.body_shapes(r, f)]
    return out


@pytest.mark.parametrize("spec,heads,f", SPECS, ids=[s[0].name for s in SPECS])
def test_loss_gradients_and_eval_match_oracle(spec, heads, f):
    ctx = make_ctx(spec, heads, f)
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    assert ctx.param_count() == pi.param_count(spec) + L * tb.body_floats_per_layer(r, f)
    # seeded initial state: LayerNorm gains 1, biases 0, W_up 0, lambda 0.5
    P0, T0 = tb.unflatten(ctx.get_params(), L, d, r, C, f)
    assert (T0.g1 == 1).all() and (T0.g2 == 1).all() and not T0.b1.any() and not T0.c1.any() and not T0.c2.any()
    assert not P0.W_up.any() and (P0.lam == 0.5).all() and abs(T0.Wq.std() * r ** 0.5 - 1) < 0.2 and abs(T0.W2.std() * f ** 0.5 - 1) < 0.2
    flat = random_flat(spec, f, 3)
    ctx.set_params(flat)
    ids = [spec.N - 1, 0, 5, 5, 2][:spec.B]
    Hc = pi.cache_samples(spec, 0, ids, "cpu").float().numpy()
    lab = pi.labels(spec, 0, "cpu").numpy().astype(np.int64)[ids]
    P, T = tb.unflatten(flat, L, d, r, C, f)
    out = torch.zeros((len(ids), C), dtype=torch.float32, device="cuda")
    ctx.eval_logits(ids, out)
    ctx.sync()
    assert rel_l2(out.cpu().numpy(), tb.eval_logits(P, T, Hc, heads)) < 1e-4
    loss = ctx.train_step(ids)
    g = ctx.get_grads()
    ref_loss, (rg, rG), _ = tb.loss_and_grads_cls(P, T, Hc, lab, heads)
    ref = tb.flatten(rg, rG)
    assert abs(loss - ref_loss) <= 1e-4 * abs(ref_loss)
    o = 0
    for name, size in block_names(spec, f):
        nrm = np.linalg.norm(ref[o:o + size])
        if nrm == 0:        # with one token the softmax is constant: Wq and Wk receive exactly no gradient
            assert spec.S == 1 and name[:2] in ("Wq", "Wk") and np.abs(g[o:o + size]).max() < 1e-7, name
        else:
            assert rel_l2(g[o:o + size], ref[o:o + size]) < 1e-4, (name, rel_l2(g[o:o + size], ref[o:o + size]))
        o += size
    assert o == g.size
    ctx.close()


def test_ten_adamw_steps_match_oracle():
    import paper_2408_10746_b200 as pac
    spec, heads, f = SPECS[0]
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    ctx = make_ctx(spec, heads, f)
    flat = random_flat(spec, f, 4)
    ctx.set_params(flat)
    hp = po.AdamW()
    perm = np.concatenate([pi.epoch_permutation(spec.N, 2, epoch=e) for e in range(3)])[:10 * spec.B]
    losses = ctx.train_epoch(perm, spec.B, pac.AdamW(hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay))
    cache = pi.cache_full(spec, 0, "cpu").float().numpy()
    labels = pi.labels(spec, 0, "cpu").numpy().astype(np.int64)
    theta = flat.copy()
    m, v = np.zeros_like(theta), np.zeros_like(theta)
    ref_losses = []
    for s in range(10):
        ids = perm[s * spec.B:(s + 1) * spec.B]
        P, T = tb.unflatten(theta, L, d, r, C, f)
        loss, (rg, rG), _ = tb.loss_and_grads_cls(P, T, po.gather(cache, ids), labels[ids], heads)
        ref_losses.append(loss)
        theta, m, v = po.adamw_step(theta, tb.flatten(rg, rG), m, v, s + 1, hp, tb.decay_mask(P, T).astype(np.float32))
    p = ctx.get_params()
    assert np.all(np.abs(losses - np.array(ref_losses)) <= 1e-4 * np.abs(ref_losses))
    assert rel_l2(p, theta) < 1e-4
    assert rel_l2(p - flat, theta - flat) < 1e-2
    assert ctx.get_opt_state()[2] == 10
    ctx.close()


def test_transformer_body_argument_checks():
    import paper_2408_10746_b200 as pac
    spec = SPECS[0][0]
    cache = pi.cache_full(spec, 0, "cuda")
    labels = pi.labels(spec, 0, "cuda")
    for kw in (dict(n_heads=3, ffn_width=8), dict(n_heads=0, ffn_width=8), dict(n_heads=2, ffn_width=0)):
        ctx = pac.PacContext(0)
        ctx.cache_register(cache, labels)
        with pytest.raises(pac.PacError) as e:
            ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=2, body=1, **kw)
        assert e.value.status_name == "PAC_ERR_INVALID_ARG"
        ctx.close()
