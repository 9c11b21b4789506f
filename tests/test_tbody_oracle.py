"""Pins of the transformer-body oracle (no GPU): finite differences of every parameter block,
torch autograd of a separately typed forward, a scalar evaluation of one attention row, softmax
rows, the one-token case, and the identity-body case that must reproduce the point-wise oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import pac_oracle as po
from oracle import tbody_oracle as tb

B, L, S, d, r, C, H, F = 2, 2, 5, 7, 4, 3, 2, 6


def make(seed=0, dtype=np.float64, S_=S):
    rng = np.random.default_rng(seed)
    P = po.AdapterParams(W_down=rng.normal(0, 0.5, (L, d, r)), lam=rng.uniform(0.3, 0.8, L), W_up=rng.normal(0, 0.4, (r, d)),
                         W_head=rng.normal(0, 0.5, (d, C)), b_head=rng.normal(0, 0.1, C)).astype(dtype)
    T = tb.BodyParams(g1=1 + rng.normal(0, 0.1, (L, r)), b1=rng.normal(0, 0.1, (L, r)),
                      Wq=rng.normal(0, 0.5, (L, r, r)), Wk=rng.normal(0, 0.5, (L, r, r)), Wv=rng.normal(0, 0.5, (L, r, r)),
                      Wo=rng.normal(0, 0.5, (L, r, r)), g2=1 + rng.normal(0, 0.1, (L, r)), b2=rng.normal(0, 0.1, (L, r)),
                      W1=rng.normal(0, 0.5, (L, r, F)), c1=rng.normal(0, 0.3, (L, F)), W2=rng.normal(0, 0.5, (L, F, r)),
                      c2=rng.normal(0, 0.1, (L, r)))
    T = tb.BodyParams(**{n: getattr(T, n).astype(dtype) for n in tb.BodyParams.NAMES})
    Hc = rng.normal(0, 1, (B, L, S_, d)).astype(dtype)
    labels = rng.integers(0, C, B)
    return P, T, Hc, labels


def test_flat_layout_round_trip_and_decay_mask():
    P, T, _, _ = make()
    flat = tb.flatten(P, T)
    per = tb.body_floats_per_layer(r, F)
    assert per == 2 * r + 4 * r * r + 2 * r + r * F + F + F * r + r
    assert flat.size == po.flatten(P).size + L * per
    P2, T2 = tb.unflatten(flat, L, d, r, C, F)
    assert np.array_equal(tb.flatten(P2, T2), flat)
    # layer-major body block: the first body entry is g1 of layer 0, and layer 1 starts `per` later
    nb = po.flatten(P).size
    assert np.array_equal(flat[nb:nb + r], T.g1[0]) and np.array_equal(flat[nb + per:nb + per + r], T.g1[1])
    mask = tb.decay_mask(P, T)
    assert mask[:nb].tolist() == po.decay_mask(P).tolist()
    assert mask[nb:nb + 2 * r].sum() == 0 and mask[nb + 2 * r:nb + 2 * r + 4 * r * r].all()


def test_finite_differences_of_every_block():
    P, T, Hc, labels = make(1)
    loss, (g, G), _ = tb.loss_and_grads_cls(P, T, Hc, labels, H)
    flat = tb.flatten(P, T)
    gflat = tb.flatten(g, G)
    rng = np.random.default_rng(5)
    eps = 1e-6
    # every block is probed: a few random entries of each named array
    o = 0
    blocks = [(n, getattr(P, n).size) for n in ("W_down", "lam", "W_up", "W_head", "b_head")]
    for l in range(L):
        blocks += [(f"{n}[{l}]", getattr(T, n)[l].size) for n in tb.BodyParams.NAMES]
    for name, size in blocks:
        for i in rng.choice(size, size=min(4, size), replace=False):
            fp, fm = flat.copy(), flat.copy()
            fp[o + i] += eps
            fm[o + i] -= eps
            lp = tb.loss_and_grads_cls(*tb.unflatten(fp, L, d, r, C, F), Hc, labels, H)[0]
            lm = tb.loss_and_grads_cls(*tb.unflatten(fm, L, d, r, C, F), Hc, labels, H)[0]
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - gflat[o + i]) <= 1e-6 * max(1.0, abs(fd)), (name, i, fd, gflat[o + i])
        o += size
    assert o == flat.size


def torch_forward(P, T, Hc, labels):
    """The same model typed independently with torch ops (layer_norm, softmax, relu from the library)."""
    t = lambda x: torch.tensor(x, dtype=torch.float64, requires_grad=True)
    tp = {n: t(getattr(P, n)) for n in ("W_down", "lam", "W_up", "W_head", "b_head")}
    tt = {n: t(getattr(T, n)) for n in tb.BodyParams.NAMES}
    Ht = torch.tensor(Hc, dtype=torch.float64)
    a = torch.zeros((B, Hc.shape[2], r), dtype=torch.float64)
    for l in range(L):
        x = tp["lam"][l] * (Ht[:, l] @ tp["W_down"][l]) + (1 - tp["lam"][l]) * a
        n1 = torch.nn.functional.layer_norm(x, (r,), tt["g1"][l], tt["b1"][l], eps=1e-5)
        q, k, v = n1 @ tt["Wq"][l], n1 @ tt["Wk"][l], n1 @ tt["Wv"][l]
        outs = []
        dh = r // H
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            att = torch.softmax(q[..., sl] @ k[..., sl].transpose(1, 2) / math.sqrt(dh), dim=-1)
            outs.append(att @ v[..., sl])
        x1 = x + torch.cat(outs, dim=-1) @ tt["Wo"][l]
        n2 = torch.nn.functional.layer_norm(x1, (r,), tt["g2"][l], tt["b2"][l], eps=1e-5)
        a = x1 + torch.relu(n2 @ tt["W1"][l] + tt["c1"][l]) @ tt["W2"][l] + tt["c2"][l]
    y = Ht[:, L - 1] + a @ tp["W_up"]
    logits = y.mean(dim=1) @ tp["W_head"] + tp["b_head"]
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(labels))
    return loss, logits, tp, tt


def test_against_torch_autograd():
    P, T, Hc, labels = make(2)
    loss, (g, G), logits = tb.loss_and_grads_cls(P, T, Hc, labels, H)
    tl, tlog, tp, tt = torch_forward(P, T, Hc, labels)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12 and np.allclose(logits, tlog.detach().numpy(), atol=1e-12)
    for n in ("W_down", "lam", "W_up", "W_head", "b_head"):
        assert np.allclose(getattr(g, n), tp[n].grad.numpy(), rtol=1e-9, atol=1e-12), n
    for n in tb.BodyParams.NAMES:
        assert np.allclose(getattr(G, n), tt[n].grad.numpy(), rtol=1e-9, atol=1e-12), n


def test_one_attention_row_by_scalar_loops_and_softmax_rows():
    P, T, Hc, _ = make(3)
    x = 0.7 * (Hc[:, 0] @ P.W_down[0])
    a, sv = tb.body_forward(T, 0, x, H)
    assert np.allclose(sv["P"].sum(axis=-1), 1.0, atol=1e-14) and (sv["P"] >= 0).all()
    # sample 1, token 2: layer norm, projections, both heads, output projection, with python floats only
    b_, s_ = 1, 2
    dh = r // H

    def ln(vec, g, bb):
        mu = sum(vec) / len(vec)
        var = sum((v - mu) ** 2 for v in vec) / len(vec)
        return [(v - mu) / math.sqrt(var + 1e-5) * g[i] + bb[i] for i, v in enumerate(vec)]

    n1 = [ln(list(x[b_, t]), list(T.g1[0]), list(T.b1[0])) for t in range(S)]
    proj = lambda vec, W: [sum(vec[i] * W[i][j] for i in range(r)) for j in range(r)]
    q = proj(n1[s_], T.Wq[0])
    ks = [proj(n1[t], T.Wk[0]) for t in range(S)]
    vs = [proj(n1[t], T.Wv[0]) for t in range(S)]
    o = []
    for h in range(H):
        sc = [sum(q[h * dh + i] * ks[t][h * dh + i] for i in range(dh)) / math.sqrt(dh) for t in range(S)]
        m = max(sc)
        e = [math.exp(v - m) for v in sc]
        p = [v / sum(e) for v in e]
        o += [sum(p[t] * vs[t][h * dh + i] for t in range(S)) for i in range(dh)]
    x1 = [x[b_, s_, j] + sum(o[i] * T.Wo[0][i][j] for i in range(r)) for j in range(r)]
    n2 = ln(x1, list(T.g2[0]), list(T.b2[0]))
    hid = [max(0.0, sum(n2[i] * T.W1[0][i][j] for i in range(r)) + T.c1[0][j]) for j in range(F)]
    want = [x1[j] + sum(hid[i] * T.W2[0][i][j] for i in range(F)) + T.c2[0][j] for j in range(r)]
    assert np.allclose(a[b_, s_], want, rtol=1e-12, atol=1e-12)


def test_single_token_attention_reduces_to_value_projection():
    P, T, Hc, _ = make(4, S_=1)
    x = Hc[:, 0] @ P.W_down[0]
    a, sv = tb.body_forward(T, 0, x, H)
    assert np.array_equal(sv["P"], np.ones_like(sv["P"]))          # softmax over one key
    n1, _, _ = tb._layer_norm(x, T.g1[0], T.b1[0])
    x1 = x + (n1 @ T.Wv[0]) @ T.Wo[0]
    n2, _, _ = tb._layer_norm(x1, T.g2[0], T.b2[0])
    assert np.allclose(a, x1 + np.maximum(n2 @ T.W1[0] + T.c1[0], 0) @ T.W2[0] + T.c2[0], atol=1e-13)


def test_identity_body_reproduces_the_pointwise_oracle():
    """Wo = 0, W2 = 0, c2 = 0 make every body the identity map, so the model is the point-wise
    adapter with the identity activation: loss, logits and the shared gradient blocks agree exactly."""
    P, T, Hc, labels = make(6)
    for n in ("Wo", "W2", "c2"):
        getattr(T, n)[...] = 0
    loss, (g, G), logits = tb.loss_and_grads_cls(P, T, Hc, labels, H)
    ref_loss, ref_g, ref_logits = po.loss_and_grads_cls(P, Hc, labels, po.ACT_IDENTITY)
    assert np.allclose(logits, ref_logits, rtol=1e-13, atol=1e-13) and abs(loss - ref_loss) < 1e-13
    for n in ("W_down", "lam", "W_up", "W_head", "b_head"):
        assert np.allclose(getattr(g, n), getattr(ref_g, n), rtol=1e-11, atol=1e-13), n
    assert np.array_equal(tb.eval_logits(P, T, Hc, H), logits)
