"""CPU oracle for Parallel Adapters whose body is a reduced-width transformer layer.

TEST INFRASTRUCTURE ONLY (same rules as pac_oracle.py: used by tests, the smoke check and
the benchmark's CPU leg; shares no code with the CUDA path).

What it follows (PAC+, arXiv 2408.10746):

* Section IV-A, "Parallel Adapters Architecture": the side network "is developed as a
  lightweight version of the backbone transformer-based LLM": L adapters of hidden width d / rho,
  adapter i fed with  lambda_i * down(b) + (1 - lambda_i) * a  (lambda initialised to 0.5), a final
  W_up back to width d.
* Section VI-A, implementation details: "all weights and hidden state dimensions of the Parallel
  Adapters are 1/rho times the corresponding weights and hidden states of the backbone model", one
  adapter at the end of each transformer layer.

So adapter l is ONE transformer layer at width r = d / rho acting on the S tokens of a sample
(tokens of a sample now interact; samples stay independent).  Readings taken where the paper is
silent (stated again in the repository's design notes):

* pre-norm encoder layer, bidirectional self-attention (no mask), no dropout:
      x   = lambda_l u_l + (1 - lambda_l) a_{l-1},      u_l = b_l W_down^l,  a_0 = 0
      n1  = LayerNorm(x; g1, b1)                         over the r features, eps = 1e-5
      q, k, v = n1 Wq, n1 Wk, n1 Wv                      r x r each, no bias; H heads of width r / H
      P_h = softmax(q_h k_h^T / sqrt(r / H))             over the keys
      x'  = x + concat_h(P_h v_h) Wo
      n2  = LayerNorm(x'; g2, b2)
      a_l = x' + relu(n2 W1 + c1) W2 + c2                W1: r x f, W2: f x r
* y = b_L + a_L W_up and the heads / losses are those of pac_oracle.py.
* the paper initialises these layers by pruning the backbone's; without backbone weights the
  initial values are Gaussian (Section IV-C evaluates that initialisation too).

Arithmetic in the dtype of the parameters handed in (float64 for finite differences).  matmul is
used as a library primitive; nothing is blocked or fused.  The backward pass is derived by hand.

Pins (tests/test_tbody_oracle.py, no GPU): central finite differences of every parameter block in
float64; torch autograd of an independently typed forward; a pure-Python scalar evaluation of one
attention row; softmax rows summing to one; S = 1 (attention reduces to v Wo); Wo = 0, W2 = 0,
c2 = 0 (the body is the identity, so the model equals pac_oracle's identity-activation model).
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

from . import pac_oracle as po

LN_EPS = 1e-5


@dataclasses.dataclass
class BodyParams:
    """Per-layer transformer-body weights, stacked over the L adapters."""
    g1: np.ndarray   # [L][r]
    b1: np.ndarray   # [L][r]
    Wq: np.ndarray   # [L][r][r]
    Wk: np.ndarray   # [L][r][r]
    Wv: np.ndarray   # [L][r][r]
    Wo: np.ndarray   # [L][r][r]
    g2: np.ndarray   # [L][r]
    b2: np.ndarray   # [L][r]
    W1: np.ndarray   # [L][r][f]
    c1: np.ndarray   # [L][f]
    W2: np.ndarray   # [L][f][r]
    c2: np.ndarray   # [L][r]

    NAMES = ("g1", "b1", "Wq", "Wk", "Wv", "Wo", "g2", "b2", "W1", "c1", "W2", "c2")
    DECAYS = ("Wq", "Wk", "Wv", "Wo", "W1", "W2")      # weight matrices take decoupled decay


def body_shapes(r: int, f: int):
    return [("g1", (r,)), ("b1", (r,)), ("Wq", (r, r)), ("Wk", (r, r)), ("Wv", (r, r)), ("Wo", (r, r)),
            ("g2", (r,)), ("b2", (r,)), ("W1", (r, f)), ("c1", (f,)), ("W2", (f, r)), ("c2", (r,))]


def body_floats_per_layer(r: int, f: int) -> int:
    return sum(int(np.prod(s)) for _, s in body_shapes(r, f))


def unflatten(flat: np.ndarray, L: int, d: int, r: int, C: Optional[int], f: int):
    """Flat layout: the point-wise model's vector (pac_oracle.flatten) followed by, for every layer
    l = 0..L-1, that layer's g1 | b1 | Wq | Wk | Wv | Wo | g2 | b2 | W1 | c1 | W2 | c2."""
    n_base = L * d * r + L + r * d + (0 if C is None else d * C + C)
    P = po.unflatten(flat[:n_base], L, d, r, C)
    per = body_floats_per_layer(r, f)
    assert flat.size == n_base + L * per, "flat vector has the wrong length"
    stacks = {n: [] for n, _ in body_shapes(r, f)}
    o = n_base
    for _ in range(L):
        for name, shp in body_shapes(r, f):
            k = int(np.prod(shp))
            stacks[name].append(flat[o:o + k].reshape(shp).copy())
            o += k
    return P, BodyParams(**{n: np.stack(v) for n, v in stacks.items()})


def flatten(P: po.AdapterParams, T: BodyParams) -> np.ndarray:
    parts = [po.flatten(P)]
    L = T.g1.shape[0]
    for l in range(L):
        for name in BodyParams.NAMES:
            parts.append(getattr(T, name)[l].ravel())
    return np.concatenate(parts)


def decay_mask(P: po.AdapterParams, T: BodyParams) -> np.ndarray:
    parts = [po.decay_mask(P)]
    L = T.g1.shape[0]
    for l in range(L):
        for name in BodyParams.NAMES:
            x = getattr(T, name)[l]
            parts.append(np.ones(x.size) if name in BodyParams.DECAYS else np.zeros(x.size))
    return np.concatenate(parts)


# ---------------------------------------------------------------------------
# One transformer layer at width r on x [B][S][r]
# ---------------------------------------------------------------------------
def _layer_norm(x, g, b):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + x.dtype.type(LN_EPS))
    xhat = (x - mu) * rstd
    return xhat * g + b, xhat, rstd


def _layer_norm_backward(dn, xhat, rstd, g):
    """d/dx of LayerNorm given d/dn; also returns dg, db."""
    dxhat = dn * g
    dx = (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True)) * rstd
    red = tuple(range(dn.ndim - 1))
    return dx, (dn * xhat).sum(axis=red), dn.sum(axis=red)


def _split_heads(x, H):
    B, S, r = x.shape
    return x.reshape(B, S, H, r // H).transpose(0, 2, 1, 3)          # [B][H][S][dh]


def _merge_heads(x):
    B, H, S, dh = x.shape
    return x.transpose(0, 2, 1, 3).reshape(B, S, H * dh)


def body_forward(T: BodyParams, l: int, x: np.ndarray, H: int):
    """a = TransformerLayer_l(x); returns a and what the backward pass needs."""
    dt = x.dtype
    r = x.shape[-1]
    n1, xhat1, rstd1 = _layer_norm(x, T.g1[l], T.b1[l])
    q, k, v = n1 @ T.Wq[l], n1 @ T.Wk[l], n1 @ T.Wv[l]
    qh, kh, vh = _split_heads(q, H), _split_heads(k, H), _split_heads(v, H)
    scale = dt.type(1.0 / np.sqrt(r // H))
    s = (qh @ kh.transpose(0, 1, 3, 2)) * scale                       # [B][H][S][S]
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    P = e / e.sum(axis=-1, keepdims=True)                             # softmax over the keys
    o = _merge_heads(P @ vh)                                          # [B][S][r]
    x1 = x + o @ T.Wo[l]
    n2, xhat2, rstd2 = _layer_norm(x1, T.g2[l], T.b2[l])
    pre = n2 @ T.W1[l] + T.c1[l]
    hid = np.where(pre > 0, pre, np.zeros_like(pre))
    a = x1 + hid @ T.W2[l] + T.c2[l]
    saved = dict(xhat1=xhat1, rstd1=rstd1, n1=n1, qh=qh, kh=kh, vh=vh, P=P, o=o, xhat2=xhat2, rstd2=rstd2, n2=n2,
                 pre=pre, hid=hid, scale=scale)
    return a, saved


def body_backward(T: BodyParams, l: int, da: np.ndarray, sv: dict, H: int, G: BodyParams):
    """Given dLoss/da, fills layer l of the gradient stacks G and returns dLoss/dx."""
    B, S, r = da.shape
    M = B * S
    # a = x1 + hid W2 + c2
    G.c2[l] = da.reshape(M, r).sum(axis=0)
    G.W2[l] = sv["hid"].reshape(M, -1).T @ da.reshape(M, r)
    dhid = da @ T.W2[l].T
    dpre = dhid * (sv["pre"] > 0)
    G.c1[l] = dpre.reshape(M, -1).sum(axis=0)
    G.W1[l] = sv["n2"].reshape(M, r).T @ dpre.reshape(M, -1)
    dn2 = dpre @ T.W1[l].T
    dx1_ln, G.g2[l], G.b2[l] = _layer_norm_backward(dn2, sv["xhat2"], sv["rstd2"], T.g2[l])
    dx1 = da + dx1_ln
    # x1 = x + o Wo
    G.Wo[l] = sv["o"].reshape(M, r).T @ dx1.reshape(M, r)
    do = _split_heads(dx1 @ T.Wo[l].T, H)                             # [B][H][S][dh]
    P, qh, kh, vh = sv["P"], sv["qh"], sv["kh"], sv["vh"]
    dP = do @ vh.transpose(0, 1, 3, 2)                                # [B][H][S][S]
    dvh = P.transpose(0, 1, 3, 2) @ do
    ds = P * (dP - (dP * P).sum(axis=-1, keepdims=True))              # softmax backward, row-wise
    dqh = (ds @ kh) * sv["scale"]
    dkh = (ds.transpose(0, 1, 3, 2) @ qh) * sv["scale"]
    dq, dk, dv = _merge_heads(dqh), _merge_heads(dkh), _merge_heads(dvh)
    n1 = sv["n1"].reshape(M, r)
    G.Wq[l] = n1.T @ dq.reshape(M, r)
    G.Wk[l] = n1.T @ dk.reshape(M, r)
    G.Wv[l] = n1.T @ dv.reshape(M, r)
    dn1 = dq @ T.Wq[l].T + dk @ T.Wk[l].T + dv @ T.Wv[l].T
    dx_ln, G.g1[l], G.b1[l] = _layer_norm_backward(dn1, sv["xhat1"], sv["rstd1"], T.g1[l])
    return dx1 + dx_ln


# ---------------------------------------------------------------------------
# The side network with transformer bodies
# ---------------------------------------------------------------------------
def adapter_forward(P: po.AdapterParams, T: BodyParams, Hc: np.ndarray, heads: int):
    """Hc: [B][L][S][d] gathered cache.  Returns y [B][S][d] and the per-layer saved state."""
    dt = P.dtype
    Hc = Hc.astype(dt, copy=False)
    B, L, S, d = Hc.shape
    r = P.W_down.shape[2]
    a_prev = np.zeros((B, S, r), dt)                                  # a_0 = 0
    saved = []
    for l in range(L):
        lam = P.lam[l]
        u = Hc[:, l] @ P.W_down[l]                                    # down-projection of b_l
        x = lam * u + (dt.type(1) - lam) * a_prev                     # lambda-merge: the input of adapter l
        a, sv = body_forward(T, l, x, heads)
        sv["u"], sv["a_prev"] = u, a_prev
        saved.append(sv)
        a_prev = a
    y = Hc[:, L - 1] + a_prev @ P.W_up
    return y, a_prev, saved


def _zeros_like_body(T: BodyParams) -> BodyParams:
    return BodyParams(**{n: np.zeros_like(getattr(T, n)) for n in BodyParams.NAMES})


def _backward(P, T, Hc, a_L, saved, dy, heads):
    dt = P.dtype
    B, L, S, d = Hc.shape
    g = po.AdapterParams(np.zeros_like(P.W_down), np.zeros_like(P.lam), np.zeros_like(P.W_up))
    G = _zeros_like_body(T)
    g.W_up = a_L.reshape(B * S, -1).T @ dy.reshape(B * S, d)
    da = dy @ P.W_up.T
    for l in range(L - 1, -1, -1):
        sv = saved[l]
        dx = body_backward(T, l, da, sv, heads, G)
        lam = P.lam[l]
        g.lam[l] = np.sum(dx * (sv["u"] - sv["a_prev"]), dtype=dt)    # d x / d lambda = u - a_prev
        du = lam * dx
        g.W_down[l] = Hc[:, l].reshape(B * S, d).T @ du.reshape(B * S, -1)
        da = (dt.type(1) - lam) * dx
    return g, G


def loss_and_grads_cls(P: po.AdapterParams, T: BodyParams, Hc: np.ndarray, labels, heads: int):
    """Mean-pool classifier head: returns (loss, (g, G), logits)."""
    dt = P.dtype
    Hc = Hc.astype(dt, copy=False)
    B, L, S, d = Hc.shape
    y, a_L, saved = adapter_forward(P, T, Hc, heads)
    pooled, logits = po.cls_head(P, y)
    loss = po.cross_entropy_mean(logits, labels)
    dlogits = po._softmax_minus_onehot(logits, labels)
    dpooled = dlogits @ P.W_head.T
    dy = np.ascontiguousarray(np.broadcast_to((dpooled / dt.type(S))[:, None, :], (B, S, d)))
    g, G = _backward(P, T, Hc, a_L, saved, dy, heads)
    g.W_head = pooled.T @ dlogits
    g.b_head = dlogits.sum(axis=0)
    return loss, (g, G), logits


def eval_logits(P: po.AdapterParams, T: BodyParams, Hc: np.ndarray, heads: int):
    y, _, _ = adapter_forward(P, T, Hc.astype(P.dtype, copy=False), heads)
    return po.cls_head(P, y)[1]
