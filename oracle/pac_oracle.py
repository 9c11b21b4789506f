"""CPU oracle for training Parallel Adapters over an activation cache.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
path computes; it exists so that the CUDA library can be checked against it.
Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may use
it.  It shares no code with the CUDA path and imports nothing from it.

What it follows (PAC+, arXiv 2408.10746):

* Section IV-A, "Parallel Adapters Architecture": a backbone with L layers emits
  b_1..b_L (n tokens x d); the side network has L adapters with states a_1..a_L of
  width d/rho.  A learned linear map W_down^i brings b to the adapter width, the
  result is mixed with the running adapter state by a learnable scalar
  lambda_i (initialised to 0.5) as  lambda_i * down(b) + (1 - lambda_i) * a,  the
  mix feeds adapter i, and a final linear map W_up returns to width d "to match
  the original language-model head".  No gradient enters the backbone.
* Section IV-B, "Activation Cache": the b_l of a sample never change because the
  backbone is frozen, so they are stored once and later epochs train the side
  network from the stored copies alone.
* Section V-B: phase 2 trains only the adapter parameters, one minibatch at a
  time, from the cached activations.

Readings taken where the paper leaves a choice open (all stated again in the
design notes of the repository):

* adapter l (1..L) consumes b_l and a_{l-1} and produces a_l;  a_0 = 0;
* the adapter body is the minimal member of the "linear down/up projection"
  family the section names: a point-wise activation phi (ReLU, phi'(0)=0, or the
  identity), so  u_l = b_l W_down^l,  z_l = lambda_l u_l + (1-lambda_l) a_{l-1},
  a_l = phi(z_l);
* the side network's output is added to the backbone's last hidden state (the
  side-tuning sum the section builds on):  y = b_L + a_L W_up;
* heads: a trainable mean-pool linear classifier  logits = mean_s(y) W_head +
  b_head  with mean softmax cross-entropy over the batch, or a frozen LM head
  logits = y W_lm^T with mean cross-entropy over all B*S positions;
* no biases on W_down / W_up; lambda is a raw scalar;
* the optimizer is AdamW with decoupled decay on the weight matrices only.

Arithmetic is carried out in the dtype of the parameters handed in (float32 for
parity runs, float64 for finite-difference checks).  Matrix products use numpy's
matmul as a library primitive; nothing is blocked, fused or reordered beyond the
equations above.

Pins (tests/test_oracle_*.py, no GPU): central finite differences of every
gradient in float64; an independent scalar per-row recursion; closed forms for a
one-layer linear adapter; W_up = 0 reproduces the head-only model exactly and
zeroes dW_down and dlambda; zero head gives loss ln C; lambda = 1 and lambda = 0
special cases; batch-mean and duplicate-id structure; AdamW against closed forms
and torch.optim.AdamW; frozen inputs left untouched; cache byte accounting
against the storage-cost paragraph of Section V-B.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

ACT_RELU = 0
ACT_IDENTITY = 1


@dataclasses.dataclass
class AdapterParams:
    """Trainable state of the side network (+ classifier head when present)."""
    W_down: np.ndarray                 # [L][d][r]
    lam: np.ndarray                    # [L]
    W_up: np.ndarray                   # [r][d]
    W_head: Optional[np.ndarray] = None  # [d][C]   (classifier head only)
    b_head: Optional[np.ndarray] = None  # [C]

    @property
    def dtype(self):
        return self.W_down.dtype

    def copy(self) -> "AdapterParams":
        return AdapterParams(*[None if x is None else x.copy() for x in dataclasses.astuple(self)])

    def astype(self, dt) -> "AdapterParams":
        return AdapterParams(*[None if x is None else x.astype(dt) for x in dataclasses.astuple(self)])


def param_shapes(L: int, d: int, r: int, C: Optional[int]):
    shapes = [("W_down", (L, d, r)), ("lam", (L,)), ("W_up", (r, d))]
    if C is not None:
        shapes += [("W_head", (d, C)), ("b_head", (C,))]
    return shapes


def unflatten(flat: np.ndarray, L: int, d: int, r: int, C: Optional[int]) -> AdapterParams:
    """Flat layout: W_down[L][d][r] | lambda[L] | W_up[r][d] | W_head[d][C] | b_head[C]."""
    out, o = {}, 0
    for name, shp in param_shapes(L, d, r, C):
        k = int(np.prod(shp))
        out[name] = flat[o:o + k].reshape(shp).copy()
        o += k
    assert o == flat.size, "flat vector has the wrong length"
    return AdapterParams(**out)


def flatten(P: AdapterParams) -> np.ndarray:
    parts = [P.W_down.ravel(), P.lam.ravel(), P.W_up.ravel()]
    if P.W_head is not None:
        parts += [P.W_head.ravel(), P.b_head.ravel()]
    return np.concatenate(parts)


def decay_mask(P: AdapterParams) -> np.ndarray:
    """1 where decoupled weight decay applies (weight matrices), 0 for lambda and b_head."""
    parts = [np.ones(P.W_down.size), np.zeros(P.lam.size), np.ones(P.W_up.size)]
    if P.W_head is not None:
        parts += [np.ones(P.W_head.size), np.zeros(P.b_head.size)]
    return np.concatenate(parts)


# ---------------------------------------------------------------------------
# Section IV-B: the cache and its gather
# ---------------------------------------------------------------------------
def gather(cache: np.ndarray, sample_ids) -> np.ndarray:
    """H[b][l] = cache[ids[b]][l]  for a cache laid out [N][L][S][d].  Pure
    indexing: the result holds copies of the stored values, bit for bit."""
    ids = np.asarray(sample_ids, dtype=np.int64)
    if ids.ndim != 1:
        raise ValueError("sample_ids must be one-dimensional")
    if ids.size and (ids.min() < 0 or ids.max() >= cache.shape[0]):
        raise IndexError("sample id out of range")
    return cache[ids]


def cache_bytes_per_sequence(s: int, h: int, l: int, elem_bytes: int) -> int:
    """Storage cost  s x h x l  elements per sequence (Section V-B, storage cost analysis)."""
    return s * h * l * elem_bytes


# ---------------------------------------------------------------------------
# Section IV-A: forward of the side network
# ---------------------------------------------------------------------------
def _phi(z, act):
    if act == ACT_RELU:
        return np.where(z > 0, z, np.zeros_like(z))
    if act == ACT_IDENTITY:
        return z
    raise ValueError("unknown activation")


def _dphi(z, act):
    if act == ACT_RELU:
        return (z > 0).astype(z.dtype)
    if act == ACT_IDENTITY:
        return np.ones_like(z)
    raise ValueError("unknown activation")


def adapter_forward(P: AdapterParams, H: np.ndarray, act: int = ACT_RELU):
    """H: [B][L][S][d] gathered cache (b_1..b_L per sample).  Returns u, z, a as
    [L][B][S][r] stacks and y [B][S][d]."""
    dt = P.dtype
    H = H.astype(dt, copy=False)
    B, L, S, d = H.shape
    r = P.W_down.shape[2]
    u = np.zeros((L, B, S, r), dt)
    z = np.zeros((L, B, S, r), dt)
    a = np.zeros((L, B, S, r), dt)
    a_prev = np.zeros((B, S, r), dt)                       # a_0 = 0
    for l in range(L):
        lam = P.lam[l]
        u[l] = H[:, l] @ P.W_down[l]                       # down-projection of b_l
        z[l] = lam * u[l] + (dt.type(1) - lam) * a_prev    # lambda-merge with the running state
        a[l] = _phi(z[l], act)                             # adapter body
        a_prev = a[l]
    y = H[:, L - 1] + a_prev @ P.W_up                      # up-projection, summed with b_L
    return u, z, a, y


def _logsumexp(x):
    m = x.max(axis=-1, keepdims=True)
    return (m + np.log(np.exp(x - m).sum(axis=-1, keepdims=True)))[..., 0]


def cls_head(P: AdapterParams, y: np.ndarray):
    pooled = y.mean(axis=1)                                # [B][d], mean over tokens
    return pooled, pooled @ P.W_head + P.b_head            # [B][C]


def cross_entropy_mean(logits: np.ndarray, targets: np.ndarray):
    """Mean over all leading positions of  logsumexp(logits) - logits[target]."""
    flat = logits.reshape(-1, logits.shape[-1])
    t = np.asarray(targets, dtype=np.int64).reshape(-1)
    per = _logsumexp(flat) - flat[np.arange(flat.shape[0]), t]
    return per.mean(dtype=logits.dtype)


def lm_head_logits(W_lm: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Frozen head: logits[b][s][v] = <y[b][s], W_lm[v]>."""
    return y @ W_lm.astype(y.dtype, copy=False).T


# ---------------------------------------------------------------------------
# Loss and gradients (adapters only; nothing flows toward H)
# ---------------------------------------------------------------------------
def _softmax_minus_onehot(logits, targets):
    flat = logits.reshape(-1, logits.shape[-1])
    t = np.asarray(targets, dtype=np.int64).reshape(-1)
    m = flat.max(axis=-1, keepdims=True)
    e = np.exp(flat - m)
    p = e / e.sum(axis=-1, keepdims=True)
    p[np.arange(flat.shape[0]), t] -= 1
    return (p / flat.shape[0]).reshape(logits.shape)       # gradient of the MEAN loss


def _adapter_backward(P, H, u, z, a, dy, act):
    """Given dy = dLoss/dy [B][S][d], walk the side network from layer L to 1."""
    dt = P.dtype
    B, L, S, d = H.shape
    g = AdapterParams(np.zeros_like(P.W_down), np.zeros_like(P.lam), np.zeros_like(P.W_up))
    aL = a[L - 1].reshape(B * S, -1)
    g.W_up = aL.T @ dy.reshape(B * S, d)                    # dW_up = a_L^T dy
    da = dy @ P.W_up.T                                      # da_L
    for l in range(L - 1, -1, -1):
        lam = P.lam[l]
        a_prev = a[l - 1] if l > 0 else np.zeros_like(a[0])
        dz = da * _dphi(z[l], act)
        g.lam[l] = np.sum(dz * (u[l] - a_prev), dtype=dt)   # d z / d lambda = u - a_prev
        du = lam * dz
        g.W_down[l] = H[:, l].reshape(B * S, d).T @ du.reshape(B * S, -1)   # dW_down^l = b_l^T du_l
        da = (dt.type(1) - lam) * dz
    return g


def loss_and_grads_cls(P: AdapterParams, H: np.ndarray, labels, act: int = ACT_RELU):
    """Classifier head: returns (loss, grads, logits)."""
    dt = P.dtype
    H = H.astype(dt, copy=False)
    B, L, S, d = H.shape
    u, z, a, y = adapter_forward(P, H, act)
    pooled, logits = cls_head(P, y)
    loss = cross_entropy_mean(logits, labels)
    dlogits = _softmax_minus_onehot(logits, labels)         # [B][C]
    dpooled = dlogits @ P.W_head.T                          # [B][d]
    dy = np.broadcast_to((dpooled / dt.type(S))[:, None, :], (B, S, d))
    g = _adapter_backward(P, H, u, z, a, np.ascontiguousarray(dy), act)
    g.W_head = pooled.T @ dlogits
    g.b_head = dlogits.sum(axis=0)
    return loss, g, logits


def loss_and_grads_lm(P: AdapterParams, H: np.ndarray, targets, W_lm: np.ndarray, act: int = ACT_RELU):
    """Frozen LM head: returns (loss, grads, logits).  targets: [B][S] token ids."""
    dt = P.dtype
    H = H.astype(dt, copy=False)
    u, z, a, y = adapter_forward(P, H, act)
    logits = lm_head_logits(W_lm, y)
    loss = cross_entropy_mean(logits, targets)
    dlogits = _softmax_minus_onehot(logits, targets)        # [B][S][V]
    dy = dlogits @ W_lm.astype(dt, copy=False)              # [B][S][d]; W_lm itself gets no gradient
    g = _adapter_backward(P, H, u, z, a, dy, act)
    return loss, g, logits


def eval_logits(P: AdapterParams, H: np.ndarray, act: int = ACT_RELU, W_lm: Optional[np.ndarray] = None):
    _, _, _, y = adapter_forward(P, H.astype(P.dtype, copy=False), act)
    if W_lm is None:
        return cls_head(P, y)[1]
    return lm_head_logits(W_lm, y)


# ---------------------------------------------------------------------------
# AdamW (decoupled weight decay, Loshchilov & Hutter), on the flat vector
# ---------------------------------------------------------------------------
@dataclasses.dataclass
class AdamW:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01


def adamw_step(theta, g, m, v, t: int, hp: AdamW, wd_mask):
    """One update at step t = 1, 2, ...; returns new (theta, m, v).

    m <- b1 m + (1-b1) g ;  v <- b2 v + (1-b2) g^2 ;  mhat = m/(1-b1^t) ;
    vhat = v/(1-b2^t) ;  theta <- theta - lr*wd*theta - lr*mhat/(sqrt(vhat)+eps),
    the decay acting on the value before the update and eps outside the root.
    """
    dt = theta.dtype.type
    b1, b2 = dt(hp.beta1), dt(hp.beta2)
    m = b1 * m + (dt(1) - b1) * g
    v = b2 * v + (dt(1) - b2) * g * g
    mhat = m / dt(1.0 - hp.beta1 ** t)
    vhat = v / dt(1.0 - hp.beta2 ** t)
    decay = dt(hp.lr) * dt(hp.weight_decay) * wd_mask.astype(theta.dtype) * theta
    theta = theta - decay - dt(hp.lr) * mhat / (np.sqrt(vhat) + dt(hp.eps))
    return theta, m, v


class Trainer:
    """Phase-2 loop: gather -> forward -> loss -> backward -> AdamW, adapters only."""

    def __init__(self, cache: np.ndarray, labels: np.ndarray, P: AdapterParams, act: int = ACT_RELU,
                 W_lm: Optional[np.ndarray] = None, hp: Optional[AdamW] = None):
        self.cache, self.labels, self.P, self.act, self.W_lm = cache, labels, P, act, W_lm
        self.hp = hp or AdamW()
        self.m = np.zeros_like(flatten(P))
        self.v = np.zeros_like(self.m)
        self.t = 0
        self.grads: Optional[AdapterParams] = None

    def _dims(self):
        L, d, r = self.P.W_down.shape
        C = None if self.P.W_head is None else self.P.W_head.shape[1]
        return L, d, r, C

    def train_step(self, sample_ids) -> float:
        H = gather(self.cache, sample_ids)
        lab = self.labels[np.asarray(sample_ids, dtype=np.int64)]
        if self.W_lm is None:
            loss, g, _ = loss_and_grads_cls(self.P, H, lab, self.act)
        else:
            loss, g, _ = loss_and_grads_lm(self.P, H, lab, self.W_lm, self.act)
        self.grads = g
        return float(loss)

    def adam_step(self):
        self.t += 1
        theta, self.m, self.v = adamw_step(flatten(self.P), flatten(self.grads), self.m, self.v, self.t,
                                           self.hp, decay_mask(self.P))
        self.P = unflatten(theta, *self._dims())

    def eval_logits(self, sample_ids):
        return eval_logits(self.P, gather(self.cache, sample_ids), self.act, self.W_lm)
