"""Pins for the CPU oracle: each test fixes it to something other than itself
(finite differences, closed forms, an independent scalar recursion, library
routines, invariants), so that a dropped term, a wrong sign or a transposed
operand somewhere in oracle/pac_oracle.py fails at least one of them."""
import math

import numpy as np
import pytest
import torch

from oracle import pac_oracle as po


def rand_params(rng, L, d, r, C, dt=np.float64, up=0.3):
    return po.AdapterParams(
        W_down=(rng.standard_normal((L, d, r)) / math.sqrt(d)).astype(dt),
        lam=(0.5 + 0.2 * rng.standard_normal(L)).astype(dt),
        W_up=(up * rng.standard_normal((r, d))).astype(dt),
        W_head=None if C is None else (rng.standard_normal((d, C)) / math.sqrt(d)).astype(dt),
        b_head=None if C is None else (0.1 * rng.standard_normal(C)).astype(dt),
    )


# ---------------------------------------------------------------------------
# independent scalar routine: one (sample, token) row at a time, python floats
# ---------------------------------------------------------------------------
def scalar_row_forward(P, rows, act):
    """rows: list over l of python lists (length d).  Returns (a_L, y) as lists."""
    L, d, r = P.W_down.shape
    a = [0.0] * r
    for l in range(L):
        nxt = []
        for j in range(r):
            acc = 0.0
            for k in range(d):
                acc += rows[l][k] * float(P.W_down[l, k, j])
            zz = float(P.lam[l]) * acc + (1.0 - float(P.lam[l])) * a[j]
            nxt.append(zz if (act == po.ACT_IDENTITY or zz > 0) else 0.0)
        a = nxt
    y = []
    for k in range(d):
        acc = rows[L - 1][k]
        for j in range(r):
            acc += a[j] * float(P.W_up[j, k])
        y.append(acc)
    return a, y


def scalar_cls_loss(P, H, labels, act):
    B, L, S, d = H.shape
    C = P.W_head.shape[1]
    total = 0.0
    all_logits = []
    for b in range(B):
        pooled = [0.0] * d
        for s in range(S):
            _, y = scalar_row_forward(P, [list(map(float, H[b, l, s])) for l in range(L)], act)
            for k in range(d):
                pooled[k] += y[k] / S
        logits = [float(P.b_head[c]) + sum(pooled[k] * float(P.W_head[k, c]) for k in range(d)) for c in range(C)]
        mx = max(logits)
        lse = mx + math.log(sum(math.exp(x - mx) for x in logits))
        total += lse - logits[int(labels[b])]
        all_logits.append(logits)
    return total / B, np.array(all_logits)


def scalar_lm_loss(P, H, targets, W_lm, act):
    B, L, S, d = H.shape
    V = W_lm.shape[0]
    total = 0.0
    for b in range(B):
        for s in range(S):
            _, y = scalar_row_forward(P, [list(map(float, H[b, l, s])) for l in range(L)], act)
            logits = [sum(y[k] * float(W_lm[v, k]) for k in range(d)) for v in range(V)]
            mx = max(logits)
            total += mx + math.log(sum(math.exp(x - mx) for x in logits)) - logits[int(targets[b, s])]
    return total / (B * S)


@pytest.mark.parametrize("act", [po.ACT_RELU, po.ACT_IDENTITY])
def test_forward_matches_scalar_recursion_cls(act):
    rng = np.random.default_rng(1)
    B, L, S, d, r, C = 2, 3, 3, 5, 4, 3
    P = rand_params(rng, L, d, r, C)
    H = rng.standard_normal((B, L, S, d))
    labels = rng.integers(0, C, B)
    loss, _, logits = po.loss_and_grads_cls(P, H, labels, act)
    ref_loss, ref_logits = scalar_cls_loss(P, H, labels, act)
    assert abs(loss - ref_loss) < 1e-12
    np.testing.assert_allclose(logits, ref_logits, rtol=0, atol=1e-12)


def test_forward_matches_scalar_recursion_lm():
    rng = np.random.default_rng(2)
    B, L, S, d, r, V = 2, 2, 3, 4, 3, 7
    P = rand_params(rng, L, d, r, None)
    H = rng.standard_normal((B, L, S, d))
    W_lm = rng.standard_normal((V, d))
    targets = rng.integers(0, V, (B, S))
    loss, _, _ = po.loss_and_grads_lm(P, H, targets, W_lm)
    assert abs(loss - scalar_lm_loss(P, H, targets, W_lm, po.ACT_RELU)) < 1e-12


# ---------------------------------------------------------------------------
# finite differences (float64): every gradient block, both heads, both bodies
# ---------------------------------------------------------------------------
def fd_check(loss_fn, P, g, L, d, r, C, h=1e-6, rtol=2e-6):
    theta = po.flatten(P)
    gflat = po.flatten(g)
    num = np.zeros_like(theta)
    for i in range(theta.size):
        tp, tm = theta.copy(), theta.copy()
        tp[i] += h
        tm[i] -= h
        num[i] = (loss_fn(po.unflatten(tp, L, d, r, C)) - loss_fn(po.unflatten(tm, L, d, r, C))) / (2 * h)
    # per parameter block, so a block that is wrong cannot hide behind a large one
    o = 0
    for name, shp in po.param_shapes(L, d, r, C):
        k = int(np.prod(shp))
        a, b = gflat[o:o + k], num[o:o + k]
        assert np.linalg.norm(b) > 0, f"{name}: FD gradient is identically zero, test is vacuous"
        err = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert err < rtol, f"{name}: rel err {err}"
        o += k


def _kink_free(P, H, act, margin=1e-3):
    _, z, _, _ = po.adapter_forward(P, H, act)
    return act == po.ACT_IDENTITY or np.abs(z).min() > margin


@pytest.mark.parametrize("act", [po.ACT_RELU, po.ACT_IDENTITY])
def test_gradients_finite_difference_cls(act):
    B, L, S, d, r, C = 2, 3, 3, 5, 4, 3
    for seed in range(3, 40):
        rng = np.random.default_rng(seed)
        P = rand_params(rng, L, d, r, C)
        H = rng.standard_normal((B, L, S, d)) * (1 + 0.1 * np.arange(L))[None, :, None, None]
        if _kink_free(P, H, act):
            break
    labels = rng.integers(0, C, B)
    loss, g, _ = po.loss_and_grads_cls(P, H, labels, act)
    fd_check(lambda Q: po.loss_and_grads_cls(Q, H, labels, act)[0], P, g, L, d, r, C)


@pytest.mark.parametrize("act", [po.ACT_RELU, po.ACT_IDENTITY])
def test_gradients_finite_difference_lm(act):
    B, L, S, d, r, V = 2, 3, 2, 5, 4, 6
    for seed in range(5, 40):
        rng = np.random.default_rng(seed)
        P = rand_params(rng, L, d, r, None)
        H = rng.standard_normal((B, L, S, d))
        if _kink_free(P, H, act):
            break
    W_lm = rng.standard_normal((V, d))
    targets = rng.integers(0, V, (B, S))
    loss, g, _ = po.loss_and_grads_lm(P, H, targets, W_lm, act)
    fd_check(lambda Q: po.loss_and_grads_lm(Q, H, targets, W_lm, act)[0], P, g, L, d, r, None)


def test_gradients_against_torch_autograd():
    """The hand-derived backward against reverse-mode autodiff of an independently
    typed forward (torch CPU, float64)."""
    rng = np.random.default_rng(11)
    B, L, S, d, r, C = 3, 4, 5, 6, 3, 4
    P = rand_params(rng, L, d, r, C)
    H = rng.standard_normal((B, L, S, d))
    labels = rng.integers(0, C, B)
    _, g, _ = po.loss_and_grads_cls(P, H, labels)
    t = {k: torch.tensor(getattr(P, k), requires_grad=True) for k in ["W_down", "lam", "W_up", "W_head", "b_head"]}
    Ht = torch.tensor(H)
    state = torch.zeros(B, S, r, dtype=torch.float64)
    for l in range(L):
        state = torch.relu(t["lam"][l] * (Ht[:, l] @ t["W_down"][l]) + (1 - t["lam"][l]) * state)
    y = Ht[:, L - 1] + state @ t["W_up"]
    logits = y.mean(1) @ t["W_head"] + t["b_head"]
    torch.nn.functional.cross_entropy(logits, torch.tensor(labels)).backward()
    for k in t:
        np.testing.assert_allclose(getattr(g, k), t[k].grad.numpy(), rtol=1e-10, atol=1e-13)


# ---------------------------------------------------------------------------
# special cases the paper and the algebra fix
# ---------------------------------------------------------------------------
def test_zero_up_projection_reproduces_head_only_model():
    """Section IV-C rationale (B = 0 keeps the initial model equal to the
    pretrained one): with W_up = 0 the logits are those of the head on b_L, and
    no gradient reaches W_down or lambda."""
    rng = np.random.default_rng(7)
    B, L, S, d, r, C = 4, 3, 6, 8, 4, 3
    P = rand_params(rng, L, d, r, C, dt=np.float32)
    P.W_up[:] = 0
    H = rng.standard_normal((B, L, S, d)).astype(np.float32)
    labels = rng.integers(0, C, B)
    loss, g, logits = po.loss_and_grads_cls(P, H, labels)
    head_only = H[:, L - 1].mean(axis=1) @ P.W_head + P.b_head
    assert np.array_equal(logits, head_only)            # bit for bit: adding a_L @ 0 changes nothing
    assert not g.W_down.any() and not g.lam.any()
    assert g.W_up.any() and g.W_head.any() and g.b_head.any()


@pytest.mark.parametrize("C", [2, 3, 5])
def test_zero_head_gives_log_C(C):
    rng = np.random.default_rng(8)
    B, L, S, d, r = 4, 2, 3, 6, 3
    P = rand_params(rng, L, d, r, C)
    P.W_head[:] = 0
    P.b_head[:] = 0
    H = rng.standard_normal((B, L, S, d))
    loss, _, _ = po.loss_and_grads_cls(P, H, rng.integers(0, C, B))
    assert abs(loss - math.log(C)) < 1e-14


def test_zero_lm_logits_give_log_V():
    rng = np.random.default_rng(9)
    B, L, S, d, r, V = 2, 2, 3, 4, 3, 32
    P = rand_params(rng, L, d, r, None)
    H = rng.standard_normal((B, L, S, d))
    loss, _, _ = po.loss_and_grads_lm(P, H, rng.integers(0, V, (B, S)), np.zeros((V, d)))
    assert abs(loss - math.log(V)) < 1e-14


def test_lambda_one_uses_only_last_layer():
    rng = np.random.default_rng(10)
    B, L, S, d, r, C = 3, 4, 3, 6, 3, 3
    P = rand_params(rng, L, d, r, C)
    P.lam[:] = 1.0
    H = rng.standard_normal((B, L, S, d))
    labels = rng.integers(0, C, B)
    _, _, a, _ = po.adapter_forward(P, H)
    np.testing.assert_allclose(a[L - 1], np.maximum(H[:, L - 1] @ P.W_down[L - 1], 0), atol=1e-15)
    _, g, _ = po.loss_and_grads_cls(P, H, labels)
    assert not g.W_down[:L - 1].any() and g.W_down[L - 1].any()


def test_lambda_zero_is_head_only_but_lambda_still_learns():
    rng = np.random.default_rng(12)
    B, L, S, d, r, C = 3, 3, 3, 6, 3, 3
    P = rand_params(rng, L, d, r, C)
    P.lam[:] = 0.0
    H = rng.standard_normal((B, L, S, d))
    labels = rng.integers(0, C, B)
    loss, g, logits = po.loss_and_grads_cls(P, H, labels, act=po.ACT_IDENTITY)
    np.testing.assert_allclose(logits, H[:, L - 1].mean(1) @ P.W_head + P.b_head, atol=1e-15)
    assert not g.W_down.any()
    # dz/dlambda = u - a_prev is non-zero even at lambda = 0 (last layer sees it directly)
    assert g.lam[L - 1] != 0.0


def test_single_linear_layer_closed_form():
    """L = 1, identity body, lambda = 1:  y = h (I + W_down W_up), a textbook
    low-rank linear model; logits and gradients from explicit triple loops."""
    rng = np.random.default_rng(13)
    B, S, d, r, C = 3, 2, 4, 2, 3
    P = rand_params(rng, 1, d, r, C)
    P.lam[:] = 1.0
    H = rng.standard_normal((B, 1, S, d))
    labels = rng.integers(0, C, B)
    loss, g, logits = po.loss_and_grads_cls(P, H, labels, act=po.ACT_IDENTITY)
    Wd, Wu, Wh = P.W_down[0], P.W_up, P.W_head
    hbar = H[:, 0].mean(axis=1)                                   # [B][d]
    A = np.eye(d) + Wd @ Wu
    ref_logits = hbar @ A @ Wh + P.b_head
    np.testing.assert_allclose(logits, ref_logits, atol=1e-14)
    e = np.exp(ref_logits - ref_logits.max(1, keepdims=True))
    G = e / e.sum(1, keepdims=True)
    G[np.arange(B), labels] -= 1
    G /= B
    dWd = np.zeros((d, r)); dWu = np.zeros((r, d))
    for b in range(B):
        for k in range(d):
            for j in range(r):
                for c in range(C):
                    # d logits[b,c] / d Wd[k,j] = hbar[b,k] * (Wu Wh)[j,c]
                    dWd[k, j] += G[b, c] * hbar[b, k] * sum(Wu[j, q] * Wh[q, c] for q in range(d))
                    # d logits[b,c] / d Wu[j,k] = (hbar Wd)[b,j] * Wh[k,c]
                    dWu[j, k] += G[b, c] * sum(hbar[b, q] * Wd[q, j] for q in range(d)) * Wh[k, c]
    np.testing.assert_allclose(g.W_down[0], dWd, atol=1e-14)
    np.testing.assert_allclose(g.W_up, dWu, atol=1e-14)
    np.testing.assert_allclose(g.W_head, (hbar @ A).T @ G, atol=1e-14)
    np.testing.assert_allclose(g.b_head, G.sum(0), atol=1e-14)


def test_batch_gradient_is_mean_of_single_sample_gradients_and_duplicates_count_twice():
    rng = np.random.default_rng(14)
    N, L, S, d, r, C = 5, 3, 3, 6, 3, 3
    P = rand_params(rng, L, d, r, C)
    cache = rng.standard_normal((N, L, S, d))
    labels = rng.integers(0, C, N)
    ids = [3, 1, 3, 0]                                            # id 3 twice
    H = po.gather(cache, ids)
    loss, g, _ = po.loss_and_grads_cls(P, H, labels[ids])
    singles = [po.loss_and_grads_cls(P, po.gather(cache, [i]), labels[[i]]) for i in ids]
    assert abs(loss - np.mean([s[0] for s in singles])) < 1e-14
    np.testing.assert_allclose(po.flatten(g), np.mean([po.flatten(s[1]) for s in singles], axis=0), atol=1e-14)
    # permuting ids inside the batch changes nothing but rounding
    perm = [0, 3, 3, 1]
    loss2, g2, _ = po.loss_and_grads_cls(P, po.gather(cache, perm), labels[perm])
    assert abs(loss - loss2) < 1e-14
    np.testing.assert_allclose(po.flatten(g), po.flatten(g2), atol=1e-14)


def test_gather_is_pure_indexing_and_checks_range():
    rng = np.random.default_rng(15)
    cache = rng.standard_normal((6, 2, 3, 4)).astype(np.float32)
    ids = [5, 0, 5, 2]
    H = po.gather(cache, ids)
    for b, i in enumerate(ids):
        assert H[b].tobytes() == cache[i].tobytes()
    with pytest.raises(IndexError):
        po.gather(cache, [6])
    with pytest.raises(IndexError):
        po.gather(cache, [-1])


def test_frozen_inputs_are_never_modified():
    """The backbone is frozen (Section IV-B): a training step may not touch the
    cache, the labels or the LM head."""
    rng = np.random.default_rng(16)
    N, L, S, d, r, V = 4, 2, 3, 5, 3, 6
    cache = rng.standard_normal((N, L, S, d)).astype(np.float32)
    targets = rng.integers(0, V, (N, S))
    W_lm = rng.standard_normal((V, d)).astype(np.float32)
    snap = (cache.tobytes(), targets.tobytes(), W_lm.tobytes())
    tr = po.Trainer(cache, targets, rand_params(rng, L, d, r, None, np.float32), W_lm=W_lm)
    for _ in range(3):
        tr.train_step([0, 3])
        tr.adam_step()
    tr.eval_logits([1, 2])
    assert (cache.tobytes(), targets.tobytes(), W_lm.tobytes()) == snap


def test_cache_storage_cost_matches_paper_example():
    """Section V-B, storage cost: s*h*l per sequence; T5-Base (h=768, l=12),
    500 samples of length 30 in FP32 stay below 1 GB."""
    per = po.cache_bytes_per_sequence(30, 768, 12, 4)
    assert per == 30 * 768 * 12 * 4
    assert 0.5e9 < 500 * per < 1e9


def test_param_count_and_flat_layout():
    L, d, r, C = 12, 768, 64, 3
    P = po.unflatten(np.arange(L * d * r + L + r * d + d * C + C, dtype=np.float64), L, d, r, C)
    assert po.flatten(P).size == 641295                      # adapters + classifier head only
    assert P.W_down[0, 0, 1] == 1 and P.W_down[0, 1, 0] == r
    assert P.lam[0] == L * d * r
    assert P.W_up[0, 1] == L * d * r + L + 1 and P.W_up[1, 0] == L * d * r + L + d
    assert P.b_head[-1] == po.flatten(P).size - 1
    assert np.array_equal(po.flatten(P), np.arange(641295, dtype=np.float64))


# ---------------------------------------------------------------------------
# AdamW
# ---------------------------------------------------------------------------
def test_adamw_first_step_closed_form():
    hp = po.AdamW(lr=1e-3, weight_decay=0.01)
    th = np.array([0.5, -2.0, 3.0]); g = np.array([0.3, -1e-3, 7.0])
    mask = np.array([1.0, 0.0, 1.0])
    new, m, v = po.adamw_step(th, g, np.zeros(3), np.zeros(3), 1, hp, mask)
    ref = th * (1 - hp.lr * hp.weight_decay * mask) - hp.lr * g / (np.abs(g) + hp.eps)
    np.testing.assert_allclose(new, ref, rtol=1e-12)


def test_adamw_constant_gradient_and_pure_decay():
    hp = po.AdamW(lr=1e-2, weight_decay=0.1)
    g = np.array([0.25, -4.0])
    th, m, v = np.array([1.0, 1.0]), np.zeros(2), np.zeros(2)
    for t in range(1, 8):
        th, m, v = po.adamw_step(th, g, m, v, t, hp, np.zeros(2))
        np.testing.assert_allclose(m / (1 - hp.beta1 ** t), g, rtol=1e-12)
        np.testing.assert_allclose(v / (1 - hp.beta2 ** t), g * g, rtol=1e-12)
    np.testing.assert_allclose(th, 1.0 - 7 * hp.lr * np.sign(g), rtol=1e-6)
    th, m, v = np.array([2.0, -3.0]), np.zeros(2), np.zeros(2)
    for t in range(1, 6):
        th, m, v = po.adamw_step(th, np.zeros(2), m, v, t, hp, np.array([1.0, 0.0]))
    np.testing.assert_allclose(th, [2.0 * (1 - hp.lr * hp.weight_decay) ** 5, -3.0], rtol=1e-13)


def test_adamw_matches_torch_optimizer():
    rng = np.random.default_rng(17)
    n = 50
    th0 = rng.standard_normal(n)
    grads = [rng.standard_normal(n) * 10.0 ** rng.integers(-4, 2) for _ in range(10)]
    hp = po.AdamW(lr=3e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05)
    th, m, v = th0.copy(), np.zeros(n), np.zeros(n)
    p = torch.tensor(th0.copy(), requires_grad=True)
    opt = torch.optim.AdamW([p], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps, weight_decay=hp.weight_decay)
    for t, g in enumerate(grads, 1):
        th, m, v = po.adamw_step(th, g, m, v, t, hp, np.ones(n))
        p.grad = torch.tensor(g)
        opt.step()
    np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-10, atol=1e-12)


def test_trainer_ten_steps_reduce_loss_on_learnable_labels():
    """End-to-end sanity of the loop: labels that depend on the cached last layer
    are learnable, so ten steps from the zero-up-projection start lower the loss."""
    rng = np.random.default_rng(18)
    N, L, S, d, r, C = 32, 2, 4, 8, 4, 2
    cache = rng.standard_normal((N, L, S, d)).astype(np.float32)
    labels = (cache[:, L - 1].mean(axis=1)[:, 0] > 0).astype(np.int64)
    P = rand_params(rng, L, d, r, C, np.float32)
    P.W_up[:] = 0
    tr = po.Trainer(cache, labels, P, hp=po.AdamW(lr=5e-2))
    ids = np.arange(N)
    first = tr.train_step(ids)
    for _ in range(20):
        tr.adam_step()
        last = tr.train_step(ids)
    assert last < first - 0.05
