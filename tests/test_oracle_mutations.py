"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source
(never in the CUDA path) and requires that at least one pin of tests/test_oracle_pins.py fails."""
import importlib.util
import os
import sys
import types

import pytest

from tests import test_oracle_pins as pins

ORACLE = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "pac_oracle.py")

MUTATIONS = {
    "merge drops the running state": ("z[l] = lam * u[l] + (dt.type(1) - lam) * a_prev", "z[l] = lam * u[l]"),
    "merge weights swapped": ("z[l] = lam * u[l] + (dt.type(1) - lam) * a_prev", "z[l] = (dt.type(1) - lam) * u[l] + lam * a_prev"),
    "no residual with the backbone output": ("y = H[:, L - 1] + a_prev @ P.W_up", "y = a_prev @ P.W_up"),
    "residual from the wrong layer": ("y = H[:, L - 1] + a_prev @ P.W_up", "y = H[:, 0] + a_prev @ P.W_up"),
    "dlambda forgets a_prev": ("np.sum(dz * (u[l] - a_prev), dtype=dt)", "np.sum(dz * u[l], dtype=dt)"),
    "du not scaled by lambda": ("du = lam * dz", "du = dz"),
    "da uses lambda instead of 1 - lambda": ("da = (dt.type(1) - lam) * dz", "da = lam * dz"),
    "dW_down from the wrong layer's activations": ("g.W_down[l] = H[:, l].reshape", "g.W_down[l] = H[:, 0].reshape"),
    "pooling gradient misses 1/S": ("(dpooled / dt.type(S))[:, None, :]", "dpooled[:, None, :]"),
    "loss gradient not averaged": ("return (p / flat.shape[0]).reshape(logits.shape)", "return p.reshape(logits.shape)"),
    "softmax without the one-hot": ("p[np.arange(flat.shape[0]), t] -= 1", "pass"),
    "ReLU derivative always one": ("return (z > 0).astype(z.dtype)", "return np.ones_like(z)"),
    "head bias gradient is a mean": ("g.b_head = dlogits.sum(axis=0)", "g.b_head = dlogits.mean(axis=0)"),
    "W_head gradient from unpooled wrong operand": ("g.W_head = pooled.T @ dlogits", "g.W_head = (pooled * 0 + 1).T @ dlogits"),
    "LM dy through the transposed head": ("dy = dlogits @ W_lm.astype(dt, copy=False)", "dy = dlogits @ np.roll(W_lm.astype(dt, copy=False), 1, axis=0)"),
    "Adam epsilon inside the root": ("(np.sqrt(vhat) + dt(hp.eps))", "np.sqrt(vhat + dt(hp.eps))"),
    "Adam without bias correction of v": ("vhat = v / dt(1.0 - hp.beta2 ** t)", "vhat = v"),
    "weight decay with the wrong sign": ("theta = theta - decay - dt(hp.lr)", "theta = theta + decay - dt(hp.lr)"),
    "second moment uses |g|": ("(dt(1) - b2) * g * g", "(dt(1) - b2) * np.abs(g)"),
    "gather off by one": ("return cache[ids]", "return cache[(ids + 1) % cache.shape[0]]"),
}

PINS = [
    lambda: pins.test_forward_matches_scalar_recursion_cls(0),
    lambda: pins.test_forward_matches_scalar_recursion_lm(),
    lambda: pins.test_gradients_finite_difference_cls(0),
    lambda: pins.test_gradients_finite_difference_cls(1),
    lambda: pins.test_gradients_finite_difference_lm(0),
    lambda: pins.test_gradients_against_torch_autograd(),
    lambda: pins.test_zero_up_projection_reproduces_head_only_model(),
    lambda: pins.test_lambda_one_uses_only_last_layer(),
    lambda: pins.test_single_linear_layer_closed_form(),
    lambda: pins.test_batch_gradient_is_mean_of_single_sample_gradients_and_duplicates_count_twice(),
    lambda: pins.test_gather_is_pure_indexing_and_checks_range(),
    lambda: pins.test_adamw_first_step_closed_form(),
    lambda: pins.test_adamw_constant_gradient_and_pure_decay(),
    lambda: pins.test_adamw_matches_torch_optimizer(),
]


def load_mutant(old: str, new: str) -> types.ModuleType:
    src = open(ORACLE).read()
    assert src.count(old) == 1, f"mutation anchor not unique: {old!r}"
    spec = importlib.util.spec_from_loader("pac_oracle_mutant", loader=None)
    mod = importlib.util.module_from_spec(spec)
    sys.modules["pac_oracle_mutant"] = mod          # dataclasses look their module up
    exec(compile(src.replace(old, new), ORACLE + " (mutant)", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, monkeypatch):
    mutant = load_mutant(*MUTATIONS[name])
    monkeypatch.setattr(pins, "po", mutant)
    caught = 0
    for pin in PINS:
        try:
            pin()
        except Exception:
            caught += 1
    assert caught >= 1, f"no pin noticed: {name}"


def test_unmutated_oracle_passes_every_pin_used_here():
    for pin in PINS:
        pin()
