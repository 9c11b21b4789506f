"""Pins for oracle/quant_oracle.py (block-wise absmax INT8, paper Eq. 1-2)."""
import json
import os

import numpy as np

from oracle import quant_oracle as qo


def test_hand_worked_example_of_eq1_and_eq2():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "quant_eq1_example.json")))
    x = np.array(g["x"], dtype=np.float32)
    q, c = qo.quantize_absmax(x, block=8)
    assert q.tolist() == g["codes"] and c.tolist() == [g["c"]]
    np.testing.assert_allclose(qo.dequantize_absmax(q, c, 8), np.array(g["dequant"]), rtol=1e-6)


def test_extremes_map_to_127_and_round_trip_error_is_half_a_step():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(10_000) * rng.uniform(0.01, 50, 10_000)).astype(np.float32)
    for block in (1, 7, 64, 4096, 10_000):
        q, c = qo.quantize_absmax(x, block)
        xr = qo.dequantize_absmax(q, c, block)
        for j in range(c.size):
            seg, segr, segq = x[j * block:(j + 1) * block], xr[j * block:(j + 1) * block], q[j * block:(j + 1) * block]
            amax = np.abs(seg).max()
            assert np.abs(segq).max() == 127 and np.abs(segq[np.abs(seg) == amax]).min() == 127
            assert np.abs(seg - segr).max() <= amax / 254 * (1 + 1e-5)


def test_power_of_two_scaling_leaves_codes_unchanged_and_blocks_are_independent():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(1000).astype(np.float32)
    q, c = qo.quantize_absmax(x, 100)
    q2, c2 = qo.quantize_absmax(x * np.float32(8), 100)
    assert np.array_equal(q, q2) and np.allclose(c2 * 8, c)
    y = x.copy()
    y[250:260] *= 100                                   # disturb block 2 only
    qy, cy = qo.quantize_absmax(y, 100)
    keep = np.r_[0:200, 300:1000]
    assert np.array_equal(q[keep], qy[keep]) and np.array_equal(np.delete(c, 2), np.delete(cy, 2))


def test_outlier_costs_precision_only_inside_its_block():
    """The motivation the section gives for block-wise quantisation."""
    rng = np.random.default_rng(2)
    x = rng.standard_normal(4096).astype(np.float32)
    x[17] = 1000.0
    err_whole = np.abs(x - qo.dequantize_absmax(*qo.quantize_absmax(x, 4096), 4096))
    err_block = np.abs(x - qo.dequantize_absmax(*qo.quantize_absmax(x, 64), 64))
    assert err_whole[64:].mean() > 20 * err_block[64:].mean()
    assert np.allclose(err_whole[:64].mean(), err_block[:64].mean(), rtol=0.5)


def test_zero_block_and_ragged_tail():
    x = np.zeros(10, dtype=np.float32)
    x[9] = -3.0
    q, c = qo.quantize_absmax(x, 4)                      # blocks: zeros, zeros, [0, -3]
    assert c.tolist()[:2] == [0.0, 0.0] and q[:8].tolist() == [0] * 8 and q[9] == -127
    assert qo.dequantize_absmax(q, c, 4).tolist() == x.tolist()
