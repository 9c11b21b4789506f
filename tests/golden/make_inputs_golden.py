"""Writes tests/golden/inputs_golden.json from pac_inputs alone (no CUDA, no oracle)."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import pac_inputs as pi  # noqa: E402

spec = pi.CONFIGS["tiny_fp32"]
x = pi.cache_samples(spec, 0, [0, 255])
gold = {
    "cache_n0_first4": x[0, 0, 0, :4].tolist(),
    "cache_n255_last4": x[1, 3, 31, -4:].tolist(),
    "labels_first16": pi.labels(spec, 0)[:16].tolist(),
    "perm_first8": pi.epoch_permutation(256, 2)[:8].tolist(),
    "init_first4": pi.init_params(spec, 1)[:4].tolist(),
}
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "inputs_golden.json"), "w") as f:
    json.dump(gold, f, indent=1)
print(gold)
