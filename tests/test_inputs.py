"""The seeded generators: determinism, slab/whole consistency, value law, ranges."""
import numpy as np
import torch

import pac_inputs as pi


def test_mix64_int_and_tensor_agree():
    xs = [0, 1, 2**63 - 1, 2**63, 2**64 - 1, 0x123456789ABCDEF]
    t = torch.tensor([pi._s64(x) for x in xs], dtype=torch.int64)
    got = pi._mix64_t(t).tolist()
    assert [g & pi._MASK64 for g in got] == [pi._mix64_i(x) for x in xs]


def test_slabs_equal_slices_of_full_cache_and_are_deterministic():
    spec = pi.CONFIGS["tiny_fp32"].scaled(N=16)
    full = pi.cache_full(spec, 0, chunk_elems=3 * spec.sample_elems)
    ids = [15, 0, 7, 7]
    slab = pi.cache_samples(spec, 0, ids)
    assert torch.equal(slab, full[ids])
    assert torch.equal(pi.cache_full(spec, 0), full)
    assert not torch.equal(pi.cache_full(spec, 1), full)


def test_value_law_unit_normal_with_layer_growth():
    spec = pi.CONFIGS["tiny_fp32"].scaled(N=64)
    x = pi.cache_full(spec, 0).double()
    for l in range(spec.L):
        s = x[:, l].std().item()
        assert abs(s / (1 + 0.1 * l) - 1) < 0.01
        assert abs(x[:, l].mean().item()) < 0.01
    z = x[:, 0].flatten()
    assert abs(((z ** 4).mean() / (z ** 2).mean() ** 2).item() - 2.9) < 0.05   # Irwin-Hall(12) kurtosis
    assert z.abs().max() < 6.0001


def test_bf16_cache_is_rounded_fp32_and_outlier_channels():
    spec = pi.CONFIGS["t5_large"].scaled(N=2, L=2, S=8, d=256)
    x = pi.cache_full(spec, 0)
    assert x.dtype == torch.bfloat16
    out = pi.outlier_channels(spec, 0)
    assert out.size == 3                                   # ceil(0.01 * 256)
    stds = x.float()[:, 0].reshape(-1, spec.d).std(0)
    big = set(np.nonzero(stds.numpy() > 4)[0].tolist())
    assert big == set(out.tolist())
    f32 = pi.cache_full(spec.scaled(dtype="f32"), 0)
    assert torch.equal(f32.to(torch.bfloat16), x)


def test_labels_targets_and_lm_head():
    spec = pi.CONFIGS["t5_base"].scaled(N=3000)
    lab = pi.labels(spec, 0)
    assert lab.dtype == torch.int32 and lab.shape == (3000,)
    counts = torch.bincount(lab.long(), minlength=3)
    assert lab.min() >= 0 and lab.max() < 3 and counts.min() > 900
    lm = pi.CONFIGS["llama_7b"].scaled(N=4, S=16, d=64, n_out=1000, L=3)
    tg = pi.labels(lm, 0)
    assert tg.shape == (4, 16) and tg.min() >= 0 and tg.max() < 1000
    W = pi.lm_head(lm, 0, chunk_rows=300)
    assert W.shape == (1000, 64) and W.dtype == torch.bfloat16
    assert torch.equal(W, pi.lm_head(lm, 0, chunk_rows=1000))
    assert abs(W.float().std().item() * (64 ** 0.5) * 1.2 - 1) < 0.02


def test_params_and_permutation():
    spec = pi.CONFIGS["tiny_fp32"]
    assert pi.param_count(spec) == 20998
    assert pi.param_count(pi.CONFIGS["t5_base"]) == 641295
    assert pi.param_count(pi.CONFIGS["llama_7b"]) == 8650784
    p0 = pi.init_params(spec, 1)
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    o = L * d * r
    assert np.all(p0[o:o + L] == 0.5) and not p0[o + L:o + L + r * d].any() and not p0[-C:].any()
    assert abs(p0[:o].std() * d ** 0.5 - 1) < 0.02
    assert np.array_equal(p0, pi.init_params(spec, 1)) and not np.array_equal(p0, pi.init_params(spec, 2))
    pr = pi.random_params(spec, 3)
    assert pr[o + L:o + L + r * d].any()
    perm = pi.epoch_permutation(1000, 2)
    assert perm.dtype == np.int32 and sorted(perm.tolist()) == list(range(1000))
    assert not np.array_equal(perm, np.arange(1000)) and np.array_equal(perm, pi.epoch_permutation(1000, 2))
    assert not np.array_equal(perm, pi.epoch_permutation(1000, 2, epoch=1))


def test_golden_first_values():
    """A few stored values (written by tests/golden/make_inputs_golden.py from this
    module alone) so that a change to the generator cannot go unnoticed."""
    import json, os
    with open(os.path.join(os.path.dirname(__file__), "golden", "inputs_golden.json")) as f:
        gold = json.load(f)
    spec = pi.CONFIGS["tiny_fp32"]
    x = pi.cache_samples(spec, 0, [0, 255])
    assert x[0, 0, 0, :4].tolist() == gold["cache_n0_first4"]
    assert x[1, 3, 31, -4:].tolist() == gold["cache_n255_last4"]
    assert pi.labels(spec, 0)[:16].tolist() == gold["labels_first16"]
    assert pi.epoch_permutation(256, 2)[:8].tolist() == gold["perm_first8"]
    assert pi.init_params(spec, 1)[:4].tolist() == gold["init_first4"]
