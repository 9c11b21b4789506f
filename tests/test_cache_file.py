"""Cache files (paper Section IV-B: activations are recorded during the first epoch; Section V-B:
they live on storage and are reloaded per micro-batch).  Without a GPU: the writer stores host
slabs in any order and the file holds exactly the oracle's gather of them.  With a GPU: samples go
from device memory into the file, the file is registered as the cache, and gather / evaluation / a
train step match the oracle."""
import os

import numpy as np
import pytest
import torch

import pac_inputs as pi
from oracle import pac_oracle as po
from tests.common import rel_l2

SPEC = pi.CacheSpec("file_cache", N=20, L=3, S=19, d=104, dtype="bf16", r=12, n_out=3, B=5)
SPEC_F32 = pi.CONFIGS["tiny_fp32"].scaled(N=24, name="file_cache_f32")


def read_file_payload(path, spec):
    """The cache and label arrays as stored, decoded with numpy alone (header: 64 bytes; labels at the
    next multiple of 64 bytes behind the data)."""
    raw = np.fromfile(path, dtype=np.uint8)
    assert bytes(raw[:8]) == b"PACCACHE"
    n_el = spec.N * spec.L * spec.S * spec.d
    eb = 2 if spec.dtype == "bf16" else 4
    data = raw[64:64 + n_el * eb]
    lab_off = 64 + ((n_el * eb + 63) // 64) * 64
    labels = raw[lab_off:lab_off + 4 * spec.N].view(np.int32)
    return data, labels


@pytest.mark.parametrize("spec", [SPEC, SPEC_F32], ids=lambda s: s.name)
def test_writer_stores_host_slabs_bit_exact_in_any_order(tmp_path, spec):
    import paper_2408_10746_b200 as pac
    path = str(tmp_path / "cache.pac")
    cache = pi.cache_full(spec, 0, "cpu")
    labels = pi.labels(spec, 0, "cpu").numpy()
    order = pi.epoch_permutation(spec.N, 5).tolist()
    with pac.CacheWriter(path, cache.dtype, spec.N, spec.L, spec.S, spec.d) as w:
        for n in order:
            w.store(n, cache[n].contiguous(), [labels[n]])
        w.store(order[0], cache[order[0]].contiguous(), [labels[order[0]]])        # storing twice is allowed
        with pytest.raises(pac.PacError) as e:
            w.store(spec.N, cache[0].contiguous(), [0])
        assert e.value.status_name == "PAC_ERR_SAMPLE_ID_RANGE"
    dt, N, L, S, d, per = pac.cache_file_info(path)
    assert (N, L, S, d, per) == (spec.N, spec.L, spec.S, spec.d, 1) and dt == (pac.PAC_BF16 if spec.dtype == "bf16" else pac.PAC_F32)
    data, lab = read_file_payload(path, spec)
    want = po.gather(cache.view(torch.uint8).numpy().reshape(spec.N, -1), range(spec.N))    # pure indexing
    assert np.array_equal(data, want.ravel()) and np.array_equal(lab, labels)
    # a foreign or truncated file is refused
    bad = str(tmp_path / "bad.pac")
    with open(bad, "wb") as f:
        f.write(b"NOTACACHE" + bytes(100))
    with pytest.raises(pac.PacError):
        pac.cache_file_info(bad)
    with open(path, "rb") as f, open(bad, "wb") as g:
        g.write(f.read()[:-8])
    with pytest.raises(pac.PacError):
        pac.cache_file_info(bad)
    with pytest.raises(pac.PacError):
        pac.CacheWriter(str(tmp_path / "x.pac"), cache.dtype, 0, 1, 1, 1)


@pytest.mark.gpu
@pytest.mark.parametrize("spec", [SPEC, SPEC_F32], ids=lambda s: s.name)
def test_file_cache_from_device_slabs_matches_oracle(tmp_path, spec):
    import paper_2408_10746_b200 as pac
    path = str(tmp_path / "cache.pac")
    dev_cache = pi.cache_full(spec, 0, "cuda")
    labels = pi.labels(spec, 0, "cpu").numpy()
    with pac.CacheWriter(path, dev_cache.dtype, spec.N, spec.L, spec.S, spec.d) as w:
        for n in pi.epoch_permutation(spec.N, 7).tolist():          # the order a first epoch would visit them in
            w.store(n, dev_cache[n], [labels[n]])
    ctx = pac.PacContext(0)
    ctx.cache_register_file(path)
    ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B)
    flat = pi.random_params(spec, 3)
    ctx.set_params(flat)
    ids = [spec.N - 1, 0, 7, 7, 3][:spec.B]
    # gather: the oracle's gather of the generator's cache, bit for bit
    cache_np = pi.cache_full(spec, 0, "cpu")
    got = torch.empty((spec.L, len(ids), spec.S, spec.d), dtype=dev_cache.dtype, device="cuda")
    ctx.gather(ids, got)
    ctx.sync()
    want = po.gather(cache_np.view(torch.uint8).numpy().reshape(spec.N, spec.L, -1), ids)       # [B][L][bytes]
    assert np.array_equal(got.cpu().view(torch.uint8).numpy().reshape(spec.L, len(ids), -1), want.transpose(1, 0, 2))
    # evaluation and one train step against the oracle
    P = po.unflatten(flat, spec.L, spec.d, spec.r, spec.n_out)
    H = po.gather(cache_np.float().numpy(), ids)
    tight = spec.dtype == "f32"
    out = torch.zeros((len(ids), spec.n_out), dtype=torch.float32, device="cuda")
    ctx.eval_logits(ids, out)
    ctx.sync()
    assert rel_l2(out.cpu().numpy(), po.eval_logits(P, H, 0)) < (1e-4 if tight else 3e-3)
    loss = ctx.train_step(ids)
    ref_loss, ref_g, _ = po.loss_and_grads_cls(P, H, labels[ids].astype(np.int64))
    assert abs(loss - ref_loss) <= (1e-4 if tight else 2e-2) * abs(ref_loss)
    assert rel_l2(ctx.get_grads(), po.flatten(ref_g)) < (1e-4 if tight else 1e-2)
    # a whole epoch through the file equals the same epoch on the device-resident cache, bit for bit
    hp = pac.AdamW()
    perm = pi.epoch_permutation(spec.N, 2)[:(spec.N // spec.B) * spec.B]
    losses_file = ctx.train_epoch(perm, spec.B, hp)
    dev = pac.PacContext(0)
    dev.cache_register(dev_cache, pi.labels(spec, 0, "cuda"))
    dev.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B)
    dev.set_params(flat)
    losses_dev = dev.train_epoch(perm, spec.B, hp)
    assert np.array_equal(losses_file, losses_dev) and np.array_equal(ctx.get_params(), dev.get_params())
    with pytest.raises(pac.PacError):
        pac.PacContext(0).cache_register_file(str(tmp_path / "missing.pac"))
    ctx.close(); dev.close()
