"""The allocation-free evaluation entry point (pac_eval_logits_static), for callers that may
not allocate device memory: its scratch is a fixed array inside the library.  Collected last on
purpose, so that a run that stops at the first failure has already run every other test.

Checked against the context-based pac_eval_logits and against the CPU oracle on the same inputs, on two calls in a row (the
second with other ids and a smaller batch, so stale scratch from the first call would show)."""
import numpy as np
import pytest
import torch

import pac_inputs as pi
from oracle import pac_oracle as po
from tests.common import Case, rel_l2

pytestmark = pytest.mark.gpu


def run_pair(spec, force_simt, tol):
    import paper_2408_10746_b200 as pac
    case = Case(spec, materialize_cpu=False)
    ctx = case.context(max_batch=spec.B, force_simt=force_simt)
    flat = pi.random_params(spec, 4)
    ctx.set_params(flat)
    dev_params = torch.from_numpy(flat).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    for ids in (list(range(spec.B)), [spec.N - 1, 2, 2, 0, 5][:max(1, spec.B - 3)]):
        want = torch.zeros((len(ids), spec.n_out), dtype=torch.float32, device="cuda")
        ctx.eval_logits(ids, want)
        ctx.sync()
        got = torch.full((len(ids), spec.n_out), float("nan"), dtype=torch.float32, device="cuda")
        dev_ids = torch.tensor(ids, dtype=torch.int32, device="cuda")
        pac.eval_logits_static(case.cache, dev_params, spec.r, spec.n_out, dev_ids, got, stream=stream)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert rel_l2(got.cpu().numpy(), want.cpu().numpy()) < tol
        # and against the oracle itself, not only against the other CUDA entry point
        ref = po.eval_logits(case.oracle_params(flat), case.H(ids), 0)
        assert rel_l2(got.cpu().numpy(), ref) < tol
    ctx.close()


def test_static_eval_matches_context_eval_fp32():
    run_pair(pi.CONFIGS["tiny_fp32"], False, 1e-4)


def test_static_eval_matches_context_eval_bf16():
    run_pair(pi.CacheSpec("ragged_bf16", N=24, L=3, S=19, d=100, dtype="bf16", r=12, n_out=3, B=5), True, 1e-4)


def test_static_eval_rejects_sizes_beyond_the_fixed_scratch():
    import paper_2408_10746_b200 as pac
    spec = pi.CONFIGS["t5_base"].scaled(N=40)
    cache = torch.zeros((spec.N, spec.L, spec.S, spec.d), dtype=torch.bfloat16, device="cuda")
    params = torch.zeros(pi.param_count(spec), dtype=torch.float32, device="cuda")
    ids = torch.arange(32, dtype=torch.int32, device="cuda")
    out = torch.zeros((32, 3), dtype=torch.float32, device="cuda")
    with pytest.raises(pac.PacError) as e:
        pac.eval_logits_static(cache, params, spec.r, spec.n_out, ids, out)      # 25 MB of intermediates
    assert e.value.status_name == "PAC_ERR_UNSUPPORTED" and "scratch" in str(e.value)
    pac.eval_logits_static(cache, params, spec.r, spec.n_out, ids[:8], out[:8])  # 6.3 MB fits
    torch.cuda.synchronize()
    assert torch.equal(out[:8], torch.zeros_like(out[:8]))                       # zero parameters, zero cache
