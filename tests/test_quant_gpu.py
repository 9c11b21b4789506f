"""GPU parity of the block-wise absmax INT8 codec (paper Eq. 1-2) against the CPU oracle:
integer codes, constants and dequantised values must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import quant_oracle as qo

pytestmark = pytest.mark.gpu


def make(n, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(n, generator=g) * torch.exp(2 * torch.randn(n, generator=g))
    x[::97] = 0.0
    return x


@pytest.mark.parametrize("n,block", [(1, 1), (1000, 64), (4096 * 3 + 5, 4096), (100_003, 64), (50_000, 8192), (257, 1000),
                                     (1 << 20, 256), (1 << 18, 16), (4096 * 5 + 64, 128), (3072 * 7, 3072), (2048 * 3 + 1024, 2048)])
def test_codes_constants_and_round_trip_bit_exact(n, block):
    import paper_2408_10746_b200 as pac
    x = make(n, n + block)
    if n > 10:
        x[block // 2: block // 2 + min(block, n)] = 0          # an all-zero block where it fits
    q, c = pac.quantize_absmax(x.cuda(), block)
    out = pac.dequantize_absmax(q, c, block)
    torch.cuda.synchronize()
    rq, rc = qo.quantize_absmax(x.numpy(), block)
    assert np.array_equal(q.cpu().numpy(), rq)
    assert np.array_equal(c.cpu().numpy().view(np.uint32), rc.view(np.uint32))
    assert np.array_equal(out.cpu().numpy().view(np.uint32), qo.dequantize_absmax(rq, rc, block).view(np.uint32))


def test_bad_arguments_are_rejected():
    import paper_2408_10746_b200 as pac
    lib = pac.load_library()
    x = torch.zeros(8, device="cuda")
    assert lib.pac_quantize_absmax(0, None, x.data_ptr(), 8, 0, x.data_ptr(), x.data_ptr()) == 1
    assert lib.pac_quantize_absmax(0, None, None, 8, 4, x.data_ptr(), x.data_ptr()) == 1
    assert lib.pac_dequantize_absmax(0, None, x.data_ptr(), x.data_ptr(), 0, 4, x.data_ptr()) == 1
