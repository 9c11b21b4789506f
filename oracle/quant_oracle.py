"""CPU oracle for block-wise absmax INT8 quantisation (PAC+ Section IV-D, Eq. 1 and Eq. 2).

TEST INFRASTRUCTURE ONLY (see pac_oracle.py for who may use it).  Shares no code with the CUDA path.

Eq. 1:  X8 = round( 127 / absmax(X32) * X32 ) = round( c * X32 ),  c the quantisation constant.
Eq. 2:  dequant(c, X8) = X8 / c.
Block-wise variant (same section): the input is cut into contiguous blocks of `block` elements
(the last one may be shorter) and each block is quantised independently with Eq. 1.

Readings where the section is silent: arithmetic in fp32, as the superscripts of the equations
say; `round` is round-to-nearest with ties to even (the IEEE default, numpy's rint); a block that
is all zeros gets c = 0, codes 0 and dequantises to 0 (its absmax is 0, so Eq. 1 has no value).

Pins (tests/test_quant_oracle.py): a hand-worked example of Eq. 1; codes of +-absmax are +-127;
round-trip error at most absmax/254 per block element (half a quantisation step); invariance
under scaling by powers of two; independence of blocks; the outlier example of the section (one
large value ruins a whole tensor's precision but only its own block's).
"""
from __future__ import annotations

import numpy as np


def quantize_absmax(x: np.ndarray, block: int):
    """x: 1-D float32.  Returns (codes int8 [n], constants float32 [ceil(n/block)])."""
    x = np.ascontiguousarray(x, dtype=np.float32).ravel()
    n = x.size
    nb = (n + block - 1) // block
    q = np.zeros(n, dtype=np.int8)
    c = np.zeros(nb, dtype=np.float32)
    for j in range(nb):
        seg = x[j * block:(j + 1) * block]
        amax = np.float32(np.max(np.abs(seg))) if seg.size else np.float32(0)
        if amax > 0:
            c[j] = np.float32(127.0) / amax                      # quantisation constant (Eq. 1)
            q[j * block:(j + 1) * block] = np.rint(c[j] * seg).astype(np.int8)
    return q, c


def dequantize_absmax(q: np.ndarray, c: np.ndarray, block: int) -> np.ndarray:
    """Eq. 2 per block: X8 / c (0 where c == 0)."""
    q = np.asarray(q, dtype=np.int8).ravel()
    out = np.zeros(q.size, dtype=np.float32)
    for j in range(c.size):
        if c[j] != 0:
            out[j * block:(j + 1) * block] = q[j * block:(j + 1) * block].astype(np.float32) / np.float32(c[j])
    return out
