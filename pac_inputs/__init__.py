"""Seeded synthetic inputs for the adapter-over-cache path.

This module only manufactures *data*: activation caches, labels, a frozen LM
head, initial adapter parameters and epoch permutations.  It holds none of the
method's arithmetic (no projection, merge, loss, gradient or optimizer code) and
is the one module both the CPU oracle's tests and the CUDA path's tests/bench may
import.

Everything is a pure function of (seed, element index) built from 64-bit integer
mixing, so any slab of a cache can be regenerated anywhere without the rest of
it, and the values are bit-identical on CPU and on a CUDA device: the generator
uses only wrapping int64 arithmetic, one int->float conversion, one IEEE fp32
multiply and (for bf16 caches) one round-to-nearest-even narrowing, all done with
ordinary torch element-wise ops.

The paper measures on GLUE activations of T5-Base / BART-Large / T5-Large
(Section VI, table of model specifications); those are not available here, so the
caches below are Gaussian stand-ins of the same shapes with a per-layer growth of
the standard deviation and, optionally, a few large "outlier" channels.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Sequence

import numpy as np
import torch

# ---------------------------------------------------------------------------
# 64-bit integer mixing (the splitmix64 output function of Steele/Lea/Flood,
# "Fast splittable pseudorandom number generators", OOPSLA 2014), written for
# torch's signed int64: multiplication wraps, and a logical right shift is an
# arithmetic shift followed by a mask.
# ---------------------------------------------------------------------------
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_GOLD = 0x9E3779B97F4A7C15
_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Two's-complement reinterpretation of an unsigned 64-bit python int."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    return (x >> k) & ((1 << (64 - k)) - 1)


def _mix64_t(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _s64(_M1)
    x = (x ^ _lsr(x, 27)) * _s64(_M2)
    return x ^ _lsr(x, 31)


def _mix64_i(x: int) -> int:
    """The same mixing on a python int (unsigned 64-bit domain)."""
    x &= _MASK64
    x = ((x ^ (x >> 30)) * _M1) & _MASK64
    x = ((x ^ (x >> 27)) * _M2) & _MASK64
    return x ^ (x >> 31)


def stream_key(seed: int, tag: int) -> int:
    """Key of an independent random stream `tag` under `seed` (unsigned 64-bit)."""
    return _mix64_i(_mix64_i(seed & _MASK64) ^ ((tag * _GOLD) & _MASK64))


# stream tags
TAG_CACHE, TAG_LABEL, TAG_LMHEAD, TAG_PARAM, TAG_PERM, TAG_OUTLIER, TAG_TARGET = 1, 2, 3, 4, 5, 6, 7


def unit_normal_from_index(key: int, idx: torch.Tensor) -> torch.Tensor:
    """Approximately N(0,1) fp32 values, one per int64 element index.

    Three mixed 64-bit words per element give twelve 16-bit uniform fields; their
    sum minus its mean is a centred Irwin-Hall(12) integer g with |g| < 2**24
    (exact in fp32) and variance 65536**2 - 1; g * 2**-16 is an exact scaling to
    unit variance (support +-6 sigma).
    """
    base = idx * 3
    total = torch.zeros_like(idx)
    for j in range(3):
        w = _mix64_t((base + j) * _s64(_GOLD) + _s64(key))
        total = total + (w & 0xFFFF) + (_lsr(w, 16) & 0xFFFF) + (_lsr(w, 32) & 0xFFFF) + _lsr(w, 48)
    g = total - 6 * 65535
    return g.to(torch.float32) * (2.0 ** -16)


def uniform_int_from_index(key: int, idx: torch.Tensor, modulus: int) -> torch.Tensor:
    """Integers in [0, modulus) from the top 31 bits of one mixed word per index."""
    w = _mix64_t(idx * _s64(_GOLD) + _s64(key))
    return (_lsr(w, 33) % modulus).to(torch.int32)


# ---------------------------------------------------------------------------
# Workload description
# ---------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class CacheSpec:
    """Shape and value law of one synthetic activation cache [N][L][S][d]."""
    name: str
    N: int
    L: int
    S: int
    d: int
    dtype: str            # "f32" or "bf16"
    r: int                # adapter width
    n_out: int            # classes C, or vocabulary V for the LM head
    B: int                # minibatch size
    head: str = "cls"     # "cls" (mean-pool classifier) or "lm" (frozen LM head)
    outlier_frac: float = 0.0
    outlier_gain: float = 8.0
    layer_growth: float = 0.1
    steps: Optional[int] = None   # None: one shuffled epoch (N // B steps)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def sample_elems(self) -> int:
        return self.L * self.S * self.d

    @property
    def cache_bytes(self) -> int:
        return self.N * self.sample_elems * self.elem_bytes

    @property
    def n_steps(self) -> int:
        return self.steps if self.steps is not None else self.N // self.B

    def scaled(self, **kw) -> "CacheSpec":
        return dataclasses.replace(self, **kw)


# The five workloads (shapes follow the paper's model-specification table for
# T5-Base, BART-Large and T5-Large, plus a LLaMA-7B-shaped decoder stack).
CONFIGS = {
    "tiny_fp32": CacheSpec("tiny_fp32", N=256, L=4, S=32, d=256, dtype="f32", r=16, n_out=2, B=8, steps=10),
    "t5_base": CacheSpec("t5_base", N=4096, L=12, S=128, d=768, dtype="bf16", r=64, n_out=3, B=32),
    "bart_large": CacheSpec("bart_large", N=4096, L=24, S=128, d=1024, dtype="bf16", r=64, n_out=2, B=32),
    "t5_large": CacheSpec("t5_large", N=4096, L=24, S=256, d=1024, dtype="bf16", r=128, n_out=5, B=64,
                          outlier_frac=0.01),
    "llama_7b": CacheSpec("llama_7b", N=256, L=32, S=512, d=4096, dtype="bf16", r=64, n_out=32000, B=16,
                          head="lm"),
}


def outlier_channels(spec: CacheSpec, seed: int) -> np.ndarray:
    """Indices of the ceil(outlier_frac * d) channels that carry the large gain.

    Channels are ranked by a mixed hash of (seed, channel); the lowest ranks win,
    so the set is fixed across samples and layers.
    """
    k = int(math.ceil(spec.outlier_frac * spec.d)) if spec.outlier_frac > 0 else 0
    if k == 0:
        return np.zeros(0, dtype=np.int64)
    key = stream_key(seed, TAG_OUTLIER)
    ranks = [(_mix64_i((c * _GOLD + key) & _MASK64), c) for c in range(spec.d)]
    ranks.sort()
    return np.array(sorted(c for _, c in ranks[:k]), dtype=np.int64)


def scale_table(spec: CacheSpec, seed: int) -> torch.Tensor:
    """fp32 [L][d] table: (1 + growth*l) * (outlier gain or 1), rounded once to fp32."""
    tab = np.ones((spec.L, spec.d), dtype=np.float64)
    tab *= (1.0 + spec.layer_growth * np.arange(spec.L, dtype=np.float64))[:, None]
    out = outlier_channels(spec, seed)
    if out.size:
        tab[:, out] *= spec.outlier_gain
    return torch.from_numpy(tab.astype(np.float32))


def cache_samples(spec: CacheSpec, seed: int, sample_ids: Sequence[int] | torch.Tensor,
                  device: str | torch.device = "cpu") -> torch.Tensor:
    """Slabs [len(ids)][L][S][d] of the cache for the given sample ids, in spec.dtype."""
    dev = torch.device(device)
    ids = torch.as_tensor(sample_ids, dtype=torch.int64, device=dev).reshape(-1)
    key = stream_key(seed, TAG_CACHE)
    per = spec.sample_elems
    within = torch.arange(per, dtype=torch.int64, device=dev)
    idx = ids[:, None] * per + within[None, :]
    x = unit_normal_from_index(key, idx).view(ids.numel(), spec.L, spec.S, spec.d)
    x = x * scale_table(spec, seed).to(dev)[None, :, None, :]
    return x.to(spec.torch_dtype)


def cache_full(spec: CacheSpec, seed: int, device: str | torch.device = "cpu",
               chunk_elems: int = 1 << 25) -> torch.Tensor:
    """The whole cache [N][L][S][d], filled in chunks of whole samples."""
    dev = torch.device(device)
    out = torch.empty((spec.N, spec.L, spec.S, spec.d), dtype=spec.torch_dtype, device=dev)
    per_chunk = max(1, chunk_elems // spec.sample_elems)
    for n0 in range(0, spec.N, per_chunk):
        n1 = min(spec.N, n0 + per_chunk)
        out[n0:n1] = cache_samples(spec, seed, torch.arange(n0, n1, device=dev), dev)
    return out


def labels(spec: CacheSpec, seed: int, device: str | torch.device = "cpu") -> torch.Tensor:
    """int32 labels: [N] uniform in [0,C) for the classifier head, [N][S] uniform
    token targets in [0,V) for the LM head."""
    dev = torch.device(device)
    if spec.head == "cls":
        idx = torch.arange(spec.N, dtype=torch.int64, device=dev)
        return uniform_int_from_index(stream_key(seed, TAG_LABEL), idx, spec.n_out)
    idx = torch.arange(spec.N * spec.S, dtype=torch.int64, device=dev)
    return uniform_int_from_index(stream_key(seed, TAG_TARGET), idx, spec.n_out).view(spec.N, spec.S)


def lm_head(spec: CacheSpec, seed: int, device: str | torch.device = "cpu",
            chunk_rows: int = 4096) -> torch.Tensor:
    """Frozen LM head [V][d] in bf16, N(0, sigma^2) with sigma chosen so that the
    logits of the last cached layer have about unit variance."""
    dev = torch.device(device)
    V, d = spec.n_out, spec.d
    sigma = np.float32(1.0 / (math.sqrt(d) * (1.0 + spec.layer_growth * (spec.L - 1))))
    key = stream_key(seed, TAG_LMHEAD)
    out = torch.empty((V, d), dtype=torch.bfloat16, device=dev)
    for v0 in range(0, V, chunk_rows):
        v1 = min(V, v0 + chunk_rows)
        idx = torch.arange(v0 * d, v1 * d, dtype=torch.int64, device=dev)
        out[v0:v1] = (unit_normal_from_index(key, idx) * float(sigma)).view(v1 - v0, d).to(torch.bfloat16)
    return out


def param_count(spec: CacheSpec) -> int:
    n = spec.L * spec.d * spec.r + spec.L + spec.r * spec.d
    if spec.head == "cls":
        n += spec.d * spec.n_out + spec.n_out
    return n


def random_params(spec: CacheSpec, seed: int, up_std: float = 0.02, lam_jitter: float = 0.2) -> np.ndarray:
    """A flat fp32 parameter vector with every block non-zero (for gradient parity
    tests, where a zero up-projection would make most gradients vanish).

    Layout: W_down[L][d][r] | lambda[L] | W_up[r][d] | W_head[d][C] | b_head[C]
    (the last two only for the classifier head).
    """
    key = stream_key(seed, TAG_PARAM)
    n = param_count(spec)
    z = unit_normal_from_index(key, torch.arange(n, dtype=torch.int64)).numpy().astype(np.float32)
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    o = 0
    out = np.empty(n, dtype=np.float32)
    k = L * d * r
    out[o:o + k] = z[o:o + k] * np.float32(1.0 / math.sqrt(d)); o += k
    out[o:o + L] = np.float32(0.5) + np.float32(lam_jitter) * z[o:o + L]; o += L
    k = r * d
    out[o:o + k] = z[o:o + k] * np.float32(up_std); o += k
    if spec.head == "cls":
        k = d * C
        out[o:o + k] = z[o:o + k] * np.float32(1.0 / math.sqrt(d)); o += k
        out[o:o + C] = np.float32(0.1) * z[o:o + C]; o += C
    assert o == n
    return out


def init_params(spec: CacheSpec, seed: int, lambda_init: float = 0.5) -> np.ndarray:
    """The library's seeded initial state restated from its documented law:
    W_down ~ N(0, 1/d), lambda = lambda_init, W_up = 0, W_head ~ N(0, 1/d),
    b_head = 0, with element i of the flat vector drawn from stream
    (seed, TAG_PARAM) at index i."""
    key = stream_key(seed, TAG_PARAM)
    n = param_count(spec)
    z = unit_normal_from_index(key, torch.arange(n, dtype=torch.int64)).numpy().astype(np.float32)
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    out = np.zeros(n, dtype=np.float32)
    inv = np.float32(1.0 / math.sqrt(d))
    o = 0
    k = L * d * r
    out[o:o + k] = z[o:o + k] * inv; o += k
    out[o:o + L] = np.float32(lambda_init); o += L
    o += r * d
    if spec.head == "cls":
        k = d * C
        out[o:o + k] = z[o:o + k] * inv; o += k
    return out


def epoch_permutation(n: int, seed: int, epoch: int = 0) -> np.ndarray:
    """Seeded Fisher-Yates shuffle of 0..n-1 (int32), driven by mixed counters."""
    key = stream_key(seed, TAG_PERM) ^ _mix64_i(epoch + 1)
    perm = np.arange(n, dtype=np.int32)
    for i in range(n - 1, 0, -1):
        w = _mix64_i((i * _GOLD + key) & _MASK64)
        j = (w >> 11) % (i + 1)
        perm[i], perm[j] = perm[j], perm[i]
    return perm
