"""Shared helpers for the parity tests: build a synthetic case on the GPU and the
matching numpy view for the oracle (inputs come from pac_inputs only)."""
from __future__ import annotations

import numpy as np
import torch

import pac_inputs as pi
from oracle import pac_oracle as po


def rel_l2(x, ref):
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    n = np.linalg.norm(ref)
    return np.linalg.norm(x - ref) / n if n > 0 else np.linalg.norm(x - ref)


class Case:
    """A cache on `device` plus what the oracle needs for any subset of sample ids."""

    def __init__(self, spec: pi.CacheSpec, seed: int = 0, device: str = "cuda", materialize_cpu: bool = True):
        self.spec, self.seed = spec, seed
        self.cache = pi.cache_full(spec, seed, device)
        self.labels = pi.labels(spec, seed, device)
        self.lm = pi.lm_head(spec, seed, device) if spec.head == "lm" else None
        self.labels_np = pi.labels(spec, seed, "cpu").numpy().astype(np.int64)
        self.lm_np = pi.lm_head(spec, seed, "cpu").float().numpy() if spec.head == "lm" else None
        self.cache_np = pi.cache_full(spec, seed, "cpu").float().numpy() if materialize_cpu else None

    def H(self, ids):
        """Oracle-side gathered slabs [B][L][S][d] as float32, regenerated on the CPU."""
        if self.cache_np is not None:
            return po.gather(self.cache_np, ids)
        return pi.cache_samples(self.spec, self.seed, list(ids), "cpu").float().numpy()

    def context(self, max_batch=None, act=0, force_simt=False, seed=1, kernel_path=0):
        import paper_2408_10746_b200 as pac
        s = self.spec
        ctx = pac.PacContext(0)
        if force_simt:
            ctx.set_option(0, 1)
        elif kernel_path:
            ctx.set_option(0, kernel_path)
        ctx.cache_register(self.cache, self.labels)
        ctx.adapter_init(r=s.r, n_out=s.n_out, max_batch=max_batch or s.B, act=act,
                         head=pac.PAC_HEAD_FROZEN_LM if s.head == "lm" else pac.PAC_HEAD_MEANPOOL_CLS,
                         lm_head=self.lm, seed=seed)
        return ctx

    def oracle_params(self, flat, dtype=np.float32):
        s = self.spec
        return po.unflatten(np.asarray(flat, dtype=dtype), s.L, s.d, s.r, s.n_out if s.head == "cls" else None)

    def oracle_loss_grads(self, flat, ids, act=0, dtype=np.float32):
        P = self.oracle_params(flat, dtype)
        H = self.H(ids).astype(dtype)
        lab = self.labels_np[np.asarray(ids)]
        if self.spec.head == "cls":
            return po.loss_and_grads_cls(P, H, lab, act)
        return po.loss_and_grads_lm(P, H, lab, self.lm_np.astype(dtype), act)

    def oracle_trainer(self, flat, act=0, hp=None, ids_universe=None):
        """Trainer over a CPU cache; with ids_universe only those samples are generated
        and the returned map translates real ids to rows of the small cache."""
        s = self.spec
        if self.cache_np is not None:
            cache, remap = self.cache_np, None
            labels = self.labels_np
        else:
            uni = sorted(set(int(i) for i in ids_universe))
            cache = pi.cache_samples(s, self.seed, uni, "cpu").float().numpy()
            remap = {g: i for i, g in enumerate(uni)}
            labels = self.labels_np[uni]
        tr = po.Trainer(cache, labels, self.oracle_params(flat), act, self.lm_np, hp or po.AdamW())
        return tr, remap


def block_slices(spec: pi.CacheSpec):
    L, d, r, C = spec.L, spec.d, spec.r, spec.n_out
    out, o = {}, 0
    for name, k in [("W_down", L * d * r), ("lam", L), ("W_up", r * d)] + \
                   ([("W_head", d * C), ("b_head", C)] if spec.head == "cls" else []):
        out[name] = slice(o, o + k)
        o += k
    return out
