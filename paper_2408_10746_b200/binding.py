"""ctypes binding of the C ABI in include/pac.h: argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  There is no CPU
fallback: if libpac_b200.so is missing or no CUDA device is usable, loading or
pac_create fails loudly.  torch is used only to own device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import Optional, Sequence

import numpy as np

PAC_F32, PAC_BF16 = 0, 1
PAC_ACT_RELU, PAC_ACT_IDENTITY = 0, 1
PAC_HEAD_MEANPOOL_CLS, PAC_HEAD_FROZEN_LM = 0, 1
PAC_BODY_POINTWISE, PAC_BODY_TRANSFORMER = 0, 1
PAC_OPT_KERNEL_PATH = 0
PAC_OPT_KERNEL_TIMING = 1
STATUS_NAMES = ["PAC_OK", "PAC_ERR_INVALID_ARG", "PAC_ERR_BAD_STATE", "PAC_ERR_SAMPLE_ID_RANGE",
                "PAC_ERR_UNSUPPORTED", "PAC_ERR_NOMEM", "PAC_ERR_CUDA", "PAC_ERR_TIMEOUT"]

# every symbol include/pac.h declares
EXPORTS = ["pac_create", "pac_destroy", "pac_cache_register", "pac_cache_register_host", "pac_cache_register_file",
           "pac_cache_writer_create", "pac_cache_writer_store", "pac_cache_writer_close", "pac_cache_file_info", "pac_adapter_init", "pac_train_step", "pac_train_step_dev_loss", "pac_set_grad_scale", "pac_train_step_async",
           "pac_adam_step", "pac_eval_logits", "pac_gather", "pac_train_epoch", "pac_train_epoch_dev",
           "pac_param_count", "pac_get_params", "pac_set_params", "pac_get_grads", "pac_get_opt_state",
           "pac_set_opt_state", "pac_set_option", "pac_device_buffers", "pac_params_changed", "pac_kernel_times", "pac_stream_phase_times", "pac_launch_count", "pac_sync", "pac_selftest_wait_expiry", "pac_last_error",
           "pac_kernel_path", "pac_eval_logits_static", "pac_quantize_absmax", "pac_dequantize_absmax"]


class PacError(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = status
        self.status_name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{self.status_name}: {message}")


class _AdapterCfg(C.Structure):
    _fields_ = [("r", C.c_int), ("act", C.c_int), ("head", C.c_int), ("n_out", C.c_int),
                ("lambda_init", C.c_float), ("max_batch", C.c_int), ("lm_head", C.c_void_p),
                ("body", C.c_int), ("n_heads", C.c_int), ("ffn_width", C.c_int)]


class _AdamW(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float)]


@dataclasses.dataclass
class AdamW:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01

    def _c(self) -> _AdamW:
        return _AdamW(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay)


_LIB: Optional[C.CDLL] = None


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpac_b200.so")


def load_library() -> C.CDLL:
    """Loads libpac_b200.so (built by `python -m paper_2408_10746_b200.build`)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2408_10746_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(path)
    P, I, LL, F = C.c_void_p, C.c_int, C.c_longlong, C.c_float
    sig = {
        "pac_create": [C.POINTER(P), I, P], "pac_destroy": [P],
        "pac_cache_register": [P, P, I, LL, I, I, I, P, I],
        "pac_cache_register_host": [P, P, I, LL, I, I, I, P, I],
        "pac_adapter_init": [P, C.POINTER(_AdapterCfg), C.c_ulonglong],
        "pac_train_step": [P, P, I, C.POINTER(F)], "pac_train_step_async": [P, P, I, C.POINTER(_AdamW), P], "pac_adam_step": [P, C.POINTER(_AdamW)],
        "pac_eval_logits": [P, P, I, P], "pac_gather": [P, P, I, P],
        "pac_train_epoch": [P, P, LL, I, C.POINTER(_AdamW), P],
        "pac_train_epoch_dev": [P, P, LL, I, C.POINTER(_AdamW), P],
        "pac_param_count": [P, C.POINTER(LL)], "pac_get_params": [P, P], "pac_set_params": [P, P],
        "pac_get_grads": [P, P], "pac_get_opt_state": [P, P, P, C.POINTER(LL)],
        "pac_set_opt_state": [P, P, P, LL], "pac_set_option": [P, I, I],
        "pac_launch_count": [P, C.POINTER(LL)], "pac_sync": [P],
        "pac_kernel_times": [P, C.POINTER(C.c_double), C.POINTER(LL)],
        "pac_stream_phase_times": [P, C.POINTER(C.c_double), C.POINTER(LL)],
        "pac_device_buffers": [P, C.POINTER(P), C.POINTER(P)], "pac_params_changed": [P],
        "pac_selftest_wait_expiry": [P, C.c_ulonglong],
        "pac_train_step_dev_loss": [P, P, I, P], "pac_set_grad_scale": [P, F],
        "pac_cache_register_file": [P, C.c_char_p],
        "pac_cache_writer_create": [C.POINTER(P), C.c_char_p, I, LL, I, I, I, I],
        "pac_cache_writer_store": [P, LL, P, I, P, P], "pac_cache_writer_close": [P],
        "pac_cache_file_info": [C.c_char_p, C.POINTER(I), C.POINTER(LL), C.POINTER(I), C.POINTER(I), C.POINTER(I), C.POINTER(I)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = I
    lib.pac_eval_logits_static.argtypes = [I, P, P, I, LL, I, I, I, P, I, I, I, P, I, P, C.c_char_p, I]
    lib.pac_eval_logits_static.restype = I
    lib.pac_quantize_absmax.argtypes = [I, P, P, LL, I, P, P]
    lib.pac_quantize_absmax.restype = I
    lib.pac_dequantize_absmax.argtypes = [I, P, P, P, LL, I, P]
    lib.pac_dequantize_absmax.restype = I
    lib.pac_last_error.argtypes = [P]
    lib.pac_last_error.restype = C.c_char_p
    lib.pac_kernel_path.argtypes = [P]
    lib.pac_kernel_path.restype = C.c_char_p
    _LIB = lib
    return lib


def _ids(ids: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(ids, dtype=np.int32).reshape(-1))


def _ptr(t) -> int:
    """Device (torch tensor) or host (numpy array) address."""
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


class PacContext:
    """One trainer context on one GPU.  Methods mirror the C calls one to one."""

    def __init__(self, device: int = 0, stream: Optional[int] = None):
        self._lib = load_library()
        h = C.c_void_p()
        st = self._lib.pac_create(C.byref(h), device, C.c_void_p(stream) if stream else None)
        if st != 0:
            raise PacError(st, "pac_create failed (is a CUDA device visible? there is no CPU fallback)")
        self._h = h
        self._keep = []          # borrowed tensors must outlive the context

    def _ck(self, st: int):
        if st != 0:
            raise PacError(st, self._lib.pac_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self._lib.pac_destroy(self._h)
            self._h = None
            self._keep = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- the calls -----------------------------------------------------------
    def cache_register(self, cache, labels):
        """cache: CUDA tensor [N][L][S][d] (float32 or bfloat16); labels: CUDA int32 [N] or [N][S]."""
        import torch
        assert cache.is_cuda and labels.is_cuda and cache.is_contiguous() and labels.is_contiguous()
        assert labels.dtype == torch.int32
        N, L, S, d = cache.shape
        dt = {torch.float32: PAC_F32, torch.bfloat16: PAC_BF16}[cache.dtype]
        per = 1 if labels.dim() == 1 else labels.shape[1]
        self._ck(self._lib.pac_cache_register(self._h, cache.data_ptr(), dt, N, L, S, d, labels.data_ptr(), per))
        self._keep += [cache, labels]
        self.shape = (N, L, S, d)
        self.cache_dtype = cache.dtype

    def cache_register_host(self, cache, labels):
        """cache: CPU tensor [N][L][S][d] (float32 or bfloat16), ideally page-locked; labels: CPU int32
        [N] or [N][S].  The cache stays in host memory; every step reloads its minibatch."""
        import torch
        assert not cache.is_cuda and not labels.is_cuda and cache.is_contiguous() and labels.is_contiguous()
        assert labels.dtype == torch.int32
        N, L, S, d = cache.shape
        dt = {torch.float32: PAC_F32, torch.bfloat16: PAC_BF16}[cache.dtype]
        per = 1 if labels.dim() == 1 else labels.shape[1]
        self._ck(self._lib.pac_cache_register_host(self._h, cache.data_ptr(), dt, N, L, S, d, labels.data_ptr(), per))
        self._keep += [cache, labels]
        self.shape = (N, L, S, d)
        self.cache_dtype = cache.dtype

    def cache_register_file(self, path: str):
        """A cache file written by CacheWriter: mapped read-only and reloaded per minibatch."""
        import torch
        dt, N, L, S, d, per = cache_file_info(path)
        self._ck(self._lib.pac_cache_register_file(self._h, path.encode()))
        self.shape = (N, L, S, d)
        self.cache_dtype = {PAC_F32: torch.float32, PAC_BF16: torch.bfloat16}[dt]

    def adapter_init(self, r: int, n_out: int, max_batch: int, act: int = PAC_ACT_RELU,
                     head: int = PAC_HEAD_MEANPOOL_CLS, lambda_init: float = 0.5, lm_head=None, seed: int = 1,
                     body: int = 0, n_heads: int = 0, ffn_width: int = 0):
        """body = 1 (PAC_BODY_TRANSFORMER): every adapter is a width-r transformer layer with n_heads
        attention heads and a feed-forward layer of ffn_width."""
        cfg = _AdapterCfg(r, act, head, n_out, lambda_init, max_batch, lm_head.data_ptr() if lm_head is not None else None,
                          body, n_heads, ffn_width)
        self._ck(self._lib.pac_adapter_init(self._h, C.byref(cfg), seed))
        if lm_head is not None:
            self._keep.append(lm_head)
        self.r, self.n_out, self.head = r, n_out, head

    def set_option(self, option: int, value: int):
        self._ck(self._lib.pac_set_option(self._h, option, value))

    def train_step(self, sample_ids, want_loss: bool = True) -> Optional[float]:
        ids = _ids(sample_ids)
        loss = C.c_float()
        self._ck(self._lib.pac_train_step(self._h, ids.ctypes.data, ids.size, C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def train_step_dev_loss(self, sample_ids, dev_loss_ptr: int = 0):
        """Enqueues forward + backward of one minibatch and returns at once; the mean loss goes to the
        device float at dev_loss_ptr (0: kept inside the context)."""
        ids = _ids(sample_ids)
        st = self._lib.pac_train_step_dev_loss(self._h, ids.ctypes.data, ids.size, dev_loss_ptr or None)
        if st != 0:
            self._ck(st)

    def set_grad_scale(self, scale: float):
        self._ck(self._lib.pac_set_grad_scale(self._h, scale))

    def train_step_async(self, sample_ids, hp: AdamW, loss_out_ptr: int = 0):
        """Enqueues one whole step (forward, backward, AdamW) and returns at once.  loss_out_ptr: address
        of one host float (page-locked for a truly asynchronous copy) that receives the loss, or 0."""
        ids = _ids(sample_ids)
        if getattr(self, "_hp_src", None) is not hp:                   # marshal the hyper-parameters once per object
            self._hp_src, self._hp_c = hp, hp._c()
        st = self._lib.pac_train_step_async(self._h, ids.ctypes.data, ids.size, self._hp_c, loss_out_ptr or None)
        if st != 0:
            self._ck(st)

    def adam_step(self, hp: AdamW):
        self._ck(self._lib.pac_adam_step(self._h, C.byref(hp._c())))

    def eval_logits(self, sample_ids, out):
        ids = _ids(sample_ids)
        self._ck(self._lib.pac_eval_logits(self._h, ids.ctypes.data, ids.size, out.data_ptr()))
        return out

    def gather(self, sample_ids, out):
        ids = _ids(sample_ids)
        self._ck(self._lib.pac_gather(self._h, ids.ctypes.data, ids.size, out.data_ptr()))
        return out

    def train_epoch(self, perm, B: int, hp: AdamW, want_losses: bool = True, losses_out: Optional[np.ndarray] = None):
        """perm: host int32 ids (n a multiple of B).  losses_out: optional host float32 array of n/B
        entries to receive the losses (e.g. a view of pinned memory); otherwise one is allocated."""
        ids = _ids(perm)
        losses = None
        if want_losses:
            losses = losses_out if losses_out is not None else np.empty(max(1, ids.size // max(B, 1)), dtype=np.float32)
            assert losses.dtype == np.float32 and losses.size >= ids.size // max(B, 1)
        self._ck(self._lib.pac_train_epoch(self._h, ids.ctypes.data, ids.size, B, C.byref(hp._c()),
                                           losses.ctypes.data if want_losses else None))
        return losses

    def train_epoch_dev(self, dev_perm, B: int, hp: AdamW, dev_losses=None):
        self._ck(self._lib.pac_train_epoch_dev(self._h, dev_perm.data_ptr(), dev_perm.numel(), B, C.byref(hp._c()),
                                               dev_losses.data_ptr() if dev_losses is not None else None))

    def param_count(self) -> int:
        n = C.c_longlong()
        self._ck(self._lib.pac_param_count(self._h, C.byref(n)))
        return n.value

    def get_params(self) -> np.ndarray:
        out = np.empty(self.param_count(), dtype=np.float32)
        self._ck(self._lib.pac_get_params(self._h, out.ctypes.data))
        return out

    def set_params(self, flat: np.ndarray):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        assert flat.size == self.param_count()
        self._ck(self._lib.pac_set_params(self._h, flat.ctypes.data))

    def get_grads(self) -> np.ndarray:
        out = np.empty(self.param_count(), dtype=np.float32)
        self._ck(self._lib.pac_get_grads(self._h, out.ctypes.data))
        return out

    def get_opt_state(self):
        n = self.param_count()
        m, v, step = np.empty(n, np.float32), np.empty(n, np.float32), C.c_longlong()
        self._ck(self._lib.pac_get_opt_state(self._h, m.ctypes.data, v.ctypes.data, C.byref(step)))
        return m, v, step.value

    def set_opt_state(self, m: np.ndarray, v: np.ndarray, step: int):
        m = np.ascontiguousarray(m, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        self._ck(self._lib.pac_set_opt_state(self._h, m.ctypes.data, v.ctypes.data, step))

    def kernel_times(self):
        """(ms_total, launches) per kernel group of the train step since the last call."""
        ms = (C.c_double * 4)()
        cnt = (C.c_longlong * 4)()
        self._ck(self._lib.pac_kernel_times(self._h, ms, cnt))
        names = ["down_projection", "chain_head", "dw_down", "finalize"]
        return {n: (ms[i], cnt[i]) for i, n in enumerate(names)}

    def stream_phase_times(self):
        """(ms_total, launches) of the two cache passes' stream phases (device timestamps) since the last call."""
        ms = (C.c_double * 2)()
        cnt = (C.c_longlong * 2)()
        self._ck(self._lib.pac_stream_phase_times(self._h, ms, cnt))
        return {"first_pass": (ms[0], cnt[0]), "second_pass": (ms[1], cnt[1])}

    def device_buffers(self):
        """Zero-copy torch views (CUDA, fp32) of the context's parameter and gradient vectors."""
        import torch
        pp, gp = C.c_void_p(), C.c_void_p()
        self._ck(self._lib.pac_device_buffers(self._h, C.byref(pp), C.byref(gp)))
        n = self.param_count()

        class _View:
            def __init__(self, ptr):
                self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<f4", "data": (ptr, False), "version": 2}

        return torch.as_tensor(_View(pp.value), device="cuda"), torch.as_tensor(_View(gp.value), device="cuda")

    def params_changed(self):
        self._ck(self._lib.pac_params_changed(self._h))

    def launch_count(self) -> int:
        n = C.c_longlong()
        self._ck(self._lib.pac_launch_count(self._h, C.byref(n)))
        return n.value

    def sync(self):
        self._ck(self._lib.pac_sync(self._h))

    def selftest_wait_expiry(self, limit_ns: int = 100_000):
        """Runs the bounded-wait self-test (a wait nobody satisfies gives up after limit_ns); the next
        sync() then raises PAC_ERR_TIMEOUT once."""
        self._ck(self._lib.pac_selftest_wait_expiry(self._h, limit_ns))

    def kernel_path(self) -> str:
        return self._lib.pac_kernel_path(self._h).decode()


STATIC_SCRATCH_BYTES = 8 << 20


def cache_file_info(path: str):
    """(dtype, N, L, S, d, labels_per_sample) from a cache file's header."""
    lib = load_library()
    dt, L, S, d, per = C.c_int(), C.c_int(), C.c_int(), C.c_int(), C.c_int()
    N = C.c_longlong()
    st = lib.pac_cache_file_info(path.encode(), C.byref(dt), C.byref(N), C.byref(L), C.byref(S), C.byref(d), C.byref(per))
    if st != 0:
        raise PacError(st, f"{path} is not a complete cache file")
    return dt.value, N.value, L.value, S.value, d.value, per.value


class CacheWriter:
    """Writer side of a cache file: store(sample_id, slabs, labels) records one sample's [L][S][d]
    activations (a CUDA or CPU tensor) and its labels, in any order, as a backbone's first epoch would."""

    def __init__(self, path: str, dtype, N: int, L: int, S: int, d: int, labels_per_sample: int = 1):
        import torch
        self._lib = load_library()
        dt = {torch.float32: PAC_F32, torch.bfloat16: PAC_BF16}[dtype]
        h = C.c_void_p()
        st = self._lib.pac_cache_writer_create(C.byref(h), path.encode(), dt, N, L, S, d, labels_per_sample)
        if st != 0:
            raise PacError(st, f"pac_cache_writer_create({path}) failed")
        self._h, self.shape, self.per = h, (L, S, d), labels_per_sample

    def store(self, sample_id: int, slabs, labels, stream: Optional[int] = None):
        assert tuple(slabs.shape) == self.shape and slabs.is_contiguous()
        lab = np.ascontiguousarray(np.asarray(labels, dtype=np.int32).reshape(-1))
        assert lab.size == self.per
        st = self._lib.pac_cache_writer_store(self._h, sample_id, slabs.data_ptr(), 1 if slabs.is_cuda else 0,
                                              lab.ctypes.data, C.c_void_p(stream) if stream else None)
        if st != 0:
            raise PacError(st, f"pac_cache_writer_store(sample {sample_id}) failed")

    def close(self):
        if getattr(self, "_h", None):
            st = self._lib.pac_cache_writer_close(self._h)
            self._h = None
            if st != 0:
                raise PacError(st, "pac_cache_writer_close failed")

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def eval_logits_static(cache, dev_params, r: int, n_out: int, dev_sample_ids, out, act: int = PAC_ACT_RELU,
                       device: int = 0, stream: Optional[int] = None):
    """Classifier-head logits [B][C] without a context and without any allocation inside the
    library (pac_eval_logits_static): for callers that may not allocate device memory - an
    application that owns all of it through its own pool, a serving loop that must stay clear of the
    allocator, a plugin that only ever receives raw buffers.  Intermediates live in a fixed 8 MiB
    array inside the library, so sizes are limited (PacError PAC_ERR_UNSUPPORTED beyond that) and
    calls that overlap on the GPU must be ordered by the caller.  All tensors are CUDA tensors the
    caller owns: cache [N][L][S][d], dev_params flat fp32, dev_sample_ids int32 [B], out fp32 [B][C].
    The work is enqueued on `stream` (default stream if None)."""
    import torch
    lib = load_library()
    N, L, S, d = cache.shape
    dt = {torch.float32: PAC_F32, torch.bfloat16: PAC_BF16}[cache.dtype]
    assert dev_params.dtype == torch.float32 and dev_sample_ids.dtype == torch.int32 and out.dtype == torch.float32
    err = C.create_string_buffer(512)
    st = lib.pac_eval_logits_static(device, C.c_void_p(stream) if stream else None, cache.data_ptr(), dt, N, L, S, d,
                                    dev_params.data_ptr(), r, act, n_out, dev_sample_ids.data_ptr(),
                                    dev_sample_ids.numel(), out.data_ptr(), err, 512)
    if st != 0:
        raise PacError(st, err.value.decode())
    return out


def quantize_absmax(x, block: int, device: int = 0, stream: Optional[int] = None):
    """Block-wise absmax INT8 codes and constants of a CUDA fp32 tensor (paper Eq. 1)."""
    import torch
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    n = x.numel()
    q = torch.empty(n, dtype=torch.int8, device=x.device)
    c = torch.empty((n + block - 1) // block, dtype=torch.float32, device=x.device)
    st = load_library().pac_quantize_absmax(device, C.c_void_p(stream) if stream else None, x.data_ptr(), n, block,
                                            q.data_ptr(), c.data_ptr())
    if st != 0:
        raise PacError(st, "pac_quantize_absmax failed")
    return q, c


def dequantize_absmax(q, c, block: int, device: int = 0, stream: Optional[int] = None):
    """fp32 tensor from codes and constants (paper Eq. 2)."""
    import torch
    out = torch.empty(q.numel(), dtype=torch.float32, device=q.device)
    st = load_library().pac_dequantize_absmax(device, C.c_void_p(stream) if stream else None, q.data_ptr(), c.data_ptr(),
                                              q.numel(), block, out.data_ptr())
    if st != 0:
        raise PacError(st, "pac_dequantize_absmax failed")
    return out
