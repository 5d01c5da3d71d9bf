"""ctypes binding of libfda (see include/fda.h for the contract of every call).

The functions keep the names of the C entry points (``fda_local_state`` ...) as methods of
:class:`FdaContext`; they pass ``tensor.data_ptr()`` and the current torch stream through and
do nothing else.  There is no fallback: if the shared library is missing or a call fails,
an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

FDA_STATE_NORM, FDA_STATE_LINEAR, FDA_STATE_SKETCH = 1, 2, 4
FDA_VARIANT_LINEAR, FDA_VARIANT_SKETCH = 0, 1
FDA_AVG_BROADCAST, FDA_AVG_UNCONDITIONAL = 1, 2
FDA_MAX_ROWS = 16

_STATUS = {0: "FDA_OK", 1: "FDA_ERR_INVALID_ARG", 2: "FDA_ERR_UNSUPPORTED", 3: "FDA_ERR_CUDA",
           4: "FDA_ERR_NOMEM"}

EXPORTS = ("fda_create", "fda_create_limited", "fda_context_info", "fda_destroy", "fda_state_len", "fda_last_error", "fda_local_state", "fda_mean_state",
           "fda_combine_estimate", "fda_average_models", "fda_average_models_xi", "fda_round_host", "fda_debug_hash", "fda_debug_read_probe", "fda_debug_last_kernel", "fda_debug_last_launches", "fda_debug_schedule",
           "fda_local_state_linear_noalloc")
FDA_NOALLOC_MAX_WORKERS = 64


class FdaError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__("%s failed with %s%s" % (where, _STATUS.get(status, status),
                                                   (": " + detail) if detail else ""))


class Estimate(ctypes.Structure):
    """Mirror of ``fda_estimate``."""
    _fields_ = [("mean_sq_norm", ctypes.c_float), ("est_sq_norm_of_mean", ctypes.c_float),
                ("H", ctypes.c_float), ("theta", ctypes.c_float), ("trigger", ctypes.c_int32),
                ("l", ctypes.c_int32), ("row_sq_norm", ctypes.c_float * FDA_MAX_ROWS)]

    def as_dict(self):
        return {"mean_sq": self.mean_sq_norm, "est": self.est_sq_norm_of_mean, "H": self.H,
                "theta": self.theta, "trigger": bool(self.trigger),
                "rows": np.array(self.row_sq_norm[:self.l], dtype=np.float32)}


_lib = None


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libfda.so")


def load_library():
    """Load libfda.so from the package directory (never from anywhere else)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise FdaError(3, "load_library", "%s not found - run `python -m paper_2405_20988_b200.build`" % path)
    lib = ctypes.CDLL(path)
    vp, i64, c_int, u32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint32, ctypes.c_float
    lib.fda_create.argtypes = [ctypes.POINTER(vp), c_int, c_int, c_int, vp, i64, c_int]
    lib.fda_create_limited.argtypes = [ctypes.POINTER(vp), c_int, c_int, c_int, vp, i64, c_int, i64]
    lib.fda_create_limited.restype = c_int
    lib.fda_context_info.argtypes = [vp, vp]
    lib.fda_context_info.restype = c_int
    lib.fda_destroy.argtypes = [vp]
    lib.fda_state_len.argtypes = [vp]
    lib.fda_state_len.restype = ctypes.c_size_t
    lib.fda_last_error.argtypes = [vp]
    lib.fda_last_error.restype = ctypes.c_char_p
    lib.fda_local_state.argtypes = [vp, vp, i64, c_int, i64, vp, vp, u32, vp, vp]
    lib.fda_mean_state.argtypes = [vp, vp, i64, c_int, i64, vp, vp, u32, vp, vp]
    lib.fda_mean_state.restype = c_int
    lib.fda_combine_estimate.argtypes = [vp, vp, c_int, c_int, f32, f32, vp, vp, vp]
    lib.fda_average_models.argtypes = [vp, vp, i64, c_int, i64, vp, vp, u32, vp]
    lib.fda_average_models_xi.argtypes = [vp, vp, i64, c_int, i64, vp, vp, vp, u32, vp]
    lib.fda_average_models_xi.restype = c_int
    lib.fda_round_host.argtypes = [vp, vp, i64, c_int, i64, vp, vp, u32, c_int, f32, f32, u32, vp, vp, vp]
    lib.fda_debug_hash.argtypes = [vp, i64, i64, vp, vp, vp]
    lib.fda_debug_read_probe.argtypes = [vp, vp, i64, vp, vp]
    lib.fda_debug_read_probe.restype = c_int
    lib.fda_debug_schedule.argtypes = [vp, i64, vp, ctypes.c_size_t, vp]
    lib.fda_debug_schedule.restype = c_int
    lib.fda_debug_last_kernel.argtypes = [vp]
    lib.fda_debug_last_kernel.restype = ctypes.c_char_p
    lib.fda_debug_last_launches.argtypes = [vp]
    lib.fda_debug_last_launches.restype = ctypes.c_int
    lib.fda_local_state_linear_noalloc.argtypes = [c_int, vp, i64, c_int, i64, vp, vp, u32, vp, vp]
    lib.fda_local_state_linear_noalloc.restype = c_int
    for name in ("fda_create", "fda_destroy", "fda_local_state", "fda_combine_estimate",
                 "fda_average_models", "fda_round_host", "fda_debug_hash"):
        getattr(lib, name).restype = c_int
    _lib = lib
    return lib


def _dev_ptr(t, dtype=None, name="tensor"):
    """Device pointer of a CUDA torch tensor (None passes NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must have dtype %s" % (name, dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _rows(w, name="w"):
    """(pointer, row_stride, K, d) of a 2-D float32 tensor/array whose rows are contiguous."""
    if w.dim() != 2 or (w.shape[1] > 1 and w.stride(1) != 1):
        raise ValueError("%s must be 2-D with contiguous rows" % name)
    K, d = w.shape
    stride = w.stride(0) if K > 1 else max(w.stride(0), d)
    return stride, K, d


def fda_local_state_linear_noalloc(w, w_t0, xi, flags: int, states, stream=None):
    """states[K, 2] <- (||u_k||^2, <xi,u_k>) of the K rows of ``w`` without a context.

    For code that must not allocate device memory when it runs (for instance a hook inside a
    training step, where the framework's allocator already holds all free memory): the C
    entry point of the same name keeps its scratch in a fixed array inside the library and
    this wrapper creates no tensor either - ``states`` is supplied by the caller.  K may not
    exceed FDA_NOALLOC_MAX_WORKERS.  Calls that overlap on the device race on that scratch.
    """
    import torch
    lib = load_library()
    stride, K, d = _rows(w)
    if states.dim() != 2 or states.shape[0] != K or states.shape[1] != 2 or not states.is_contiguous():
        raise ValueError("states must be a contiguous K x 2 tensor")
    st = lib.fda_local_state_linear_noalloc(w.device.index or 0, _dev_ptr(w, torch.float32, "w"), stride, K, d,
                                            _dev_ptr(w_t0, torch.float32, "w_t0"),
                                            _dev_ptr(xi, torch.float32, "xi"), flags,
                                            _dev_ptr(states, torch.float32, "states"), _stream_ptr(stream))
    if st != 0:
        raise FdaError(st, "fda_local_state_linear_noalloc",
                       "K exceeds FDA_NOALLOC_MAX_WORKERS" if st == 2 else "")


class FdaContext:
    """Owner of an ``fda_ctx``.  Methods mirror the C entry points one to one."""

    def __init__(self, l: int, m: int, hash_coeffs, d_max: int, K_max: int, device: int = 0,
                 schedule_limit_bytes: int | None = None):
        """``schedule_limit_bytes``: None calls ``fda_create``; a number calls ``fda_create_limited``."""
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        coeffs = None
        if l > 0:
            coeffs = np.ascontiguousarray(hash_coeffs, dtype=np.uint64).reshape(-1)
            if coeffs.size != 6 * l:
                raise ValueError("hash_coeffs must hold 6*l values")
        self._coeffs = coeffs
        ptr = coeffs.ctypes.data_as(ctypes.c_void_p) if coeffs is not None else None
        if schedule_limit_bytes is None:
            st = self._lib.fda_create(ctypes.byref(self._h), device, l, m, ptr, d_max, K_max)
        else:
            st = self._lib.fda_create_limited(ctypes.byref(self._h), device, l, m, ptr, d_max, K_max,
                                              int(schedule_limit_bytes))
        if st != 0:
            self._h = ctypes.c_void_p()
            raise FdaError(st, "fda_create")
        self.l, self.m, self.d_max, self.K_max, self.device = l, m if l > 0 else 0, d_max, K_max, device

    # -- helpers ---------------------------------------------------------------------------
    def _check(self, st: int, where: str):
        if st != 0:
            raise FdaError(st, where, self._lib.fda_last_error(self._h).decode())

    @property
    def state_len(self) -> int:
        return int(self._lib.fda_state_len(self._h))

    def fda_last_error(self) -> str:
        return self._lib.fda_last_error(self._h).decode()

    def fda_context_info(self) -> dict:
        """What the context holds: see ``fda_context_info`` in include/fda.h."""
        info = (ctypes.c_int64 * 8)()
        self._check(self._lib.fda_context_info(self._h, info), "fda_context_info")
        keys = ("device_bytes", "schedule_bytes", "list_kernel", "tile_indices", "schedule_dropped_bytes",
                "table_bytes", "schedule_build_us", "other_lazy_bytes")
        return dict(zip(keys, (int(v) for v in info)))

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.fda_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- the C entry points ----------------------------------------------------------------
    def fda_local_state(self, w, w_t0, xi, flags: int, states, stream=None):
        """states[K, state_len] <- local states of the K rows of w (device tensors)."""
        import torch
        stride, K, d = _rows(w)
        st = self._lib.fda_local_state(self._h, _dev_ptr(w, torch.float32, "w"), stride, K, d,
                                       _dev_ptr(w_t0, torch.float32, "w_t0"),
                                       _dev_ptr(xi, torch.float32, "xi"), flags,
                                       _dev_ptr(states, torch.float32, "states"), _stream_ptr(stream))
        self._check(st, "fda_local_state")

    def fda_mean_state(self, w, w_t0, xi, flags: int, mean_state, stream=None):
        """mean_state[state_len] <- averaged state S-bar of the K rows of w (device tensors)."""
        import torch
        stride, K, d = _rows(w)
        st = self._lib.fda_mean_state(self._h, _dev_ptr(w, torch.float32, "w"), stride, K, d,
                                      _dev_ptr(w_t0, torch.float32, "w_t0"),
                                      _dev_ptr(xi, torch.float32, "xi"), flags,
                                      _dev_ptr(mean_state, torch.float32, "mean_state"), _stream_ptr(stream))
        self._check(st, "fda_mean_state")

    def fda_combine_estimate(self, states, K: int, variant: int, epsilon: float, theta: float,
                             est_dev, want_host: bool = True, stream=None):
        """est_dev: uint8 CUDA tensor of sizeof(fda_estimate) bytes.  Returns an Estimate
        (host copy, synchronises the stream) when ``want_host``, else None."""
        import torch
        host = Estimate() if want_host else None
        st = self._lib.fda_combine_estimate(self._h, _dev_ptr(states, torch.float32, "states"), K,
                                            variant, epsilon, theta, _dev_ptr(est_dev, torch.uint8, "est_dev"),
                                            ctypes.byref(host) if host is not None else None,
                                            _stream_ptr(stream))
        self._check(st, "fda_combine_estimate")
        return host

    def fda_average_models(self, w, w_t0, est_dev, flags: int, stream=None):
        import torch
        stride, K, d = _rows(w)
        st = self._lib.fda_average_models(self._h, _dev_ptr(w, torch.float32, "w"), stride, K, d,
                                          _dev_ptr(w_t0, torch.float32, "w_t0"),
                                          _dev_ptr(est_dev, torch.uint8, "est_dev"), flags,
                                          _stream_ptr(stream))
        self._check(st, "fda_average_models")

    def fda_average_models_xi(self, w, w_t0, xi_out, est_dev, flags: int, stream=None):
        """fda_average_models that also writes the refreshed unit direction xi_out (d floats)."""
        import torch
        stride, K, d = _rows(w)
        st = self._lib.fda_average_models_xi(self._h, _dev_ptr(w, torch.float32, "w"), stride, K, d,
                                             _dev_ptr(w_t0, torch.float32, "w_t0"),
                                             _dev_ptr(xi_out, torch.float32, "xi_out"),
                                             _dev_ptr(est_dev, torch.uint8, "est_dev"), flags,
                                             _stream_ptr(stream))
        self._check(st, "fda_average_models_xi")

    def fda_round_host(self, w_host, w_t0_host, xi_host, state_flags: int, variant: int,
                       epsilon: float, theta: float, avg_flags: int, states_host=None, stream=None):
        """Whole round on HOST tensors (CPU torch tensors, ideally pinned).  Returns Estimate."""
        stride, K, d = _rows(w_host, "w_host")
        est = Estimate()

        def hp(t):
            return None if t is None else ctypes.c_void_p(t.data_ptr())

        st = self._lib.fda_round_host(self._h, hp(w_host), stride, K, d, hp(w_t0_host), hp(xi_host),
                                      state_flags, variant, epsilon, theta, avg_flags,
                                      hp(states_host), ctypes.byref(est), _stream_ptr(stream))
        self._check(st, "fda_round_host")
        return est

    def fda_debug_hash(self, j0: int, n: int, buckets, signs, stream=None):
        """buckets: uint16[l, n] (torch.int16 storage is accepted), signs: int8[l, n]."""
        st = self._lib.fda_debug_hash(self._h, j0, n, ctypes.c_void_p(buckets.data_ptr()),
                                      ctypes.c_void_p(signs.data_ptr()), _stream_ptr(stream))
        self._check(st, "fda_debug_hash")

    def fda_debug_read_probe(self, src, sum_out, stream=None):
        """src: float32 CUDA tensor (contiguous); sum_out: float32[1] CUDA tensor."""
        if not src.is_contiguous():
            raise ValueError("src must be contiguous")
        st = self._lib.fda_debug_read_probe(self._h, _dev_ptr(src, name="src"), src.numel(),
                                            _dev_ptr(sum_out, name="sum_out"), _stream_ptr(stream))
        self._check(st, "fda_debug_read_probe")

    def fda_debug_schedule(self, tile: int):
        """(record bytes as a numpy uint8 array, info dict) of the list schedule's record of a tile."""
        info = (ctypes.c_int64 * 8)()
        probe = (ctypes.c_uint8 * 16)()
        st = self._lib.fda_debug_schedule(self._h, tile, probe, 16, info)
        self._check(st, "fda_debug_schedule")
        buf = np.zeros(int(info[3]), dtype=np.uint8)
        st = self._lib.fda_debug_schedule(self._h, tile, buf.ctypes.data_as(ctypes.c_void_p), buf.size, info)
        self._check(st, "fda_debug_schedule")
        keys = ("tile_indices", "slots", "max_len", "record_bytes", "tiles", "pad_rows", "lanes_per_pass",
                "schedule_bytes")
        return buf, dict(zip(keys, (int(v) for v in info)))

    def fda_debug_last_kernel(self) -> str:
        """Name of the kernel that served the last fda_local_state call on this context."""
        return self._lib.fda_debug_last_kernel(self._h).decode()

    def fda_debug_last_launches(self) -> int:
        """Kernels that the last fda_local_state call on this context launched."""
        return int(self._lib.fda_debug_last_launches(self._h))

    @staticmethod
    def new_estimate_buffer(device="cuda"):
        import torch
        return torch.zeros(ctypes.sizeof(Estimate), dtype=torch.uint8, device=device)
