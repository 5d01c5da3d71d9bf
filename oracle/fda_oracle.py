"""ctypes wrapper around the C oracle (``fda_oracle.c``).  Test infrastructure only.

Each function marshals numpy arrays into the C routine of the same purpose and returns
fp64 results.  The arithmetic lives in the C file; this module holds none.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

P61 = (1 << 61) - 1  # the prime field of the hash family

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fda_oracle.c")
_LIB = os.path.join(_HERE, "libfda_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, no fast-math) if it is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=gnu11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_i64, c_int, c_dbl = ctypes.c_int64, ctypes.c_int, ctypes.c_double
        vp = ctypes.c_void_p
        lib.fda_oracle_hash.argtypes = [vp, c_int, c_int, c_i64, c_i64, vp, vp]
        lib.fda_oracle_local_state.argtypes = [vp, c_i64, c_int, c_i64, vp, vp, vp, c_int,
                                               c_int, c_int, c_int, vp]
        lib.fda_oracle_combine.argtypes = [vp, c_int, c_int, c_int, c_int, c_dbl, c_dbl, vp]
        lib.fda_oracle_average.argtypes = [vp, c_i64, c_int, c_i64, c_i64, c_i64, vp]
        lib.fda_oracle_variance.argtypes = [vp, c_i64, c_int, c_i64, vp, vp]
        lib.fda_oracle_direction.argtypes = [vp, vp, c_i64, vp]
        lib.fda_oracle_direction.restype = c_int
        for f in (lib.fda_oracle_hash, lib.fda_oracle_local_state, lib.fda_oracle_combine,
                  lib.fda_oracle_average, lib.fda_oracle_variance):
            f.restype = c_int
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32_rows(w):
    w = np.asarray(w)
    if w.dtype != np.float32 or w.ndim != 2:
        raise ValueError("w must be a 2-D float32 array")
    if w.shape[0] == 1:                      # a single row has no meaningful pitch
        w = np.ascontiguousarray(w)
        return w, w.shape[1]
    if w.strides[1] != 4 or w.strides[0] % 4:
        raise ValueError("w must have contiguous rows")
    return w, w.strides[0] // 4


def _f32_vec(v, d, name):
    if v is None:
        return None
    v = np.ascontiguousarray(v, dtype=np.float32)
    if v.shape != (d,):
        raise ValueError("%s must have shape (d,)" % name)
    return v


def _coeffs(coeffs, l):
    c = np.ascontiguousarray(coeffs, dtype=np.uint64).reshape(-1)
    if c.size != 6 * l:
        raise ValueError("coefficient table must hold 6*l values")
    return c


def state_len(l: int, m: int) -> int:
    return 2 + l * m


def hash_dump(coeffs, l: int, m: int, j0: int, n: int):
    """(buckets[l, n] int32, signs[l, n] int8) for indices j0 .. j0+n-1."""
    c = _coeffs(coeffs, l)
    b = np.empty((l, n), dtype=np.int32)
    s = np.empty((l, n), dtype=np.int8)
    rc = _load().fda_oracle_hash(_ptr(c), l, m, j0, n, _ptr(b), _ptr(s))
    if rc:
        raise ValueError("fda_oracle_hash rejected its arguments")
    return b, s


def local_state(w, w_t0, xi, coeffs, l: int, m: int, workers=None, threads: int = 1):
    """fp64 local states, shape (K, 2 + l*m).  ``w`` is (K, d) float32 (rows may be padded:
    pass a view ``buf[:, :d]``).  ``workers`` restricts the computation to some rows (the
    others stay NaN); ``threads`` runs that many workers at a time, each single-threaded.
    """
    w, stride = _f32_rows(w)
    K, d = w.shape
    w_t0 = _f32_vec(w_t0, d, "w_t0")
    xi = _f32_vec(xi, d, "xi")
    c = _coeffs(coeffs, l) if l > 0 else None
    states = np.full((K, state_len(l, m)), np.nan, dtype=np.float64)
    ks = list(range(K)) if workers is None else [int(k) for k in workers]
    lib = _load()

    def one(k):
        rc = lib.fda_oracle_local_state(_ptr(w), stride, K, d, _ptr(w_t0), _ptr(xi), _ptr(c),
                                        l, m, k, k + 1, _ptr(states))
        if rc:
            raise ValueError("fda_oracle_local_state rejected its arguments")

    if threads <= 1 or len(ks) <= 1:
        for k in ks:
            one(k)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, ks))
    return states


def combine(states, l: int, m: int, variant: int, epsilon: float, theta: float):
    """dict(mean_sq, est, H, trigger, rows) from a (K, 2 + l*m) array of states."""
    s = np.ascontiguousarray(states, dtype=np.float64)
    if s.ndim != 2 or s.shape[1] != state_len(l, m):
        raise ValueError("states must have shape (K, 2 + l*m)")
    out = np.zeros(4 + max(l, 0), dtype=np.float64)
    rc = _load().fda_oracle_combine(_ptr(s), s.shape[0], l, m, variant, float(epsilon),
                                    float(theta), _ptr(out))
    if rc:
        raise ValueError("fda_oracle_combine rejected its arguments")
    return {"mean_sq": out[0], "est": out[1], "H": out[2], "trigger": bool(out[3]),
            "rows": out[4:4 + l].copy()}


def average(w, j_begin: int = 0, j_end: int | None = None):
    """fp64 average model over the K rows of ``w`` for indices [j_begin, j_end)."""
    w, stride = _f32_rows(w)
    K, d = w.shape
    j_end = d if j_end is None else j_end
    out = np.empty(j_end - j_begin, dtype=np.float64)
    rc = _load().fda_oracle_average(_ptr(w), stride, K, d, j_begin, j_end, _ptr(out))
    if rc:
        raise ValueError("fda_oracle_average rejected its arguments")
    return out


def variance(w, w_t0):
    """(Var by Eq. 2, mean_k ||u_k||^2, ||u-bar||^2) in fp64 by brute force."""
    w, stride = _f32_rows(w)
    K, d = w.shape
    w_t0 = _f32_vec(w_t0, d, "w_t0")
    out = np.zeros(3, dtype=np.float64)
    rc = _load().fda_oracle_variance(_ptr(w), stride, K, d, _ptr(w_t0), _ptr(out))
    if rc:
        raise ValueError("fda_oracle_variance rejected its arguments")
    return float(out[0]), float(out[1]), float(out[2])


def direction(w_new, w_old):
    """Unit direction of the global step, (w_new - w_old)/||.||, in fp64 (zero step -> zeros)."""
    w_new = np.ascontiguousarray(w_new, dtype=np.float64)
    w_old = np.ascontiguousarray(w_old, dtype=np.float32)
    if w_new.shape != w_old.shape or w_new.ndim != 1:
        raise ValueError("w_new and w_old must be vectors of equal length")
    out = np.empty_like(w_new)
    rc = _load().fda_oracle_direction(_ptr(w_new), _ptr(w_old), w_new.size, _ptr(out))
    if rc:
        raise ValueError("fda_oracle_direction rejected its arguments")
    return out
