"""Seeded synthetic inputs for the FDA monitoring / averaging path.

This module only draws random numbers and lays them out in float32 buffers; it holds none
of the method's arithmetic (no drift norms, sketches, hashes, estimates or averages), so
that the CPU oracle and the CUDA library can both be fed from it without sharing any code
of the method.

Recipe.  Every item of a workload has its own counter-based stream, numpy's Philox
generator keyed by ``(seed, item)``, so any item can be regenerated on its own:

    item 0       w_t0, the last synchronised model:  N(0, 0.05^2)
    item 1       xi: standard normal vector, scaled to unit L2 norm in fp64, stored as fp32
    item 2       hash coefficients: 6 per sketch row, uniform in [0, 2^61-2] by rejection,
                 the two leading coefficients (a and c3) redrawn until non-zero
    item 3       shared drift component (drift kind "shared")
    item 4       per-worker drift scales (drift kind "scaled")
    item 16 + k  the private draws of worker k

Vectors are drawn in consecutive chunks of ``CHUNK`` elements; within a chunk a worker
draws its normals first, then (drift kind "heavy") one uniform per coordinate for the
replacement mask and one Student-t value per masked coordinate.  Model k is
``fp32(w_t0 + drift_k)`` evaluated in float32.

The five workloads mirror the parameter counts and worker counts of the models the paper
trains (LeNet-5, a small CNN, DenseNet121, DenseNet201, ConvNeXt-Large); no dataset or
trained weight is involved.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

CHUNK = 1 << 22
P61 = (1 << 61) - 1

ITEM_W_T0, ITEM_XI, ITEM_COEFFS, ITEM_SHARED, ITEM_SCALES, ITEM_WORKER0 = 0, 1, 2, 3, 4, 16


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    K: int
    l: int
    m: int
    epsilon: float
    thetas: tuple
    seed: int
    drift: str          # "iid" | "shared" | "scaled" | "heavy"
    sigma: float = 1e-3  # std of the private normal component
    note: str = ""


WORKLOADS = {
    1: Workload("lenet5", 61_706, 5, 5, 250, 0.06, (1e-4, 1e-3, 1e-2), 0, "iid", 1e-3,
                "LeNet-5-sized, iid drift"),
    2: Workload("smallcnn", 1_199_882, 10, 5, 250, 0.06, (1e-2,), 1, "shared", 1e-3,
                "small-CNN-sized, shared N(0,5e-4^2) + private N(0,1e-3^2)"),
    3: Workload("densenet121", 6_964_106, 30, 5, 250, 0.06, (1e-2,), 2, "scaled", 1.0,
                "DenseNet121-sized, per-worker scale log-uniform in [1e-4,1e-2]"),
    4: Workload("densenet201", 20_013_928, 60, 7, 500, 0.06 * (250.0 / 500.0) ** 0.5, (1e-2,), 3,
                "heavy", 1e-3, "DenseNet201-sized, 1% of coordinates replaced by 1e-2*t(nu=2)"),
    5: Workload("convnextlarge", 197_767_336, 8, 5, 250, 0.06, (1e-2,), 4, "iid", 1e-4,
                "ConvNeXt-Large-sized, iid drift"),
    # a second shape (Table 2: VGG16* with 2.6M parameters; Section 3.3 leaves other sketch
    # sizes open): the recommended sketch and a larger one
    6: Workload("vgg16star", 2_600_000, 20, 5, 250, 0.06, (1e-2,), 11, "shared", 1e-3,
                "VGG16*-sized, shared + private drift"),
    7: Workload("vgg16star-8x1000", 2_600_000, 20, 8, 1000, 0.06 * (250.0 / 1000.0) ** 0.5, (1e-2,), 11,
                "shared", 1e-3, "VGG16*-sized, shared + private drift, 8 x 1000 sketch"),
}

SHARED_SIGMA = 5e-4
SCALE_LO, SCALE_HI = 1e-4, 1e-2
HEAVY_FRACTION, HEAVY_SCALE, HEAVY_NU = 0.01, 1e-2, 2.0
W_T0_SIGMA = 0.05


def _rng(seed: int, item: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(item)]))


def row_stride(d: int) -> int:
    """Row pitch (in elements) used for the K x d model tensor: d rounded up to 32."""
    return (d + 31) // 32 * 32


def hash_coefficients(seed: int, l: int) -> np.ndarray:
    """uint64[6*l] table, rows of {a, b, c3, c2, c1, c0}, every value in [0, 2^61-2]."""
    rng = _rng(seed, ITEM_COEFFS)

    def draw(nonzero: bool) -> int:
        while True:
            v = int(rng.integers(0, 1 << 61, dtype=np.uint64))
            if v < P61 and (v != 0 or not nonzero):
                return v

    out = np.empty(6 * l, dtype=np.uint64)
    for i in range(l):
        for c in range(6):
            out[6 * i + c] = draw(nonzero=(c == 0 or c == 2))
    return out


def _chunks(d: int):
    for lo in range(0, d, CHUNK):
        yield lo, min(d, lo + CHUNK)


def last_global_model(wl: Workload) -> np.ndarray:
    """w_t0: float32[d]."""
    rng = _rng(wl.seed, ITEM_W_T0)
    out = np.empty(wl.d, dtype=np.float32)
    for lo, hi in _chunks(wl.d):
        out[lo:hi] = rng.standard_normal(hi - lo, dtype=np.float32) * np.float32(W_T0_SIGMA)
    return out


def unit_direction(wl: Workload) -> np.ndarray:
    """xi: float32[d], a normal vector scaled to unit length in fp64 before rounding."""
    rng = _rng(wl.seed, ITEM_XI)
    g = np.empty(wl.d, dtype=np.float32)
    for lo, hi in _chunks(wl.d):
        g[lo:hi] = rng.standard_normal(hi - lo, dtype=np.float32)
    scale = 1.0 / np.sqrt(np.sum(g.astype(np.float64) ** 2))
    return (g.astype(np.float64) * scale).astype(np.float32)


def worker_scales(wl: Workload) -> np.ndarray:
    """Per-worker drift scale of kind "scaled": log-uniform in [SCALE_LO, SCALE_HI]."""
    u = _rng(wl.seed, ITEM_SCALES).random(wl.K)
    return np.exp(np.log(SCALE_LO) + u * (np.log(SCALE_HI) - np.log(SCALE_LO)))


def worker_model(wl: Workload, k: int, w_t0: np.ndarray, out: np.ndarray | None = None) -> np.ndarray:
    """w_k = fp32(w_t0 + drift_k): float32[d] (written into ``out`` when given)."""
    d = wl.d
    if out is None:
        out = np.empty(d, dtype=np.float32)
    rng = _rng(wl.seed, ITEM_WORKER0 + k)
    shared = _rng(wl.seed, ITEM_SHARED) if wl.drift == "shared" else None
    scale = np.float32(worker_scales(wl)[k] if wl.drift == "scaled" else wl.sigma)
    for lo, hi in _chunks(d):
        n = hi - lo
        drift = rng.standard_normal(n, dtype=np.float32)
        drift *= scale
        if wl.drift == "shared":
            drift += shared.standard_normal(n, dtype=np.float32) * np.float32(SHARED_SIGMA)
        elif wl.drift == "heavy":
            mask = rng.random(n, dtype=np.float32) < np.float32(HEAVY_FRACTION)
            cnt = int(mask.sum())
            drift[mask] = (rng.standard_t(HEAVY_NU, size=cnt) * HEAVY_SCALE).astype(np.float32)
        np.add(w_t0[lo:hi], drift, out=out[lo:hi])
    return out


def worker_models(wl: Workload, w_t0: np.ndarray, workers=None, out: np.ndarray | None = None,
                  threads: int = 8) -> np.ndarray:
    """Model tensor of shape (len(workers), row_stride(d)) float32; columns >= d are zero.
    Row r holds worker ``workers[r]`` (all K workers by default).  Use ``buf[:, :d]`` as the
    K x d view."""
    ks = list(range(wl.K)) if workers is None else [int(k) for k in workers]
    stride = row_stride(wl.d)
    if out is None:
        out = np.zeros((len(ks), stride), dtype=np.float32)
    else:
        out[:, wl.d:] = 0
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        list(ex.map(lambda rk: worker_model(wl, rk[1], w_t0, out[rk[0], :wl.d]), enumerate(ks)))
    return out


def small_workload(seed: int, d: int, K: int, l: int = 5, m: int = 250, drift: str = "iid",
                   sigma: float = 1e-3, epsilon: float = 0.06) -> Workload:
    """A workload of arbitrary small shape drawn by the same recipe (parity and edge cases)."""
    return Workload("small", d, K, l, m, epsilon, (1e-2,), seed, drift, sigma, "test shape")
