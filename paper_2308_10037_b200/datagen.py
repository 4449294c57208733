"""Seeded synthetic workloads for full-batch gradient-descent logistic regression.

This module only *draws inputs*: a design matrix ``X`` (fp32, row-major), a planted
parameter pair ``(w*, b*)`` and 0/1 labels ``y`` sampled from the planted model
``P(y=1|x) = 1/(1+exp(-w*.x - b*))`` (model equation of Section II-A).  It holds none of the
training arithmetic (no loss, gradient, update or thresholding); both the CUDA path and the
CPU checker consume the arrays it returns, bit for bit.

The paper's only workload is HIGGS (11 M rows x 28 dense features, Section IV-A); that data
is not available offline, so the workloads below are tall dense stand-ins with the same
character (dense fp32 rows, binary labels), plus a wide image-like case.

Determinism: every random array is drawn from numpy's counter-based Philox generator keyed by
``(seed, stream id, chunk index)``.  Rows are generated in fixed chunks of ``CHUNK_ROWS`` rows,
so the result does not depend on the number of worker threads.
"""
from __future__ import annotations

import dataclasses
import math
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

CHUNK_ROWS = 1 << 16

# stream ids (second Philox key word, high half)
_S_X, _S_SCALE, _S_SELECT, _S_WSTAR, _S_LABEL, _S_BIN = 1, 2, 3, 4, 5, 6


@dataclasses.dataclass(frozen=True)
class Workload:
    """One named training problem: shape, value recipe and the GD run parameters."""
    name: str
    m: int
    n: int
    lr: float
    iters: int
    x_dist: str            # "normal" | "scaled_normal" | "uniform01" | "normal_binary_tail"
    wstar: str             # "dense_unit" | "sparse10" | "std002"
    bstar: float | None    # None -> solved so that the positive rate hits `pos_rate`
    pos_rate: float | None = None
    predict_thr: float | None = None
    seed: int = 0


# The five workloads, in the order the benchmark refers to them (cfg1..cfg5).
WORKLOADS = {
    "cfg1": Workload("cfg1", 10_000, 32, 0.1, 100, "normal", "dense_unit", 0.1),
    "cfg2": Workload("cfg2", 1_000_000, 100, 0.5, 200, "scaled_normal", "dense_unit", 0.0),
    "cfg3": Workload("cfg3", 4_000_000, 256, 0.5, 100, "normal", "sparse10", -0.5),
    "cfg4": Workload("cfg4", 100_000, 4096, 0.05, 100, "uniform01", "std002", None, pos_rate=0.5),
    "cfg5": Workload("cfg5", 16_000_000, 64, 1.0, 300, "normal_binary_tail", "dense_unit", None,
                     pos_rate=0.01, predict_thr=0.5),
    # HIGGS-shaped stand-in (Section IV-A: 11 M events x 28 features, binary target).
    "higgs_like": Workload("higgs_like", 11_000_000, 28, 0.1, 100, "scaled_normal", "dense_unit", 0.0,
                           predict_thr=0.5),
}


def scaled(wl: Workload, m: int, name: str | None = None) -> Workload:
    """Same recipe with a different row count (used by the small parity cases)."""
    return dataclasses.replace(wl, m=int(m), name=name or f"{wl.name}_m{m}")


def _gen(seed: int, stream: int, chunk: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), (np.uint64(stream) << np.uint64(32)) | np.uint64(chunk)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _feature_scale(wl: Workload) -> np.ndarray | None:
    if wl.x_dist != "scaled_normal":
        return None
    return _gen(wl.seed, _S_SCALE, 0).uniform(0.5, 2.0, size=wl.n).astype(np.float32)


def _n_binary(wl: Workload) -> int:
    return int(round(0.3 * wl.n)) if wl.x_dist == "normal_binary_tail" else 0


def _x_chunk(wl: Workload, chunk: int, rows: int, scale: np.ndarray | None) -> np.ndarray:
    g = _gen(wl.seed, _S_X, chunk)
    if wl.x_dist == "uniform01":
        return g.random((rows, wl.n), dtype=np.float32)
    x = g.standard_normal((rows, wl.n), dtype=np.float32)
    if scale is not None:
        x *= scale[None, :]
    nb = _n_binary(wl)
    if nb:
        u = _gen(wl.seed, _S_BIN, chunk).random((rows, nb), dtype=np.float32)
        x[:, wl.n - nb:] = (u < np.float32(0.1)).astype(np.float32)
    return x


def planted_w(wl: Workload) -> np.ndarray:
    """The planted weight vector w* (float64)."""
    g = _gen(wl.seed, _S_WSTAR, 0)
    z = g.standard_normal(wl.n)
    if wl.wstar == "dense_unit":
        return z / math.sqrt(wl.n)
    if wl.wstar == "std002":
        return 0.02 * z
    if wl.wstar == "sparse10":
        k = int(round(0.1 * wl.n))
        keep = _gen(wl.seed, _S_SELECT, 0).permutation(wl.n)[:k]
        w = np.zeros(wl.n)
        w[keep] = z[keep]
        return w
    raise ValueError(wl.wstar)


def _planted_prob(zlin: np.ndarray) -> np.ndarray:
    # P(y=1|x) of the planted model, evaluated without overflow
    e = np.exp(-np.abs(zlin))
    return np.where(zlin >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


def _solve_bstar(wl: Workload, wstar: np.ndarray, scale: np.ndarray | None) -> float:
    """b* such that the mean planted probability over the first min(m, 2^20) rows is pos_rate."""
    rows_left = min(wl.m, 1 << 20)
    zs, chunk = [], 0
    while rows_left > 0:
        r = min(rows_left, CHUNK_ROWS, wl.m - chunk * CHUNK_ROWS)
        zs.append(_x_chunk(wl, chunk, r, scale).astype(np.float64) @ wstar)
        rows_left -= r
        chunk += 1
    zlin = np.concatenate(zs)
    lo, hi = -50.0, 50.0
    for _ in range(64):
        mid = 0.5 * (lo + hi)
        if _planted_prob(zlin + mid).mean() < wl.pos_rate:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def generate(wl: Workload, threads: int | None = None, x_out: np.ndarray | None = None):
    """Draw the workload.  Returns ``(X fp32 [m,n] C-order, y fp32 [m] in {0,1}, w* f64 [n], b* float)``.

    ``x_out`` may be a preallocated fp32 C-contiguous [m, n] array (for example a view of pinned
    host memory) that receives X.
    """
    m, n = wl.m, wl.n
    scale = _feature_scale(wl)
    wstar = planted_w(wl)
    bstar = float(wl.bstar) if wl.bstar is not None else _solve_bstar(wl, wstar, scale)
    X = x_out if x_out is not None else np.empty((m, n), dtype=np.float32)
    assert X.shape == (m, n) and X.dtype == np.float32 and X.flags.c_contiguous
    y = np.empty(m, dtype=np.float32)
    nchunks = (m + CHUNK_ROWS - 1) // CHUNK_ROWS

    def work(c: int) -> None:
        r0 = c * CHUNK_ROWS
        r = min(CHUNK_ROWS, m - r0)
        xc = _x_chunk(wl, c, r, scale)
        X[r0:r0 + r] = xc
        p = _planted_prob(xc.astype(np.float64) @ wstar + bstar)
        u = _gen(wl.seed, _S_LABEL, c).random(r)
        y[r0:r0 + r] = (u < p).astype(np.float32)

    threads = threads or min(32, os.cpu_count() or 1)
    if threads > 1 and nchunks > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(nchunks)))
    else:
        for c in range(nchunks):
            work(c)
    return X, y, wstar, bstar


def random_problem(m: int, n: int, seed: int = 0, wscale: float = 1.0):
    """Small unstructured test problem: X ~ N(0,1), w ~ N(0, wscale^2/n), b ~ N(0,1)/4, y ~ Bernoulli(0.5).

    Returns fp32 ``X, y, w, b`` (b as a python float holding an fp32 value).
    """
    g = _gen(seed, 99, 0)
    X = g.standard_normal((m, n), dtype=np.float32)
    y = (g.random(m) < 0.5).astype(np.float32)
    w = (wscale * g.standard_normal(n) / math.sqrt(max(n, 1))).astype(np.float32)
    b = float(np.float32(0.25 * g.standard_normal()))
    return X, y, w, b
