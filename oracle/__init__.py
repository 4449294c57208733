"""Python face of the CPU checker in ``lr_oracle.c`` (float64, plain loops).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg.  The product (CUDA) path never imports this package and this package never imports the
product.  The C file's header lists what each routine follows in the paper and how it is pinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lr_oracle.c")
_SO = os.path.join(_HERE, "liblr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``lr_oracle.c`` with gcc (-O2, OpenMP, no fast-math) if the shared object is stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P, I64, I32, D = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_double
        lib.oracle_threads.restype = ctypes.c_int
        lib.oracle_set_threads.argtypes = [ctypes.c_int]
        lib.oracle_loss_grad.argtypes = [P, P, I64, I32, P, D, P, P, P]
        lib.oracle_fit.argtypes = [P, P, I64, I32, D, I32, P, P, P, P, P, ctypes.c_int]
        lib.oracle_predict.argtypes = [P, I64, I32, P, D, D, P, P]
        lib.oracle_fit_opt.argtypes = [P, P, I64, I32, D, I32, D, D, ctypes.c_int, P, P, P, P]
        lib.oracle_fit_sgd.argtypes = [P, P, I64, I32, D, I64, I32, I64, P, P, P]
        lib.oracle_fit_tol.argtypes = [P, P, I64, I32, D, D, I32, P, P, P, P, P, P]
        lib.oracle_f1.argtypes = [P, P, I64, P, P, P, P]
        lib.oracle_round_bf16.argtypes = [P, I64, P, P]
        _lib = lib
    return _lib


def _f32(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.float32)
    if shape is not None:
        assert a.shape == shape, (a.shape, shape)
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def threads() -> int:
    return int(_load().oracle_threads())


def set_threads(t: int) -> None:
    _load().oracle_set_threads(int(t))


def loss_grad(X, y, w, b):
    """(loss, grad_w[n], grad_b) in float64 at parameters (w, b); X, y are fp32 arrays."""
    X = _f32(X)
    m, n = X.shape
    y = _f32(y, (m,))
    w = np.ascontiguousarray(w, dtype=np.float64)
    assert w.shape == (n,)
    loss, gb = np.zeros(1), np.zeros(1)
    gw = np.zeros(n)
    rc = _load().oracle_loss_grad(_ptr(X), _ptr(y), m, n, _ptr(w), float(b), _ptr(loss), _ptr(gw), _ptr(gb))
    if rc != 0:
        raise ValueError("oracle_loss_grad: bad arguments")
    return float(loss[0]), gw, float(gb[0])


def fit(X, y, lr, iters, w0=None, b0=0.0, history=False, round_to_fp32=False):
    """Run ``iters`` full-batch GD steps from (w0, b0) (zeros by default).

    Returns ``(w, b, loss_hist)``; with ``history=True`` also ``w_hist[(iters+1), n]`` and
    ``b_hist[iters+1]``.  ``loss_hist[t]`` is the loss before update t.
    """
    X = _f32(X)
    m, n = X.shape
    y = _f32(y, (m,))
    w = np.zeros(n) if w0 is None else np.array(w0, dtype=np.float64).copy()
    assert w.shape == (n,)
    b = np.array([float(b0)])
    lh = np.zeros(max(iters, 1))
    wh = np.zeros((iters + 1, n)) if history else None
    bh = np.zeros(iters + 1) if history else None
    rc = _load().oracle_fit(_ptr(X), _ptr(y), m, n, float(lr), int(iters), _ptr(w), _ptr(b), _ptr(lh),
                            _ptr(wh), _ptr(bh), int(bool(round_to_fp32)))
    if rc != 0:
        raise ValueError("oracle_fit: bad arguments")
    lh = lh[:iters]
    if history:
        return w, float(b[0]), lh, wh, bh
    return w, float(b[0]), lh


def fit_tol(X, y, lr, eps, max_iters, w0=None, b0=0.0):
    """GD with the stopping rule ||grad||_2 <= eps tested after each update (at most ``max_iters`` updates).

    Returns ``(w, b, iters_done, grad_norm, loss_hist[:iters_done], gnorm_hist[:iters_done])``.
    """
    X = _f32(X)
    m, n = X.shape
    y = _f32(y, (m,))
    w = np.zeros(n) if w0 is None else np.array(w0, dtype=np.float64).copy()
    b = np.array([float(b0)])
    lh, gh = np.zeros(max(max_iters, 1)), np.zeros(max(max_iters, 1))
    done = ctypes.c_int32()
    nrm = ctypes.c_double()
    rc = _load().oracle_fit_tol(_ptr(X), _ptr(y), m, n, float(lr), float(eps), int(max_iters), _ptr(w), _ptr(b), _ptr(lh),
                                _ptr(gh), ctypes.byref(done), ctypes.byref(nrm))
    if rc != 0:
        raise ValueError("oracle_fit_tol: bad arguments")
    k = done.value
    return w, float(b[0]), k, nrm.value, lh[:k], gh[:k]


def fit_opt(X, y, lr, iters, l2=0.0, momentum=0.0, nesterov=False, w0=None, b0=0.0, vel0=None):
    """GD with an L2 penalty and momentum.  Returns ``(w, b, vel[n+1], loss_hist)``."""
    X = _f32(X)
    m, n = X.shape
    y = _f32(y, (m,))
    w = np.zeros(n) if w0 is None else np.array(w0, dtype=np.float64).copy()
    b = np.array([float(b0)])
    vel = np.zeros(n + 1) if vel0 is None else np.array(vel0, dtype=np.float64).copy()
    lh = np.zeros(max(iters, 1))
    rc = _load().oracle_fit_opt(_ptr(X), _ptr(y), m, n, float(lr), int(iters), float(l2), float(momentum), int(bool(nesterov)),
                                _ptr(w), _ptr(b), _ptr(vel), _ptr(lh))
    if rc != 0:
        raise ValueError("oracle_fit_opt: bad arguments")
    return w, float(b[0]), vel, lh[:iters]


def fit_sgd(X, y, lr, batch_rows, steps, first_batch=0, w0=None, b0=0.0):
    """Mini-batch GD over contiguous row blocks (no shuffling).  Returns ``(w, b, loss_hist)``."""
    X = _f32(X)
    m, n = X.shape
    y = _f32(y, (m,))
    w = np.zeros(n) if w0 is None else np.array(w0, dtype=np.float64).copy()
    b = np.array([float(b0)])
    lh = np.zeros(max(steps, 1))
    rc = _load().oracle_fit_sgd(_ptr(X), _ptr(y), m, n, float(lr), int(batch_rows), int(steps), int(first_batch), _ptr(w),
                                _ptr(b), _ptr(lh))
    if rc != 0:
        raise ValueError("oracle_fit_sgd: bad arguments")
    return w, float(b[0]), lh[:steps]


def predict(X, w, b, thr, return_z=False):
    """uint8 labels[m]: 1 iff sigmoid(x.w + b) >= thr (decided as z >= logit(thr))."""
    X = _f32(X)
    m, n = X.shape
    w = np.ascontiguousarray(w, dtype=np.float64)
    assert w.shape == (n,)
    labels = np.zeros(m, dtype=np.uint8)
    z = np.zeros(m) if return_z else None
    rc = _load().oracle_predict(_ptr(X), m, n, _ptr(w), float(b), float(thr), _ptr(labels), _ptr(z))
    if rc != 0:
        raise ValueError("oracle_predict: bad arguments")
    return (labels, z) if return_z else labels


def f1_score(labels, y):
    """(f1, tp, fp, fn) of uint8 labels against fp32 0/1 targets."""
    labels = np.ascontiguousarray(labels, dtype=np.uint8)
    y = _f32(y, labels.shape)
    tp, fp, fn = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    f1 = ctypes.c_double()
    rc = _load().oracle_f1(_ptr(labels), _ptr(y), labels.shape[0], ctypes.byref(tp), ctypes.byref(fp),
                           ctypes.byref(fn), ctypes.byref(f1))
    if rc != 0:
        raise ValueError("oracle_f1: bad arguments")
    return f1.value, tp.value, fp.value, fn.value


def round_bf16(x):
    """Rounds fp32 values to bfloat16 (round to nearest, ties to even).

    Returns ``(bits, values)``: the uint16 patterns and the same numbers widened back to fp32, both shaped like ``x``.
    The other routines of this module take ``values`` wherever the CUDA path is given the bfloat16 matrix.
    """
    x = _f32(x)
    bits = np.zeros(x.shape, dtype=np.uint16)
    values = np.zeros(x.shape, dtype=np.float32)
    rc = _load().oracle_round_bf16(_ptr(x), x.size, _ptr(bits), _ptr(values))
    if rc != 0:
        raise ValueError("oracle_round_bf16: bad arguments")
    return bits, values
