"""Thin ctypes binding over the C-ABI library ``liblrgd.so`` (declared in ``include/lrgd.h``).

Argument marshalling only: every step of the computation runs in the CUDA kernels behind the C
entry points.  PyTorch supplies device memory and the current stream.  Loading fails loudly when the
library has not been built; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("LRGD_LIB") or os.path.join(_HERE, "liblrgd.so")   # LRGD_LIB: another build of the same library

LR_OK = 0
LR_ERR_NULL, LR_ERR_SHAPE, LR_ERR_ALIGNMENT, LR_ERR_VALUE, LR_ERR_CUDA, LR_ERR_TIMEOUT, LR_ERR_NOMEM = range(-1, -8, -1)

EXPORTS = ["lr_plan_query", "lr_create", "lr_destroy", "lr_loss_grad", "lr_fit", "lr_predict", "lr_shard_sums",
           "lr_apply_sums", "lr_fit_host",
           "lr_predict_host", "lr_profile_enable", "lr_profile_read", "lr_launch_count", "lr_last_device_status",
           "lr_last_cuda_error", "lr_status_string", "lr_loss_grad_noalloc", "lr_fit_tol", "lr_fit_opt", "lr_selftest_wait", "lr_set_persistent", "lr_fit_sgd", "lr_set_l2_keep",
           "lr_convert_bf16", "lr_loss_grad_bf16", "lr_fit_bf16", "lr_predict_bf16", "lr_plan_query_bf16",
           "lr_fit_tol_bf16", "lr_fit_opt_bf16", "lr_fit_sgd_bf16", "lr_shard_sums_bf16", "lr_set_overlap",
           "lr_fit_host_bf16", "lr_predict_host_bf16", "lr_exchange_bytes", "lr_fit_sharded", "lr_fit_sharded_bf16", "lr_fit_sharded_local", "lr_set_sm_limit",
           "lr_set_cluster", "lr_cluster_ctas", "lr_f1_counts", "lr_check_guards"]


class LrPlan(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("variant", "lanes_per_row", "vec_per_lane", "rows_per_batch", "tile_rows",
                                              "stages", "grid", "threads", "smem_bytes")]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class LrOpt(ctypes.Structure):
    _fields_ = [("l2", ctypes.c_float), ("momentum", ctypes.c_float), ("nesterov", ctypes.c_int32)]


class LrError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (code {code}){detail}")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (run ``python -m paper_2308_10037_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2308_10037_b200.build` "
                              "(nvcc, sm_100a).  There is no CPU fallback.")
        L = ctypes.CDLL(LIB_PATH)
        P, I64, I32, F = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
        L.lr_plan_query.argtypes = [I64, I32, I32, I32, ctypes.POINTER(LrPlan)]
        L.lr_create.argtypes = [ctypes.POINTER(P), I32, I32]
        L.lr_destroy.argtypes = [P]
        L.lr_loss_grad.argtypes = [P, P, P, I64, I32, P, P, P, P, P, P]
        L.lr_fit.argtypes = [P, P, P, I64, I32, F, I32, P, P, P, P]
        L.lr_predict.argtypes = [P, P, I64, I32, P, P, F, P, P]
        L.lr_shard_sums.argtypes = [P, P, P, I64, I32, P, P, P, P]
        L.lr_f1_counts.argtypes = [P, P, P, I64, P, P]
        L.lr_check_guards.argtypes = [P, ctypes.POINTER(I32)]
        L.lr_convert_bf16.argtypes = [P, P, I64, P, P]
        L.lr_loss_grad_bf16.argtypes = L.lr_loss_grad.argtypes
        L.lr_fit_bf16.argtypes = L.lr_fit.argtypes
        L.lr_predict_bf16.argtypes = L.lr_predict.argtypes
        L.lr_plan_query_bf16.argtypes = L.lr_plan_query.argtypes
        L.lr_apply_sums.argtypes = [P, P, I32, I64, I32, F, P, P, P, P]
        L.lr_fit_tol.argtypes = [P, P, P, I64, I32, F, F, I32, I32, P, P, P, P, ctypes.POINTER(I32),
                                 ctypes.POINTER(F), P]
        L.lr_fit_opt.argtypes = [P, P, P, I64, I32, F, I32, ctypes.POINTER(LrOpt), P, P, P, P, P]
        L.lr_selftest_wait.argtypes = [P, I32, I32, P]
        L.lr_fit_sgd.argtypes = [P, P, P, I64, I32, F, I64, I32, I64, P, P, P, P]
        L.lr_fit_tol_bf16.argtypes = L.lr_fit_tol.argtypes
        L.lr_fit_opt_bf16.argtypes = L.lr_fit_opt.argtypes
        L.lr_fit_sgd_bf16.argtypes = L.lr_fit_sgd.argtypes
        L.lr_shard_sums_bf16.argtypes = L.lr_shard_sums.argtypes
        L.lr_set_persistent.argtypes = [P, I32]
        L.lr_set_overlap.argtypes = [P, I32]
        L.lr_set_l2_keep.argtypes = [P, I64]
        L.lr_set_sm_limit.argtypes = [P, I32]
        L.lr_set_cluster.argtypes = [P, I32]
        L.lr_cluster_ctas.argtypes = [I64, I32, I32, I32, I32]
        L.lr_cluster_ctas.restype = I32
        L.lr_exchange_bytes.argtypes = [I32, I32, ctypes.POINTER(I64)]
        L.lr_fit_sharded.argtypes = [P, P, P, I64, I64, I32, F, I32, P, P, P, I32, I32, ctypes.POINTER(P), I64, I32, P]
        L.lr_fit_sharded_bf16.argtypes = L.lr_fit_sharded.argtypes
        L.lr_fit_sharded_local.argtypes = [P, I32, ctypes.POINTER(P), ctypes.POINTER(P), ctypes.POINTER(I64), I32, F, I32,
                                           ctypes.POINTER(P), ctypes.POINTER(P), ctypes.POINTER(P), ctypes.POINTER(P), I64, I32, P]
        L.lr_loss_grad_noalloc.argtypes = [I32, P, P, I64, I32, P, P, P, P, P, P, P]
        L.lr_fit_host.argtypes = [P, P, P, I64, I32, F, I32, P, P, P]
        L.lr_predict_host.argtypes = [P, P, I64, I32, P, P, F, P]
        L.lr_fit_host_bf16.argtypes = L.lr_fit_host.argtypes
        L.lr_predict_host_bf16.argtypes = L.lr_predict_host.argtypes
        L.lr_profile_enable.argtypes = [P, I32]
        L.lr_profile_read.argtypes = [P, ctypes.POINTER(I32), ctypes.POINTER(ctypes.c_double)]
        L.lr_launch_count.argtypes = [P, ctypes.POINTER(I64)]
        L.lr_last_device_status.argtypes = [P, ctypes.POINTER(I32)]
        L.lr_last_cuda_error.argtypes = [P]
        L.lr_status_string.argtypes = [ctypes.c_int]
        L.lr_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name != "lr_status_string":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().lr_status_string(int(code)).decode()


def plan_query(m: int, n: int, x_aligned16: bool = True, sm_count: int = 148, bf16: bool = False) -> dict:
    """Host-only view of the launch plan for an m-by-n problem (no CUDA call); ``bf16``: X stored as bfloat16."""
    p = LrPlan()
    fn = lib().lr_plan_query_bf16 if bf16 else lib().lr_plan_query
    rc = fn(int(m), int(n), int(bool(x_aligned16)), int(sm_count), ctypes.byref(p))
    if rc != LR_OK:
        raise LrError(rc, "lr_plan_query")
    return p.as_dict()


def cluster_ctas(m: int, n: int, x_aligned16: bool = True, sm_count: int = 148, bf16: bool = False) -> int:
    """Cluster size the single-cluster form of ``fit`` would use for an m-by-n problem, 0 if it has none (host only)."""
    return int(lib().lr_cluster_ctas(int(m), int(n), int(bool(x_aligned16)), int(sm_count), int(bool(bf16))))


def exchange_bytes(world: int, n: int) -> int:
    """Size of one rank's exchange buffer for a row-sharded fit over ``world`` ranks and ``n`` columns."""
    v = ctypes.c_int64()
    rc = lib().lr_exchange_bytes(int(world), int(n), ctypes.byref(v))
    if rc != LR_OK:
        raise LrError(rc, "lr_exchange_bytes")
    return v.value


def _dev_ptr(t: torch.Tensor | None, dtype, name: str, count: int | None = None, device: int | None = None):
    """Device address of ``t`` after checking what the C side cannot see behind a bare pointer.

    ``count`` is the number of elements the call reads or writes through the pointer: a shorter tensor would be an
    out-of-bounds access on the device, so it is refused here with ValueError.  ``device`` is the index of the device
    the call runs on; a tensor that lives on another one is refused as well.  None passes through (optional arguments).
    """
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    if count is not None and t.numel() < count:
        raise ValueError(f"{name}: {t.numel()} elements, the call needs {count}")
    if device is not None and t.device.index != device:
        raise ValueError(f"{name}: lives on cuda:{t.device.index}, the call runs on cuda:{device}")
    return ctypes.c_void_p(t.data_ptr())


def _shape2(X, name: str = "X"):
    if not isinstance(X, (torch.Tensor, np.ndarray)) or X.ndim != 2 or X.shape[0] < 1 or X.shape[1] < 1:
        raise ValueError(f"{name}: expected a 2-D array with at least one row and one column")
    return int(X.shape[0]), int(X.shape[1])


def _host_ptr(a, dtype, name: str, count: int | None = None):
    """Host address of a CPU tensor or numpy array holding at least ``count`` elements of ``dtype``."""
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous() or a.dtype != dtype:
            raise TypeError(f"{name}: expected a contiguous CPU tensor of dtype {dtype}")
        if count is not None and a.numel() < count:
            raise ValueError(f"{name}: {a.numel()} elements, the call needs {count}")
        return ctypes.c_void_p(a.data_ptr())
    npdt = {torch.float32: np.float32, torch.uint8: np.uint8}[dtype]
    if not (isinstance(a, np.ndarray) and a.dtype == npdt and a.flags.c_contiguous):
        raise TypeError(f"{name}: expected a C-contiguous numpy array of dtype {npdt}")
    if count is not None and a.size < count:
        raise ValueError(f"{name}: {a.size} elements, the call needs {count}")
    return ctypes.c_void_p(a.ctypes.data)


class Context:
    """Owns one ``lr_ctx``: workspace for problems of up to ``n_max`` columns on one device."""

    def __init__(self, n_max: int = 4096, device: int | None = None):
        self._h = ctypes.c_void_p()
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.n_max = int(n_max)
        rc = lib().lr_create(ctypes.byref(self._h), self.device, self.n_max)
        if rc != LR_OK:
            self._h = ctypes.c_void_p()
            raise LrError(rc, "lr_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().lr_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != LR_OK:
            detail = f"; cudaError {lib().lr_last_cuda_error(self._h)}" if rc == LR_ERR_CUDA else ""
            raise LrError(rc, where, detail)

    def _stream(self):
        return ctypes.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    # ---- device-pointer entry points -------------------------------------------------------------
    # X may be a float32 tensor (lr_loss_grad / lr_fit / lr_predict) or a bfloat16 tensor (the *_bf16 entry points).
    @staticmethod
    def _x_kind(X):
        if isinstance(X, torch.Tensor) and X.dtype == torch.bfloat16:
            return torch.bfloat16, "_bf16"
        return torch.float32, ""

    def _p(self, t, dtype, name, count=None):
        """``_dev_ptr`` for an argument of a call on this context: also checks that the tensor is on the context's device."""
        return _dev_ptr(t, dtype, name, count, self.device)

    def convert_bf16(self, X, out=None):
        """Rounds a float32 CUDA tensor to bfloat16 (nearest, ties to even) with the library's kernel."""
        px = self._p(X, torch.float32, "X")
        count = X.numel()
        Xh = torch.empty(X.shape, dtype=torch.bfloat16, device=X.device) if out is None else out
        rc = lib().lr_convert_bf16(self._h, px, count, self._p(Xh, torch.bfloat16, "Xh", count), self._stream())
        self._check(rc, "lr_convert_bf16")
        return Xh

    def loss_grad(self, X, y, w, b):
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32 = torch.float32
        inputs = (self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n, self._p(w, F32, "w", n), self._p(b, F32, "b", 1))
        loss = torch.empty(1, dtype=F32, device=X.device)
        gw = torch.empty(n, dtype=F32, device=X.device)
        gb = torch.empty(1, dtype=F32, device=X.device)
        rc = getattr(lib(), "lr_loss_grad" + sfx)(self._h, *inputs, self._p(loss, F32, "loss", 1),
                                self._p(gw, F32, "grad_w", n), self._p(gb, F32, "grad_b", 1), self._stream())
        self._check(rc, "lr_loss_grad" + sfx)
        return loss, gw, gb

    def fit(self, X, y, lr, iters, w, b, loss_hist=None):
        """In place on ``w`` [n] and ``b`` [1]; ``loss_hist`` is None or a float32 CUDA tensor [iters]."""
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32, iters = torch.float32, int(iters)
        rc = getattr(lib(), "lr_fit" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n, float(lr), iters,
                          self._p(w, F32, "w", n), self._p(b, F32, "b", 1), self._p(loss_hist, F32, "loss_hist", max(iters, 0)),
                          self._stream())
        self._check(rc, "lr_fit" + sfx)

    def fit_tol(self, X, y, lr, eps, max_iters, w, b, check_every=16, loss_hist=None, gnorm_hist=None):
        """GD until ||grad||_2 <= eps (at most ``max_iters`` updates), in place on w, b.  Returns (updates, last norm)."""
        m, n = _shape2(X)
        done, nrm = ctypes.c_int32(), ctypes.c_float()
        xdt, sfx = self._x_kind(X)
        F32, cap = torch.float32, max(int(max_iters), 0)
        rc = getattr(lib(), "lr_fit_tol" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n, float(lr),
                              float(eps), int(max_iters), int(check_every), self._p(w, F32, "w", n), self._p(b, F32, "b", 1),
                              self._p(loss_hist, F32, "loss_hist", cap), self._p(gnorm_hist, F32, "gnorm_hist", cap),
                              ctypes.byref(done), ctypes.byref(nrm), self._stream())
        self._check(rc, "lr_fit_tol" + sfx)
        return done.value, nrm.value

    def fit_opt(self, X, y, lr, iters, w, b, l2=0.0, momentum=0.0, nesterov=False, velocity=None, loss_hist=None):
        """GD with an L2 penalty and (Nesterov) momentum, in place on w, b (and ``velocity`` [n+1] when given)."""
        m, n = _shape2(X)
        opt = LrOpt(float(l2), float(momentum), int(bool(nesterov)))
        xdt, sfx = self._x_kind(X)
        F32, iters = torch.float32, int(iters)
        rc = getattr(lib(), "lr_fit_opt" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n, float(lr),
                              iters, ctypes.byref(opt), self._p(w, F32, "w", n), self._p(b, F32, "b", 1),
                              self._p(velocity, F32, "velocity", n + 1), self._p(loss_hist, F32, "loss_hist", max(iters, 0)),
                              self._stream())
        self._check(rc, "lr_fit_opt" + sfx)

    def fit_sgd(self, X, y, lr, batch_rows, steps, w, b, first_batch=0, loss_hist=None):
        """Mini-batch GD over contiguous row blocks (block (first_batch + s) mod count at step s), in place on w, b."""
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32, steps = torch.float32, int(steps)
        rc = getattr(lib(), "lr_fit_sgd" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n, float(lr),
                              int(batch_rows), steps, int(first_batch), self._p(w, F32, "w", n), self._p(b, F32, "b", 1),
                              self._p(loss_hist, F32, "loss_hist", max(steps, 0)), self._stream())
        self._check(rc, "lr_fit_sgd" + sfx)

    def predict(self, X, w, b, thr, out=None):
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32 = torch.float32
        px, pw, pb = self._p(X, xdt, "X"), self._p(w, F32, "w", n), self._p(b, F32, "b", 1)
        labels = torch.empty(m, dtype=torch.uint8, device=X.device) if out is None else out
        rc = getattr(lib(), "lr_predict" + sfx)(self._h, px, m, n, pw, pb, float(thr),
                                                self._p(labels, torch.uint8, "labels", m), self._stream())
        self._check(rc, "lr_predict" + sfx)
        return labels

    def f1_counts_async(self, labels, y, counts):
        """Enqueues the confusion counts of uint8 ``labels`` against 0/1 targets ``y`` into ``counts`` (int64 CUDA tensor
        [3]: tp, fp, fn) without reading them back."""
        if not isinstance(labels, torch.Tensor) or labels.dim() != 1:
            raise ValueError("labels: expected a 1-D uint8 CUDA tensor")
        m = labels.numel()
        rc = lib().lr_f1_counts(self._h, self._p(labels, torch.uint8, "labels", m) if m else None,
                                self._p(y, torch.float32, "y", m) if m else None, m,
                                self._p(counts, torch.int64, "counts", 3), self._stream())
        self._check(rc, "lr_f1_counts")

    def f1_counts(self, labels, y):
        """``(f1, tp, fp, fn)`` of uint8 ``labels`` against 0/1 targets ``y``, counted on the device; f1 = 2tp / (2tp + fp
        + fn), 0 when tp == 0.  Reads the three counters back, so it waits for the stream."""
        counts = torch.empty(3, dtype=torch.int64, device=labels.device if isinstance(labels, torch.Tensor) else None)
        self.f1_counts_async(labels, y, counts)
        tp, fp, fn = (int(v) for v in counts.tolist())
        return (2.0 * tp / (2.0 * tp + fp + fn) if tp > 0 else 0.0), tp, fp, fn

    def shard_sums(self, X, y, w, b, sums):
        """Unnormalised fp64 sums [n+2] of the local rows into ``sums`` (float64 CUDA tensor)."""
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32 = torch.float32
        rc = getattr(lib(), "lr_shard_sums" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, n,
                                 self._p(w, F32, "w", n), self._p(b, F32, "b", 1),
                                 self._p(sums, torch.float64, "sums", n + 2), self._stream())
        self._check(rc, "lr_shard_sums" + sfx)

    def apply_sums(self, sums_all, m_total, lr, w, b, loss=None):
        """Adds the ``parts`` rows of ``sums_all`` [parts, n+2] in order and applies the update to w, b in place."""
        parts, n2 = _shape2(sums_all, "sums_all")
        if n2 < 3:
            raise ValueError("sums_all: expected [parts, n+2] with n >= 1")
        F32, n = torch.float32, n2 - 2
        rc = lib().lr_apply_sums(self._h, self._p(sums_all, torch.float64, "sums_all"), parts, int(m_total), n,
                                 float(lr), self._p(w, F32, "w", n), self._p(b, F32, "b", 1), self._p(loss, F32, "loss", 1),
                                 self._stream())
        self._check(rc, "lr_apply_sums")

    # ---- row shards with the exchange inside the kernel ------------------------------------------
    def fit_sharded(self, X, y, m_total, lr, iters, w, b, rank, world, exchange_ptrs, epoch=0, wait_ms=10_000, loss_hist=None):
        """This rank's part of a row-sharded fit (see ``lr_fit_sharded``), in place on w, b.

        ``exchange_ptrs``: the ``world`` exchange buffers as this rank addresses them (integers, or CUDA tensors for
        buffers of this process); ``exchange_ptrs[rank]`` is this rank's own.  ``epoch``: steps these buffers have carried.
        """
        m, n = _shape2(X)
        xdt, sfx = self._x_kind(X)
        F32, iters = torch.float32, int(iters)
        if len(exchange_ptrs) != int(world):
            raise ValueError("exchange_ptrs: one buffer per rank")
        need = exchange_bytes(int(world), n)
        ptrs = (ctypes.c_void_p * int(world))()
        for r, e in enumerate(exchange_ptrs):
            if isinstance(e, torch.Tensor):
                if not e.is_cuda or e.numel() * e.element_size() < need:
                    raise ValueError(f"exchange_ptrs[{r}]: a CUDA tensor of at least {need} bytes is needed")
                e = e.data_ptr()
            ptrs[r] = ctypes.c_void_p(int(e))
        rc = getattr(lib(), "lr_fit_sharded" + sfx)(self._h, self._p(X, xdt, "X"), self._p(y, F32, "y", m), m, int(m_total), n,
                                  float(lr), iters, self._p(w, F32, "w", n), self._p(b, F32, "b", 1),
                                  self._p(loss_hist, F32, "loss_hist", max(iters, 0)), int(rank), int(world), ptrs,
                                  int(epoch), int(wait_ms), self._stream())
        self._check(rc, "lr_fit_sharded" + sfx)

    def fit_sharded_local(self, Xs, ys, lr, iters, ws, bs, exchange, epoch=0, wait_ms=10_000, loss_hists=None):
        """All ranks of a row-sharded fit as CTA groups of one launch on this GPU (see ``lr_fit_sharded_local``).

        ``Xs``, ``ys``, ``ws``, ``bs``, ``exchange`` (and ``loss_hists``) are lists with one CUDA tensor per rank.
        """
        world = len(Xs)
        if not (len(ys) == len(ws) == len(bs) == len(exchange) == world) or (loss_hists is not None and len(loss_hists) != world):
            raise ValueError("one entry per rank in every list")
        F32, iters = torch.float32, int(iters)
        n = _shape2(Xs[0])[1]
        need = exchange_bytes(world, n)
        PA = ctypes.c_void_p * world
        pX, py, pw, pb, ph, pe = PA(), PA(), PA(), PA(), PA(), PA()
        ms = (ctypes.c_int64 * world)()
        for r in range(world):
            m, nr = _shape2(Xs[r], f"Xs[{r}]")
            if nr != n:
                raise ValueError("all shards need the same number of columns")
            ms[r] = m
            pX[r] = self._p(Xs[r], F32, f"Xs[{r}]")
            py[r] = self._p(ys[r], F32, f"ys[{r}]", m)
            pw[r] = self._p(ws[r], F32, f"ws[{r}]", n)
            pb[r] = self._p(bs[r], F32, f"bs[{r}]", 1)
            ph[r] = self._p(loss_hists[r], F32, f"loss_hists[{r}]", max(iters, 0)) if loss_hists is not None else None
            e = exchange[r]
            if not (isinstance(e, torch.Tensor) and e.is_cuda and e.numel() * e.element_size() >= need):
                raise ValueError(f"exchange[{r}]: a CUDA tensor of at least {need} bytes is needed")
            pe[r] = ctypes.c_void_p(e.data_ptr())
        rc = lib().lr_fit_sharded_local(self._h, world, pX, py, ms, n, float(lr), iters, pw, pb,
                                        ph if loss_hists is not None else None, pe, int(epoch), int(wait_ms), self._stream())
        self._check(rc, "lr_fit_sharded_local")

    def set_sm_limit(self, sms: int | None):
        """Launch plans of this context use at most ``sms`` SMs (None or 0: all of them)."""
        self._check(lib().lr_set_sm_limit(self._h, int(sms or 0)), "lr_set_sm_limit")

    # ---- host-pointer entry points ---------------------------------------------------------------
    def fit_host(self, X, y, lr, iters, w, b, loss_hist=None, store_bf16=False):
        """X, y, w, b (and loss_hist) are CPU tensors or numpy arrays; w, b are updated in place.

        ``store_bf16``: X (fp32 on the host) is rounded to bfloat16 on the device after the copy and the fit streams that.
        """
        m, n = _shape2(X)
        F32, iters = torch.float32, int(iters)
        fn = lib().lr_fit_host_bf16 if store_bf16 else lib().lr_fit_host
        rc = fn(self._h, _host_ptr(X, F32, "X"), _host_ptr(y, F32, "y", m), m, n, float(lr), iters,
                _host_ptr(w, F32, "w", n), _host_ptr(b, F32, "b", 1), _host_ptr(loss_hist, F32, "loss_hist", max(iters, 0)))
        self._check(rc, "lr_fit_host_bf16" if store_bf16 else "lr_fit_host")

    def predict_host(self, X, w, b, thr, labels, store_bf16=False):
        m, n = _shape2(X)
        F32 = torch.float32
        fn = lib().lr_predict_host_bf16 if store_bf16 else lib().lr_predict_host
        rc = fn(self._h, _host_ptr(X, F32, "X"), m, n, _host_ptr(w, F32, "w", n), _host_ptr(b, F32, "b", 1),
                float(thr), _host_ptr(labels, torch.uint8, "labels", m))
        self._check(rc, "lr_predict_host_bf16" if store_bf16 else "lr_predict_host")

    # ---- measurement / status --------------------------------------------------------------------
    def profile_enable(self, on: bool = True):
        self._check(lib().lr_profile_enable(self._h, int(bool(on))), "lr_profile_enable")

    def profile_read(self):
        n, ms = ctypes.c_int32(), ctypes.c_double()
        self._check(lib().lr_profile_read(self._h, ctypes.byref(n), ctypes.byref(ms)), "lr_profile_read")
        return n.value, ms.value

    def check_guards(self) -> int:
        """Number of guard regions around the context's device workspaces that no longer hold their pattern (0 = no kernel
        wrote outside its array).  Waits for the device."""
        v = ctypes.c_int32()
        self._check(lib().lr_check_guards(self._h, ctypes.byref(v)), "lr_check_guards")
        return v.value

    def launch_count(self) -> int:
        v = ctypes.c_int64()
        self._check(lib().lr_launch_count(self._h, ctypes.byref(v)), "lr_launch_count")
        return v.value

    def set_l2_keep(self, nbytes: int):
        """Ask for the first ``nbytes`` of X to be kept in L2 across the passes of a fit (0 = off)."""
        self._check(lib().lr_set_l2_keep(self._h, int(nbytes)), "lr_set_l2_keep")

    def set_persistent(self, on: bool | None):
        """Form of ``fit`` / ``fit_tol``: True = the single-launch persistent kernel wherever the shape allows, False = two
        kernels per iteration, None = the library chooses (default; small problems may then run on one thread-block
        cluster, see ``set_cluster``).  True and False give identical results."""
        self._check(lib().lr_set_persistent(self._h, -1 if on is None else int(bool(on))), "lr_set_persistent")

    def set_cluster(self, on: bool):
        """Allow (default) or forbid the single-cluster form of ``fit`` for small problems; same results either way."""
        self._check(lib().lr_set_cluster(self._h, int(bool(on))), "lr_set_cluster")

    def set_overlap(self, on: bool):
        """Allow (default) or forbid launching consecutive kernels of a call as programmatic dependents; same results."""
        self._check(lib().lr_set_overlap(self._h, int(bool(on))), "lr_set_overlap")

    def selftest_wait(self, arm: bool, limit_ms: int = 20):
        """Enqueue the bounded-wait probe (see ``lr_selftest_wait``); read the outcome with ``device_status``."""
        self._check(lib().lr_selftest_wait(self._h, int(bool(arm)), int(limit_ms), self._stream()), "lr_selftest_wait")

    def device_status(self) -> int:
        v = ctypes.c_int32()
        self._check(lib().lr_last_device_status(self._h, ctypes.byref(v)), "lr_last_device_status")
        return v.value


_default_ctx: dict[int, Context] = {}


def _ctx_for(X: torch.Tensor, ctx: Context | None) -> Context:
    if ctx is not None:
        return ctx
    dev = X.device.index if X.device.index is not None else torch.cuda.current_device()
    n = int(X.shape[1])
    c = _default_ctx.get(dev)
    if c is None or c.n_max < n:
        if c is not None:
            c.close()
        c = _default_ctx[dev] = Context(n_max=max(4096, n), device=dev)
    return c


def _as_b(b, device) -> torch.Tensor:
    if isinstance(b, torch.Tensor):
        return b.reshape(1)
    return torch.tensor([float(b)], dtype=torch.float32, device=device)


def lr_loss_grad(X, y, w, b, ctx: Context | None = None):
    """(loss[1], grad_w[n], grad_b[1]) as float32 CUDA tensors at the parameters (w, b)."""
    return _ctx_for(X, ctx).loss_grad(X, y, w, _as_b(b, X.device))


def lr_fit(X, y, lr, iters, w0=None, b0=None, return_history=False, ctx: Context | None = None):
    """``iters`` full-batch gradient-descent steps from (w0, b0) (zeros by default).  Returns (w, b[, loss_hist])."""
    n = int(X.shape[1])
    w = torch.zeros(n, dtype=torch.float32, device=X.device) if w0 is None else w0.detach().clone()
    b = torch.zeros(1, dtype=torch.float32, device=X.device) if b0 is None else _as_b(b0, X.device).clone()
    hist = torch.empty(int(iters), dtype=torch.float32, device=X.device) if return_history else None
    _ctx_for(X, ctx).fit(X, y, lr, iters, w, b, hist)
    return (w, b, hist) if return_history else (w, b)


def lr_predict(X, w, b, thr, ctx: Context | None = None):
    """uint8 CUDA tensor [m]: 1 where sigmoid(x.w + b) >= thr."""
    return _ctx_for(X, ctx).predict(X, w, _as_b(b, X.device), thr)


LR_NOALLOC_MAX_N = 1022


def lr_loss_grad_noalloc(X, y, w, b, loss, grad_w, grad_b, status=None):
    """Allocation-free ``lr_loss_grad``: no context, no workspace allocation inside the library.

    For callers that cannot allocate device memory when they call (latency-critical loops, processes whose
    device memory is fully owned by another allocator, hosts with a no-allocation-after-start rule).  The
    caller passes every buffer, outputs included: ``loss`` [1], ``grad_w`` [n], ``grad_b`` [1] float32 and
    optionally ``status`` [1] int32, all CUDA tensors that already exist.  Scratch lives in a fixed array
    inside the library (n <= LR_NOALLOC_MAX_N); calls that overlap on the GPU race on it.
    """
    m, n = _shape2(X)
    if not (isinstance(X, torch.Tensor) and X.is_cuda):
        raise TypeError("X: expected a contiguous CUDA tensor of dtype torch.float32")
    dev = X.device.index if X.device.index is not None else torch.cuda.current_device()
    F32 = torch.float32
    rc = lib().lr_loss_grad_noalloc(int(dev), _dev_ptr(X, F32, "X", None, dev), _dev_ptr(y, F32, "y", m, dev), m, n,
                                    _dev_ptr(w, F32, "w", n, dev), _dev_ptr(b, F32, "b", 1, dev),
                                    _dev_ptr(loss, F32, "loss", 1, dev), _dev_ptr(grad_w, F32, "grad_w", n, dev),
                                    _dev_ptr(grad_b, F32, "grad_b", 1, dev), _dev_ptr(status, torch.int32, "status", 1, dev),
                                    ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream))
    if rc != LR_OK:
        raise LrError(rc, "lr_loss_grad_noalloc")
