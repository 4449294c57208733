"""The Python binding refuses arguments whose sizes or devices do not fit the call, before anything is launched.

CPU only.  The C side sees bare pointers, so a y with fewer than m entries, a w shorter than n, a history shorter than
the iteration count or a tensor on another GPU would become an out-of-bounds access on the device.  The binding has to
turn each of them into a Python exception.  The library is replaced by a recorder that fails the test if a call gets
through, and CUDA tensors are imitated by CPU tensors that claim to live on a GPU (nothing dereferences them).
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2308_10037_b200 import api


class FakeCuda(torch.Tensor):
    """A CPU tensor that reports itself as living on cuda:<index>."""

    @staticmethod
    def __new__(cls, data, index=0):
        t = torch.Tensor._make_subclass(cls, data)
        t._index = index
        return t

    is_cuda = property(lambda self: True)
    device = property(lambda self: torch.device("cuda", self._index))


def fake(shape, dtype=torch.float32, index=0):
    return FakeCuda(torch.zeros(shape, dtype=dtype), index)


class Recorder:
    """Stands in for the loaded library: remembers which entry points were reached."""

    def __init__(self):
        self.calls = []

    def __getattr__(self, name):
        def call(*args):
            self.calls.append(name)
            return api.LR_OK
        return call


@pytest.fixture
def ctx(monkeypatch):
    rec = Recorder()
    monkeypatch.setattr(api, "lib", lambda: rec)
    monkeypatch.setattr(api.Context, "_stream", lambda self: ctypes.c_void_p(0))
    c = api.Context.__new__(api.Context)
    c._h, c.device, c.n_max = ctypes.c_void_p(1), 0, 4096
    c.rec = rec
    yield c
    c._h = ctypes.c_void_p()


M, N = 64, 8


def good():
    return dict(X=fake((M, N)), y=fake(M), w=fake(N), b=fake(1))


def test_well_formed_calls_get_through(ctx):
    a = good()
    ctx.fit(a["X"], a["y"], 0.1, 5, a["w"], a["b"], fake(5))
    ctx.predict(a["X"], a["w"], a["b"], 0.5, out=fake(M, torch.uint8))
    ctx.shard_sums(a["X"], a["y"], a["w"], a["b"], fake(N + 2, torch.float64))
    ctx.apply_sums(fake((3, N + 2), torch.float64), 3 * M, 0.1, a["w"], a["b"], fake(1))
    ctx.fit_tol(a["X"], a["y"], 0.1, 1e-3, 7, a["w"], a["b"], loss_hist=fake(7), gnorm_hist=fake(7))
    ctx.fit_opt(a["X"], a["y"], 0.1, 4, a["w"], a["b"], velocity=fake(N + 1), loss_hist=fake(4))
    ctx.fit_sgd(a["X"], a["y"], 0.1, 16, 6, a["w"], a["b"], loss_hist=fake(6))
    assert ctx.rec.calls == ["lr_fit", "lr_predict", "lr_shard_sums", "lr_apply_sums", "lr_fit_tol", "lr_fit_opt", "lr_fit_sgd"]


@pytest.mark.parametrize("what,change", [
    ("y shorter than m", dict(y=fake(M - 1))),
    ("w shorter than n", dict(w=fake(N - 1))),
    ("b empty", dict(b=fake(0))),
    ("X not two-dimensional", dict(X=fake(M * N))),
    ("y on another GPU", dict(y=fake(M, index=1))),
    ("w on another GPU", dict(w=fake(N, index=1))),
    ("X on another GPU", dict(X=fake((M, N), index=1))),
])
def test_bad_inputs_never_reach_the_library(ctx, what, change):
    a = dict(good(), **change)
    for call in (lambda: ctx.fit(a["X"], a["y"], 0.1, 3, a["w"], a["b"]),
                 lambda: ctx.loss_grad(a["X"], a["y"], a["w"], a["b"]),
                 lambda: ctx.predict(a["X"], a["w"], a["b"], 0.5) if "y" not in change else ctx.fit(a["X"], a["y"], 0.1, 1, a["w"], a["b"]),
                 lambda: ctx.fit_tol(a["X"], a["y"], 0.1, 1e-3, 5, a["w"], a["b"]),
                 lambda: ctx.fit_opt(a["X"], a["y"], 0.1, 3, a["w"], a["b"]),
                 lambda: ctx.fit_sgd(a["X"], a["y"], 0.1, 8, 3, a["w"], a["b"]),
                 lambda: ctx.shard_sums(a["X"], a["y"], a["w"], a["b"], fake(N + 2, torch.float64))):
        with pytest.raises(ValueError):
            call()
    assert ctx.rec.calls == [], what


def test_outputs_that_are_too_short_are_refused(ctx):
    a = good()
    with pytest.raises(ValueError):
        ctx.fit(a["X"], a["y"], 0.1, 10, a["w"], a["b"], fake(9))                       # history shorter than iters
    with pytest.raises(ValueError):
        ctx.predict(a["X"], a["w"], a["b"], 0.5, out=fake(M - 1, torch.uint8))          # labels shorter than m
    with pytest.raises(ValueError):
        ctx.fit_tol(a["X"], a["y"], 0.1, 1e-3, 12, a["w"], a["b"], gnorm_hist=fake(11))
    with pytest.raises(ValueError):
        ctx.fit_opt(a["X"], a["y"], 0.1, 3, a["w"], a["b"], velocity=fake(N))           # velocity needs n + 1
    with pytest.raises(ValueError):
        ctx.shard_sums(a["X"], a["y"], a["w"], a["b"], fake(N + 1, torch.float64))
    with pytest.raises(ValueError):
        ctx.apply_sums(fake((2, N + 2), torch.float64), 2 * M, 0.1, fake(N - 1), a["b"])
    with pytest.raises(ValueError):
        ctx.convert_bf16(fake((M, N)), out=fake((M, N - 1), torch.bfloat16))
    assert ctx.rec.calls == []


def test_wrong_dtype_or_layout_is_a_type_error(ctx):
    a = good()
    with pytest.raises(TypeError):
        ctx.fit(a["X"], fake(M, torch.float64), 0.1, 3, a["w"], a["b"])
    with pytest.raises(TypeError):
        ctx.fit(FakeCuda(torch.zeros((N, M)).t()), a["y"], 0.1, 3, a["w"], a["b"])      # a transposed view is not contiguous
    with pytest.raises(TypeError):
        ctx.fit(torch.zeros((M, N)), a["y"], 0.1, 3, a["w"], a["b"])                    # a CPU tensor
    assert ctx.rec.calls == []


def test_no_allocation_entry_point_checks_every_buffer(monkeypatch):
    rec = Recorder()
    monkeypatch.setattr(api, "lib", lambda: rec)
    monkeypatch.setattr(torch.cuda, "current_stream", lambda dev=None: type("S", (), {"cuda_stream": 0})())
    a = good()
    out = dict(loss=fake(1), grad_w=fake(N), grad_b=fake(1), status=fake(1, torch.int32))
    api.lr_loss_grad_noalloc(a["X"], a["y"], a["w"], a["b"], **out)
    assert rec.calls == ["lr_loss_grad_noalloc"]
    for key, bad in (("grad_w", fake(N - 1)), ("loss", fake(0)), ("grad_b", fake(0)), ("status", fake(0, torch.int32)),
                     ("grad_w", fake(N, index=1))):
        with pytest.raises(ValueError):
            api.lr_loss_grad_noalloc(a["X"], a["y"], a["w"], a["b"], **dict(out, **{key: bad}))
    with pytest.raises(ValueError):
        api.lr_loss_grad_noalloc(a["X"], fake(M - 1), a["w"], a["b"], **out)
    assert rec.calls == ["lr_loss_grad_noalloc"]


def test_host_entry_points_check_sizes(ctx):
    X, y = np.zeros((M, N), dtype=np.float32), np.zeros(M, dtype=np.float32)
    w, b = np.zeros(N, dtype=np.float32), np.zeros(1, dtype=np.float32)
    ctx.fit_host(X, y, 0.1, 3, w, b, np.zeros(3, dtype=np.float32))
    with pytest.raises(ValueError):
        ctx.fit_host(X, y[:-1], 0.1, 3, w, b)
    with pytest.raises(ValueError):
        ctx.fit_host(X, y, 0.1, 3, w, b, np.zeros(2, dtype=np.float32))
    with pytest.raises(ValueError):
        ctx.predict_host(X, w, b, 0.5, np.zeros(M - 1, dtype=np.uint8))
    assert ctx.rec.calls == ["lr_fit_host"]
