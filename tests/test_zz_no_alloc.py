"""The allocation-free entry point ``lr_loss_grad_noalloc`` against ``lr_loss_grad`` and the float64 CPU checker.

Some callers cannot allocate device memory at the moment they need a loss/gradient pass (a loop that
must not take the allocator's lock or trigger a device-wide synchronisation, a process whose device
memory is already fully owned by another allocator, a host with a no-allocation-after-start rule).
For them the library keeps the scratch of the pass in a fixed array of its device image.  These tests
call that entry point through the C-ABI binding, twice in a row on different inputs (the second call
finds the first call's leftovers in the shared array), and compare with the context-based entry point and, since
that one runs the same kernels, also with the float64 CPU checker at the stated bars (loss 1e-6 absolute, gradient
1e-5 relative L2).

This file sorts last on purpose: a run that stops at the first failure has then already run every other
test.  It also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu

GRAD_TOL, LOSS_TOL = 1e-5, 1e-6


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _rel_l2(a, b):
    a, b = a.double().cpu().numpy().ravel(), b.double().cpu().numpy().ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def _run_pair(ctx, m, n, seed, shift=0):
    X, y, w, b = datagen.random_problem(m, n, seed=seed, wscale=1.5)
    dy, dw, db = _dev(y), _dev(w), _dev(np.array([b], dtype=np.float32))
    if shift:
        # a view that starts `shift` floats into an allocation: X is then 4-byte aligned only
        buf = torch.full((X.size + 8,), float("nan"), dtype=torch.float32, device="cuda")
        buf[shift:shift + X.size] = _dev(X).ravel()
        dX = buf[shift:shift + X.size].view(m, n)
        assert dX.data_ptr() % 16 == 4 * shift
    else:
        dX = _dev(X)
    # every buffer the call touches exists before the call
    loss = torch.full((1,), float("nan"), device="cuda")
    gw = torch.full((n,), float("nan"), device="cuda")
    gb = torch.full((1,), float("nan"), device="cuda")
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    api.lr_loss_grad_noalloc(dX, dy, dw, db, loss, gw, gb, status)
    ref_loss, ref_gw, ref_gb = ctx.loss_grad(dX, dy, dw, db)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert abs(loss.item() - ref_loss.item()) <= LOSS_TOL
    assert _rel_l2(torch.cat([gw, gb]), torch.cat([ref_gw, ref_gb])) <= GRAD_TOL
    # and against the float64 checker
    L, g, g0 = oracle.loss_grad(X, y, w.astype(np.float64), float(b))
    assert abs(loss.item() - L) <= LOSS_TOL
    got = torch.cat([gw, gb]).double().cpu().numpy()
    ref = np.concatenate([g, [g0]])
    assert np.linalg.norm(got - ref) <= GRAD_TOL * np.linalg.norm(ref)


def test_two_calls_in_a_row_match_the_context_entry_point_and_the_checker():
    from paper_2308_10037_b200 import build
    build.build()
    ctx = api.Context(n_max=1024, device=0)
    try:
        # first call: 256 columns, many CTAs; second call: fewer columns and CTAs, so stale rows and columns of the first
        # call are still in the shared array when the second one runs
        _run_pair(ctx, 150_001, 256, seed=901)
        _run_pair(ctx, 3_001, 100, seed=902)
        # the other instantiations of the two narrow-row staged kernels the entry point can take, again back to back
        _run_pair(ctx, 70_003, 32, seed=903)        # 16-byte groups, 8 lanes per row
        _run_pair(ctx, 20_000, 30, seed=904)        # n % 4 != 0: the element-wise staged kernel
        _run_pair(ctx, 900, 1020, seed=905)         # 16-byte groups, eight warps per CTA
        _run_pair(ctx, 800, 1022, seed=906)         # the largest n, not a whole number of 16-byte groups: CTA-wide stages
        _run_pair(ctx, 2_001, 777, seed=909, shift=1)    # the same kernel on a matrix that is 4-byte aligned only
        _run_pair(ctx, 40_001, 449, seed=907, shift=1)   # X 4-byte aligned only: element-wise kernel, head and tail by plain loads
        _run_pair(ctx, 5_003, 64, seed=908, shift=3)
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_sizes_beyond_the_fixed_array_are_rejected():
    n = api.LR_NOALLOC_MAX_N + 2
    X = torch.zeros((8, n), device="cuda")
    y = torch.zeros(8, device="cuda")
    w = torch.zeros(n, device="cuda")
    b = torch.zeros(1, device="cuda")
    loss, gw, gb = torch.zeros(1, device="cuda"), torch.zeros(n, device="cuda"), torch.zeros(1, device="cuda")
    with pytest.raises(api.LrError) as e:
        api.lr_loss_grad_noalloc(X, y, w, b, loss, gw, gb)
    assert e.value.code == api.LR_ERR_SHAPE
