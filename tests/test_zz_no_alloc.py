"""The allocation-free entry point ``lr_loss_grad_noalloc`` against ``lr_loss_grad``.

Some callers cannot allocate device memory at the moment they need a loss/gradient pass (a loop that
must not take the allocator's lock or trigger a device-wide synchronisation, a process whose device
memory is already fully owned by another allocator, a host with a no-allocation-after-start rule).
For them the library keeps the scratch of the pass in a fixed array of its device image.  These tests
call that entry point through the C-ABI binding, twice in a row on different inputs (the second call
finds the first call's leftovers in the shared array), and compare with the context-based entry point.

This file sorts last on purpose: a run that stops at the first failure has then already run every other
test.  It also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu

GRAD_TOL, LOSS_TOL = 1e-5, 1e-6


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _rel_l2(a, b):
    a, b = a.double().cpu().numpy().ravel(), b.double().cpu().numpy().ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def _run_pair(ctx, m, n, seed):
    X, y, w, b = datagen.random_problem(m, n, seed=seed, wscale=1.5)
    dX, dy, dw, db = _dev(X), _dev(y), _dev(w), _dev(np.array([b], dtype=np.float32))
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


def test_two_calls_in_a_row_match_the_context_entry_point():
    from paper_2308_10037_b200 import build
    build.build()
    ctx = api.Context(n_max=1024, device=0)
    try:
        # first call: wide rows, many CTAs; second call: fewer columns and CTAs, so stale rows and columns of the first
        # call are still in the shared array when the second one runs
        _run_pair(ctx, 150_001, 256, seed=901)
        _run_pair(ctx, 3_001, 100, seed=902)
        # shapes served by the other kernel variants, again back to back
        _run_pair(ctx, 70_003, 32, seed=903)
        _run_pair(ctx, 20_000, 30, seed=904)        # n % 4 != 0: unstaged kernel, its grid is capped by the array size
        _run_pair(ctx, 900, 1020, seed=905)         # wide rows: the row-split kernel
        _run_pair(ctx, 800, 1022, seed=906)
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
