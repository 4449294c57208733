"""Seeded random shapes through every entry point that computes, against the float64 checker.

The shape list is drawn once from a fixed seed, so the test is reproducible; it mixes the three kernel families
(narrow staged rows of whole groups and of any length, wide rows, unstaged), tiny and ragged row counts, and iteration counts that make the
persistent fit kernel wrap its stages across iteration boundaries in every phase.
"""
import numpy as np
import pytest
import torch

import oracle
from _parity import GRAD_TOL, LABEL_AGREE, LOSS_TOL, W_TOL, rel_l2
from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu


def _shapes():
    g = np.random.Generator(np.random.Philox(key=np.array([2308, 10037], dtype=np.uint64)))
    out = []
    for k in range(36):
        family = k % 3
        if family == 0:
            n = int(g.integers(1, 129)) * 4                     # staged narrow rows: 4 .. 512
        elif family == 1:
            n = int(g.integers(129, 2049)) * 4                  # wide rows: 516 .. 8192 (eight-warp and row-split kernels)
        else:
            n = int(g.integers(1, 700))                         # anything, mostly not a multiple of 4
        budget = 6_000_000 // n                                 # keep each case at a few MB
        m = int(g.integers(1, max(2, min(budget, 60_000))))
        iters = int(g.integers(2, 9))
        out.append((m, n, iters, 7000 + k))
    for k in range(36, 40):                                     # rows beyond 8192 columns: CTA-wide stages, one row per batch
        n = int(g.integers(8193, 16385))
        out.append((int(g.integers(1, 500)), n, int(g.integers(2, 6)), 7000 + k))
    return out


@pytest.fixture(scope="module")
def ctx():
    from paper_2308_10037_b200 import build
    build.build()
    c = api.Context(n_max=16384, device=0)
    yield c
    assert c.device_status() == 0
    assert c.check_guards() == 0                   # no kernel of the module wrote outside a workspace array
    c.close()


@pytest.mark.parametrize("m,n,iters,seed", _shapes())
def test_random_shape(ctx, m, n, iters, seed):
    X, y, w, b = datagen.random_problem(m, n, seed=seed, wscale=1.0)
    dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    dw, db = torch.from_numpy(w).cuda(), torch.tensor([b], device="cuda")
    # one pass
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    dl, dg, dg0 = ctx.loss_grad(dX, dy, dw, db)
    assert abs(dl.item() - L) <= LOSS_TOL
    assert rel_l2(np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()]), np.concatenate([g, [g0]])) <= GRAD_TOL
    # a short fit from that point (lr small enough for any of these shapes)
    lr = 0.05
    w_ref, b_ref, lh_ref = oracle.fit(X, y, lr, iters, w0=w, b0=b)
    ctx.set_persistent(True)                       # the persistent kernel wherever the shape allows it ...
    try:
        wf, bf, hf = api.lr_fit(dX, dy, lr, iters, w0=dw, b0=db, return_history=True, ctx=ctx)
    finally:
        ctx.set_persistent(None)
    wa, ba, ha = api.lr_fit(dX, dy, lr, iters, w0=dw, b0=db, return_history=True, ctx=ctx)   # ... and the library's own choice
    assert torch.equal(wf, wa) and torch.equal(bf, ba) and torch.equal(hf, ha)
    assert rel_l2(np.concatenate([wf.cpu().numpy(), bf.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(hf.cpu().numpy() - lh_ref)) <= LOSS_TOL
    # labels at the checker's parameters
    w32 = w_ref.astype(np.float32)
    ref, z = oracle.predict(X, w32.astype(np.float64), float(np.float32(b_ref)), 0.4, return_z=True)
    got = ctx.predict(dX, torch.from_numpy(w32).cuda(), torch.tensor([np.float32(b_ref)], device="cuda"), 0.4).cpu().numpy()
    clear = np.abs(z - np.log(0.4 / 0.6)) > 1e-4 * (1 + np.abs(z))
    assert np.array_equal(got[clear], ref[clear])
    assert (got == ref).mean() >= LABEL_AGREE or (got != ref).sum() <= 1
