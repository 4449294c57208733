"""GPU parity for gradient descent with an L2 penalty and momentum (``lr_fit_opt``) against the checker's ``fit_opt``."""
import numpy as np
import pytest
import torch

import oracle
from _parity import LOSS_TOL, W_TOL, rel_l2
from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2308_10037_b200 import build
    build.build()
    c = api.Context(n_max=4096, device=0)
    yield c
    assert c.device_status() == 0
    assert c.check_guards() == 0                   # no kernel of the module wrote outside a workspace array
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_fit(ctx, dX, dy, n, lr, iters, **kw):
    w = torch.zeros(n, device="cuda")
    b = torch.zeros(1, device="cuda")
    lh = torch.empty(iters, device="cuda")
    ctx.fit_opt(dX, dy, lr, iters, w, b, loss_hist=lh, **kw)
    return w, b, lh


CASES = [("cfg1", 10_000, None, dict(l2=0.1, momentum=0.9)), ("cfg3", 40_003, None, dict(l2=0.01, momentum=0.5, nesterov=True)),
         ("cfg5", 90_001, None, dict(l2=0.0, momentum=0.8)), ("cfg2", 30_000, None, dict(l2=0.3, momentum=0.0)),
         ("cfg3", 5_003, 4096, dict(l2=0.05, momentum=0.6, nesterov=True)), ("cfg2", 9_000, 30, dict(l2=0.02, momentum=0.7))]


@pytest.mark.parametrize("name,m,n,opt", CASES)
def test_fit_opt_matches_oracle(ctx, name, m, n, opt):
    import dataclasses
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    if n is not None:
        wl = dataclasses.replace(wl, n=n)
    lr = min(wl.lr, 0.25)                      # momentum amplifies the step; keep the iteration a contraction
    iters = 30
    X, y, _, _ = datagen.generate(wl)
    w_ref, b_ref, v_ref, lh_ref = oracle.fit_opt(X, y, lr, iters, **opt)
    w, b, lh = gpu_fit(ctx, dev(X), dev(y), wl.n, lr, iters, **opt)
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(lh.cpu().numpy() - lh_ref)) <= LOSS_TOL


@pytest.mark.parametrize("name,m,n,batch", [("cfg3", 50_003, None, 8_192), ("cfg5", 120_001, None, 30_000), ("cfg2", 9_000, 30, 2_500),
                                            ("cfg3", 6_001, 2048, 1_000), ("cfg1", 10_000, None, 10_000)])
def test_minibatch_descent_matches_oracle(ctx, name, m, n, batch):
    import dataclasses
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    if n is not None:
        wl = dataclasses.replace(wl, n=n)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    steps, lr = 17, 0.2
    w_ref, b_ref, lh_ref = oracle.fit_sgd(X, y, lr, batch, steps)
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    lh = torch.empty(steps, device="cuda")
    ctx.fit_sgd(dX, dy, lr, batch, steps, w, b, loss_hist=lh)
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(lh.cpu().numpy() - lh_ref)) <= LOSS_TOL
    # split across two calls with first_batch: the same bits
    w2 = torch.zeros(wl.n, device="cuda")
    b2 = torch.zeros(1, device="cuda")
    ctx.fit_sgd(dX, dy, lr, batch, 6, w2, b2)
    ctx.fit_sgd(dX, dy, lr, batch, steps - 6, w2, b2, first_batch=6)
    assert torch.equal(w2, w) and torch.equal(b2, b)
    if batch == m:
        wf, bf = api.lr_fit(dX, dy, lr, steps, ctx=ctx)
        assert torch.equal(wf, w) and torch.equal(bf, b)        # one block per step is the plain fit
    with pytest.raises(api.LrError):
        ctx.fit_sgd(dX, dy, lr, m + 1, 1, w2, b2)


def test_defaults_reproduce_plain_fit_and_velocity_resumes(ctx):
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 20_000)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    w0, b0, lh0 = gpu_fit(ctx, dX, dy, wl.n, wl.lr, 11)
    wf, bf, hf = api.lr_fit(dX, dy, wl.lr, 11, return_history=True, ctx=ctx)
    assert torch.equal(w0, wf) and torch.equal(b0, bf) and torch.equal(lh0, hf)
    # a caller-owned velocity lets a run be split: 4 + 5 steps equal 9 steps bit for bit
    kw = dict(l2=0.02, momentum=0.8, nesterov=True)
    v = torch.zeros(wl.n + 1, device="cuda")
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    ctx.fit_opt(dX, dy, 0.2, 4, w, b, velocity=v, **kw)
    ctx.fit_opt(dX, dy, 0.2, 5, w, b, velocity=v, **kw)
    w9, b9, _ = gpu_fit(ctx, dX, dy, wl.n, 0.2, 9, **kw)
    assert torch.equal(w, w9) and torch.equal(b, b9)
    _, _, v_ref, _ = oracle.fit_opt(X, y, 0.2, 9, **kw)
    assert rel_l2(v.cpu().numpy(), v_ref) <= 1e-3       # the velocity is a gradient-sized quantity near convergence
    for bad in (dict(l2=-1.0), dict(momentum=1.0), dict(momentum=-0.1)):
        with pytest.raises(api.LrError) as e:
            ctx.fit_opt(dX, dy, 0.2, 1, w, b, **bad)
        assert e.value.code == api.LR_ERR_VALUE
