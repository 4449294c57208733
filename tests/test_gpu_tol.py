"""GPU parity for gradient descent with the paper's stopping rule (Algorithm 7): ``lr_fit_tol`` against the checker's
``fit_tol`` on the same seeded inputs.

The number of updates is an integer decided by a floating-point comparison.  Both sides decide in float64 from their
own gradient; the tests pick tolerances that sit clearly between two consecutive gradient norms of the checker's run
(far outside the fp32 noise of the GPU's gradient), where the count is unique, and check the norm history itself to
the gradient bar.
"""
import numpy as np
import pytest
import torch

import oracle
from _parity import GRAD_TOL, LOSS_TOL, W_TOL, rel_l2
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


def run_gpu(ctx, dX, dy, n, lr, eps, max_iters, check_every=16):
    w = torch.zeros(n, device="cuda")
    b = torch.zeros(1, device="cuda")
    lh = torch.full((max_iters,), float("nan"), device="cuda")
    gh = torch.full((max_iters,), float("nan"), device="cuda")
    k, nrm = ctx.fit_tol(dX, dy, lr, eps, max_iters, w, b, check_every=check_every, loss_hist=lh, gnorm_hist=gh)
    return w, b, k, nrm, lh.cpu().numpy(), gh.cpu().numpy()


# cfg4's own recipe (uncentred features, lr 0.05) makes GD oscillate, so its gradient norm never settles below a
# threshold; the wide-row kernels are exercised with the cfg3 recipe widened to 2048 and 4096 columns instead
CASES = [("cfg1", 10_000, 60, None), ("cfg3", 40_003, 40, None), ("cfg5", 120_001, 40, None), ("cfg3", 6_001, 40, 2048),
         ("cfg3", 5_003, 30, 4096), ("cfg2", 20_000, 40, 30), ("higgs_like", 90_007, 60, None),
         # problems that fit one thread-block cluster (the library's own choice of form then differs from the forced ones)
         ("cfg5", 12_001, 40, None), ("cfg3", 1_500, 40, None), ("cfg1", 4_100, 60, None)]


@pytest.mark.parametrize("name,m,max_iters,n", CASES)
def test_stops_at_the_same_iteration_as_the_checker(ctx, name, m, max_iters, n):
    import dataclasses
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    if n is not None:
        wl = dataclasses.replace(wl, n=n)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    _, _, _, _, lh_all, gh_all = oracle.fit_tol(X, y, wl.lr, 0.0, max_iters)
    # a stopping index whose norm is a new minimum, and a tolerance halfway (in log) to the previous minimum
    run_min = np.minimum.accumulate(gh_all)
    cands = [t for t in range(2, max_iters) if gh_all[t] < 0.98 * run_min[t - 1]]
    assert cands, "no clearly decreasing norm to stop at"
    t_stop = cands[len(cands) // 2]
    eps = float(np.sqrt(gh_all[t_stop] * run_min[t_stop - 1]))
    w_ref, b_ref, k_ref, n_ref, lh_ref, gh_ref = oracle.fit_tol(X, y, wl.lr, eps, max_iters)
    assert k_ref == t_stop + 1

    ctx.set_persistent(True)                                               # the rule inside the persistent kernel (narrow rows)
    try:
        w, b, k, nrm, lh, gh = run_gpu(ctx, dX, dy, wl.n, wl.lr, eps, max_iters)
    finally:
        ctx.set_persistent(None)
    assert k == k_ref
    assert abs(nrm - n_ref) <= 1e-4 * n_ref
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(lh[:k] - lh_ref)) <= LOSS_TOL
    assert np.max(np.abs(gh[:k] - gh_ref) / gh_ref) <= 10 * GRAD_TOL       # free-running iterates: parameters differ by <= W_TOL
    assert np.isnan(lh[k:]).all() and np.isnan(gh[k:]).all()               # nothing is written after the stop

    # the library's own choice of form (one thread-block cluster where the problem fits one): the same bits, one launch
    n0 = ctx.launch_count()
    w1, b1, k1, nrm1, lh1, gh1 = run_gpu(ctx, dX, dy, wl.n, wl.lr, eps, max_iters)
    if api.plan_query(wl.m, wl.n)["variant"] == 0:
        assert ctx.launch_count() == n0 + 1
    assert k1 == k and nrm1 == nrm and torch.equal(w1, w) and torch.equal(b1, b)
    assert np.array_equal(gh1[:k], gh[:k]) and np.isnan(gh1[k:]).all()
    assert np.array_equal(lh1[:k], lh[:k]) and np.isnan(lh1[k:]).all()

    # narrow rows stop inside one persistent launch; the two-kernel form (a device flag turns later launches into no-ops)
    # must give the same bits, however often the host looks at the flag
    ctx.set_persistent(False)
    try:
        for ce in (1, 5, 1000):
            w2, b2, k2, nrm2, lh2, gh2 = run_gpu(ctx, dX, dy, wl.n, wl.lr, eps, max_iters, check_every=ce)
            assert k2 == k and nrm2 == nrm and torch.equal(w2, w) and torch.equal(b2, b)
            assert np.array_equal(gh2[:k], gh[:k]) and np.isnan(gh2[k:]).all()
            assert np.array_equal(lh2[:k], lh[:k]) and np.isnan(lh2[k:]).all()
    finally:
        ctx.set_persistent(None)


def test_limits_of_the_rule(ctx):
    wl = datagen.scaled(datagen.WORKLOADS["cfg2"], 30_000)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    # eps = 0 never stops early and equals lr_fit bit for bit
    w, b, k, nrm, lh, gh = run_gpu(ctx, dX, dy, wl.n, wl.lr, 0.0, 23, check_every=4)
    wf, bf, hf = api.lr_fit(dX, dy, wl.lr, 23, return_history=True, ctx=ctx)
    assert k == 23 and torch.equal(w, wf) and torch.equal(b, bf) and np.array_equal(lh, hf.cpu().numpy())
    # a huge tolerance still applies exactly one update (Algorithm 7 tests after updating)
    w1, b1, k1, nrm1, _, gh1 = run_gpu(ctx, dX, dy, wl.n, wl.lr, 1e9, 23)
    w1f, b1f = api.lr_fit(dX, dy, wl.lr, 1, ctx=ctx)
    assert k1 == 1 and torch.equal(w1, w1f) and torch.equal(b1, b1f) and nrm1 == gh1[0]
    _, g, g0 = oracle.loss_grad(X, y, np.zeros(wl.n), 0.0)
    assert abs(nrm1 - np.sqrt(g @ g + g0 * g0)) <= GRAD_TOL * nrm1
    # no iterations
    w0 = torch.ones(wl.n, device="cuda")
    b0 = torch.ones(1, device="cuda")
    assert ctx.fit_tol(dX, dy, wl.lr, 1.0, 0, w0, b0) == (0, -1.0) and bool((w0 == 1).all())
    for bad in (dict(eps=-1.0), dict(eps=float("nan")), dict(check_every=0)):
        kw = dict(eps=0.1, check_every=4)
        kw.update(bad)
        with pytest.raises(api.LrError):
            ctx.fit_tol(dX, dy, wl.lr, kw["eps"], 5, w0, b0, check_every=kw["check_every"])


@pytest.mark.parametrize("lr,eps", [(0.1, 0.01), (0.01, 0.008)])
def test_higgs_shaped_runs_with_the_papers_hyperparameters(ctx, lr, eps):
    # the two (alpha, epsilon) settings of the paper's Tables I and II on a 28-feature stand-in (the HIGGS data itself is
    # not available): both sides must stop after the same number of updates unless the crossing is within fp32 noise
    wl = datagen.scaled(datagen.WORKLOADS["higgs_like"], 300_000)
    X, y, _, _ = datagen.generate(wl)
    w_ref, b_ref, k_ref, n_ref, lh_ref, gh_ref = oracle.fit_tol(X, y, lr, eps, 3000)
    w, b, k, nrm, lh, gh = run_gpu(ctx, dev(X), dev(y), wl.n, lr, eps, 3000, check_every=32)
    margin = min(abs(gh_ref[-1] - eps), abs(gh_ref[-2] - eps) if k_ref > 1 else 1.0) / eps
    if margin > 1e-4:
        assert k == k_ref
    else:
        assert abs(k - k_ref) <= 1
    assert nrm <= eps or k == 3000
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= 10 * W_TOL
