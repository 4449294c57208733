"""Full-size parity on the five benchmark workloads, in the launch configuration the benchmark times.

Each workload is generated once (seed 0), fitted on the GPU through ``lr_fit`` for its configured number of
iterations and by the float64 CPU checker on the same bits, and compared on: the loss history (abs <= 1e-6),
the final parameters (relative L2 <= 1e-4), teacher-forced gradients at checker iterates (relative L2 <= 1e-5, with the
fp32 noise floor of ``_parity`` for converged iterates),
and predicted labels (>= 99.99 % agreement; F1 for the imbalanced workload).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu

from _parity import (LABEL_AGREE, LOSS_TOL, W_TOL, allowed_drift, assert_grad_close, grad_noise_floor, record,
                     rel_l2)

# Workloads whose last iterates are converged so far that the fp32 noise floor of ``_parity`` may be the binding bound
# on the gradient.  Everywhere else the plain relative bar has to hold on its own.
FLOOR_ALLOWED = {"cfg2"}


@pytest.fixture(scope="module")
def ctx():
    from paper_2308_10037_b200 import build
    build.build()
    c = api.Context(n_max=4096, device=0)
    yield c
    assert c.device_status() == 0
    assert c.check_guards() == 0                   # no kernel of the module wrote outside a workspace array
    c.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_workload(ctx, name):
    wl = datagen.WORKLOADS[name]
    X, y, _, _ = datagen.generate(wl)
    dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()

    # the launch plan is the one the benchmark runs (same entry point, same shape)
    plan = api.plan_query(wl.m, wl.n, sm_count=torch.cuda.get_device_properties(0).multi_processor_count)
    assert plan["grid"] >= 1

    w, b, hist = api.lr_fit(dX, dy, wl.lr, wl.iters, return_history=True, ctx=ctx)
    torch.cuda.synchronize()
    w_ref, b_ref, hist_ref, wh, bh = oracle.fit(X, y, wl.lr, wl.iters, history=True)
    got = np.concatenate([w.cpu().numpy(), b.cpu().numpy()])
    ref = np.concatenate([w_ref, [b_ref]])

    # per-iteration parity at the checker's own iterates (no compounding)
    floor = grad_noise_floor(X)
    its = wl.iters
    for t in sorted({0, 1, its // 4, its // 2, 3 * its // 4, its - 10, its - 1}):
        w32, b32 = wh[t].astype(np.float32), np.float32(bh[t])
        L, g, g0 = oracle.loss_grad(X, y, w32.astype(np.float64), float(b32))
        dl, dg, dg0 = ctx.loss_grad(dX, dy, torch.from_numpy(w32).cuda(), torch.tensor([b32], device="cuda"))
        loss_err = abs(dl.item() - L)
        assert loss_err <= max(LOSS_TOL, abs(L) * 2.0 ** -23), (name, t)
        g_ref = np.concatenate([g, [g0]])
        rel, used_floor = assert_grad_close(np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()]), g_ref, floor, (name, t),
                                            floor_allowed=name in FLOOR_ALLOWED)
        record("full_size_iterate", workload=name, t=t, grad_rel_l2=rel, grad_norm=float(np.linalg.norm(g_ref)),
               bound="floor" if used_floor else "1e-5*|g|", floor=floor, grad_abs_err=rel * float(np.linalg.norm(g_ref)),
               loss=L, loss_abs_err=loss_err)

    w_rel = rel_l2(got, ref)
    hist_err = float(np.max(np.abs(hist.cpu().numpy().astype(np.float64) - hist_ref)))
    if name == "cfg4":
        # Not a contraction at lr = 0.05 (uncentred U[0,1) features: the top Hessian eigenvalue is ~250, 2/lr is 40): the
        # loss oscillates between ~4.7 and ~8 and deviations are amplified along the trajectory.  The final parameters are
        # nevertheless held to the plain bar.  The loss history is held to the drift the checker itself shows when one
        # tolerance-sized deviation is injected (see allowed_drift), and never below one fp32 spacing of the values
        # (the history is stored as fp32 and the values reach 8: spacing 9.5e-7).
        w_r, b_r, _ = oracle.fit(X, y, wl.lr, wl.iters, round_to_fp32=True)
        own = rel_l2(np.concatenate([w_r, [b_r]]), ref)
        drift_w, drift_l = allowed_drift(X, y, wl, ref, hist_ref)
        hist_bound = max(LOSS_TOL, float(np.max(np.abs(hist_ref))) * 2.0 ** -23, drift_l)
        record("full_size_fit", workload=name, w_rel_l2=w_rel, w_bound=W_TOL, loss_hist_max_abs_err=hist_err,
               loss_hist_bound=hist_bound, checker_fp32_rounded_rerun_rel_l2=own, checker_drift_w=drift_w,
               checker_drift_loss=drift_l)
        assert w_rel <= W_TOL, (w_rel, own, drift_w)
        assert hist_err <= hist_bound, (hist_err, hist_bound)
    else:
        record("full_size_fit", workload=name, w_rel_l2=w_rel, w_bound=W_TOL, loss_hist_max_abs_err=hist_err,
               loss_hist_bound=LOSS_TOL)
        assert w_rel <= W_TOL
        assert hist_err <= LOSS_TOL

    # labels: both sides predict at the checker's fitted parameters (rounded to fp32, the storage type of the GPU path);
    # the imbalanced workload is also scored near its 1 % base rate, where positives are actually predicted
    w32, b32 = w_ref.astype(np.float32), np.float32(b_ref)
    dw32, db32 = torch.from_numpy(w32).cuda(), torch.tensor([b32], device="cuda")
    for thr in ([wl.predict_thr or 0.5] + ([0.05] if name == "cfg5" else [])):
        labels = ctx.predict(dX, dw32, db32, thr).cpu().numpy()
        lab_ref = oracle.predict(X, w32.astype(np.float64), float(b32), thr)
        agree = float((labels == lab_ref).mean())
        record("full_size_labels", workload=name, thr=thr, agreement=agree, rows_differing=int((labels != lab_ref).sum()),
               f1_gpu=oracle.f1_score(labels, y)[0], f1_checker=oracle.f1_score(lab_ref, y)[0])
        assert agree >= LABEL_AGREE, (name, thr)
        assert abs(oracle.f1_score(labels, y)[0] - oracle.f1_score(lab_ref, y)[0]) <= 1e-3
    # and free-running: labels from the GPU's own fit against labels from the checker's own fit
    own_labels = api.lr_predict(dX, w, b, 0.5, ctx=ctx).cpu().numpy()
    agree = float((own_labels == oracle.predict(X, w_ref, b_ref, 0.5)).mean())
    record("full_size_labels_free_running", workload=name, thr=0.5, agreement=agree)
    assert agree >= LABEL_AGREE


def test_more_than_2_to_31_elements(ctx):
    # 36,000,007 x 64 = 2.3e9 elements (9.2 GB): element offsets pass 2^31 and byte offsets pass 2^33, with a ragged tail.
    # One pass at non-trivial parameters against the checker, and labels on the last rows (the ones with the largest offsets).
    import dataclasses
    wl = dataclasses.replace(datagen.WORKLOADS["cfg5"], m=36_000_007, name="cfg5_big")
    X, y, wstar, bstar = datagen.generate(wl)
    dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    w32 = (0.5 * wstar).astype(np.float32)
    b32 = np.float32(0.5 * bstar)
    dw, db = torch.from_numpy(w32).cuda(), torch.tensor([b32], device="cuda")
    L, g, g0 = oracle.loss_grad(X, y, w32.astype(np.float64), float(b32))
    dl, dg, dg0 = ctx.loss_grad(dX, dy, dw, db)
    assert abs(dl.item() - L) <= LOSS_TOL
    assert_grad_close(np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()]), np.concatenate([g, [g0]]), 0.0, "big")
    labels = ctx.predict(dX, dw, db, 0.02).cpu().numpy()
    tail = slice(wl.m - 2_000_000, wl.m)
    ref = oracle.predict(X[tail], w32.astype(np.float64), float(b32), 0.02)
    assert (labels[tail] == ref).mean() >= LABEL_AGREE
    del dX, dy
    torch.cuda.empty_cache()
