"""GPU parity for the bfloat16 storage variant of X, through the C-ABI binding.

The conversion kernel is compared bit for bit with the checker's rounding.  The three bfloat16 entry points are compared
with the float64 checker run on the SAME values (the rounded matrix widened back to fp32), so the tolerances are those
of the fp32 path: gradient relative L2 <= 1e-5, loss absolute <= 1e-6, fitted parameters relative L2 <= 1e-4, labels
agreeing on >= 99.99 % of rows.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_10037_b200 import api, datagen

pytestmark = pytest.mark.gpu

from _parity import GRAD_TOL, LABEL_AGREE, LOSS_TOL, W_TOL, assert_grad_close, grad_noise_floor, record, rel_l2


@pytest.fixture(scope="module")
def ctx():
    from paper_2308_10037_b200 import build
    build.build()
    c = api.Context(n_max=16400, device=0)
    yield c
    assert c.device_status() == 0
    assert c.check_guards() == 0                   # no kernel of the module wrote outside a workspace array
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_bf16(bits):
    """uint16 bfloat16 patterns (numpy) -> a CUDA bfloat16 tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_conversion_is_bit_exact(ctx):
    rng = np.random.default_rng(5)
    # random patterns (all exponents, subnormals, infinities, NaNs), a sweep across ties, and a ragged tail
    x = rng.integers(0, 1 << 32, size=1_000_003, dtype=np.uint64).astype(np.uint32)
    top = rng.integers(0, 1 << 16, size=20_000, dtype=np.uint64).astype(np.uint32) << 16
    x = np.concatenate([x, top | 0x7FFF, top | 0x8000, top | 0x8001]).view(np.float32)
    want, _ = oracle.round_bf16(x)
    got = ctx.convert_bf16(dev(x)).view(torch.int16).cpu().numpy().view(np.uint16)
    nan = np.isnan(x)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.all((got[nan] & 0x7FFF) > 0x7F80) and np.array_equal(got[nan] >> 15, want[nan] >> 15)   # NaN stays NaN, sign kept
    # unaligned source and destination take the element-wise path; an empty input is accepted
    buf = torch.zeros(x.size + 1, dtype=torch.float32, device="cuda")
    buf[1:] = dev(x)
    out = torch.zeros(x.size + 1, dtype=torch.bfloat16, device="cuda")
    ctx.convert_bf16(buf[1:], out=out[1:])
    got2 = out[1:].view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got2[~nan], want[~nan])
    ctx.convert_bf16(torch.empty(0, dtype=torch.float32, device="cuda"))


def check_loss_grad(ctx, Xv, dXh, y, w, b, loss_tol=LOSS_TOL):
    L, g, g0 = oracle.loss_grad(Xv, y, np.asarray(w, dtype=np.float64), float(b))
    dl, dg, dg0 = ctx.loss_grad(dXh, dev(y), dev(np.asarray(w, dtype=np.float32)), dev(np.array([b], dtype=np.float32)))
    torch.cuda.synchronize()
    assert abs(dl.item() - L) <= loss_tol, (dl.item(), L)
    got = np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()])
    assert rel_l2(got, np.concatenate([g, [g0]])) <= GRAD_TOL
    return got


# every staged instantiation for 8-column groups (n/8 <= 8, 16, 32, 64), partly filled lane groups, the wide-row kernel
# (n/8 > 64: full and partly idle warp slices), rows beyond 8192 columns (CTA-wide stages, one row per batch), the unstaged kernel (n > 16384), tiny / ragged / many-tile rows
SHAPES = [(1, 8), (7, 8), (9, 5), (33, 56), (1000, 64), (4097, 64), (5003, 128), (2500, 72), (3001, 100), (9999, 256),
          (777, 200), (1500, 512), (2049, 264), (640, 30), (300, 1), (50, 8200), (301, 8193), (97, 16384), (20, 16392), (20011, 16), (1025, 36),
          (200_003, 256), (400_001, 64), (200_002, 128), (150_001, 24), (60_001, 512), (90_001, 200), (120_007, 104),
          (5_001, 4096), (20_003, 1024), (2_500, 520), (1_203, 2056), (701, 4088), (9_000, 2048), (3, 8192), (130, 8192),
          (1_001, 6000)]


@pytest.mark.parametrize("m,n", SHAPES)
def test_loss_grad_matches_oracle(ctx, m, n):
    X, y, w, b = datagen.random_problem(m, n, seed=2000 + m + n, wscale=1.5)
    bits, Xv = oracle.round_bf16(X)
    check_loss_grad(ctx, Xv, dev_bf16(bits), y, w, b)


# both sides of every boundary between the bfloat16 kernel shapes
@pytest.mark.parametrize("n", [8, 16, 64, 72, 128, 136, 256, 264, 512, 520, 1024, 1032, 2048, 2056, 4096, 4104, 8192, 8200, 12288, 12296, 16384, 16392, 9, 65,
                               257, 511, 516])
def test_shape_boundaries_bf16(ctx, n):
    m = max(40, min(60_001, 24_000_000 // n)) + 3
    X, y, w, b = datagen.random_problem(m, n, seed=6500 + n, wscale=1.0)
    bits, Xv = oracle.round_bf16(X)
    check_loss_grad(ctx, Xv, dev_bf16(bits), y, w, b)


def test_library_conversion_feeds_the_pass(ctx):
    # fp32 on the device -> lr_convert_bf16 -> lr_loss_grad_bf16, against the checker on its own rounding of the same X
    X, y, w, b = datagen.random_problem(30_011, 256, seed=31, wscale=1.0)
    _, Xv = oracle.round_bf16(X)
    check_loss_grad(ctx, Xv, ctx.convert_bf16(dev(X)), y, w, b)


@pytest.mark.parametrize("m,n,shift", [(1201, 64, 1), (90_001, 30, 3), (40_001, 449, 5), (7, 3, 7), (20_001, 520, 1), (2_001, 1032, 1)])
def test_bf16_views_that_are_only_2_byte_aligned(ctx, m, n, shift):
    # narrow rows stay on a staged kernel (element-wise; the first batch is completed with plain loads instead of reading
    # in front of the matrix, which is surrounded by NaN here); wide rows run unstaged
    X, y, w, b = datagen.random_problem(m, n, seed=13 + m + n)
    bits, Xv = oracle.round_bf16(X)
    buf = torch.full((bits.size + 16,), float("nan"), dtype=torch.bfloat16, device="cuda")
    buf[shift:shift + bits.size] = dev_bf16(bits).ravel()
    Xh = buf[shift:shift + bits.size].view(m, n)
    assert Xh.data_ptr() % 16 == 2 * shift
    assert api.plan_query(m, n, x_aligned16=False, bf16=True)["variant"] == (3 if n <= 512 else 4)
    check_loss_grad(ctx, Xv, Xh, y, w, b)


# bfloat16 rows whose length is not a multiple of eight: every element-wise instantiation, batches that start off a
# 16-byte boundary, ragged tails, stage reuse; pass, labels and a short fit
@pytest.mark.parametrize("m,n", [(33, 7), (1, 3), (40_003, 13), (150_001, 30), (100_001, 100), (200_003, 255), (2_758, 449),
                                 (60_001, 449), (50_002, 508), (5, 510), (17, 257), (30_001, 1020), (20_003, 777),
                                 (9_001, 4100), (3_001, 8191), (20_001, 1025), (7, 8190), (12_001, 2049)])
def test_bf16_rows_of_any_length(ctx, m, n):
    assert api.plan_query(m, n, bf16=True)["variant"] == (3 if n <= 512 else 4)
    X, y, w, b = datagen.random_problem(m, n, seed=3500 + m + n, wscale=1.5)
    bits, Xv = oracle.round_bf16(X)
    dXh = dev_bf16(bits)
    check_loss_grad(ctx, Xv, dXh, y, w, b)
    dw, db = dev(w), dev(np.array([b], dtype=np.float32))
    ref, z = oracle.predict(Xv, w, b, 0.4, return_z=True)
    got = ctx.predict(dXh, dw, db, 0.4).cpu().numpy()
    clear = np.abs(z - np.log(0.4 / 0.6)) > 1e-4 * (1 + np.abs(z))
    assert np.array_equal(got[clear], ref[clear])
    iters, lr = 6, 0.1
    w_ref, b_ref, lh_ref = oracle.fit(Xv, y, lr, iters, w0=w, b0=b)
    hist = torch.empty(iters, device="cuda")
    ctx.fit(dXh, dev(y), lr, iters, dw, db, hist)
    assert rel_l2(np.concatenate([dw.cpu().numpy(), db.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(hist.cpu().numpy() - lh_ref)) <= LOSS_TOL


SMALL_WORKLOADS = [("cfg1", 10_000), ("cfg3", 30_011), ("cfg4", 3_000), ("cfg5", 100_003)]


@pytest.mark.parametrize("name,m", SMALL_WORKLOADS)
def test_teacher_forced_trajectory(ctx, name, m):
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    iters = min(wl.iters, 40)
    _, _, lh, wh, bh = oracle.fit(Xv, y, wl.lr, iters, history=True)
    dXh, dy = dev_bf16(bits), dev(y)
    floor = grad_noise_floor(Xv)
    for t in sorted({0, 1, 2, iters // 2, iters - 1}):
        w32 = wh[t].astype(np.float32)
        b32 = np.float32(bh[t])
        L, g, g0 = oracle.loss_grad(Xv, y, w32.astype(np.float64), float(b32))
        dl, dg, dg0 = ctx.loss_grad(dXh, dy, dev(w32), dev(np.array([b32])))
        assert abs(dl.item() - L) <= LOSS_TOL, (t, dl.item(), L)
        got = np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()])
        assert_grad_close(got, np.concatenate([g, [g0]]), floor, (name, t))


@pytest.mark.parametrize("name,m", [("cfg1", 10_000), ("cfg3", 30_011), ("cfg5", 100_003)])
def test_fit_and_predict_match_oracle(ctx, name, m):
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    iters = min(wl.iters, 60)
    w_ref, b_ref, lh_ref = oracle.fit(Xv, y, wl.lr, iters)
    dXh, dy = dev_bf16(bits), dev(y)
    hist = torch.empty(iters, dtype=torch.float32, device="cuda")
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    ctx.set_persistent(True)
    ctx.fit(dXh, dy, wl.lr, iters, w, b, hist)                    # one persistent launch
    got = np.concatenate([w.cpu().numpy(), b.cpu().numpy()])
    assert rel_l2(got, np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(hist.cpu().numpy() - lh_ref)) <= LOSS_TOL
    # the two-kernel form gives the same bits
    ctx.set_persistent(False)
    w2 = torch.zeros(wl.n, device="cuda")
    b2 = torch.zeros(1, device="cuda")
    ctx.fit(dXh, dy, wl.lr, iters, w2, b2)
    ctx.set_persistent(None)
    assert torch.equal(w, w2) and torch.equal(b, b2)
    # predict at two thresholds; rows within fp32 noise of the cut may fall on either side
    for thr in (0.5, 0.3):
        lab_ref, z = oracle.predict(Xv, w.cpu().numpy().astype(np.float64), float(b.item()), thr, return_z=True)
        lab = ctx.predict(dXh, w, b, thr).cpu().numpy()
        cut = np.log(thr / (1 - thr))
        clear = np.abs(z - cut) > 1e-4 * (1.0 + np.abs(z))
        assert np.array_equal(lab[clear], lab_ref[clear])
        assert (lab == lab_ref).mean() >= LABEL_AGREE


def test_host_entry_points_with_bfloat16_storage(ctx):
    # fp32 rows on the host, rounded to bfloat16 on the device after the copy: the result is the device-pointer fit on the
    # library's own conversion, bit for bit, and the checker's fit on its own rounding within the tolerances
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 30_011)
    X, y, _, _ = datagen.generate(wl)
    iters = 9
    w = np.zeros(wl.n, dtype=np.float32)
    b = np.zeros(1, dtype=np.float32)
    hist = np.zeros(iters, dtype=np.float32)
    ctx.fit_host(X, y, wl.lr, iters, w, b, hist, store_bf16=True)
    dXh = ctx.convert_bf16(dev(X))
    dw = torch.zeros(wl.n, device="cuda")
    db = torch.zeros(1, device="cuda")
    dh = torch.empty(iters, device="cuda")
    ctx.fit(dXh, dev(y), wl.lr, iters, dw, db, dh)
    assert np.array_equal(w, dw.cpu().numpy()) and np.array_equal(b, db.cpu().numpy()) and np.array_equal(hist, dh.cpu().numpy())
    _, Xv = oracle.round_bf16(X)
    w_ref, b_ref, lh_ref = oracle.fit(Xv, y, wl.lr, iters)
    assert rel_l2(np.concatenate([w, b]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(hist - lh_ref)) <= LOSS_TOL
    labels = np.zeros(wl.m, dtype=np.uint8)
    ctx.predict_host(X, w, b, 0.4, labels, store_bf16=True)
    assert np.array_equal(labels, ctx.predict(dXh, dw, db, 0.4).cpu().numpy())
    assert (labels == oracle.predict(Xv, w.astype(np.float64), float(b[0]), 0.4)).mean() >= LABEL_AGREE


def test_wide_rows_fit(ctx):
    # the wide-row kernel iterates as two kernels per step
    wl = datagen.scaled(datagen.WORKLOADS["cfg4"], 3_000)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    iters = 8
    w_ref, b_ref, lh_ref = oracle.fit(Xv, y, wl.lr, iters)
    hist = torch.empty(iters, dtype=torch.float32, device="cuda")
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    ctx.fit(dev_bf16(bits), dev(y), wl.lr, iters, w, b, hist)
    # this workload is not a contraction (the iterates oscillate), so early iterates are compared, loosely on w
    assert np.max(np.abs(hist.cpu().numpy()[:3] - lh_ref[:3])) <= 1e-5 * max(1.0, float(np.max(lh_ref[:3])))
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= 1e-2


def test_argument_checks(ctx):
    Xh = torch.zeros((16, 8), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(16, device="cuda")
    w = torch.zeros(8, device="cuda")
    b = torch.zeros(1, device="cuda")
    L = api.lib()
    import ctypes
    P = lambda t: ctypes.c_void_p(t.data_ptr() if t is not None else None)
    out = torch.zeros(10, device="cuda")
    assert L.lr_loss_grad_bf16(ctx._h, None, P(y), 16, 8, P(w), P(b), P(out), P(out[1:]), P(out[9:]), None) == api.LR_ERR_NULL
    assert L.lr_loss_grad_bf16(ctx._h, ctypes.c_void_p(Xh.data_ptr() + 1), P(y), 16, 8, P(w), P(b), P(out), P(out[1:]),
                               P(out[9:]), None) == api.LR_ERR_ALIGNMENT
    assert L.lr_fit_bf16(ctx._h, P(Xh), P(y), 16, 16408, 0.1, 1, P(w), P(b), None, None) == api.LR_ERR_SHAPE
    assert L.lr_predict_bf16(ctx._h, P(Xh), 16, 8, P(w), P(b), 1.5, P(out), None) == api.LR_ERR_VALUE
    assert L.lr_convert_bf16(ctx._h, P(out), -1, P(Xh), None) == api.LR_ERR_SHAPE


@pytest.mark.parametrize("name", ["cfg3", "cfg5"])
def test_full_size_workload_bf16(ctx, name):
    """The benchmark's bfloat16 runs at full size: conversion on the device, the workload's own fit, labels."""
    wl = datagen.WORKLOADS[name]
    X, y, _, _ = datagen.generate(wl)
    dX32 = torch.from_numpy(X).cuda()
    dXh = ctx.convert_bf16(dX32)
    del dX32
    bits, Xv = oracle.round_bf16(X)
    del X
    # conversion: bit-exact on a strided sample of rows plus the last rows (largest offsets)
    got_bits = dXh.view(torch.int16)
    for sl in (slice(0, wl.m, 997), slice(wl.m - 4096, wl.m)):
        assert np.array_equal(got_bits[sl].cpu().numpy().view(np.uint16), bits[sl])
    del bits
    dy = dev(y)
    iters = wl.iters
    hist = torch.empty(iters, dtype=torch.float32, device="cuda")
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    ctx.fit(dXh, dy, wl.lr, iters, w, b, hist)
    torch.cuda.synchronize()
    w_ref, b_ref, hist_ref, wh, bh = oracle.fit(Xv, y, wl.lr, iters, history=True)
    w_rel = rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]]))
    hist_err = float(np.max(np.abs(hist.cpu().numpy().astype(np.float64) - hist_ref)))
    record("full_size_fit", workload=name + "_bf16", w_rel_l2=w_rel, w_bound=W_TOL, loss_hist_max_abs_err=hist_err,
           loss_hist_bound=LOSS_TOL)
    assert w_rel <= W_TOL
    assert hist_err <= LOSS_TOL
    floor = grad_noise_floor(Xv)
    for t in sorted({0, 1, iters // 2, iters - 1}):
        w32, b32 = wh[t].astype(np.float32), np.float32(bh[t])
        L, g, g0 = oracle.loss_grad(Xv, y, w32.astype(np.float64), float(b32))
        dl, dg, dg0 = ctx.loss_grad(dXh, dy, dev(w32), dev(np.array([b32])))
        loss_err = abs(dl.item() - L)
        assert loss_err <= LOSS_TOL, (name, t)
        g_ref = np.concatenate([g, [g0]])
        rel, used_floor = assert_grad_close(np.concatenate([dg.cpu().numpy(), dg0.cpu().numpy()]), g_ref, floor, (name, t),
                                            floor_allowed=False)       # these two workloads are far from converged
        record("full_size_iterate", workload=name + "_bf16", t=t, grad_rel_l2=rel, grad_norm=float(np.linalg.norm(g_ref)),
               bound="floor" if used_floor else "1e-5*|g|", floor=floor, grad_abs_err=rel * float(np.linalg.norm(g_ref)),
               loss=L, loss_abs_err=loss_err)
    w32, b32 = w_ref.astype(np.float32), np.float32(b_ref)
    for thr in ([0.5] + ([0.05] if name == "cfg5" else [])):
        labels = ctx.predict(dXh, dev(w32), dev(np.array([b32])), thr).cpu().numpy()
        lab_ref = oracle.predict(Xv, w32.astype(np.float64), float(b32), thr)
        agree = float((labels == lab_ref).mean())
        record("full_size_labels", workload=name + "_bf16", thr=thr, agreement=agree,
               rows_differing=int((labels != lab_ref).sum()))
        assert agree >= LABEL_AGREE, (name, thr)
    del dXh
    torch.cuda.empty_cache()


# ---- the other fits on a bfloat16-stored X: stopping rule, penalty + momentum, mini-batches, row shards ----

def test_stopping_rule_bf16(ctx):
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 40_003)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    max_iters = 40
    _, _, _, _, _, gh_all = oracle.fit_tol(Xv, y, wl.lr, 0.0, max_iters)
    run_min = np.minimum.accumulate(gh_all)
    cands = [t for t in range(2, max_iters) if gh_all[t] < 0.98 * run_min[t - 1]]
    t_stop = cands[len(cands) // 2]
    eps = float(np.sqrt(gh_all[t_stop] * run_min[t_stop - 1]))      # clearly between two consecutive norms
    w_ref, b_ref, k_ref, n_ref, lh_ref, gh_ref = oracle.fit_tol(Xv, y, wl.lr, eps, max_iters)
    dXh, dy = dev_bf16(bits), dev(y)
    results = []
    for persistent in (True, False):
        ctx.set_persistent(persistent)
        try:
            w = torch.zeros(wl.n, device="cuda")
            b = torch.zeros(1, device="cuda")
            lh = torch.full((max_iters,), float("nan"), device="cuda")
            k, nrm = ctx.fit_tol(dXh, dy, wl.lr, eps, max_iters, w, b, check_every=7, loss_hist=lh)
        finally:
            ctx.set_persistent(None)
        assert k == k_ref == t_stop + 1 and abs(nrm - n_ref) <= 1e-4 * n_ref
        assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
        lhc = lh.cpu().numpy()
        assert np.max(np.abs(lhc[:k] - lh_ref)) <= LOSS_TOL and np.isnan(lhc[k:]).all()
        results.append((w, b))
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])   # both forms, same bits


@pytest.mark.parametrize("name,m,n,opt", [("cfg3", 40_003, None, dict(l2=0.01, momentum=0.5, nesterov=True)),
                                          ("cfg5", 90_001, None, dict(l2=0.1, momentum=0.9)),
                                          ("cfg3", 5_003, 4096, dict(l2=0.05, momentum=0.6))])
def test_fit_opt_bf16(ctx, name, m, n, opt):
    import dataclasses
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    if n is not None:
        wl = dataclasses.replace(wl, n=n)
    lr, iters = min(wl.lr, 0.25), 30
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    w_ref, b_ref, _, lh_ref = oracle.fit_opt(Xv, y, lr, iters, **opt)
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    lh = torch.empty(iters, device="cuda")
    ctx.fit_opt(dev_bf16(bits), dev(y), lr, iters, w, b, loss_hist=lh, **opt)
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(lh.cpu().numpy() - lh_ref)) <= LOSS_TOL


@pytest.mark.parametrize("m,n,batch", [(50_003, 256, 8_192), (9_000, 24, 2_501), (6_001, 2048, 1_000)])
def test_minibatch_descent_bf16(ctx, m, n, batch):
    # 2,501 rows of 24 bfloat16 columns: the second block starts 8 bytes off a 16-byte boundary (unstaged kernel)
    import dataclasses
    wl = dataclasses.replace(datagen.scaled(datagen.WORKLOADS["cfg3"], m), n=n)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    steps, lr = 12, 0.2
    w_ref, b_ref, lh_ref = oracle.fit_sgd(Xv, y, lr, batch, steps, first_batch=1)
    w = torch.zeros(n, device="cuda")
    b = torch.zeros(1, device="cuda")
    lh = torch.empty(steps, device="cuda")
    ctx.fit_sgd(dev_bf16(bits), dev(y), lr, batch, steps, w, b, first_batch=1, loss_hist=lh)
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(lh.cpu().numpy() - lh_ref)) <= LOSS_TOL


def test_row_shards_bf16(ctx):
    from paper_2308_10037_b200.parallel import shard_rows
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 50_003)
    X, y, _, _ = datagen.generate(wl)
    bits, Xv = oracle.round_bf16(X)
    parts, steps = 3, 5
    shards = [shard_rows(wl.m, r, parts) for r in range(parts)]
    dXs = [dev_bf16(bits[a:b]) for a, b in shards]
    dys = [dev(y[a:b]) for a, b in shards]
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    sums = torch.empty((parts, wl.n + 2), dtype=torch.float64, device="cuda")
    loss = torch.empty(steps, device="cuda")
    for t in range(steps):
        for r in range(parts):
            ctx.shard_sums(dXs[r], dys[r], w, b, sums[r])
        ctx.apply_sums(sums, wl.m, wl.lr, w, b, loss[t:t + 1])
    w_ref, b_ref, lh_ref = oracle.fit(Xv, y, wl.lr, steps)
    assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(loss.cpu().numpy() - lh_ref)) <= LOSS_TOL
