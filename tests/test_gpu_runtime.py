"""Runtime behaviour around the kernels: the bounded-wait give-up path, and the row-sharded driver on a real
process group (one rank: the only size a single GPU allows).

Nothing here faults, traps or hangs the device: the give-up test waits a few milliseconds on a barrier that
nothing completes, the kernel then returns normally with the status word set, and the context stays usable.
"""
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
    c = api.Context(n_max=512, device=0)
    yield c
    c.close()


def test_bounded_wait_gives_up_and_reports(ctx):
    ctx.selftest_wait(arm=True, limit_ms=20)                 # the barrier completes: no status
    assert ctx.device_status() == 0
    ctx.selftest_wait(arm=False, limit_ms=20)                # nothing completes it: the kernel gives up after 20 ms
    assert ctx.device_status() == api.LR_ERR_TIMEOUT
    assert api.status_string(api.LR_ERR_TIMEOUT) == "a bounded device-side wait expired"
    assert ctx.device_status() == 0                          # reading clears the word
    # the context and the device are still fine
    X, y, w, b = datagen.random_problem(5000, 64, seed=21)
    dl, dg, dg0 = ctx.loss_grad(torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(w).cuda(),
                                torch.tensor([b], device="cuda"))
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    assert abs(dl.item() - L) <= LOSS_TOL and rel_l2(dg.cpu().numpy(), g) <= 1e-5
    assert ctx.device_status() == 0
    with pytest.raises(api.LrError):
        ctx.selftest_wait(arm=False, limit_ms=5000)          # limits above one second are refused


def test_an_unread_status_does_not_disturb_later_fits(ctx):
    # the status word is a sticky report: a give-up that nobody has read yet must not end the persistent kernel of a later
    # call (which has an abort flag of its own, cleared at every launch), nor change any result
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 40_001)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    ctx.set_persistent(False)
    w_ref, b_ref, h_ref = api.lr_fit(dX, dy, wl.lr, 6, return_history=True, ctx=ctx)
    assert ctx.device_status() == 0
    ctx.selftest_wait(arm=False, limit_ms=20)                # leaves LR_ERR_TIMEOUT in the status word, unread
    try:
        ctx.set_persistent(True)
        w, b, h = api.lr_fit(dX, dy, wl.lr, 6, return_history=True, ctx=ctx)
        assert torch.equal(w, w_ref) and torch.equal(b, b_ref) and torch.equal(h, h_ref)
        wt = torch.zeros(wl.n, device="cuda")
        bt = torch.zeros(1, device="cuda")
        done, nrm = ctx.fit_tol(dX, dy, wl.lr, 0.0, 6, wt, bt)     # eps = 0 never stops early: six updates, same bits
        assert done == 6 and torch.equal(wt, w_ref) and torch.equal(bt, b_ref)
        ctx.set_persistent(False)
        wt.zero_(); bt.zero_()
        done, nrm = ctx.fit_tol(dX, dy, wl.lr, 0.0, 6, wt, bt, check_every=2)
        assert done == 6 and torch.equal(wt, w_ref) and torch.equal(bt, b_ref)
    finally:
        ctx.set_persistent(None)
    assert ctx.device_status() == api.LR_ERR_TIMEOUT         # the old report is still there, and reading clears it
    assert ctx.device_status() == 0


def test_sharded_driver_on_a_one_rank_nccl_group(ctx):
    import torch.distributed as dist
    from paper_2308_10037_b200 import parallel
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29871", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 30_001)
        X, y, _, _ = datagen.generate(wl)
        dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        w = torch.zeros(wl.n, device="cuda")
        b = torch.zeros(1, device="cuda")
        hist = torch.empty(8, device="cuda")
        parallel.fit_sharded_cuda(ctx, dX, dy, wl.m, wl.lr, 8, w, b, loss_hist=hist)
        torch.cuda.synchronize()
        w_ref, b_ref, lh_ref = oracle.fit(X, y, wl.lr, 8)
        assert rel_l2(np.concatenate([w.cpu().numpy(), b.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
        assert np.max(np.abs(hist.cpu().numpy() - lh_ref)) <= LOSS_TOL
        # one shard, one rank: the same kernels and the same summation order as lr_fit -> identical bits
        wf, bf = api.lr_fit(dX, dy, wl.lr, 8, ctx=ctx)
        assert torch.equal(w, wf) and torch.equal(b, bf)
        # and the fused form on the same one-rank group: exchange buffer in symmetric memory, one launch for all steps
        try:
            ex = parallel.ExchangeBuffers(wl.n, torch.device("cuda", 0))
        except Exception as err:                                  # symmetric memory is not available everywhere
            ex = None
            print("symmetric memory unavailable:", err)
        if ex is not None:
            w2 = torch.zeros(wl.n, device="cuda")
            b2 = torch.zeros(1, device="cuda")
            parallel.fit_sharded_fused(ctx, dX, dy, wl.m, wl.lr, 5, w2, b2, ex)
            parallel.fit_sharded_fused(ctx, dX, dy, wl.m, wl.lr, 3, w2, b2, ex)
            torch.cuda.synchronize()
            assert ex.epoch == 8 and torch.equal(w2, wf) and torch.equal(b2, bf)
            assert ctx.device_status() == 0
    finally:
        dist.destroy_process_group()


def test_c_example_program_runs():
    # a plain C program linked against the shared library, no Python in between
    import os
    import shutil
    import subprocess
    import tempfile
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    pkg = os.path.join(root, "paper_2308_10037_b200")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "fit_host")
        subprocess.check_call([gcc, "-std=c99", "-O2", "-I", os.path.join(root, "include"), os.path.join(pkg, "examples", "fit_host.c"),
                               "-L", pkg, "-llrgd", f"-Wl,-rpath,{pkg}", "-lm", "-o", exe])
        out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
        assert out.returncode == 0, out.stdout + out.stderr
        assert "device status 0" in out.stdout


def test_guard_regions_stay_clean_at_the_context_limit(ctx):
    """Every workspace array sits between two guard regions; runs at the widest row the context allows (n = n_max), in every
    fit form that uses a workspace (partial rows, gradient buffer, context-owned velocity, optimiser scratch), must leave all
    eight regions untouched.  A clean context reports 0 to begin with."""
    fresh = api.Context(n_max=512, device=0)
    assert fresh.check_guards() == 0
    fresh.close()
    for m, n in [(30_011, 512), (2_001, 511), (150_001, 28), (9, 512)]:
        X, y, w, b = datagen.random_problem(m, n, seed=31 + n)
        dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        zeros = lambda: (torch.zeros(n, device="cuda"), torch.zeros(1, device="cuda"))
        ctx.loss_grad(dX, dy, torch.from_numpy(w).cuda(), torch.tensor([b], device="cuda"))
        for persistent in (None, True, False):
            ctx.set_persistent(persistent)
            ctx.fit(dX, dy, 0.05, 4, *zeros())
            ctx.fit_tol(dX, dy, 0.05, 1e-9, 5, *zeros(), check_every=2)
            ctx.fit_opt(dX, dy, 0.05, 4, *zeros(), l2=1e-3, momentum=0.9, nesterov=True)
        ctx.set_persistent(None)
        ctx.fit_sgd(dX, dy, 0.05, max(1, m // 3), 5, *zeros())
        ctx.predict(dX, torch.from_numpy(w).cuda(), torch.tensor([b], device="cuda"), 0.5)
    assert ctx.device_status() == 0
    assert ctx.check_guards() == 0
