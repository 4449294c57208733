"""Row-sharded fits with the exchange inside the persistent kernel (``lr_fit_sharded``, ``lr_fit_sharded_local``).

One GPU is all these tests need and all they use:
  * a world of one rank must reproduce ``lr_fit`` bit for bit (the exchange path runs, with one rank in it);
  * a rank whose peer never shows up must give up after its bound, report LR_ERR_TIMEOUT and leave the context usable
    (the wait simply runs out: nothing faults, traps or hangs);
  * several ranks run as CTA groups of ONE cooperative launch (all CTAs resident together, so the ranks' waits on each
    other always end) must agree bit for bit among themselves and with the lr_shard_sums / lr_apply_sums loop, and match
    the float64 checker's unsharded fit within the stated tolerances.
"""
import numpy as np
import pytest
import torch

import oracle
from _parity import LOSS_TOL, W_TOL, rel_l2
from paper_2308_10037_b200 import api, datagen
from paper_2308_10037_b200.parallel import shard_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2308_10037_b200 import build
    build.build()
    c = api.Context(n_max=1024, device=0)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def exchange_buffer(world, n):
    return torch.zeros(api.exchange_bytes(world, n) // 8, dtype=torch.float64, device="cuda")


@pytest.mark.parametrize("name,m", [("cfg3", 60_001), ("cfg3", 20_003), ("cfg1", 10_000), ("cfg2", 150_007), ("higgs_like", 90_001)])
def test_a_world_of_one_rank_is_lr_fit(ctx, name, m):
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    iters = 9
    w_ref, b_ref, h_ref = api.lr_fit(dX, dy, wl.lr, iters, return_history=True, ctx=ctx)
    buf = exchange_buffer(1, wl.n)
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    h = torch.empty(iters, device="cuda")
    n0 = ctx.launch_count()
    ctx.fit_sharded(dX, dy, wl.m, wl.lr, 5, w, b, rank=0, world=1, exchange_ptrs=[buf], epoch=0, loss_hist=h[:5])
    ctx.fit_sharded(dX, dy, wl.m, wl.lr, 4, w, b, rank=0, world=1, exchange_ptrs=[buf], epoch=5, loss_hist=h[5:])
    assert ctx.launch_count() == n0 + 2                      # one persistent launch per call
    torch.cuda.synchronize()
    assert torch.equal(w, w_ref) and torch.equal(b, b_ref) and torch.equal(h, h_ref)
    assert ctx.device_status() == 0


def test_a_missing_peer_ends_in_a_timeout_not_a_hang(ctx):
    wl = datagen.scaled(datagen.WORKLOADS["cfg3"], 30_001)
    X, y, _, _ = datagen.generate(wl)
    dX, dy = dev(X), dev(y)
    own, peer = exchange_buffer(2, wl.n), exchange_buffer(2, wl.n)   # nobody ever publishes a flag for rank 1
    w = torch.full((wl.n,), 0.25, device="cuda")
    b = torch.full((1,), -0.5, device="cuda")
    ctx.fit_sharded(dX, dy, 2 * wl.m, wl.lr, 5, w, b, rank=0, world=2, exchange_ptrs=[own, peer], epoch=0, wait_ms=50)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.LR_ERR_TIMEOUT
    assert bool((w == 0.25).all()) and bool((b == -0.5).all())       # the parameters are left as they were
    # rank 0 did write its own sums to both buffers before it waited
    assert own.abs().sum().item() > 0 and peer.abs().sum().item() > 0
    # the context and the device are fine
    w2, b2 = api.lr_fit(dX, dy, wl.lr, 5, ctx=ctx)
    w_ref, b_ref, _ = oracle.fit(X, y, wl.lr, 5)
    assert rel_l2(np.concatenate([w2.cpu().numpy(), b2.cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert ctx.device_status() == 0


@pytest.mark.parametrize("name,m,world", [("cfg3", 120_001, 2), ("cfg3", 90_000, 3), ("cfg3", 30_011, 4), ("cfg1", 10_000, 2),
                                          ("higgs_like", 200_003, 4), ("cfg3", 400_003, 2)])
def test_ranks_as_cta_groups_of_one_launch(ctx, name, m, world):
    wl = datagen.scaled(datagen.WORKLOADS[name], m)
    X, y, _, _ = datagen.generate(wl)
    iters = 8
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    shards = [shard_rows(wl.m, r, world) for r in range(world)]
    # 16-byte aligned shards: every shard gets its own allocation
    Xs = [dev(X[a:b]) for a, b in shards]
    ys = [dev(y[a:b]) for a, b in shards]
    ws = [torch.zeros(wl.n, device="cuda") for _ in range(world)]
    bs = [torch.zeros(1, device="cuda") for _ in range(world)]
    hs = [torch.empty(iters, device="cuda") for _ in range(world)]
    bufs = [exchange_buffer(world, wl.n) for _ in range(world)]
    n0 = ctx.launch_count()
    ctx.fit_sharded_local(Xs, ys, wl.lr, 5, ws, bs, bufs, epoch=0, loss_hists=[h[:5] for h in hs])
    ctx.fit_sharded_local(Xs, ys, wl.lr, iters - 5, ws, bs, bufs, epoch=5, loss_hists=[h[5:] for h in hs])
    assert ctx.launch_count() == n0 + 2
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for r in range(1, world):                                # every rank holds the same bits
        assert torch.equal(ws[r], ws[0]) and torch.equal(bs[r], bs[0]) and torch.equal(hs[r], hs[0])
    # the float64 checker's unsharded fit
    w_ref, b_ref, lh_ref = oracle.fit(X, y, wl.lr, iters)
    assert rel_l2(np.concatenate([ws[0].cpu().numpy(), bs[0].cpu().numpy()]), np.concatenate([w_ref, [b_ref]])) <= W_TOL
    assert np.max(np.abs(hs[0].cpu().numpy() - lh_ref)) <= LOSS_TOL
    # the host-driven loop over the same shards on the same number of SMs per rank: same sums, same order, same bits
    try:
        ctx.set_sm_limit(sms // world)
        w = torch.zeros(wl.n, device="cuda")
        b = torch.zeros(1, device="cuda")
        sums = torch.empty((world, wl.n + 2), dtype=torch.float64, device="cuda")
        loss = torch.empty(iters, device="cuda")
        for t in range(iters):
            for r in range(world):
                ctx.shard_sums(Xs[r], ys[r], w, b, sums[r])
            ctx.apply_sums(sums, wl.m, wl.lr, w, b, loss[t:t + 1])
    finally:
        ctx.set_sm_limit(None)
    assert torch.equal(w, ws[0]) and torch.equal(b, bs[0]) and torch.equal(loss, hs[0])


def test_argument_checks(ctx):
    X, y, w, b = datagen.random_problem(4000, 256, seed=5)
    dX, dy, dw, db = dev(X), dev(y), dev(w), dev(np.array([b], dtype=np.float32))
    buf = exchange_buffer(2, 256)
    for kwargs, code in ((dict(rank=2, world=2), api.LR_ERR_SHAPE), (dict(rank=0, world=2, wait_ms=0), api.LR_ERR_VALUE),
                         (dict(rank=0, world=2, epoch=-1), api.LR_ERR_SHAPE)):
        kw = dict(dict(epoch=0, wait_ms=100), **kwargs)
        with pytest.raises(api.LrError) as e:
            ctx.fit_sharded(dX, dy, 8000, 0.1, 2, dw.clone(), db.clone(), exchange_ptrs=[buf, buf], **kw)
        assert e.value.code == code
    with pytest.raises(api.LrError) as e:                    # a buffer that is not 128-byte aligned
        ctx.fit_sharded(dX, dy, 4000, 0.1, 2, dw.clone(), db.clone(), rank=0, world=1, exchange_ptrs=[buf.data_ptr() + 8])
    assert e.value.code == api.LR_ERR_ALIGNMENT
    Xw = dev(np.zeros((64, 4100), dtype=np.float32))          # wide rows have no persistent kernel
    big = api.Context(n_max=4100, device=0)
    with pytest.raises(api.LrError) as e:
        big.fit_sharded(Xw, dev(np.zeros(64, dtype=np.float32)), 64, 0.1, 2, torch.zeros(4100, device="cuda"),
                        torch.zeros(1, device="cuda"), rank=0, world=1, exchange_ptrs=[exchange_buffer(1, 4100)])
    assert e.value.code == api.LR_ERR_SHAPE
    big.close()
    with pytest.raises(ValueError):                           # an exchange buffer that is too small never reaches the library
        ctx.fit_sharded(dX, dy, 4000, 0.1, 2, dw.clone(), db.clone(), rank=0, world=1,
                        exchange_ptrs=[torch.zeros(8, dtype=torch.float64, device="cuda")])
    assert ctx.device_status() == 0
