"""Row-sharded data parallelism on two CPU ranks (gloo): the orchestration in ``parallel.py`` with the float64
checker supplying the per-shard sums, against one unsharded fit by the same checker.

The CUDA entry points ``lr_shard_sums`` / ``lr_apply_sums`` do on a GPU what the two callables below do here; what this
covers is the host side: row ranges, the all-gather, rank-ordered addition and identical parameters on every rank.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, m, n, lr, iters, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2308_10037_b200 import datagen, parallel
    oracle.set_threads(1)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = datagen.scaled(datagen.WORKLOADS["cfg1"], m)
        X, y, _, _ = datagen.generate(wl, threads=1)          # every rank draws the same bits, then keeps its rows
        r0, r1 = parallel.shard_rows(m, rank, world)
        Xl, yl = X[r0:r1], y[r0:r1]
        w = np.zeros(n)
        b = [0.0]
        losses = []

        def local_sums(out):
            # unnormalised sums of the local rows: the checker returns means over the local rows
            L, g, g0 = oracle.loss_grad(Xl, yl, w, b[0])
            k = r1 - r0
            out[:n] = torch.from_numpy(g * k)
            out[n] = g0 * k
            out[n + 1] = L * k

        def apply_sums(gathered, t):
            tot = torch.zeros(n + 2, dtype=torch.float64)
            for r in range(gathered.shape[0]):              # rank order
                tot += gathered[r]
            tot /= m
            w[:] -= lr * tot[:n].numpy()
            b[0] -= lr * float(tot[n])
            losses.append(float(tot[n + 1]))

        sums = torch.zeros(n + 2, dtype=torch.float64)
        parallel.fit_sharded(local_sums, apply_sums, sums, iters)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), w=w, b=b[0], losses=np.array(losses), rows=np.array([r0, r1]))
    finally:
        dist.destroy_process_group()


def test_shard_rows_partition():
    sys.path.insert(0, ROOT)
    from paper_2308_10037_b200 import parallel
    for m, world in [(10, 3), (7, 7), (5, 8), (1_000_003, 8), (0, 2)]:
        spans = [parallel.shard_rows(m, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == m
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [b - a for a, b in spans]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        parallel.shard_rows(10, 2, 2)


def test_two_rank_fit_equals_unsharded_fit(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2308_10037_b200 import datagen
    m, n, lr, iters, world = 6001, 32, 0.1, 15, 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, m, n, lr, iters, str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"rank{k}.npz") for k in range(world)]
    assert np.array_equal(r[0]["w"], r[1]["w"]) and r[0]["b"] == r[1]["b"]          # identical on every rank, bit for bit
    assert np.array_equal(r[0]["losses"], r[1]["losses"])
    assert r[0]["rows"].tolist() == [0, 3001] and r[1]["rows"].tolist() == [3001, 6001]
    X, y, _, _ = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg1"], m), threads=1)
    w_ref, b_ref, lh_ref = oracle.fit(X, y, lr, iters)
    np.testing.assert_allclose(r[0]["w"], w_ref, rtol=0, atol=1e-13)
    assert abs(float(r[0]["b"]) - b_ref) < 1e-13
    np.testing.assert_allclose(r[0]["losses"], lh_ref, rtol=0, atol=1e-13)
