"""CPU-only pins for the float64 checker in ``oracle/``.

Each test ties the checker to a fact fixed by the paper's definitions or by mathematics, chosen so
that a dropped term, a wrong sign, a transposed operand or a missing 1/m fails at least one of them.
Nothing here touches the CUDA library.
"""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2308_10037_b200 import datagen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_form_cases.txt")


def _expr(s):
    return float(eval(s, {"__builtins__": {}}, {"log": math.log}))


def _cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, X, y, w, b, loss, gw, gb = [t.strip() for t in line.split(";")]
            X = np.array([[_expr(v) for v in row.split(",")] for row in X.split("|")], dtype=np.float32)
            y = np.array([_expr(v) for v in y.split(",")], dtype=np.float32)
            w = np.array([_expr(v) for v in w.split(",")])
            gw = np.array([_expr(v) for v in gw.split(",")])
            out.append((name, X, y, w, _expr(b), _expr(loss), gw, _expr(gb)))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c[0])
def test_closed_form_cases(case):
    _, X, y, w, b, loss, gw, gb = case
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    assert abs(L - loss) < 1e-15
    np.testing.assert_allclose(g, gw, atol=1e-15, rtol=0)
    assert abs(g0 - gb) < 1e-15


def test_closed_form_one_gd_step_and_predict():
    # asym_bias case: one step with lr = 1/2 moves (w, b) by -g/2; thresholds checked against z = (ln3, -ln2)
    _, X, y, w, b, _, gw, gb = [c for c in _cases() if c[0] == "asym_bias"][0]
    w1, b1, lh = oracle.fit(X, y, 0.5, 1, w0=w, b0=b)
    np.testing.assert_allclose(w1, [math.log(1.5) - 3 / 16, -math.log(2) + 1 / 3], atol=1e-15, rtol=0)
    assert abs(b1 - (math.log(2) - 1 / 48)) < 1e-15
    assert abs(lh[0] - (math.log(4) + math.log(3)) / 2) < 1e-15
    assert oracle.predict(X, w, b, 0.5).tolist() == [1, 0]
    assert oracle.predict(X, w, b, 0.8).tolist() == [0, 0]      # logit(0.8) = ln4 > ln3
    assert oracle.predict(X, w, b, 0.3).tolist() == [1, 1]      # logit(0.3) = ln(3/7) < -ln2


@pytest.mark.parametrize("m,n", [(1, 1), (8, 3), (1025, 7), (3000, 33)])
def test_zero_parameters(m, n):
    # at w = 0, b = 0 every p is 1/2: loss is ln 2 whatever y is, grad_w = X^T(0.5 - y)/m
    X, y, _, _ = datagen.random_problem(m, n, seed=m + n)
    L, g, g0 = oracle.loss_grad(X, y, np.zeros(n), 0.0)
    assert abs(L - math.log(2)) < 1e-13              # m rounded additions of ln 2
    ref = (X.astype(np.float64).T @ (0.5 - y.astype(np.float64))) / m
    np.testing.assert_allclose(g, ref, atol=1e-14, rtol=0)
    assert abs(g0 - np.mean(0.5 - y.astype(np.float64))) < 1e-14


def test_central_finite_differences():
    m, n = 8, 3
    X, y, w, b = datagen.random_problem(m, n, seed=5)
    w = w.astype(np.float64)
    _, g, g0 = oracle.loss_grad(X, y, w, b)
    h = 1e-5
    for j in range(n):
        d = np.zeros(n)
        d[j] = h
        fd = (oracle.loss_grad(X, y, w + d, b)[0] - oracle.loss_grad(X, y, w - d, b)[0]) / (2 * h)
        assert abs(fd - g[j]) <= 1e-7 * max(1.0, abs(g[j]))
    fd = (oracle.loss_grad(X, y, w, b + h)[0] - oracle.loss_grad(X, y, w, b - h)[0]) / (2 * h)
    assert abs(fd - g0) <= 1e-7 * max(1.0, abs(g0))


def test_label_flip_symmetry():
    # (y, w, b) -> (1-y, -w, -b) keeps the loss and negates the gradient
    X, y, w, b = datagen.random_problem(500, 6, seed=2)
    w = w.astype(np.float64)
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    L2, g2, g02 = oracle.loss_grad(X, 1.0 - y, -w, -b)
    assert abs(L - L2) < 1e-14
    np.testing.assert_allclose(g2, -g, atol=1e-14, rtol=0)
    assert abs(g02 + g0) < 1e-14


def test_row_duplication_keeps_mean_quantities():
    # pins the 1/m: stacking the data twice changes nothing
    X, y, w, b = datagen.random_problem(700, 5, seed=3)
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    L2, g2, g02 = oracle.loss_grad(np.vstack([X, X]), np.concatenate([y, y]), w, b)
    assert abs(L - L2) < 1e-14
    np.testing.assert_allclose(g2, g, atol=1e-14, rtol=0)
    assert abs(g02 - g0) < 1e-14


def test_bias_equals_constant_one_feature():
    X, y, w, b = datagen.random_problem(900, 4, seed=4)
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    X1 = np.hstack([X, np.ones((X.shape[0], 1), dtype=np.float32)])
    L1, g1, g01 = oracle.loss_grad(X1, y, np.concatenate([w.astype(np.float64), [b]]), 0.0)
    assert abs(L - L1) < 1e-14
    np.testing.assert_allclose(g1[:-1], g, atol=1e-14, rtol=0)
    assert abs(g1[-1] - g0) < 1e-14 and abs(g01 - g0) < 1e-14


def test_saturated_logits_stay_finite():
    # |z| = 40: loss term equals max(z,0) - y z up to exp(-40); err is -1, 0, 0, 1 up to exp(-40)
    X = np.array([[40.0], [40.0], [-40.0], [-40.0]], dtype=np.float32)
    y = np.array([1, 0, 1, 0], dtype=np.float32)
    L, g, g0 = oracle.loss_grad(X, y, np.array([1.0]), 0.0)
    assert abs(L - (0 + 40 + 40 + 0) / 4) < 1e-15 * 40
    np.testing.assert_allclose(g, [(40 * 1.0 + 40 * 1.0) / 4], rtol=1e-15)   # x*e: 40*(1-0) and -40*(0-1)
    assert abs(g0) < 1e-15
    X = np.array([[800.0], [-800.0]], dtype=np.float32)
    L, g, g0 = oracle.loss_grad(X, np.array([0, 1], dtype=np.float32), np.array([1.0]), 0.0)
    assert np.isfinite([L, g[0], g0]).all() and abs(L - 800.0) < 1e-12


def test_matches_float64_library_bce_with_logits_autograd():
    torch = pytest.importorskip("torch")
    X, y, w, b = datagen.random_problem(257, 9, seed=6, wscale=3.0)
    Xt = torch.from_numpy(X).double()
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    loss = torch.nn.functional.binary_cross_entropy_with_logits(Xt @ wt + bt, torch.from_numpy(y).double())
    loss.backward()
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    assert abs(L - loss.item()) < 1e-13
    np.testing.assert_allclose(g, wt.grad.numpy(), atol=1e-13, rtol=0)
    assert abs(g0 - bt.grad.item()) < 1e-13


def test_loss_decreases_monotonically_below_descent_lemma_bound():
    wl = datagen.scaled(datagen.WORKLOADS["cfg1"], 2000)
    X, y, _, _ = datagen.generate(wl, threads=1)
    A = np.hstack([X.astype(np.float64), np.ones((wl.m, 1))])
    lip = 0.25 * np.linalg.eigvalsh(A.T @ A / wl.m)[-1]
    lr = 1.0 / lip                                   # < 2/L
    w, b, lh = oracle.fit(X, y, lr, 60)
    final = oracle.loss_grad(X, y, w, b)[0]
    seq = np.concatenate([lh, [final]])
    d = np.diff(seq)
    assert (d[:12] < 0).all()                        # strict while the decrease is far above rounding
    assert (d < 4e-15).all()                         # and never an increase beyond a few ulp at the floor
    assert abs(lh[0] - math.log(2)) < 1e-13


def test_planted_weights_are_recovered():
    wl = datagen.WORKLOADS["cfg1"]                    # 10,000 x 32, lr 0.1, 100 iterations
    X, y, wstar, bstar = datagen.generate(wl, threads=1)
    w, b, _ = oracle.fit(X, y, wl.lr, wl.iters)
    assert np.corrcoef(w, wstar)[0, 1] > 0.95


def test_fit_is_resumable_and_history_is_consistent():
    X, y, _, _ = datagen.random_problem(1500, 5, seed=8)
    wa, ba, la = oracle.fit(X, y, 0.3, 7)
    wb, bb, lb = oracle.fit(X, y, 0.3, 5, w0=wa, b0=ba)
    wc, bc, lc, wh, bh = oracle.fit(X, y, 0.3, 12, history=True)
    assert np.array_equal(wb, wc) and bb == bc
    assert np.array_equal(np.concatenate([la, lb]), lc)
    assert np.array_equal(wh[7], wa) and bh[7] == ba and np.array_equal(wh[0], np.zeros(5))
    # the step itself: w_{t+1} = w_t - lr * grad(w_t)
    _, g, g0 = oracle.loss_grad(X, y, wh[3], bh[3])
    np.testing.assert_allclose(wh[4], wh[3] - 0.3 * g, atol=1e-16, rtol=0)
    assert abs(bh[4] - (bh[3] - 0.3 * g0)) < 1e-16


def test_blocked_threaded_sum_equals_plain_definition():
    # several blocks plus a ragged tail, against the definition written with numpy in float64
    X, y, w, b = datagen.random_problem(5 * 1024 + 77, 11, seed=9)
    Xd, yd, wd = X.astype(np.float64), y.astype(np.float64), w.astype(np.float64)
    z = Xd @ wd + b
    p = 1.0 / (1.0 + np.exp(-z))
    loss = -np.mean(yd * np.log(p) + (1 - yd) * np.log(1 - p))     # -l/m, straight from the log-likelihood
    L, g, g0 = oracle.loss_grad(X, y, w, b)
    assert abs(L - loss) < 1e-13
    np.testing.assert_allclose(g, Xd.T @ (p - yd) / len(yd), atol=1e-14, rtol=0)
    assert abs(g0 - np.mean(p - yd)) < 1e-15
    oracle.set_threads(1)
    try:
        L1, g1, g01 = oracle.loss_grad(X, y, w, b)
    finally:
        oracle.set_threads(os.cpu_count() or 1)
    assert L1 == L and g01 == g0 and np.array_equal(g1, g)       # thread count does not change a bit


def test_predict_brute_force_and_threshold_monotone():
    X, y, w, b = datagen.random_problem(333, 6, seed=10, wscale=2.0)
    labels, z = oracle.predict(X, w, b, 0.5, return_z=True)
    for i in range(X.shape[0]):
        zi = b + sum(float(X[i, j]) * float(w[j]) for j in range(X.shape[1]))
        assert abs(zi - z[i]) < 1e-13
        assert labels[i] == (1 if zi >= 0 else 0)                 # thr = 0.5 <=> sign of z
    prev = None
    for thr in (0.1, 0.3, 0.5, 0.7, 0.9):
        lab = oracle.predict(X, w, b, thr)
        p = 1 / (1 + np.exp(-z))
        assert np.array_equal(lab, (p >= thr).astype(np.uint8)) or np.min(np.abs(p - thr)) < 1e-12
        if prev is not None:
            assert (lab <= prev).all()
        prev = lab


def test_f1_hand_counted():
    y = np.array([1, 1, 1, 0, 0, 0, 0, 1], dtype=np.float32)
    lab = np.array([1, 1, 0, 1, 0, 0, 0, 0], dtype=np.uint8)     # TP=2 FP=1 FN=2
    f1, tp, fp, fn = oracle.f1_score(lab, y)
    assert (tp, fp, fn) == (2, 1, 2) and abs(f1 - 4 / 7) < 1e-16
    assert oracle.f1_score(np.zeros(8, np.uint8), y)[0] == 0.0   # nothing predicted positive
    assert oracle.f1_score(y.astype(np.uint8), y)[0] == 1.0


def test_bad_arguments_are_rejected():
    X, y, w, b = datagen.random_problem(4, 2, seed=1)
    with pytest.raises(ValueError):
        oracle.predict(X, w, b, 1.0)
    with pytest.raises(ValueError):
        oracle.predict(X, w, b, 0.0)


def test_stopping_rule_follows_algorithm_7():
    X, y, _, _ = datagen.random_problem(2000, 6, seed=12)
    lr = 0.5
    # eps = 0 never stops early: identical to the fixed-count fit
    w0, b0, k0, n0, lh0, gh0 = oracle.fit_tol(X, y, lr, 0.0, 25)
    wf, bf, lhf = oracle.fit(X, y, lr, 25)
    assert k0 == 25 and np.array_equal(w0, wf) and b0 == bf and np.array_equal(lh0, lhf)
    # the recorded norms are the norms of the gradients at the iterates before each update
    _, _, _, wh, bh = oracle.fit(X, y, lr, 25, history=True)
    for t in (0, 7, 24):
        _, g, g_b = oracle.loss_grad(X, y, wh[t], bh[t])
        assert abs(gh0[t] - math.sqrt(float(g @ g) + g_b * g_b)) < 1e-15
    # a tolerance between two consecutive norms stops exactly there, after applying that update
    eps = 0.5 * (gh0[9] + gh0[10])
    assert gh0[10] < eps < gh0[9]
    w1, b1, k1, n1, lh1, gh1 = oracle.fit_tol(X, y, lr, eps, 25)
    assert k1 == 11 and n1 == gh0[10] and np.array_equal(w1, wh[11]) and b1 == bh[11]
    assert len(lh1) == 11 and np.array_equal(gh1, gh0[:11])
    # a huge tolerance still applies one update (the test comes after the update)
    w2, b2, k2, n2, _, _ = oracle.fit_tol(X, y, lr, 1e9, 25)
    assert k2 == 1 and np.array_equal(w2, wh[1]) and n2 == gh0[0]
    # no iterations allowed: nothing happens
    w3, b3, k3, n3, _, _ = oracle.fit_tol(X, y, lr, 1.0, 0)
    assert k3 == 0 and n3 == -1.0 and not w3.any() and b3 == 0.0


def test_penalty_and_momentum_follow_their_definitions():
    X, y, _, _ = datagen.random_problem(1200, 5, seed=13)
    lr, l2, mu = 0.4, 0.3, 0.7
    # no penalty, no momentum: the plain fit
    w0, b0, v0, lh0 = oracle.fit_opt(X, y, lr, 9)
    wf, bf, lhf = oracle.fit(X, y, lr, 9)
    assert np.array_equal(w0, wf) and b0 == bf and np.array_equal(lh0, lhf)
    # heavy ball, three steps by hand from the plain loss/gradient routine
    w, b, v = np.zeros(5), 0.0, np.zeros(6)
    losses = []
    for _ in range(3):
        L, g, gb = oracle.loss_grad(X, y, w, b)
        losses.append(L + 0.5 * l2 * float(w @ w))
        gfull = np.concatenate([g + l2 * w, [gb]])           # the bias carries no penalty
        v = mu * v + gfull
        w, b = w - lr * v[:5], b - lr * v[5]
    w1, b1, v1, lh1 = oracle.fit_opt(X, y, lr, 3, l2=l2, momentum=mu)
    np.testing.assert_allclose(w1, w, atol=1e-15, rtol=0)
    assert abs(b1 - b) < 1e-15
    np.testing.assert_allclose(v1, v, atol=1e-15, rtol=0)
    np.testing.assert_allclose(lh1, losses, atol=1e-15, rtol=0)
    # Nesterov form, same bookkeeping
    w, b, v = np.zeros(5), 0.0, np.zeros(6)
    for _ in range(3):
        _, g, gb = oracle.loss_grad(X, y, w, b)
        gfull = np.concatenate([g + l2 * w, [gb]])
        v = mu * v + gfull
        step = gfull + mu * v
        w, b = w - lr * step[:5], b - lr * step[5]
    w2, b2, v2, _ = oracle.fit_opt(X, y, lr, 3, l2=l2, momentum=mu, nesterov=True)
    np.testing.assert_allclose(w2, w, atol=1e-15, rtol=0)
    assert abs(b2 - b) < 1e-15 and not np.allclose(w2, w1)
    # the penalised gradient is the gradient of the penalised loss (central differences)
    wp = np.array([0.3, -0.2, 0.5, 0.1, -0.4])
    _, g, _ = oracle.loss_grad(X, y, wp, 0.2)
    for j in range(5):
        d = np.zeros(5)
        d[j] = 1e-5
        f = lambda ww: oracle.loss_grad(X, y, ww, 0.2)[0] + 0.5 * l2 * float(ww @ ww)
        assert abs((f(wp + d) - f(wp - d)) / 2e-5 - (g[j] + l2 * wp[j])) < 1e-8
    # at the fixed point of the penalised problem the penalised gradient vanishes and ||w|| shrinks with the penalty
    wa, ba, _, _ = oracle.fit_opt(X, y, 1.0, 400, l2=0.5, momentum=0.5)
    _, g, gb = oracle.loss_grad(X, y, wa, ba)
    assert np.linalg.norm(np.concatenate([g + 0.5 * wa, [gb]])) < 1e-10
    wb, _, _, _ = oracle.fit_opt(X, y, 1.0, 400, l2=0.05, momentum=0.5)
    assert np.linalg.norm(wa) < np.linalg.norm(wb)
    # resuming with the returned velocity continues the same trajectory
    wa1, ba1, va1, _ = oracle.fit_opt(X, y, lr, 4, l2=l2, momentum=mu)
    wa2, ba2, va2, _ = oracle.fit_opt(X, y, lr, 3, l2=l2, momentum=mu, w0=wa1, b0=ba1, vel0=va1)
    wa3, ba3, va3, _ = oracle.fit_opt(X, y, lr, 7, l2=l2, momentum=mu)
    assert np.array_equal(wa2, wa3) and ba2 == ba3 and np.array_equal(va2, va3)


def test_minibatch_descent_walks_contiguous_blocks():
    X, y, _, _ = datagen.random_problem(1000, 4, seed=14)
    lr = 0.3
    # one block = the plain fit
    w0, b0, lh0 = oracle.fit_sgd(X, y, lr, 1000, 6)
    wf, bf, lhf = oracle.fit(X, y, lr, 6)
    assert np.array_equal(w0, wf) and b0 == bf and np.array_equal(lh0, lhf)
    # blocks of 300 rows: 300, 300, 300, 100; five steps by hand with the plain loss/gradient routine on slices
    w, b, losses = np.zeros(4), 0.0, []
    spans = [(0, 300), (300, 600), (600, 900), (900, 1000), (0, 300)]
    for a, c in spans:
        L, g, gb = oracle.loss_grad(X[a:c], y[a:c], w, b)
        losses.append(L)
        w, b = w - lr * g, b - lr * gb
    w1, b1, lh1 = oracle.fit_sgd(X, y, lr, 300, 5)
    np.testing.assert_allclose(w1, w, atol=1e-16, rtol=0)
    assert abs(b1 - b) < 1e-16
    np.testing.assert_allclose(lh1, losses, atol=1e-16, rtol=0)
    # resuming at the right block continues the same walk
    wa, ba, _ = oracle.fit_sgd(X, y, lr, 300, 3)
    wb, bb, _ = oracle.fit_sgd(X, y, lr, 300, 2, first_batch=3, w0=wa, b0=ba)
    assert np.array_equal(wb, w1) and bb == b1
    with pytest.raises(ValueError):
        oracle.fit_sgd(X, y, lr, 1001, 1)
