"""Tolerances shared by the GPU parity tests.

The stated bars (fp32 storage and accumulation against the float64 checker):
  gradient relative L2 <= 1e-5 per iteration, loss absolute <= 1e-6, fitted parameters relative L2 <= 1e-4,
  labels agreeing on >= 99.99 % of rows.

A relative bound on the gradient cannot hold once gradient descent has converged: the gradient tends to zero while
the rounding noise of an fp32 pass does not.  Each row's err = p - y carries an absolute error of a few units in the
last place of a number below one (2^-24 each from rounding z = x.w, from exp, from 1 + exp(-|z|), from the divide), and
part of it is systematic in z, hence correlated with x.  Modelling it as 8 * 2^-24 per row, independent across rows,
the sums sum_i x_ij * err_i carry a noise of 8 * 2^-24 * ||X_j||_2, and the gradient, stacked over columns and divided
by m, a noise of 8 * 2^-24 * ||[X 1]||_F / m.  The gradient bar is therefore
    ||g_gpu - g_ref||_2 <= max(1e-5 * ||g_ref||_2, 8 * 2^-24 * ||[X 1]||_F / m),
where the second term only matters at iterates whose gradient norm is below ~1e5 times that noise (the last
iterations of the fast-converging workloads).  ``test_fp32_floor.py`` shows on the CPU that even an idealised fp32
evaluation (float32 logits and sigmoid, exact float64 accumulation) misses the relative bar at such an iterate.
"""
import numpy as np

GRAD_TOL, LOSS_TOL, W_TOL, LABEL_AGREE = 1e-5, 1e-6, 1e-4, 0.9999


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64).ravel(), np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def frobenius_with_ones(X):
    """||[X 1]||_F in float64, accumulated in row chunks."""
    m = X.shape[0]
    s = float(m)
    step = 1 << 18
    for r in range(0, m, step):
        c = X[r:r + step].astype(np.float64)
        s += float(np.einsum("ij,ij->", c, c))
    return s ** 0.5


def grad_noise_floor(X, fro=None):
    fro = frobenius_with_ones(X) if fro is None else fro
    return 8.0 * 2.0 ** -24 * fro / X.shape[0]


def assert_grad_close(got, ref, floor, what=""):
    got, ref = np.asarray(got, dtype=np.float64).ravel(), np.asarray(ref, dtype=np.float64).ravel()
    err = float(np.linalg.norm(got - ref))
    bound = max(GRAD_TOL * float(np.linalg.norm(ref)), floor)
    assert err <= bound, (what, err, bound, float(np.linalg.norm(ref)))
