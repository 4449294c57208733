/*
 * CPU checker ("oracle") for full-batch gradient-descent logistic regression.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain float64 statement of what the GPU
 * library must compute.  It shares no code, header, table or helper with the CUDA path and is
 * called only from the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * What it follows (paper: "High Performance Computing Applied to Logistic Regression"):
 *   - model            p(y=1|x) = 1/(1+exp(-w.x-b))                    Section II-A, model equation
 *   - sigmoid          1/(1+e^-x)                                      Eq. 1
 *   - log-likelihood   l(w,b) = sum_i y_i log p_i + (1-y_i) log(1-p_i) Section II-A
 *   - gradient step    grad = (1/m) err.X ; W = W - alpha*grad         Algorithm 1 (sequential version)
 *   - error sign       res <- sigmoid(res) - Y, then w <- w - alpha*grad  Algorithm 7 with Algorithm 5
 *
 * Readings taken where the paper is silent or inconsistent:
 *   - "Loss" is never defined; it is taken as the mean negative log-likelihood, loss = -l/m,
 *     matching the 1/m of Algorithm 1.
 *   - Algorithm 1 writes error = Y - y_pred and still subtracts alpha*grad (which would ascend);
 *     Algorithm 7 computes y_pred - Y.  The descent reading err = p - y is used.
 *   - The model has a bias b but Algorithms 1/7 carry only W; b is kept as an explicit scalar
 *     with grad_b = (1/m) sum_i err_i and the same learning rate.
 *   - Algorithm 7 drops the 1/m; it is kept (Algorithm 1).
 *   - Prediction threshold: the caller's thr; label = 1 iff p >= thr, decided as z >= log(thr/(1-thr)).
 *   - F1 with no true positives is 0.
 *
 * Arithmetic: X and y arrive as fp32 bits and are promoted element by element; everything else is
 * double.  Per-row loss is evaluated as max(z,0) + log1p(exp(-|z|)) - y*z, which equals
 * -[y log p + (1-y) log(1-p)] for y in {0,1} and stays finite for large |z|.
 * Rows are summed in index order inside fixed blocks of ORACLE_BLOCK_ROWS rows and the block sums
 * are added in block order, so the result does not depend on the thread count.
 *
 * Pins (tests, CPU only): ln 2 at w=b=0, X^T(0.5-y)/m at w=b=0, closed-form one- and two-row cases,
 * central finite differences, label-flip symmetry, row duplication, ones-column/bias equivalence,
 * saturation at |z|=40, descent-lemma monotonicity, planted-w* recovery, float64 autograd of a
 * library BCE-with-logits, brute-force predict and hand-counted F1; the stopping rule against the fixed-count
 * trajectory and its recorded norms; the penalty/momentum update against three steps done by hand from
 * oracle_loss_grad, central differences of the penalised loss and the vanishing penalised gradient at its fixed
 * point; mini-batch descent against five steps done by hand on row slices.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_BLOCK_ROWS 1024

int oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* z_i = b + sum_j X[i][j] w[j]   (Section II-A model equation; Algorithm 1, y_pred = sigmoid(W X^T)) */
static double row_logit(const float* xi, int32_t n, const double* w, double b) {
    double z = b;
    for (int32_t j = 0; j < n; ++j) z += (double)xi[j] * w[j];
    return z;
}

/* sums over rows [r0, r1): s[0..n) = sum x_ij e_i ; s[n] = sum e_i ; s[n+1] = sum L_i */
static void block_sums(const float* X, const float* y, int64_t r0, int64_t r1, int32_t n,
                       const double* w, double b, double* s) {
    for (int32_t j = 0; j < n + 2; ++j) s[j] = 0.0;
    for (int64_t i = r0; i < r1; ++i) {
        const float* xi = X + i * (int64_t)n;
        double z = row_logit(xi, n, w, b);
        double p = 1.0 / (1.0 + exp(-z));                                   /* Eq. 1 */
        double yi = (double)y[i];
        double e = p - yi;                                                  /* Algorithm 7 with Algorithm 5 */
        double L = fmax(z, 0.0) + log1p(exp(-fabs(z))) - yi * z;            /* -log-likelihood term */
        for (int32_t j = 0; j < n; ++j) s[j] += (double)xi[j] * e;          /* err.X, Algorithm 1 */
        s[n] += e;
        s[n + 1] += L;
    }
}

/* loss = -l/m ; grad_w = X^T err / m ; grad_b = sum err / m.  Returns 0, or -1 on bad arguments / no memory. */
int oracle_loss_grad(const float* X, const float* y, int64_t m, int32_t n, const double* w, double b,
                     double* loss, double* grad_w, double* grad_b) {
    if (!X || !y || !w || !loss || !grad_w || !grad_b || m < 1 || n < 1) return -1;
    int64_t nblocks = (m + ORACLE_BLOCK_ROWS - 1) / ORACLE_BLOCK_ROWS;
    size_t stride = (size_t)n + 2;
    double* part = (double*)malloc(sizeof(double) * stride * (size_t)nblocks);
    if (!part) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < nblocks; ++k) {
        int64_t r0 = k * ORACLE_BLOCK_ROWS;
        int64_t r1 = r0 + ORACLE_BLOCK_ROWS < m ? r0 + ORACLE_BLOCK_ROWS : m;
        block_sums(X, y, r0, r1, n, w, b, part + (size_t)k * stride);
    }
    double inv_m = 1.0 / (double)m;
    for (int32_t j = 0; j < n + 2; ++j) {
        double s = 0.0;
        for (int64_t k = 0; k < nblocks; ++k) s += part[(size_t)k * stride + j];
        if (j < n) grad_w[j] = s * inv_m;
        else if (j == n) *grad_b = s * inv_m;
        else *loss = s * inv_m;
    }
    free(part);
    return 0;
}

/*
 * iters steps of  w <- w - lr*grad_w, b <- b - lr*grad_b  (Algorithm 1 update; Algorithm 7 sign).
 * w[n], b[1] in/out.  loss_hist[iters] (nullable) receives the loss at the parameters BEFORE each update.
 * w_hist[(iters+1)*n], b_hist[iters+1] (nullable) receive the whole trajectory including the start.
 * round_to_fp32 != 0 rounds w and b to fp32 after every update (sensitivity study only).
 */
int oracle_fit(const float* X, const float* y, int64_t m, int32_t n, double lr, int32_t iters,
               double* w, double* b, double* loss_hist, double* w_hist, double* b_hist, int round_to_fp32) {
    if (!X || !y || !w || !b || m < 1 || n < 1 || iters < 0) return -1;
    double* g = (double*)malloc(sizeof(double) * (size_t)n);
    if (!g) return -1;
    if (w_hist) memcpy(w_hist, w, sizeof(double) * (size_t)n);
    if (b_hist) b_hist[0] = *b;
    for (int32_t t = 0; t < iters; ++t) {
        double loss, gb;
        if (oracle_loss_grad(X, y, m, n, w, *b, &loss, g, &gb) != 0) { free(g); return -1; }
        if (loss_hist) loss_hist[t] = loss;
        for (int32_t j = 0; j < n; ++j) w[j] -= lr * g[j];
        *b -= lr * gb;
        if (round_to_fp32) {
            for (int32_t j = 0; j < n; ++j) w[j] = (double)(float)w[j];
            *b = (double)(float)*b;
        }
        if (w_hist) memcpy(w_hist + (size_t)(t + 1) * n, w, sizeof(double) * (size_t)n);
        if (b_hist) b_hist[t + 1] = *b;
    }
    free(g);
    return 0;
}

/*
 * Algorithm 7's loop: form the gradient at the current point, apply the update, then stop if the 2-norm of the
 * gradient just applied is <= eps (Algorithm 4 gives the squared norm; Algorithm 7 compares its square root).
 * Reading: the bias is part of the model, so the norm is taken over (grad_w, grad_b) stacked.
 * At most max_iters updates.  *iters_done = updates applied, *grad_norm = norm of the last applied gradient
 * (-1 when max_iters == 0).  loss_hist / gnorm_hist (nullable, [max_iters]) are filled up to the stopping iteration.
 */
int oracle_fit_tol(const float* X, const float* y, int64_t m, int32_t n, double lr, double eps, int32_t max_iters,
                   double* w, double* b, double* loss_hist, double* gnorm_hist, int32_t* iters_done, double* grad_norm) {
    if (!X || !y || !w || !b || !iters_done || !grad_norm || m < 1 || n < 1 || max_iters < 0 || !(eps >= 0.0)) return -1;
    double* g = (double*)malloc(sizeof(double) * (size_t)n);
    if (!g) return -1;
    *iters_done = 0;
    *grad_norm = -1.0;
    for (int32_t t = 0; t < max_iters; ++t) {
        double loss, gb;
        if (oracle_loss_grad(X, y, m, n, w, *b, &loss, g, &gb) != 0) { free(g); return -1; }
        for (int32_t j = 0; j < n; ++j) w[j] -= lr * g[j];
        *b -= lr * gb;
        double q = 0.0;
        for (int32_t j = 0; j < n; ++j) q += g[j] * g[j];          /* Algorithm 4 */
        q += gb * gb;
        double nrm = sqrt(q);
        if (loss_hist) loss_hist[t] = loss;
        if (gnorm_hist) gnorm_hist[t] = nrm;
        *iters_done = t + 1;
        *grad_norm = nrm;
        if (nrm <= eps) break;                                      /* Algorithm 7: test after the update */
    }
    free(g);
    return 0;
}

/*
 * Gradient descent with an L2 penalty on w and (optionally Nesterov) momentum.  The paper only names these as future
 * work (Section V); the definitions are the textbook ones:
 *   loss = data loss + (l2/2) sum_j w_j^2 ;  g_w = grad_w + l2*w ;  g_b = grad_b   (bias not penalised)
 *   v <- mu*v + g ;  (w,b) <- (w,b) - lr*v            heavy ball
 *                    (w,b) <- (w,b) - lr*(g + mu*v)   Nesterov form, v already updated
 * vel[n+1] (w entries then b) is in/out.  loss_hist (nullable) gets the penalised loss before each update.
 */
int oracle_fit_opt(const float* X, const float* y, int64_t m, int32_t n, double lr, int32_t iters, double l2, double mu,
                   int nesterov, double* w, double* b, double* vel, double* loss_hist) {
    if (!X || !y || !w || !b || !vel || m < 1 || n < 1 || iters < 0 || !(l2 >= 0.0) || !(mu >= 0.0 && mu < 1.0)) return -1;
    double* g = (double*)malloc(sizeof(double) * (size_t)n);
    if (!g) return -1;
    for (int32_t t = 0; t < iters; ++t) {
        double loss, gb;
        if (oracle_loss_grad(X, y, m, n, w, *b, &loss, g, &gb) != 0) { free(g); return -1; }
        double sq = 0.0;
        for (int32_t j = 0; j < n; ++j) sq += w[j] * w[j];
        if (loss_hist) loss_hist[t] = loss + 0.5 * l2 * sq;
        for (int32_t j = 0; j <= n; ++j) {
            double gj = j < n ? g[j] + l2 * w[j] : gb;
            double v = mu * vel[j] + gj;
            double step = nesterov ? gj + mu * v : v;
            vel[j] = v;
            if (j < n) w[j] -= lr * step; else *b -= lr * step;
        }
    }
    free(g);
    return 0;
}

/*
 * Mini-batch gradient descent over contiguous row blocks, no shuffling (an "other optimiser" in the sense of the paper's
 * Section V, defined here): the rows are cut into ceil(m/batch_rows) blocks; step s uses block (first_batch + s) mod that
 * count, takes loss and gradient over that block alone (mean over its rows) and applies the Algorithm 1 update.
 */
int oracle_fit_sgd(const float* X, const float* y, int64_t m, int32_t n, double lr, int64_t batch_rows, int32_t steps,
                   int64_t first_batch, double* w, double* b, double* loss_hist) {
    if (!X || !y || !w || !b || m < 1 || n < 1 || steps < 0 || batch_rows < 1 || batch_rows > m || first_batch < 0) return -1;
    double* g = (double*)malloc(sizeof(double) * (size_t)n);
    if (!g) return -1;
    int64_t nb = (m + batch_rows - 1) / batch_rows;
    for (int32_t s = 0; s < steps; ++s) {
        int64_t k = (first_batch + s) % nb;
        int64_t r0 = k * batch_rows;
        int64_t rows = batch_rows < m - r0 ? batch_rows : m - r0;
        double loss, gb;
        if (oracle_loss_grad(X + r0 * (int64_t)n, y + r0, rows, n, w, *b, &loss, g, &gb) != 0) { free(g); return -1; }
        if (loss_hist) loss_hist[s] = loss;
        for (int32_t j = 0; j < n; ++j) w[j] -= lr * g[j];
        *b -= lr * gb;
    }
    free(g);
    return 0;
}

/* label_i = 1 iff p_i >= thr, decided in logit space: z_i >= log(thr/(1-thr)).  z_out (nullable) gets z. */
int oracle_predict(const float* X, int64_t m, int32_t n, const double* w, double b, double thr,
                   uint8_t* labels, double* z_out) {
    if (!X || !w || !labels || m < 1 || n < 1 || !(thr > 0.0 && thr < 1.0)) return -1;
    double cut = log(thr / (1.0 - thr));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        double z = row_logit(X + i * (int64_t)n, n, w, b);
        labels[i] = (uint8_t)(z >= cut ? 1 : 0);
        if (z_out) z_out[i] = z;
    }
    return 0;
}

/* Confusion counts of labels against y (y > 0.5 is positive) and F1 = 2TP/(2TP+FP+FN), 0 when TP = 0. */
int oracle_f1(const uint8_t* labels, const float* y, int64_t m, int64_t* tp, int64_t* fp, int64_t* fn, double* f1) {
    if (!labels || !y || m < 0 || !tp || !fp || !fn || !f1) return -1;
    int64_t a = 0, c = 0, d = 0;
    for (int64_t i = 0; i < m; ++i) {
        int pos = y[i] > 0.5f, pred = labels[i] != 0;
        a += (pred && pos);
        c += (pred && !pos);
        d += (!pred && pos);
    }
    *tp = a; *fp = c; *fn = d;
    *f1 = a > 0 ? (2.0 * (double)a) / (2.0 * (double)a + (double)c + (double)d) : 0.0;
    return 0;
}

/*
 * Rounding of binary32 values to the bfloat16 format (the reduced-precision storage variant of X; the paper
 * itself does not discuss storage precision).  bfloat16 is the upper half of binary32: 1 sign bit, the same 8
 * exponent bits, the top 7 fraction bits; a pattern h stands for the binary32 value with bits h << 16.
 * Rounding is IEEE 754 roundTiesToEven, written out as the definition: the two neighbouring bfloat16 values
 * (the truncated pattern and the next pattern away from zero) are decoded to double, the nearer one wins, and an
 * exact tie goes to the pattern whose last bit is 0.  The pattern past the largest finite value counts as
 * 2^128 for the distance and yields infinity.  NaN maps to a quiet NaN of the same sign; infinities and zeros
 * keep their sign.
 * Pins (tests, CPU only): hand-worked patterns in tests/golden/bf16_rounding_cases.txt, identity on all 65,536
 * patterns, a library conversion on random and special values, the half-spacing error bound and monotonicity.
 */
static double bf16_pattern_magnitude(uint32_t h15) {         /* h15 = pattern without its sign bit */
    uint32_t e = h15 >> 7, f = h15 & 0x7fu;
    if (e == 0) return ldexp((double)f / 128.0, -126);       /* subnormal (and zero) */
    return ldexp(1.0 + (double)f / 128.0, (int)e - 127);     /* e == 255, f == 0 gives 2^128: the overflow threshold */
}

int oracle_round_bf16(const float* x, int64_t count, uint16_t* bits_out, float* values_out) {
    if (!x || count < 0 || (!bits_out && !values_out)) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        uint32_t u;
        memcpy(&u, &x[i], 4);
        uint32_t sign = u >> 31, mag = u & 0x7fffffffu;
        uint32_t h15;
        if (mag > 0x7f800000u) {
            h15 = 0x7fc0u;                                   /* NaN -> quiet NaN */
        } else if (mag == 0x7f800000u) {
            h15 = 0x7f80u;                                   /* infinity */
        } else {
            uint32_t lo = mag >> 16, hi = lo + 1u;           /* neighbours: towards zero, away from zero */
            double v = fabs((double)x[i]);
            double d_lo = v - bf16_pattern_magnitude(lo);
            double d_hi = bf16_pattern_magnitude(hi) - v;
            if (d_lo < d_hi) h15 = lo;
            else if (d_hi < d_lo) h15 = hi;
            else h15 = (lo & 1u) ? hi : lo;                  /* tie: the even pattern */
        }
        uint16_t h = (uint16_t)((sign << 15) | h15);
        if (bits_out) bits_out[i] = h;
        if (values_out) {
            uint32_t w = (uint32_t)h << 16;
            memcpy(&values_out[i], &w, 4);
        }
    }
    return 0;
}
