/*
 * lrgd -- full-batch gradient-descent logistic regression on one NVIDIA B200 (sm_100a).
 *
 * C-ABI boundary.  Plain pointers and sizes only.  Pointers named d_* are DEVICE pointers and
 * pointers named h_* are HOST pointers; both are owned by the caller.  The library never frees or
 * reallocates caller memory; it owns only the workspace inside an lr_ctx.
 *
 * Data layout: X is fp32, row-major, m rows by n columns with leading dimension n (row i starts at
 * X + i*n); y is fp32 with values 0.0f or 1.0f; w is fp32[n]; b is one fp32.  All arithmetic on the
 * m*n stream is fp32; the cross-block reduction is carried in fp64.
 *
 * What is computed (paper: "High Performance Computing Applied to Logistic Regression"):
 *   z_i = x_i.w + b, p_i = 1/(1+exp(-z_i))                 model equation of Section II-A, Eq. 1
 *   err_i = p_i - y_i                                      Algorithm 7 (sigmoid, then Substract(Y, res))
 *   loss = -(1/m) sum_i [y_i log p_i + (1-y_i) log(1-p_i)] mean negative log-likelihood, Section II-A
 *   grad_w = X^T err / m, grad_b = sum err / m             Algorithm 1 (the 1/m err.X line)
 *   w <- w - lr*grad_w, b <- b - lr*grad_b                 Algorithm 1 update, Algorithm 7 sign
 *
 * Streams: every device-pointer call enqueues its kernels on `stream` (a cudaStream_t passed as
 * void*, NULL = the legacy default stream) and returns without synchronising; outputs are valid once
 * the caller has synchronised that stream.  One lr_ctx must not be used from two streams at once.
 *
 * Errors: every call returns LR_OK (0) or a negative LR_ERR_* code; nothing is launched when
 * argument validation fails.  A wait inside a kernel that exceeds its bound makes the kernel finish
 * early and set a device status word, read back with lr_last_device_status.
 *
 * There is no CPU fallback: without a usable CUDA device lr_create fails with LR_ERR_CUDA.
 */
#ifndef LRGD_H
#define LRGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    LR_OK = 0,
    LR_ERR_NULL = -1,       /* a required pointer is NULL */
    LR_ERR_SHAPE = -2,      /* m < 1, n < 1, n > n_max of the ctx, iters < 0, m too large */
    LR_ERR_ALIGNMENT = -3,  /* a float pointer is not 4-byte aligned (a bfloat16 pointer: 2-byte) */
    LR_ERR_VALUE = -4,      /* thr outside (0,1), lr not finite */
    LR_ERR_CUDA = -5,       /* a CUDA runtime call failed; see lr_last_cuda_error */
    LR_ERR_TIMEOUT = -6,    /* a bounded device-side wait expired (reported by lr_last_device_status) */
    LR_ERR_NOMEM = -7       /* host or device allocation failed */
};

typedef struct lr_ctx lr_ctx;

/* Launch plan for a given shape, as chosen by the host logic (pure host code, no CUDA call). */
typedef struct lr_plan {
    int32_t variant;       /* 0 = row-per-lane-group staged kernel, 1 = row-split staged kernel, 2 = unstaged generic kernel,
                              3 = row-per-lane-group staged kernel for rows of any length up to 512 in a matrix aligned to its
                              element size only (a lane owns single elements: vec_per_lane counts elements, not 16-byte groups),
                              4 = row-split kernel with CTA-wide stages for such rows of 513..8192 elements and for every row of
                              8193..16384 elements */
    int32_t lanes_per_row; /* staged kernels: lanes that share one row (8, 16, 32; all threads of the CTA for the row-split kernel) */
    int32_t vec_per_lane;  /* staged kernels: 16-byte column groups owned by one lane */
    int32_t rows_per_batch;/* rows one warp (or one CTA for the row-split kernel) holds in registers at a time */
    int32_t tile_rows;     /* rows per asynchronously staged shared-memory stage */
    int32_t stages;        /* stages (copies in flight) per warp; per CTA for the row-split kernel */
    int32_t grid;          /* CTAs */
    int32_t threads;       /* threads per CTA: 512, or 256 for the shapes whose threads need more than 128 registers */
    int32_t smem_bytes;    /* dynamic shared memory per CTA */
} lr_plan;

/*
 * Host-only: fills *out with the launch plan lr_loss_grad / lr_fit / lr_predict use for an m-by-n
 * problem whose X pointer is 16-byte aligned (x_aligned16 != 0) or not, on a device with sm_count
 * multiprocessors.  Makes no CUDA call.  Returns LR_ERR_NULL / LR_ERR_SHAPE on bad arguments.
 */
int lr_plan_query(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, lr_plan* out);

/*
 * Creates a context on CUDA device `device` with workspace for problems of up to n_max columns
 * (any m: the workspace is one row of n_max + 2 sums per CTA and a few words of state, so the number of rows
 * of a problem needs no bound here).  Allocates the per-CTA partial-sum buffer and the device status word.
 * Every computing call runs inside a named NVTX range (lr_fit, lr_fit_tol, ...), visible on a profiler's timeline.
 * Errors: LR_ERR_NULL (out), LR_ERR_SHAPE (n_max < 1), LR_ERR_CUDA, LR_ERR_NOMEM.
 */
int lr_create(lr_ctx** out, int32_t device, int32_t n_max);

/* Frees the context's workspace (synchronises the device first).  NULL is accepted. */
int lr_destroy(lr_ctx* ctx);

/*
 * One full-batch pass at fixed parameters (Section II-A loss; Algorithm 1 gradient):
 *   d_loss[0] = loss, d_grad_w[0..n) = X^T err / m, d_grad_b[0] = sum err / m.
 * Inputs d_X [m*n], d_y [m], d_w [n], d_b [1] are read only.  Two kernels are enqueued: the fused
 * streaming kernel (reads X once) and the fixed-order cross-CTA reduction.
 * Which streaming kernel runs depends on the shape (lr_plan_query tells): rows of up to 16384 columns always take a staged
 * kernel (at HBM speed with d_X 16-byte aligned, n % 4 == 0 and n <= 8192; at a half to nine tenths of it for other lengths, for
 * matrices that are only 4-byte aligned and for rows beyond 8192 columns); wider rows run on a slower unstaged kernel.
 */
int lr_loss_grad(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n,
                 const float* d_w, const float* d_b,
                 float* d_loss, float* d_grad_w, float* d_grad_b, void* stream);

/*
 * `iters` gradient-descent steps (Algorithm 1 update with Algorithm 7's sign), fixed count, no
 * host synchronisation inside the loop.  d_w [n] and d_b [1] hold the start point on entry (the
 * caller zeroes them for a cold start) and the result on exit.  d_loss_hist is NULL or [iters] and
 * receives the loss at the parameters BEFORE update t.  iters == 0 is a no-op.
 * Results are bit-reproducible for a given shape and device, and fit(a) followed by fit(b) equals
 * fit(a+b) bit for bit.
 * Two forms give the same bits.  Two kernels per iteration (the pass, then the reduction with the update), each
 * launched as the programmatic dependent of the one before it (see lr_set_overlap); or, for rows of up to 256 or of
 * 388..512 columns (the shapes whose kernel runs 16 warps per CTA; 16-byte aligned X, n % 4 == 0) and iters >= 2, ONE cooperative
 * launch of a persistent kernel for the whole call: one grid barrier per iteration, after which every CTA adds up the
 * partial sums for itself and keeps its own copy of the parameters; the HBM stream continues across iterations, and a
 * problem whose rows all fit the CTAs' shared memory (up to ~28 MB) is fetched once and kept there for the whole call.
 * The library takes the persistent kernel wherever the shape allows it (it measures at least as fast everywhere).
 * lr_set_persistent(ctx, 0) forces two kernels (also used while lr_profile_enable is on, so that single launches can
 * be timed), a negative value restores the default, and a positive value asks for this persistent kernel in particular
 * (the default may take the single-cluster form below instead).  The same choice applies to lr_fit_tol and the bfloat16 calls.
 * If a bounded wait inside the persistent kernel expires, the kernel stops, the status word reports LR_ERR_TIMEOUT and
 * d_w, d_b are left as they were on entry.
 */
int lr_fit(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n,
           float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist, void* stream);
int lr_set_persistent(lr_ctx* ctx, int32_t on);
/*
 * Third form of lr_fit, for problems whose X fits the shared memory of ONE thread-block cluster of 16 (or 8) CTAs (up to
 * ~3 MB; rows of 16-byte groups as for the persistent kernel; at least one batch of rows for every CTA).  Such a
 * problem is planned on that many CTAs by every entry point (lr_plan_query shows grid = 16 or 8), so all of them divide
 * the rows the same way and all forms of the fit give the same bits.  lr_fit then runs the whole call as one launch on
 * one cluster: X is fetched once, and in every iteration each CTA pushes its partial sums into the shared memory of all
 * CTAs of the cluster with asynchronous remote stores that complete on the receiver's mbarrier, so an iteration never
 * touches global memory (10,000 x 32: 3 us per iteration where the grid-wide persistent kernel takes 4.3).
 * Taken by default where it applies, unless lr_set_persistent has asked for a particular form.  lr_set_cluster(ctx, 0)
 * switches the form off (the persistent kernel then runs on the same plan), any other value restores the default.
 * lr_fit_tol uses it too (the stopping rule is evaluated by every CTA of the cluster, same bits as the persistent kernel);
 * lr_fit_sharded does not.  A wait that expires ends the kernel as it ends the persistent one.
 * lr_cluster_ctas (host only, no CUDA call; arguments as lr_plan_query) returns the cluster size the form would use
 * for a shape, 0 if none; whether a cluster of that size can be resident is known at launch only (if not, the
 * persistent kernel runs).
 */
int lr_set_cluster(lr_ctx* ctx, int32_t on);
int32_t lr_cluster_ctas(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, int32_t bf16);

/*
 * Overlap between the kernels of one call (on by default).  Every iteration of the two-kernel form is a pass followed by
 * the reduction; with overlap on, each of them is launched as the programmatic dependent of the one before it: it is
 * scheduled while its predecessor drains, the pass stages its first rows of X (an input nothing in this library
 * writes) meanwhile, and it waits on the device for the predecessor to complete before it reads the parameters.  The
 * first kernel of a call is always an ordinary launch, so work the caller enqueued earlier on the stream is complete
 * before anything is read.  Results do not change.  lr_set_overlap(ctx, 0) launches every kernel the ordinary way.
 */
int lr_set_overlap(lr_ctx* ctx, int32_t on);

/*
 * L2 residency hint for iterated passes over the same X: the first `bytes` bytes of X (whole rows) are fetched with an
 * L2 evict-last hint and everything else with evict-first, so that across the iterations of a fit that leading part
 * of X is served from the 126 MB L2 instead of HBM.  Results do not change.  0 turns the hint off; -1 (the default)
 * lets the library choose: three quarters of the L2 for the wide-row kernel (n > 1024), where it is worth 12 % per pass
 * on 100k x 4096; a quarter of the L2 for the persistent narrow-row kernel, where the kept rows are the first ones every
 * warp needs after an iteration boundary (3 % per iteration on 1M x 100, 10 % on 250k x 256); and nothing for single
 * narrow-row passes, which measure slower with any part kept.
 */
int lr_set_l2_keep(lr_ctx* ctx, int64_t bytes);

/*
 * Gradient descent with the paper's stopping rule (Algorithm 7's loop; the norm is Algorithm 4's):
 *   repeat { grad at the current (w, b);  w <- w - lr*grad_w, b <- b - lr*grad_b;
 *            if ||(grad_w, grad_b)||_2 <= eps: stop }   -- the update is applied before the test, as in
 * Algorithm 7 -- for at most max_iters updates.  The norm is formed on the device in fp64 from the same
 * sums the update uses; once it is met a device flag turns every later launch of this call into a
 * no-op, so the result does not depend on check_every.  The host enqueues check_every iterations at a
 * time and then synchronises `stream` to read the flag (this call blocks, unlike lr_fit).  Where lr_fit would take its
 * persistent kernel (see lr_fit) the whole run is instead ONE persistent launch in which all CTAs form the norm after
 * every update and leave the loop together (check_every is not used; no launch is wasted); both forms give the same bits.
 * d_w, d_b in/out as for lr_fit; d_loss_hist / d_gnorm_hist are NULL or [max_iters] (entries past the
 * stopping iteration are left untouched); *iters_done receives the number of updates applied and
 * *grad_norm the norm of the last applied gradient (-1 if max_iters == 0).  The caller tells
 * "converged" from "ran out of iterations" by comparing *grad_norm with eps.
 * Errors as lr_fit, plus LR_ERR_SHAPE for check_every < 1 and LR_ERR_VALUE for eps < 0 or not finite.
 */
int lr_fit_tol(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n,
               float lr, float eps, int32_t max_iters, int32_t check_every,
               float* d_w, float* d_b, float* d_loss_hist, float* d_gnorm_hist,
               int32_t* iters_done, float* grad_norm, void* stream);

/*
 * Gradient descent with an L2 penalty and momentum.  The paper lists regularisation and other optimisers as future
 * work (Section V) without defining them; the textbook definitions are used:
 *   loss = data loss + (l2/2)*||w||^2 (the bias is not penalised);  g_w = X^T err/m + l2*w,  g_b = sum err/m;
 *   v <- momentum*v + g;   w, b <- w, b - lr*v,   or with nesterov != 0:  w, b - lr*(g + momentum*v)  (v updated first).
 * l2 = 0, momentum = 0 reproduces lr_fit bit for bit.  d_velocity is NULL (a context-owned velocity, zeroed at the start of
 * the call) or a device array [n+1] (w entries, then b) that is read and updated, so a run can be split across calls.
 * d_loss_hist (NULL or [iters]) receives the penalised loss at the parameters before each update.
 * Errors as lr_fit, plus LR_ERR_VALUE for l2 < 0 or momentum outside [0, 1).
 */
typedef struct lr_opt {
    float l2;
    float momentum;
    int32_t nesterov;
} lr_opt;
int lr_fit_opt(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n,
               float lr, int32_t iters, const lr_opt* opt,
               float* d_w, float* d_b, float* d_velocity, float* d_loss_hist, void* stream);

/*
 * Mini-batch gradient descent over contiguous row blocks (one of the "other optimisers" the paper leaves to future
 * work, Section V; deterministic: no shuffling).  The rows are cut into ceil(m / batch_rows) blocks of batch_rows rows
 * (the last one may be shorter); step s uses block (first_batch + s) mod that count, forms loss and gradient over that
 * block alone (scaled by 1 / rows in the block) and applies  w <- w - lr*grad_w, b <- b - lr*grad_b.
 * batch_rows == m is lr_fit.  d_loss_hist (NULL or [steps]) receives the block's loss before each update.
 * Errors as lr_fit, plus LR_ERR_SHAPE for batch_rows outside [1, m] or first_batch < 0.
 */
int lr_fit_sgd(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n,
               float lr, int64_t batch_rows, int32_t steps, int64_t first_batch,
               float* d_w, float* d_b, float* d_loss_hist, void* stream);

/*
 * d_labels[i] = 1 if sigmoid(x_i.w + b) >= thr else 0, decided in logit space as
 * z_i >= log(thr/(1-thr)) evaluated in fp32 (the paper reports f1 but states no threshold; the
 * caller supplies it).  0 < thr < 1.  d_labels is uint8 [m].
 */
int lr_predict(lr_ctx* ctx, const float* d_X, int64_t m, int32_t n,
               const float* d_w, const float* d_b, float thr, uint8_t* d_labels, void* stream);

/*
 * Confusion counts behind the f1 score that the paper reports beside every timing (Section IV, Tables I and II; it
 * does not spell the score out, so the usual definition is used).  With "predicted positive" = d_labels[i] != 0 and
 * "positive" = d_y[i] > 0.5:
 *   d_counts[0] = tp = predicted positive and positive,  d_counts[1] = fp = predicted positive and not positive,
 *   d_counts[2] = fn = not predicted positive and positive;   f1 = 2 tp / (2 tp + fp + fn), 0 when tp == 0
 * (the quotient is left to the caller: three integers are exact, a device-side double would add nothing).
 * d_labels is a DEVICE array uint8 [m] (lr_predict's output), d_y DEVICE fp32 [m], d_counts DEVICE int64 [3], 8-byte
 * aligned, overwritten (zeroed on the stream, then added to by one kernel; integer sums, so the result does not depend
 * on the order).  m == 0 gives three zeros.  Fastest with d_labels and d_y 16-byte aligned.  Errors: LR_ERR_NULL,
 * LR_ERR_SHAPE (m < 0 or beyond 2^40), LR_ERR_ALIGNMENT (d_y not 4-byte, d_counts not 8-byte aligned), LR_ERR_CUDA.
 */
int lr_f1_counts(lr_ctx* ctx, const uint8_t* d_labels, const float* d_y, int64_t m, int64_t* d_counts, void* stream);

/*
 * bfloat16 storage of X (not in the paper, which is silent on storage precision; it halves the bytes the pass has to
 * stream).  d_Xh is a DEVICE array of m*n bfloat16 patterns (uint16: the upper half of a binary32 pattern), row-major
 * with leading dimension n, 2-byte aligned.  Only X changes: y, w, b, the gradient and every sum stay as in the fp32
 * calls, each element of X is widened exactly to fp32 when it is used, so the three calls below compute exactly what
 * lr_loss_grad / lr_fit / lr_predict would compute on the fp32 matrix holding the same (bfloat16-representable) values.
 * Rows of up to 16384 columns always take a staged kernel (fastest with n % 8 == 0, d_Xh 16-byte aligned and n <= 8192); wider rows
 * run on the unstaged kernel.  lr_fit_bf16 takes the persistent kernel of lr_fit for rows of up to 512 columns with n % 8 == 0 and
 * d_Xh 16-byte aligned.  Errors as the fp32 calls.
 *
 * lr_convert_bf16 rounds `count` fp32 values to bfloat16 (round to nearest, ties to even; NaN stays NaN, values past
 * the largest finite bfloat16 become infinity) -- one elementwise kernel on `stream`; d_X and d_Xh must not overlap.
 * count == 0 is a no-op.
 * lr_plan_query_bf16 is lr_plan_query for a bfloat16 matrix (lanes and groups then count 8 columns per 16 bytes).
 */
int lr_convert_bf16(lr_ctx* ctx, const float* d_X, int64_t count, uint16_t* d_Xh, void* stream);
int lr_loss_grad_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n,
                      const float* d_w, const float* d_b,
                      float* d_loss, float* d_grad_w, float* d_grad_b, void* stream);
int lr_fit_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n,
                float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist, void* stream);
int lr_predict_bf16(lr_ctx* ctx, const uint16_t* d_Xh, int64_t m, int32_t n,
                    const float* d_w, const float* d_b, float thr, uint8_t* d_labels, void* stream);
int lr_plan_query_bf16(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, lr_plan* out);
/* lr_fit_tol, lr_fit_opt, lr_fit_sgd and lr_shard_sums on a bfloat16-stored X: same contracts, same arithmetic, d_Xh as above
 * (lr_fit_sgd_bf16's row blocks start at d_Xh + block*batch_rows*n; a block that does not start on a 16-byte boundary
 * runs on the unstaged kernel).  lr_apply_sums is independent of the storage type. */
int lr_fit_tol_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n,
                    float lr, float eps, int32_t max_iters, int32_t check_every,
                    float* d_w, float* d_b, float* d_loss_hist, float* d_gnorm_hist,
                    int32_t* iters_done, float* grad_norm, void* stream);
int lr_fit_opt_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n,
                    float lr, int32_t iters, const lr_opt* opt,
                    float* d_w, float* d_b, float* d_velocity, float* d_loss_hist, void* stream);
int lr_fit_sgd_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n,
                    float lr, int64_t batch_rows, int32_t steps, int64_t first_batch,
                    float* d_w, float* d_b, float* d_loss_hist, void* stream);
int lr_shard_sums_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m_local, int32_t n,
                       const float* d_w, const float* d_b, double* d_sums, void* stream);

/*
 * Row-sharded data parallelism (the natural split of Algorithm 1's sums over rows; the paper itself
 * runs on one device).  Each shard holds a contiguous block of rows.  lr_shard_sums runs the fused
 * pass on the local rows and writes the UNNORMALISED fp64 sums d_sums[0..n) = X^T err,
 * d_sums[n] = sum err, d_sums[n+1] = sum of per-row loss terms.  After the caller has gathered the
 * `parts` sum vectors into d_sums_all [parts][n+2] (rank order), lr_apply_sums adds them in a fixed
 * order (a pairwise tree over the parts), scales by 1/m_total and applies  w <- w - lr*grad_w, b <- b - lr*grad_b  (every rank gets
 * bit-identical parameters); d_loss (nullable) receives the global loss before the update.
 */
int lr_shard_sums(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m_local, int32_t n,
                  const float* d_w, const float* d_b, double* d_sums, void* stream);
int lr_apply_sums(lr_ctx* ctx, const double* d_sums_all, int32_t parts, int64_t m_total, int32_t n,
                  float lr, float* d_w, float* d_b, float* d_loss, void* stream);

/*
 * Row-sharded fit with the exchange inside the kernel (same split of Algorithm 1's sums over rows as lr_shard_sums /
 * lr_apply_sums, without a host round trip or a collective call per iteration).  Every rank calls lr_fit_sharded with
 * its own rows (m_local of the m_total rows), the same n, lr and iters, and the same start point in d_w, d_b.  Each
 * iteration a rank forms the n+2 sums of its rows in one persistent launch (see lr_fit), stores them into slot
 * [step parity][rank] of EVERY rank's exchange buffer with plain stores, publishes the step number in flag [rank] of
 * every buffer (system-scope release), waits until the flags of all ranks in its own buffer show the step, adds the
 * `world` vectors in the fixed order lr_apply_sums uses and applies the update.  All ranks end with bit-identical
 * parameters, and with the bits the lr_shard_sums / all-gather / lr_apply_sums loop gives.  With world == 1 the result is
 * lr_fit's, bit for bit.  d_loss_hist (NULL or [iters]) receives the global loss on every rank.
 *
 * Exchange buffers: one per rank, in that rank's own device memory, lr_exchange_bytes(world, n) bytes, 128-byte aligned,
 * ZEROED ONCE before the first use (followed by a barrier among the ranks), and mapped into every other rank's address
 * space (peer access within a process, CUDA IPC or a symmetric-memory allocation between processes).  d_exchange is a HOST
 * array of `world` device pointers as THIS rank addresses them; d_exchange[rank] is its own buffer.  Only plain loads
 * and stores touch a peer's memory.
 * epoch: the number of steps these buffers have carried so far -- 0 for the first call, then the sum of the iters of the
 * earlier calls; it must be the same on every rank (the flags count steps monotonically across calls).
 * wait_ms (1..60000): bound on every wait for the other ranks.  When it expires (a rank that died or never called), the
 * kernel stops, d_w and d_b keep their values from before the call and lr_last_device_status reports LR_ERR_TIMEOUT;
 * the buffers must then be zeroed and the epoch restarted before they are used again.
 * Shapes: those lr_fit runs as one persistent launch (rows of up to 1024 columns, 16-byte aligned X, n % 4 == 0; n % 8 for
 * bfloat16) on a device with cooperative launches; anything else returns LR_ERR_SHAPE (use lr_shard_sums / lr_apply_sums).
 * Errors: as lr_fit, plus LR_ERR_SHAPE for world outside 1..32, rank outside [0, world), m_total < m_local, epoch < 0;
 * LR_ERR_VALUE for wait_ms out of range; LR_ERR_ALIGNMENT for an exchange buffer that is not 128-byte aligned.
 */
int lr_exchange_bytes(int32_t world, int32_t n, int64_t* bytes);
int lr_fit_sharded(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m_local, int64_t m_total, int32_t n,
                   float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist,
                   int32_t rank, int32_t world, void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream);
int lr_fit_sharded_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m_local, int64_t m_total, int32_t n,
                        float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist,
                        int32_t rank, int32_t world, void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream);

/*
 * The ranks of lr_fit_sharded on ONE GPU: `world` (2..32) row shards run as `world` groups of CTAs of a single cooperative
 * launch, each group with its own rows, parameters and exchange buffer, exchanging exactly as ranks on different GPUs do.
 * Because all CTAs of a cooperative launch are resident together, ranks that wait on one another cannot starve each
 * other -- which separate launches, streams or processes on one GPU could not guarantee.  This is the way to run and
 * test the multi-rank path where a single GPU is available; it is not faster than lr_fit.
 * d_X, d_y, m_local, d_w, d_b, d_loss_hist (nullable, entries nullable) and d_exchange are HOST arrays of `world`
 * entries (device pointers / row counts); d_w[r], d_b[r] hold the common start point and receive rank r's result.
 * Every rank takes plan-SMs / world SMs (see lr_set_sm_limit).  Built for fp32 rows of up to 32 and of 132..256 columns
 * with 16-byte aligned shards; other shapes return LR_ERR_SHAPE.  The call blocks until its parameter block is on the device.
 */
int lr_fit_sharded_local(lr_ctx* ctx, int32_t world, const float* const* d_X, const float* const* d_y, const int64_t* m_local,
                         int32_t n, float lr, int32_t iters, float* const* d_w, float* const* d_b, float* const* d_loss_hist,
                         void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream);

/*
 * Limits the SMs (CTAs) the launch plans of this context use to `sms`; 0 restores the device's count.  The per-CTA
 * partial sums, hence the low bits of every result, depend on the grid: two contexts with the same limit on the same
 * kind of device give the same bits.
 */
int lr_set_sm_limit(lr_ctx* ctx, int32_t sms);

/*
 * Host-buffer variants: copy h_X, h_y (and h_w, h_b) to device buffers owned by the context
 * (allocated or grown on first use), run the same kernels, copy the results back, and synchronise.
 * h_w / h_b are in-out as for lr_fit; h_loss_hist is NULL or [iters]; h_labels is uint8 [m].
 * Pinned host memory makes the copies faster but is not required.
 */
int lr_fit_host(lr_ctx* ctx, const float* h_X, const float* h_y, int64_t m, int32_t n,
                float lr, int32_t iters, float* h_w, float* h_b, float* h_loss_hist);
int lr_predict_host(lr_ctx* ctx, const float* h_X, int64_t m, int32_t n,
                    const float* h_w, const float* h_b, float thr, uint8_t* h_labels);
/* The same with X stored as bfloat16 on the device: h_X is fp32 as above, it is copied in and rounded once on the device
 * (lr_convert_bf16), and the bfloat16 entry points run on the rounded matrix (half the bytes per pass; the result is what
 * lr_fit / lr_predict give on the matrix of rounded values). */
int lr_fit_host_bf16(lr_ctx* ctx, const float* h_X, const float* h_y, int64_t m, int32_t n,
                     float lr, int32_t iters, float* h_w, float* h_b, float* h_loss_hist);
int lr_predict_host_bf16(lr_ctx* ctx, const float* h_X, int64_t m, int32_t n,
                         const float* h_w, const float* h_b, float thr, uint8_t* h_labels);

/*
 * Per-kernel timing for measurement.  While enabled, lr_loss_grad / lr_fit / lr_predict bracket every
 * launch of the streaming kernel with CUDA events on the caller's stream (up to 4096 launches since
 * the last reset).  lr_profile_read synchronises those events and returns the number of bracketed
 * launches and the sum of their durations in milliseconds, then clears the record.
 */
int lr_profile_enable(lr_ctx* ctx, int32_t on);
int lr_profile_read(lr_ctx* ctx, int32_t* launches, double* total_ms);

/* Number of kernels this context has launched since it was created. */
int lr_launch_count(lr_ctx* ctx, int64_t* out);

/* Synchronises the device and returns in *out the device status word: LR_OK or LR_ERR_TIMEOUT.  Clears it. */
int lr_last_device_status(lr_ctx* ctx, int32_t* out);

/*
 * Bounds check of the library's own device workspaces (no counterpart in the paper).  Every array that the kernels index
 * by a computed offset -- the per-CTA partial rows, the gradient buffer of the stopping rule, the context's velocity and
 * the optimiser scratch -- is allocated between two 256-byte guard regions filled with a fixed pattern when the context
 * is created.  lr_check_guards synchronises the device, reads the guard regions back and returns in *corrupted how many of
 * them (0..8) no longer hold the pattern: anything but 0 means a kernel wrote outside its array.  It changes nothing, so it
 * can be called at any point between calls; the tests call it after every batch of shapes.
 */
int lr_check_guards(lr_ctx* ctx, int32_t* corrupted);

/*
 * Exercises the give-up path of the bounded device-side waits without harming the device: enqueues a one-warp
 * kernel that waits on an mbarrier which is completed up front (arm != 0) or never (arm == 0), for at most limit_ms
 * (1..1000) milliseconds.  When the wait runs out the kernel sets the device status word, exactly as a streaming kernel
 * whose copy never lands would, and returns; lr_last_device_status then reports LR_ERR_TIMEOUT and clears it.
 */
int lr_selftest_wait(lr_ctx* ctx, int32_t arm, int32_t limit_ms, void* stream);

/* The cudaError_t value of the most recent failing CUDA call made through this context (0 if none). */
int lr_last_cuda_error(lr_ctx* ctx);

/*
 * lr_loss_grad without any allocation.  (The paper has no counterpart; this exists for callers that
 * must not allocate.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a latency-critical loop that cannot
 * afford the allocator's lock or the device-wide synchronisation a cudaFree brings; a process whose
 * device memory has been handed in full to another allocator (a framework's caching pool), where a
 * late cudaMalloc can fail; a plug-in whose host forbids allocation after start-up.  lr_create
 * allocates a workspace, so those callers cannot use a context.
 *
 * Same computation and outputs as lr_loss_grad (d_loss[1], d_grad_w[n], d_grad_b[1]; inputs read only),
 * but no lr_ctx: the per-CTA partial sums go to a fixed array that is part of the library's device
 * image (about 2 MiB on every GPU that loads the library, until the process exits).  The call makes no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Limits: n <= LR_NOALLOC_MAX_N (else LR_ERR_SHAPE, nothing launched); device index < 64.
 * d_status is NULL or a device int32 that the call zeroes and the kernel sets to LR_ERR_TIMEOUT if a
 * bounded device-side wait expires (read it after synchronising the stream).
 * First call on a device: resolves the array's device address and reads the SM count; make that first
 * call outside any stream capture.
 * Sharing: every call on a device uses the same array and finds the previous call's contents in it;
 * the call clears what has to start from zero itself.  Two calls that overlap on the GPU (different
 * streams, or different host threads without ordering) race on the array -- order them on one stream
 * or with events.
 */
#define LR_NOALLOC_MAX_N 1022
int lr_loss_grad_noalloc(int32_t device, const float* d_X, const float* d_y, int64_t m, int32_t n,
                         const float* d_w, const float* d_b,
                         float* d_loss, float* d_grad_w, float* d_grad_b, int32_t* d_status, void* stream);

/* Static description of a status code. */
const char* lr_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* LRGD_H */
