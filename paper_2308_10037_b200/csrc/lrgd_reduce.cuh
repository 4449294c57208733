// Second stage: fixed-order reduction of the per-CTA partial rows, 1/m scaling, and either the
// gradient/loss outputs or the fused parameter update  w <- w - lr*grad_w, b <- b - lr*grad_b
// (Algorithm 1's update; descent sign as in Algorithm 7).
//
// Block = 32 columns x kRedSlices slices.  Slice s sums partial rows [s*per, (s+1)*per) of its column in
// index order in fp64; the 32 slice sums are then added pairwise in a fixed tree (slice s with s+16, then
// with s+8, s+4, s+2, s+1).  No atomics on data: bit-reproducible.
//
// Tolerance mode (Algorithm 7's stopping rule, built from Algorithm 4's norm): every block parks its fp64
// gradient entries in `gbuf`; the block that finishes last (a ticket counter) adds their squares in index
// order, records ||grad||_2, counts the update, and raises `stop` when ||grad||_2 <= eps.  Kernels enqueued
// after that see `stop` and return without touching anything, so the parameters stay exactly as they were
// after the stopping update no matter how many further iterations the host had already enqueued.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kRedSlices = 32;           // 1024 threads: few dependent L2 reads per thread keeps this stage at ~2 us

// The fixed tree in which the 32 slice sums of a column are added: v[s] + v[s+16] for s < 16, then the 16 results
// pairwise at distance 8, and so on.  slice_tree_sum works on the 32 values held by one thread; slice_tree_sum_warp
// on one value per lane (a butterfly of xor shuffles: every lane ends with the value slice_tree_sum returns, because
// each step adds the same two numbers on both partners).  Depth five instead of a chain of 32 dependent additions.
__device__ __forceinline__ double slice_tree_sum(double (&v)[kRedSlices]) {
#pragma unroll
    for (int h = kRedSlices / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int i = 0; i < h; ++i) v[i] = v[i] + v[i + h];
    return v[0];
}
__device__ __forceinline__ double slice_tree_sum_warp(double v) {
#pragma unroll
    for (int msk = kRedSlices / 2; msk >= 1; msk >>= 1) v = v + __shfl_xor_sync(0xffffffffu, v, msk);
    return v;
}

struct TolState {             // device-resident, owned by the context
    int stop;                 // 1 once the tolerance has been met
    int iters_done;           // updates applied since the state was reset
    unsigned int ticket;      // blocks of the current reduction that have finished
    int pad;
    double grad_norm;         // ||(grad_w, grad_b)||_2 of the last applied update
};

struct ReduceParams {
    const double* partial;    // [G][n+2]: n column sums, sum err, sum loss
    int G;
    int n;
    double inv_m;
    double lr;
    int update;               // 1: update w, b in place; 0: write grad_w, grad_b
    float* w;
    float* b;
    float* grad_w;
    float* grad_b;
    float* loss_out;          // nullable
    double* raw_sums;         // non-null: write the unscaled fp64 sums [n+2] here and nothing else
    // tolerance mode (all null / zero otherwise)
    TolState* tol;
    double* gbuf;             // [n+1] scratch for the gradient entries
    double eps;
    float* gnorm_out;         // nullable: ||grad||_2 of this iteration
};

__global__ void __launch_bounds__(32 * kRedSlices) k_reduce_update(const ReduceParams p) {
    __shared__ double sh[kRedSlices][33];
    __shared__ int is_last;
    grid_dependency_release();
    grid_dependency_wait();                        // the partial rows come from the kernel before this one
    if (p.tol != nullptr && *reinterpret_cast<volatile int*>(&p.tol->stop) != 0) return;   // uniform: set by an earlier kernel
    const int col = blockIdx.x * 32 + threadIdx.x;
    const int slice = threadIdx.y;
    const int stride = p.n + 2;
    const int per = (p.G + kRedSlices - 1) / kRedSlices;
    const int g0 = slice * per;
    const int g1 = g0 + per < p.G ? g0 + per : p.G;
    // the parameter this thread will update is fetched together with the partial rows (one round trip instead of two)
    float old_param = 0.f;
    if (p.update && slice == 0 && col <= p.n) old_param = col < p.n ? __ldcg(p.w + col) : __ldcg(p.b);
    double s = 0.0;
    if (col < stride) {
        const double* src = p.partial + col;
#pragma unroll 8
        for (int g = g0; g < g1; ++g) s += __ldcg(src + static_cast<size_t>(g) * stride);   // straight from L2
    }
    sh[slice][threadIdx.x] = s;
    __syncthreads();
    if (slice == 0 && col < stride) {
        double sl[kRedSlices];
#pragma unroll
        for (int k = 0; k < kRedSlices; ++k) sl[k] = sh[k][threadIdx.x];
        const double t = slice_tree_sum(sl);
        if (p.raw_sums) {
            p.raw_sums[col] = t;
        } else {
            const double v = t * p.inv_m;
            if (col < p.n) {
                if (p.update) p.w[col] = static_cast<float>(static_cast<double>(old_param) - p.lr * v);
                else p.grad_w[col] = static_cast<float>(v);
            } else if (col == p.n) {
                if (p.update) p.b[0] = static_cast<float>(static_cast<double>(old_param) - p.lr * v);
                else p.grad_b[0] = static_cast<float>(v);
            } else {
                if (p.loss_out) p.loss_out[0] = static_cast<float>(v);
            }
            if (p.tol != nullptr && col <= p.n) p.gbuf[col] = v;
        }
    }
    if (p.tol == nullptr) return;

    // ---- tolerance mode: the last block to finish forms the norm ----
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && threadIdx.y == 0) {
        const unsigned int t = atomicAdd(&p.tol->ticket, 1u);
        is_last = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!is_last || threadIdx.y != 0) return;
    __threadfence();
    const volatile double* gb = p.gbuf;
    double q = 0.0;
    for (int c = threadIdx.x; c <= p.n; c += 32) {           // lane-strided, then a fixed xor tree: one fixed order
        const double v = gb[c];
        q += v * v;
    }
#pragma unroll
    for (int msk = 16; msk >= 1; msk >>= 1) q += __shfl_xor_sync(0xffffffffu, q, msk);
    if (threadIdx.x == 0) {
        const double nrm = sqrt(q);
        p.tol->grad_norm = nrm;
        p.tol->iters_done += 1;
        if (p.gnorm_out) p.gnorm_out[0] = static_cast<float>(nrm);
        if (nrm <= p.eps) p.tol->stop = 1;
        p.tol->ticket = 0u;
    }
}

// ------------------------------------------------------------------------------------------------------
// Second stage with an L2 penalty and momentum (the paper names regularisation and other optimisers as future
// work, Section V, without defining them; the definitions used here are the textbook ones):
//   loss   = data loss + (l2/2) * ||w||^2                (the bias is not penalised)
//   g_w    = X^T err / m + l2 * w ,  g_b = sum err / m
//   v     <- mu * v + g                                   (heavy-ball velocity, one entry per parameter)
//   w, b  <- w, b - lr * v            or, with nesterov:  w, b - lr * (g + mu * v)   (v already updated)
// Same fixed-order column reduction as k_reduce_update; the block that finishes last adds the squared old
// weights in index order and writes the penalised loss.
struct OptParams {
    const double* partial;    // [G][n+2]
    int G;
    int n;
    double inv_m;
    double lr;
    double l2;
    double mu;
    int nesterov;
    float* w;
    float* b;
    float* vel;               // [n+1] in/out
    float* loss_out;          // nullable
    double* scratch;          // [n+2]: squared old weights [n], spare, data loss
    unsigned int* ticket;
};

__global__ void __launch_bounds__(32 * kRedSlices) k_reduce_opt(const OptParams p) {
    __shared__ double sh[kRedSlices][33];
    __shared__ int is_last;
    grid_dependency_release();
    grid_dependency_wait();                        // the partial rows come from the kernel before this one
    const int col = blockIdx.x * 32 + threadIdx.x;
    const int slice = threadIdx.y;
    const int stride = p.n + 2;
    const int per = (p.G + kRedSlices - 1) / kRedSlices;
    const int g0 = slice * per;
    const int g1 = g0 + per < p.G ? g0 + per : p.G;
    double s = 0.0;
    if (col < stride) {
        const double* src = p.partial + col;
#pragma unroll 8
        for (int g = g0; g < g1; ++g) s += __ldcg(src + static_cast<size_t>(g) * stride);   // straight from L2
    }
    sh[slice][threadIdx.x] = s;
    __syncthreads();
    if (slice == 0 && col < stride) {
        double sl[kRedSlices];
#pragma unroll
        for (int k = 0; k < kRedSlices; ++k) sl[k] = sh[k][threadIdx.x];
        const double mean = slice_tree_sum(sl) * p.inv_m;
        if (col <= p.n) {
            float* param = col < p.n ? p.w + col : p.b;
            const double old = static_cast<double>(*param);
            const double g = col < p.n ? mean + p.l2 * old : mean;
            const double v = p.mu * static_cast<double>(p.vel[col]) + g;
            const double step = p.nesterov ? g + p.mu * v : v;
            p.vel[col] = static_cast<float>(v);
            *param = static_cast<float>(old - p.lr * step);
            if (col < p.n) p.scratch[col] = old * old;
        } else {
            p.scratch[p.n + 1] = mean;            // data loss
        }
    }
    if (p.loss_out == nullptr) return;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && threadIdx.y == 0) {
        const unsigned int t = atomicAdd(p.ticket, 1u);
        is_last = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!is_last || threadIdx.y != 0) return;
    __threadfence();
    const volatile double* sc = p.scratch;
    double q = 0.0;
    for (int c = threadIdx.x; c < p.n; c += 32) q += sc[c];
#pragma unroll
    for (int msk = 16; msk >= 1; msk >>= 1) q += __shfl_xor_sync(0xffffffffu, q, msk);
    if (threadIdx.x == 0) {
        p.loss_out[0] = static_cast<float>(sc[p.n + 1] + 0.5 * p.l2 * q);
        *p.ticket = 0u;
    }
}

}  // namespace lrgd
