// Second stage: fixed-order reduction of the per-CTA partial rows, 1/m scaling, and either the
// gradient/loss outputs or the fused parameter update  w <- w - lr*grad_w, b <- b - lr*grad_b
// (Algorithm 1's update; descent sign as in Algorithm 7).
//
// Block = 32 columns x kRedSlices slices.  Slice s sums partial rows [s*per, (s+1)*per) of its column in
// index order in fp64; the slices are then added in slice order.  No atomics: bit-reproducible.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kRedSlices = 8;

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
};

__global__ void __launch_bounds__(32 * kRedSlices) k_reduce_update(const ReduceParams p) {
    __shared__ double sh[kRedSlices][33];
    const int col = blockIdx.x * 32 + threadIdx.x;
    const int slice = threadIdx.y;
    const int stride = p.n + 2;
    const int per = (p.G + kRedSlices - 1) / kRedSlices;
    const int g0 = slice * per;
    const int g1 = g0 + per < p.G ? g0 + per : p.G;
    double s = 0.0;
    if (col < stride) {
        const double* src = p.partial + col;
        for (int g = g0; g < g1; ++g) s += src[static_cast<size_t>(g) * stride];
    }
    sh[slice][threadIdx.x] = s;
    __syncthreads();
    if (slice != 0 || col >= stride) return;
    double t = 0.0;
#pragma unroll
    for (int k = 0; k < kRedSlices; ++k) t += sh[k][threadIdx.x];
    if (p.raw_sums) {
        p.raw_sums[col] = t;
        return;
    }
    const double v = t * p.inv_m;
    if (col < p.n) {
        if (p.update) p.w[col] = static_cast<float>(static_cast<double>(p.w[col]) - p.lr * v);
        else p.grad_w[col] = static_cast<float>(v);
    } else if (col == p.n) {
        if (p.update) p.b[0] = static_cast<float>(static_cast<double>(p.b[0]) - p.lr * v);
        else p.grad_b[0] = static_cast<float>(v);
    } else {
        if (p.loss_out) p.loss_out[0] = static_cast<float>(v);
    }
}

}  // namespace lrgd
