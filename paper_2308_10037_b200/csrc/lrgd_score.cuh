// Confusion counts of predicted labels against the targets, for the f1 score the paper reports beside every timing
// (Section IV, Tables I and II: "f1").  With "predicted positive" = label != 0 and "positive" = y > 0.5:
//   tp = #(predicted positive and positive), fp = #(predicted positive and not positive), fn = #(not predicted
//   positive and positive);  f1 = 2 tp / (2 tp + fp + fn), taken as 0 when tp = 0.
// The counts are integers, so the order of the additions does not matter: every thread counts its elements, a warp adds
// its lanes' counts with shuffles, the warps of a CTA meet in shared memory, and three threads per CTA add the totals to
// the 64-bit counters in global memory with atomics -- exact and reproducible.  HBM-bound: one byte of label and four bytes of y per row.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kScoreThreads = 256;

// vec != 0: labels and y are 16-byte aligned, so a thread takes sixteen rows per step (one 16-byte load of labels,
// four of y); the rows past the last whole sixteen are taken one by one.  counts = {tp, fp, fn}, zeroed by the host.
__global__ void __launch_bounds__(kScoreThreads) k_confusion(const unsigned char* __restrict__ labels, const float* __restrict__ y,
                                                             long long m, unsigned long long* counts, int vec) {
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    unsigned long long tp = 0, fp = 0, fn = 0;
    auto count_one = [&](unsigned int pred, float yv) {
        const unsigned int pos = yv > 0.5f ? 1u : 0u;
        tp += pred & pos;
        fp += pred & (pos ^ 1u);
        fn += (pred ^ 1u) & pos;
    };
    long long done = 0;
    if (vec) {
        const long long blocks16 = m >> 4;
        for (long long q = tid; q < blocks16; q += nthreads) {
            const uint4 lab = __ldcs(reinterpret_cast<const uint4*>(labels) + q);
            const uint32_t word[4] = {lab.x, lab.y, lab.z, lab.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float4 yv = __ldcs(reinterpret_cast<const float4*>(y) + 4 * q + j);
                count_one(((word[j] >> 0) & 0xffu) != 0u, yv.x);
                count_one(((word[j] >> 8) & 0xffu) != 0u, yv.y);
                count_one(((word[j] >> 16) & 0xffu) != 0u, yv.z);
                count_one(((word[j] >> 24) & 0xffu) != 0u, yv.w);
            }
        }
        done = blocks16 << 4;
    }
    for (long long i = done + tid; i < m; i += nthreads) count_one(labels[i] != 0, y[i]);
#pragma unroll
    for (int msk = 16; msk >= 1; msk >>= 1) {
        tp += __shfl_xor_sync(0xffffffffu, tp, msk);
        fp += __shfl_xor_sync(0xffffffffu, fp, msk);
        fn += __shfl_xor_sync(0xffffffffu, fn, msk);
    }
    // one atomic per counter and CTA: the warps' totals meet in shared memory first
    __shared__ unsigned long long part[3][kScoreThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { part[0][warp] = tp; part[1][warp] = fp; part[2][warp] = fn; }
    __syncthreads();
    if (threadIdx.x < 3) {
        unsigned long long t = 0;
#pragma unroll
        for (int wi = 0; wi < kScoreThreads / 32; ++wi) t += part[threadIdx.x][wi];
        if (t) atomicAdd(counts + threadIdx.x, t);
    }
}

}  // namespace lrgd
