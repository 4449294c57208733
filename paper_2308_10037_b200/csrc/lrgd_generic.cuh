// Unstaged kernel for the rows the staged kernels do not take: more than 16384 elements.  E is the storage type of X.
// Plain coalesced loads; X is read from HBM once and a second time through the cache hierarchy.
//
// A CTA walks chunks of `rows` (8..kGenRows) rows (chunk c belongs to CTA c mod grid; the host picks the chunk so that
// the grid fills the GPU: with 64-row chunks of 64 KB rows a 512 MB matrix gave 128 CTAs work and ran at 0.5 TB/s).  Phase 1: one warp per row
// forms z = x.w + b (model equation, Section II-A), then err and the loss term (Eq. 1, Algorithm 7,
// log-likelihood), and parks err in shared memory.  Phase 2: thread t owns columns t, t+T, ...; it sums
// x[r][c]*err[r] over the chunk's rows in fp32 and adds the result to the CTA's own fp64 partial row
// in global memory (Algorithm 1's err.X).  Only this CTA ever touches that row, so there are no atomics
// and the result is bit-reproducible.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kGenRows = 64;
constexpr int kGenThreads = 256;

struct GenericParams {
    const void* X;            // fp32 or bfloat16 [m][n], row-major
    const float* y;
    long long m;
    int n;
    const float* w;
    const float* b;
    double* partial;          // [grid][n+2]
    unsigned char* labels;    // predict mode
    float cut;
    const int* stop;          // nullable: non-zero makes the launch a no-op
    int rows;                 // rows per chunk (a multiple of 8, at most kGenRows)
};

template <class E, bool PREDICT>
__global__ void __launch_bounds__(kGenThreads) k_generic(const GenericParams p) {
    grid_dependency_release();
    grid_dependency_wait();                        // the parameters and the stop flag come from the kernel before this one
    if (p.stop != nullptr && *reinterpret_cast<const volatile int*>(p.stop) != 0) return;   // a stopping rule was met by an earlier iteration
    __shared__ float err_s[kGenRows];
    __shared__ double red_e[kGenThreads / 32], red_l[kGenThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int NWARP = kGenThreads / 32;
    const int n = p.n;
    const float bval = __ldcg(p.b);
    double* out = PREDICT ? nullptr : p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
    if constexpr (!PREDICT) {
        for (int c = threadIdx.x; c < n + 2; c += kGenThreads) out[c] = 0.0;
    }
    double dse = 0.0, dsl = 0.0;                   // lane 0 of each warp
    const int R = p.rows;
    const long long nchunks = (p.m + R - 1) / R;
    for (long long chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        const long long row0 = chunk * R;
        const int rows = static_cast<int>(p.m - row0 < R ? p.m - row0 : R);
        for (int r = warp; r < rows; r += NWARP) {
            const long long xr = (row0 + r) * n;
            float d = 0.f;
            for (int c = lane; c < n; c += 32) d = fmaf(E::load(p.X, xr + c), __ldcg(p.w + c), d);
#pragma unroll
            for (int msk = 16; msk >= 1; msk >>= 1) d += __shfl_xor_sync(0xffffffffu, d, msk);
            const float z = d + bval;
            if constexpr (PREDICT) {
                if (lane == 0) p.labels[row0 + r] = z >= p.cut ? 1 : 0;
            } else {
                float e, L;
                logistic_terms(z, __ldg(p.y + row0 + r), e, L);
                if (lane == 0) { err_s[r] = e; dse += e; dsl += L; }
            }
        }
        if constexpr (!PREDICT) {
            __syncthreads();
            for (int c = threadIdx.x; c < n; c += kGenThreads) {
                const long long xc = row0 * n + c;
                float a = 0.f;
                for (int r = 0; r < rows; ++r) a = fmaf(E::load(p.X, xc + static_cast<long long>(r) * n), err_s[r], a);
                out[c] += static_cast<double>(a);
            }
            __syncthreads();
        }
    }
    if constexpr (!PREDICT) {
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }
        __syncthreads();
        if (threadIdx.x == 0) {
            double se = 0.0, sl = 0.0;
            for (int wi = 0; wi < NWARP; ++wi) { se += red_e[wi]; sl += red_l[wi]; }
            out[n] = se;
            out[n + 1] = sl;
        }
    }
}

}  // namespace lrgd
