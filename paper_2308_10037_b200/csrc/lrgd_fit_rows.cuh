// Persistent whole-fit kernel for rows of up to 512 columns: all `iters` gradient-descent iterations in ONE
// cooperative launch (one CTA per SM, co-resident), instead of two launches per iteration.
//
// Per iteration every CTA runs the same per-warp streaming pass as k_stream_rows (same static batch map, same
// arithmetic, same summation orders), writes its fp64 partial row, and meets the other CTAs at a grid barrier; the
// columns of the reduction + update (the arithmetic of k_reduce_update, slice for slice) are then spread over all
// warps of all CTAs, and a second grid barrier publishes the new parameters.  Results are bit-identical to the two-kernel path.
//
// What the single launch buys: no launch gaps, and the HBM stream never drains -- X does not depend on w, so each warp
// keeps re-arming its stages straight across the iteration boundary (the first batches of iteration t+1 are in flight
// while the CTAs reduce iteration t).  This matters for short passes (a 400 MB pass lasts ~60 us, of which launch,
// ramp-up and tail were ~20 %) and most for L2-resident problems.
//
// With a tolerance (lr_fit_tol) the kernel also forms ||grad||_2 after every update and all CTAs leave the loop together
// once it is <= eps: the stopping rule of Algorithm 7 with no host round trip and no wasted launch.
//
// Grid barrier: a monotonic counter in global memory; thread 0 of each CTA adds one and spins (bounded, 2 s) until the
// counter reaches grid * k.  On expiry, or when another CTA has raised the status word, the CTA stops iterating, waits
// (bounded) for its own copies in flight and retires with LR_ERR_TIMEOUT in the status word.
#pragma once
#include "lrgd_common.cuh"
#include "lrgd_reduce.cuh"
#include "lrgd_stream_rows.cuh"

namespace lrgd {

constexpr int kFitCombineCols = 64;            // columns combined per pass through the CTA's combine buffer
#ifndef LRGD_FIT_L2PF
#define LRGD_FIT_L2PF 4
#endif
constexpr int kFitL2Prefetch = LRGD_FIT_L2PF;   // batches per warp pulled into L2 ahead of the next iteration (beyond the staged ones)
constexpr int kFitTailBytes = 9216;            // combine buffer / reduction slices, after the stages

struct FitParams {
    const void* X;             // fp32 or bfloat16 [m][n], row-major
    const float* y;
    long long m;
    int n;
    float* w;                  // [n] in/out
    float* b;                  // [1] in/out
    double* partial;           // [grid][n+2]
    float* loss_hist;          // nullable [iters]
    int* status;               // device status word
    unsigned int* gbar;        // grid-barrier counter, zero at launch
    int depth;
    long long num_batches;
    long long keep_rows;       // rows [0, keep_rows) are fetched with an L2 evict-last hint, the rest evict-first
    int iters;
    double lr;
    double inv_m;
    // stopping rule (all null / zero for a fixed-count fit): as in k_reduce_update's tolerance mode
    TolState* tol;
    double* gbuf;              // [n+1] gradient entries of the current iteration
    double eps;
    float* gnorm_hist;         // nullable [iters]
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// All threads of the CTA call this.  Returns false if the barrier gave up (or the CTA had already given up).
__device__ __forceinline__ bool grid_barrier(unsigned int* counter, unsigned int target, int* status, volatile int* cta_abort) {
    __syncthreads();
    if (threadIdx.x == 0 && !*cta_abort) {
        __threadfence();
        atomicAdd(counter, 1u);
        const unsigned long long t0 = global_timer_ns();
        while (ld_acquire_u32(counter) < target) {
            if (*reinterpret_cast<volatile int*>(status) != 0 || global_timer_ns() - t0 > kWaitLimitNs) {
                atomicExch(status, kStatusTimeout);
                *cta_abort = 1;
                break;
            }
        }
        __threadfence();
    }
    __syncthreads();
    return *cta_abort == 0;
}

template <class E, int NV, int LPR, int RB, int NW>
__global__ void __launch_bounds__(NW * 32, 1) k_fit_rows(const FitParams p) {
    constexpr int EPG = E::EPG;
    constexpr int RPW = 32 / LPR;
    constexpr int RPB = RB * RPW;
    constexpr int LOG_LPR = Log2<LPR>::value;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = LOG_LPR - LOG_RB;
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(SHIFT >= 0, "rows per batch slot must not exceed lanes per row");
    static_assert(E::EPG > 1, "rows of 16-byte groups only");
    static_assert(kRedSlices == 32, "one lane per reduction slice of k_reduce_update");
    static_assert(NW * kFitCombineCols * 8 + 2 * NW * 8 <= kFitTailBytes, "tail too small");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    unsigned char* data = smem + kHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth;
    const int n = p.n, n4 = n / EPG;                   // n4 = 16-byte groups per row
    const int G = gridDim.x;
    const uint32_t row_bytes = static_cast<uint32_t>(n) * E::BYTES;
    const uint32_t stage_stride = (static_cast<uint32_t>(RPB) * row_bytes + 127u) & ~127u;
    unsigned char* my_stages = data + static_cast<size_t>(warp) * D * stage_stride;
    unsigned char* tail = data + static_cast<size_t>(NW) * D * stage_stride;      // combine buffer
    uint64_t* my_bars = bars + warp * kMaxDepth;

    const long long B = p.num_batches;
    const long long Bw = B > warp ? (B - warp + NW - 1) / NW : 0;
    const int cnt = Bw > blockIdx.x ? static_cast<int>((Bw - blockIdx.x + G - 1) / G) : 0;    // batches of this warp per iteration
    const int fill_iters = cnt > 0 ? p.iters : 0;  // the fit is cnt * fill_iters stage fills for this warp, iteration-major

    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) mbar_init(&my_bars[d], 1);
        fence_mbar_init();
    }
    __syncthreads();

    const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
    const long long stride_rows = static_cast<long long>(G) * NW * RPB;
    const long long first_row = (static_cast<long long>(blockIdx.x) * NW + warp) * RPB;
    auto issue = [&](long long r0, int d) {        // lane 0 only
        const long long left = p.m - r0;
        const uint32_t rows = left < RPB ? static_cast<uint32_t>(left) : RPB;
        const uint32_t xbytes = rows * row_bytes;
        mbar_arrive_expect_tx(&my_bars[d], xbytes);
        bulk_copy_g2s(my_stages + static_cast<size_t>(d) * stage_stride,
                      static_cast<const unsigned char*>(p.X) + static_cast<size_t>(r0) * row_bytes, xbytes, &my_bars[d],
                      r0 < p.keep_rows ? pol_keep : pol_stream);
    };

    const int sub = lane & (LPR - 1), slot = lane >> LOG_LPR;
    const int myr = ((sub >> SHIFT) & (RB - 1)) * RPW + slot;
    const bool owner = (sub & ((1 << SHIFT) - 1)) == 0;
    const bool full_cols = n4 == NV * LPR;

    // the fit is one long sequence of fills (iteration-major); consecutive fills land in consecutive stages (mod D)
    int issue_i = 0, issue_t = 0;                  // batch index and iteration of the next fill to issue (warp-uniform)
    long long issue_row = first_row;               // its first row
    int inflight = 0;                              // fills issued and not yet consumed
    auto next_fill = [&]() {
        issue_row += stride_rows;
        if (++issue_i == cnt) { issue_i = 0; issue_row = first_row; ++issue_t; }
    };
    for (int f = 0; f < D && issue_t < fill_iters; ++f) {
        if (lane == 0) issue(issue_row, f);
        next_fill();
        ++inflight;
    }
    int d = 0;
    uint32_t phase = 0;
    unsigned int barrier_no = 0;
    bool alive = true;                             // CTA-uniform after every grid barrier

    for (int t = 0; t < p.iters && alive; ++t) {
        typename E::template Lane<NV> lm;          // this lane's slice of the current w and its fp32 accumulators
        lm.load_w(p.w, sub, LPR, n4, true);
        lm.zero();
        const float bval = __ldcg(p.b);
        double dacc[NV][EPG];
        float se = 0.f, sl = 0.f;
        double dse = 0.0, dsl = 0.0;
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int c = 0; c < EPG; ++c) dacc[k][c] = 0.0;
        int since_flush = 0;
        long long row0 = first_row;
        float y_next = (cnt > 0 && row0 + myr < p.m) ? __ldg(p.y + row0 + myr) : 0.f;
        bool warp_ok = true;

        for (int i = 0; i < cnt; ++i) {
            bool ok = mbar_wait_bounded(&my_bars[d], phase, abort_flag);
            ok = __all_sync(FULL, ok);
            if (!ok) { warp_ok = false; break; }

            const long long left = p.m - row0;
            const int rows = left < RPB ? static_cast<int>(left) : RPB;
            const uint4* t4 = reinterpret_cast<const uint4*>(my_stages + static_cast<size_t>(d) * stage_stride);
            uint4 x[RB][NV];
            load_row_batch<uint4, NV, LPR, RB>(x, t4, rows, n4, full_cols && rows == RPB, sub, slot);
            const bool myvalid = myr < rows;
            const float yv = y_next;
            {
                const long long rn = row0 + stride_rows + myr;
                y_next = (i + 1 < cnt && rn < p.m) ? __ldg(p.y + rn) : 0.f;
            }
            // re-arm the stage with the fill `depth` ahead in the fit-long sequence (possibly of the next iteration)
            __syncwarp();
            if (issue_t < fill_iters) {
                if (lane == 0) {
                    fence_proxy_async_smem();
                    issue(issue_row, d);
                }
                next_fill();
            } else {
                --inflight;
            }
            if (++d == D) { d = 0; phase ^= 1u; }

            const float z = batch_dot<E, NV, LPR, RB>(x, lm, lane) + bval;
            float e, L;
            logistic_terms(z, yv, e, L);
            if (!myvalid) { e = 0.f; L = 0.f; }
            if (owner) { se += e; sl += L; }
            batch_accumulate<E, NV, LPR, RB>(x, e, lm);
            if (++since_flush == kFlushBatches) {
                since_flush = 0;
                fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
            }
            row0 += stride_rows;
        }
        (void)warp_ok;                             // a failed wait has raised the CTA's abort flag; handled at the barrier

        // The grid barriers, the reduction and the parameter reload below take longer than the staged batches of the next
        // iteration last; keep HBM busy meanwhile by pulling this warp's following batches of that iteration into L2.
        if (lane == 0 && t + 1 < p.iters) {
#pragma unroll
            for (int j = 0; j < kFitL2Prefetch; ++j) {
                const int bi = D + j;
                if (bi < cnt) {
                    const long long r0 = first_row + bi * stride_rows;
                    const long long left = p.m - r0;
                    const uint32_t rows = left < RPB ? static_cast<uint32_t>(left) : RPB;
                    bulk_prefetch_l2(static_cast<const unsigned char*>(p.X) + static_cast<size_t>(r0) * row_bytes, rows * row_bytes,
                                     r0 < p.keep_rows ? pol_keep : pol_stream);
                }
            }
        }

        fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);

        // ---- fixed-order combine of the CTA's warps, kFitCombineCols columns at a time (the stages stay in use) ----
        // row slots of one warp that own the same columns: add in slot order (as k_stream_rows does)
#pragma unroll
        for (int k2 = 0; k2 < NV; ++k2)
#pragma unroll
            for (int c = 0; c < EPG; ++c) {
                double tsum = 0.0;
#pragma unroll
                for (int sidx = 0; sidx < RPW; ++sidx) tsum += __shfl_sync(FULL, dacc[k2][c], sub + sidx * LPR);
                dacc[k2][c] = tsum;
            }
#pragma unroll
        for (int msk = 16; msk >= 1; msk >>= 1) {
            dse += __shfl_xor_sync(FULL, dse, msk);
            dsl += __shfl_xor_sync(FULL, dsl, msk);
        }
        double* red = reinterpret_cast<double*>(tail);                 // [NW][kFitCombineCols]
        double* red_e = red + NW * kFitCombineCols;
        double* red_l = red_e + NW;
        double* out = p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
        __syncthreads();                                               // previous use of the tail is over
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }
        for (int c0 = 0; c0 < n; c0 += kFitCombineCols) {
#pragma unroll
            for (int k2 = 0; k2 < NV; ++k2) {
                const int idx = sub + k2 * LPR;
                const int col = idx * EPG - c0;
                if (slot == 0 && idx < n4 && col >= 0 && col < kFitCombineCols) {
#pragma unroll
                    for (int c = 0; c < EPG; ++c) red[warp * kFitCombineCols + col + c] = dacc[k2][c];
                }
            }
            __syncthreads();
            if (threadIdx.x < kFitCombineCols && c0 + threadIdx.x < n) {
                double tsum = 0.0;
                for (int wi = 0; wi < NW; ++wi) tsum += red[wi * kFitCombineCols + threadIdx.x];
                out[c0 + threadIdx.x] = tsum;
            }
            __syncthreads();
        }
        if (threadIdx.x < 2) {
            const double* src = threadIdx.x == 0 ? red_e : red_l;
            double tsum = 0.0;
            for (int wi = 0; wi < NW; ++wi) tsum += src[wi];
            out[n + threadIdx.x] = tsum;
        }

        barrier_no += 1;
        alive = grid_barrier(p.gbar, static_cast<unsigned int>(G) * barrier_no, p.status, abort_flag);
        if (!alive) break;

        // ---- reduction + update: one warp per column, columns spread over all warps of all CTAs.  Lane s plays slice s of
        // k_reduce_update (rows [s*per, (s+1)*per) in index order); lane 0 then adds the 32 slice sums in slice order ----
        {
            const int stride = n + 2;
            const int per = (G + kRedSlices - 1) / kRedSlices;
            const int g0 = lane * per;
            const int g1 = g0 + per < G ? g0 + per : G;
            for (int col = warp * G + blockIdx.x; col < stride; col += NW * G) {
                double s = 0.0;
                const double* src = p.partial + col;
                for (int g = g0; g < g1; ++g) s += __ldcg(src + static_cast<size_t>(g) * stride);
                double tsum = 0.0;
#pragma unroll
                for (int k = 0; k < kRedSlices; ++k) tsum += __shfl_sync(FULL, s, k);
                if (lane == 0) {
                    const double v = tsum * p.inv_m;
                    if (col < n) p.w[col] = static_cast<float>(static_cast<double>(__ldcg(p.w + col)) - p.lr * v);
                    else if (col == n) p.b[0] = static_cast<float>(static_cast<double>(__ldcg(p.b)) - p.lr * v);
                    else if (p.loss_hist) p.loss_hist[t] = static_cast<float>(v);
                    if (p.tol != nullptr && col <= n) p.gbuf[col] = v;
                }
            }
        }
        barrier_no += 1;
        alive = grid_barrier(p.gbar, static_cast<unsigned int>(G) * barrier_no, p.status, abort_flag);

        // ---- stopping rule (Algorithm 7): ||(grad_w, grad_b)||_2 of the update just applied, formed by every CTA in the
        // same order as k_reduce_update's last block (lane-strided squares, xor tree), so all CTAs take the same decision ----
        if (p.tol != nullptr && alive) {
            double q = 0.0;
            for (int c = lane; c <= n; c += 32) {
                const double v = __ldcg(p.gbuf + c);
                q += v * v;
            }
#pragma unroll
            for (int msk = 16; msk >= 1; msk >>= 1) q += __shfl_xor_sync(FULL, q, msk);
            const double nrm = sqrt(q);
            if (blockIdx.x == 0 && threadIdx.x == 0) {
                p.tol->grad_norm = nrm;
                p.tol->iters_done = t + 1;
                if (p.gnorm_hist) p.gnorm_hist[t] = static_cast<float>(nrm);
                if (nrm <= p.eps) p.tol->stop = 1;
            }
            if (nrm <= p.eps) break;               // uniform over the whole grid: every warp computed the same nrm
        }
    }

    // Copies still in flight when the loop ends (a give-up, or an early stop with the next iteration already being
    // prefetched) must land before the CTA retires and its shared memory is handed to another CTA.
    if (!alive || *abort_flag) {
        if (lane == 0) atomicExch(p.status, kStatusTimeout);
    }
    if (inflight > 0) {
        if (lane == 0) {
            for (int f = 0; f < inflight; ++f) {           // the oldest fill in flight sits in stage d, phase parity `phase`
                mbar_wait_drain(&my_bars[d], phase);
                if (++d == D) { d = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    }
}

}  // namespace lrgd
