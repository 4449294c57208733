// Whole-fit kernel for problems small enough to live in the shared memory of ONE thread-block cluster (up to ~3 MB of X):
// all iterations in one launch, like k_fit_rows, but nothing leaves the cluster between the first fetch of X and the
// final store of the parameters.  Where k_fit_rows goes through global memory twice per iteration (partial rows out,
// a counter, partial rows of every CTA back from L2), a CTA here PUSHES its partial row into the shared memory of every
// CTA of the cluster with asynchronous remote stores that complete on the receiver's mbarrier; a CTA waits on its own
// mbarrier only, for C rows' worth of bytes, and then finds all rows in its own shared memory.  One one-way trip through the
// cluster's interconnect per iteration instead of a barrier and a round trip.
//
// The result has the bits of k_fit_rows (and of the two-kernel form) run on a grid of C CTAs: the same batches for the
// same warps, the same order inside a warp, the same combine of a CTA's warps, and k_reduce_update's order over the C
// partial rows (a slice is a single row).
//
// Buffers and phases.  The C rows of iteration t land in slot set t & 1 and complete mbarrier t & 1 (phase (t >> 1) & 1).
// A CTA cannot send the rows of iteration t+2 (same set as t) before it has received everybody's row of t+1, and a CTA
// sends its row of t+1 only after it has read set t -- so a set is never overwritten while somebody still reads it, and
// bytes of iteration t+2 never count towards the phase of t.  Bytes may arrive before the receiver has armed the phase
// (its own arrive.expect_tx is the only arrival the phase waits for, so it cannot complete early).
//
// Every wait is bounded.  A CTA whose wait expires raises the status word and stops sending; the others then run into
// their own bound.  Nobody leaves before all CTAs have stopped sending (the cluster barrier at the end, which every CTA
// reaches because nothing before it waits without a bound).
//
// With a tolerance (lr_fit_tol) every CTA also forms ||grad||_2 of the update just applied, in k_fit_rows' order, so all CTAs
// get the same bits and leave the loop in the same iteration once it is <= eps (Algorithm 7's stopping rule).  Row shards
// stay with k_fit_rows.
#pragma once
#include <cooperative_groups.h>

#include "lrgd_common.cuh"
#include "lrgd_fit_rows.cuh"
#include "lrgd_reduce.cuh"
#include "lrgd_stream_rows.cuh"

namespace lrgd {

constexpr int kClusterMaxCtas = 16;

struct ClusterFitParams {
    const void* X;             // fp32 or bfloat16 [m][n], row-major
    const float* y;
    long long m;
    int n;
    float* w;                  // [n] in/out
    float* b;                  // [1] in/out
    float* loss_hist;          // nullable [iters]
    int* status;               // device status word
    int depth;                 // stages per warp = most batches any warp owns (all of X stays in shared memory)
    long long num_batches;
    int iters;
    double lr;
    double inv_m;
    unsigned int* abort_word;  // raised (1) if a bounded wait expired anywhere in the cluster; zero at launch
    // stopping rule (all null / zero for a fixed-count fit): as in k_fit_rows
    TolState* tol;
    double eps;
    float* gnorm_hist;         // nullable [iters]
};

// shared memory of a CTA: header and stages as k_fit_rows lays them out, its tail (combine buffer, parameters, this CTA's
// partial row), then the received rows [2][C][n+2], the two mbarriers they complete and the gradient entries [n+2] of the
// stopping rule
__host__ __device__ constexpr int cluster_fit_smem(int n, int nw, int depth, int stage_stride, int C) {
    return kHeaderBytes + nw * depth * stage_stride + fit_tail_bytes(n) + 2 * C * (n + 2) * 8 + 16 + (n + 2) * 8;
}

// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, int rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// asynchronous store of two doubles to shared memory anywhere in the cluster; the 16 bytes count on the mbarrier (which
// sits in the destination CTA) once they are written
__device__ __forceinline__ void st_async_f64x2(uint32_t cluster_addr, double a, double b, uint32_t cluster_mbar) {
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v2.f64 [%0], {%1, %2}, [%3];"
                 ::"r"(cluster_addr), "d"(a), "d"(b), "r"(cluster_mbar) : "memory");
}

template <class E, int NV, int LPR, int RB, int NW>
__global__ void __launch_bounds__(NW * 32, 1) k_fit_cluster(const __grid_constant__ ClusterFitParams p) {
    namespace cg = cooperative_groups;
    constexpr int EPG = E::EPG;
    constexpr int RPW = 32 / LPR;
    constexpr int RPB = RB * RPW;
    constexpr int LOG_LPR = Log2<LPR>::value;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = LOG_LPR - LOG_RB;
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(SHIFT >= 0 && E::EPG > 1, "shapes of the narrow-row kernel with 16-byte groups");
    static_assert(NW <= kFitMaxWarps && kRedSlices % NW == 0 && kClusterMaxCtas <= kRedSlices, "tail layout and reduction");

    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks()), cta = static_cast<int>(cluster.block_rank());

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                       // [NW][kMaxDepth]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    unsigned char* data = smem + kHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth;
    const int n = p.n, n4 = n / EPG, stride = n + 2, npairs = stride / 2;
    const uint32_t row_bytes = static_cast<uint32_t>(n) * E::BYTES;
    const uint32_t stage_stride = (static_cast<uint32_t>(RPB) * row_bytes + 127u) & ~127u;
    unsigned char* my_stages = data + static_cast<size_t>(warp) * D * stage_stride;
    unsigned char* tail = data + static_cast<size_t>(NW) * D * stage_stride;
    double* red = reinterpret_cast<double*>(tail);                     // [NW][kFitCombineCols]
    double* red_e = red + NW * kFitCombineCols;
    double* red_l = red_e + NW;
    float* w_s = reinterpret_cast<float*>(tail + kFitRedBytes);        // w[0..n), then b
    double* my_row = reinterpret_cast<double*>(tail + kFitRedBytes + fit_param_bytes(n));   // [n+2]: this CTA's partial row
    double* slots = reinterpret_cast<double*>(tail + fit_tail_bytes(n));                     // [2][C][n+2]: everybody's rows
    uint64_t* xbar = reinterpret_cast<uint64_t*>(slots + 2 * static_cast<size_t>(C) * stride);   // [2]
    double* grad_s = reinterpret_cast<double*>(xbar + 2);                                         // [n+2], tolerance mode only
    uint64_t* my_bars = bars + warp * kMaxDepth;

    const long long B = p.num_batches;
    const long long Bw = B > warp ? (B - warp + NW - 1) / NW : 0;
    const int cnt = Bw > cta ? static_cast<int>((Bw - cta + C - 1) / C) : 0;    // batches of this warp (<= D: the host checked)

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(&xbar[0], 1);
        mbar_init(&xbar[1], 1);
    }
    if (lane == 0)
        for (int d = 0; d < D; ++d) mbar_init(&my_bars[d], 1);
    fence_mbar_init();
    for (int c = threadIdx.x; c <= n; c += NW * 32) w_s[c] = c < n ? __ldcg(p.w + c) : __ldcg(p.b);
    __syncthreads();

    // batch i of this warp lives in stage i for the whole fit
    const long long stride_rows = static_cast<long long>(C) * NW * RPB;
    const long long first_row = (static_cast<long long>(cta) * NW + warp) * RPB;
    if (lane == 0) {
        const uint64_t pol = l2_policy_evict_first();
        for (int i = 0; i < cnt; ++i) {
            const long long r0 = first_row + i * stride_rows, left = p.m - r0;
            const uint32_t rows = left < RPB ? static_cast<uint32_t>(left) : RPB;
            mbar_arrive_expect_tx(&my_bars[i], rows * row_bytes);
            bulk_copy_g2s(my_stages + static_cast<size_t>(i) * stage_stride,
                          static_cast<const unsigned char*>(p.X) + static_cast<size_t>(r0) * row_bytes, rows * row_bytes, &my_bars[i], pol);
        }
    }
    const int sub = lane & (LPR - 1), slot = lane >> LOG_LPR;
    const int myr = ((sub >> SHIFT) & (RB - 1)) * RPW + slot;
    const bool owner = (sub & ((1 << SHIFT) - 1)) == 0;
    const bool full_cols = n4 == NV * LPR;
    float yreg[kMaxDepth];                         // y of this lane's row in each of the warp's batches: the same in every iteration
#pragma unroll
    for (int i = 0; i < kMaxDepth; ++i) {
        const long long r = first_row + i * stride_rows + myr;
        yreg[i] = (i < cnt && r < p.m) ? __ldg(p.y + r) : 0.f;
    }
    // where the pushes of this warp go: the slot of this CTA and the mbarrier in the CTAs warp, warp + NW, ...
    constexpr int DPW = (kClusterMaxCtas + NW - 1) / NW;
    uint32_t push_slot[DPW], push_bar[DPW];
#pragma unroll
    for (int j = 0; j < DPW; ++j) {
        const int r = warp + j * NW < C ? warp + j * NW : 0;
        push_slot[j] = map_to_cta(smem_u32(slots) + static_cast<uint32_t>(cta) * stride * 8u, r);
        push_bar[j] = map_to_cta(smem_u32(xbar), r);
    }

    cluster.sync();                                // everybody's mbarriers exist before anybody sends

    bool alive = true;                             // CTA-uniform
    bool staged = false;                           // this warp's stages have landed (they are waited for in the first iteration)
    for (int t = 0; t < p.iters && alive; ++t) {
        const int set = t & 1;
        if (threadIdx.x == 0) mbar_arrive_expect_tx(&xbar[set], static_cast<uint32_t>(C) * stride * 8u);

        typename E::template Lane<NV> lm;          // this lane's slice of the current w and its fp32 accumulators
        lm.template load_w<WSource::Shared>(w_s, sub, LPR, n4);
        lm.zero();
        const float bval = w_s[n];
        double dacc[NV][EPG];
        float se = 0.f, sl = 0.f;
        double dse = 0.0, dsl = 0.0;
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int c = 0; c < EPG; ++c) dacc[k][c] = 0.0;
        int since_flush = 0;
        long long row0 = first_row;
        bool ok = true;                            // warp-uniform until the exchange wait below

        for (int i = 0; i < cnt; ++i) {
            if (!staged) {
                ok = __all_sync(FULL, mbar_wait_bounded(&my_bars[i], 0u, abort_flag));
                if (!ok) break;                    // the CTA's abort flag is up; handled at the end of the iteration
            }
            const long long left = p.m - row0;
            const int rows = left < RPB ? static_cast<int>(left) : RPB;
            const uint4* t4 = reinterpret_cast<const uint4*>(my_stages + static_cast<size_t>(i) * stage_stride);
            uint4 x[RB][NV];
            load_row_batch<uint4, NV, LPR, RB>(x, t4, rows, n4, full_cols && rows == RPB, sub, slot);
            const bool myvalid = myr < rows;
            float yv = yreg[0];
#pragma unroll
            for (int j = 1; j < kMaxDepth; ++j) yv = i == j ? yreg[j] : yv;
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
        staged = ok;
        fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);

        // ---- fixed-order combine of the CTA's warps (as k_fit_rows and k_stream_rows do) into my_row ----
#pragma unroll
        for (int msk = 16; msk >= 1; msk >>= 1) {
            dse += __shfl_xor_sync(FULL, dse, msk);
            dsl += __shfl_xor_sync(FULL, dsl, msk);
        }
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }
        // Several row slots per warp and all of them fit the combine buffer at once (narrow fp32 rows): every lane stores its
        // sums and the combining thread adds a warp's slots in slot order itself -- the additions of slot_order_sum without
        // its shuffles (32 per warp, on a unit that issues one per clock for the whole SM).
        constexpr int NC = NV * LPR * EPG;         // columns a warp's lanes cover
        constexpr bool kSlotsInSmem = RPW > 1 && RPW * NC <= kFitCombineCols;
        if constexpr (kSlotsInSmem) {
#pragma unroll
            for (int k2 = 0; k2 < NV; ++k2)
#pragma unroll
                for (int c = 0; c < EPG; c += 2)
                    *reinterpret_cast<double2*>(red + (warp * RPW + slot) * NC + (sub + k2 * LPR) * EPG + c) = make_double2(dacc[k2][c], dacc[k2][c + 1]);
            __syncthreads();
            if (threadIdx.x < n) {
                double a[NW];                      // per warp: its slots in slot order from +0.0; then warp_tree_sum's tree
#pragma unroll
                for (int wi = 0; wi < NW; ++wi) {
                    double ws = 0.0;
#pragma unroll
                    for (int sidx = 0; sidx < RPW; ++sidx) ws += red[(wi * RPW + sidx) * NC + threadIdx.x];
                    a[wi] = ws;
                }
#pragma unroll
                for (int h = NW / 2; h >= 1; h >>= 1)
#pragma unroll
                    for (int i = 0; i < h; ++i) a[i] += a[i + h];
                my_row[threadIdx.x] = a[0] + 0.0;
            } else if (threadIdx.x >= NW * 32 - 2) {
                const int which = threadIdx.x - (NW * 32 - 2);
                my_row[n + which] = warp_tree_sum<NW>(which == 0 ? red_e : red_l, 1);
            }
            __syncthreads();
        } else {
#pragma unroll
            for (int k2 = 0; k2 < NV; ++k2)
#pragma unroll
                for (int c = 0; c < EPG; ++c) dacc[k2][c] = slot_order_sum<LPR>(dacc[k2][c], sub);
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
                    my_row[c0 + threadIdx.x] = warp_tree_sum<NW>(red + threadIdx.x, kFitCombineCols);
                } else if (c0 + kFitCombineCols >= n && threadIdx.x >= NW * 32 - 2) {   // with the last chunk: the two scalar sums
                    const int which = threadIdx.x - (NW * 32 - 2);
                    my_row[n + which] = warp_tree_sum<NW>(which == 0 ? red_e : red_l, 1);
                }
                __syncthreads();
            }
        }

        // ---- this CTA's row into slot [set][cta] of every CTA (its own included), 16 bytes per store ----
        if (*abort_flag == 0) {                    // CTA-uniform here: a CTA that gave up on its stages sends nothing more
            const uint32_t set_off = static_cast<uint32_t>(set) * C * stride * 8u;
#pragma unroll
            for (int j = 0; j < DPW; ++j) {
                if (warp + j * NW < C) {           // warp-uniform
                    for (int q = lane; q < npairs; q += 32) {
                        const double2 v = reinterpret_cast<const double2*>(my_row)[q];
                        st_async_f64x2(push_slot[j] + set_off + static_cast<uint32_t>(q) * 16u, v.x, v.y, push_bar[j] + set * 8u);
                    }
                }
            }
            // only the threads that read the rows wait for them; the others go on to the barrier below
            if (threadIdx.x < stride) ok = mbar_wait_bounded(&xbar[set], static_cast<uint32_t>(t >> 1) & 1u, abort_flag);
        } else {
            ok = false;
        }

        // ---- every CTA for itself: k_reduce_update's order over the C rows, then its update of its own copy of the
        // parameters; CTA 0 keeps the history ----
        if (ok) {
            const double* rows_in = slots + static_cast<size_t>(set) * C * stride;
            for (int c = threadIdx.x; c < stride; c += NW * 32) {
                const double v = single_row_slices_sum<NW>(C, [&](int g) { return rows_in[static_cast<size_t>(g) * stride + c]; }) * p.inv_m;
                if (c <= n) {
                    w_s[c] = static_cast<float>(static_cast<double>(w_s[c]) - p.lr * v);
                    if (p.tol != nullptr) grad_s[c] = v;               // gradient entry, for the norm below
                } else if (cta == 0 && p.loss_hist) {
                    p.loss_hist[t] = static_cast<float>(v);
                }
            }
        }
        alive = __syncthreads_and(ok) != 0;

        // ---- stopping rule (Algorithm 7): ||(grad_w, grad_b)||_2 of the update just applied, formed by every warp in the
        // order of k_fit_rows and k_reduce_update (lane-strided squares, xor tree): the same bits in every CTA ----
        if (p.tol != nullptr && alive) {
            double q = 0.0;
            for (int c = lane; c <= n; c += 32) {
                const double v = grad_s[c];
                q += v * v;
            }
#pragma unroll
            for (int msk = 16; msk >= 1; msk >>= 1) q += __shfl_xor_sync(FULL, q, msk);
            const double nrm = sqrt(q);
            if (cta == 0 && threadIdx.x == 0) {
                p.tol->grad_norm = nrm;
                p.tol->iters_done = t + 1;
                if (p.gnorm_hist) p.gnorm_hist[t] = static_cast<float>(nrm);
                if (nrm <= p.eps) p.tol->stop = 1;
            }
            if (nrm <= p.eps) break;               // uniform over the whole cluster
        }
    }

    if (!alive && threadIdx.x == 0) {
        atomicExch(p.status, kStatusTimeout);
        atomicExch(p.abort_word, 1u);
    }
    // nobody may leave while another CTA could still send to it; the outcome of every CTA is looked at together
    int* flag_s = reinterpret_cast<int*>(red);
    if (threadIdx.x == 0) *flag_s = alive ? 0 : 1;
    cluster.sync();
    bool all_ok = true;
    for (int r = 0; r < C; ++r) all_ok = all_ok && *cluster.map_shared_rank(flag_s, r) == 0;
    cluster.sync();
    if (!staged && lane == 0)                      // copies that had not landed in time must not land in freed shared memory
        for (int i = 0; i < cnt; ++i) mbar_wait_drain(&my_bars[i], 0u);
    if (all_ok && cta == 0) {                      // (otherwise the parameters are left as they were at launch)
        for (int c = threadIdx.x; c <= n; c += NW * 32) {
            if (c < n) p.w[c] = w_s[c];
            else p.b[0] = w_s[n];
        }
    }
}

}  // namespace lrgd
