// Fused single-pass streaming kernel for rows of up to 128 16-byte groups (512 fp32 or 512 bfloat16 columns; the
// row length a whole number of groups, X 16-byte aligned).  E is the storage type of X (ElemF32 / ElemBF16).
//
// Every warp runs its own small asynchronous pipeline: it owns `depth` shared-memory stages, each the
// size of one batch of rows, and its elected lane keeps them filled with 1-D bulk asynchronous copies
// (contiguous row ranges of X) that complete on the warp's own mbarriers.  The few y values of a batch are
// read with a plain load issued one batch ahead (a second, tiny bulk copy per batch measurably slows the stream).
// Stages are never shared between warps, so a barrier only ever sees consecutive fills from one
// waiter and its one-bit phase parity is unambiguous; there is no producer warp and no release barrier.
// Per batch the warp
//   1. waits for the stage, moves the batch into registers with one conflict-free 128-bit shared load
//      per element group, and immediately re-arms the stage with the copy for a later batch;
//   2. z = x.w + b: lane-local FMAs, then a transposing shuffle reduction that leaves each row's sum on
//      a distinct lane group                                          (model equation, Section II-A)
//   3. p, err, loss term, one row per lane                            (Eq. 1; Algorithm 7; log-likelihood)
//   4. X^T err: acc[c] += x[r][c] * err[r] on the same registers       (Algorithm 1's err.X)
// so X is read from HBM once and from shared memory once per pass.  Per-lane fp32 accumulators are
// folded into fp64 every kFlushBatches batches; at the end the CTA combines its warps in a fixed order
// and writes one row of partial sums [n columns | sum err | sum loss] in fp64.
//
// Batch g (rows [g*RPB, (g+1)*RPB)) belongs to warp g % NW of CTA (g / NW) % grid: a static map, so
// results are bit-reproducible.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kMaxDepth = 4;
constexpr int kHeaderBytes = 1024;     // per-warp mbarriers [NW][kMaxDepth], abort flag
constexpr int kFlushBatches = 4;

struct StreamParams {
    const void* X;            // fp32 or bfloat16 [m][n], row-major
    const float* y;
    long long m;
    int n;
    const float* w;
    const float* b;
    double* partial;          // [grid][n+2]           (loss/grad mode)
    unsigned char* labels;    // [m]                   (predict mode)
    float cut;                // predict: logit(thr)
    int* status;              // device status word
    const int* stop;          // nullable: non-zero means a stopping rule has been met and the launch is a no-op
    int depth;                // stages per warp (1..kMaxDepth)
    long long num_batches;    // ceil(m / rows per batch)
    long long keep_rows;      // rows [0, keep_rows) are fetched with an L2 evict-last hint (kept across passes), the rest evict-first
};

// Sums C values per lane across the lanes selected by masks M, M/2, ..., 1.  While more than one value
// is left, each step halves the values a lane carries (lanes with the mask bit set keep the upper half),
// so the whole reduction costs C-1 + (remaining levels) shuffles instead of C*log2(lanes).
template <int C, int M, int RB>
__device__ __forceinline__ void lane_reduce(float (&v)[RB], int lane) {
    if constexpr (M >= 1) {
        if constexpr (C > 1) {
            constexpr int H = C / 2;
            const bool upper = (lane & M) != 0;
#pragma unroll
            for (int j = 0; j < H; ++j) {
                const float send = upper ? v[j] : v[j + H];
                const float keep = upper ? v[j + H] : v[j];
                v[j] = keep + __shfl_xor_sync(0xffffffffu, send, M);
            }
            lane_reduce<H, M / 2, RB>(v, lane);
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], M);
            lane_reduce<1, M / 2, RB>(v, lane);
        }
    }
}

// ---- pieces of the per-batch work shared by the narrow-row, wide-row and persistent kernels ----
// A batch lives in registers as x[RB][NV]: RB row slots by NV 16-byte column groups per lane (raw bits; widened to
// fp32 where they are used); LPR lanes share a row.  EPG = elements per group of the storage type E.

// z partials: lane-local FMAs, then the transposing reduction; the returned value is the full dot product of the row
// (r, with r = (lane_in_group >> (log2 LPR - log2 RB)) & (RB-1)) that ends up on this lane.
template <class E, int NV, int LPR, int RB>
__device__ __forceinline__ float batch_dot(const typename E::Raw (&x)[RB][NV], const typename E::template Lane<NV>& lm, int lane) {
    float v[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) v[r] = lm.dot(x[r]);
    lane_reduce<RB, LPR / 2, RB>(v, lane);
    return v[0];
}

// acc[c] += x[r][c] * err[r]: each row's err is fetched from the lane that holds it (Algorithm 1's err.X on registers).
template <class E, int NV, int LPR, int RB>
__device__ __forceinline__ void batch_accumulate(const typename E::Raw (&x)[RB][NV], float e, typename E::template Lane<NV>& lm) {
    constexpr int SHIFT = Log2<LPR>::value - Log2<RB>::value;
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        const float er = __shfl_sync(0xffffffffu, e, r << SHIFT, LPR);
        lm.accumulate(x[r], er);
    }
}

// fp32 per-lane sums folded into their fp64 counterparts (keeps the serial fp32 chains short)
template <class E, int NV>
__device__ __forceinline__ void fold_into_fp64(typename E::template Lane<NV>& lm, double (&dacc)[NV][E::EPG], float& se, float& sl,
                                               double& dse, double& dsl) {
    lm.fold(dacc);
    dse += se; dsl += sl; se = 0.f; sl = 0.f;
}

// Sum of a value over the row slots of a warp that own the same columns (lanes sub, sub + LPR, ...), in slot order, starting
// from +0.0; every lane gets it.  With one slot per warp the value itself (it may then be -0.0 where the sum would be +0.0:
// the combine of the CTA's warps starts from +0.0 and wipes that out).
template <int LPR>
__device__ __forceinline__ double slot_order_sum(double v, int sub) {
    constexpr int RPW = 32 / LPR;
    if constexpr (RPW == 1) {
        return v;
    } else {
        double t = 0.0;
#pragma unroll
        for (int sidx = 0; sidx < RPW; ++sidx) t += __shfl_sync(0xffffffffu, v, sub + sidx * LPR);
        return t;
    }
}

// Sum of the per-warp values src[0], src[step], ..., src[(NW-1) step] in a fixed pairwise tree (warp w with w + NW/2, then
// distance NW/4, ... 1), plus +0.0 so that the result is never -0.0.  The order every narrow-row kernel uses for the combine
// of a CTA's warps: log2(NW) dependent fp64 additions instead of NW in a row (which is what a thread waits for).
template <int NW>
__device__ __forceinline__ double warp_tree_sum(const double* src, size_t step) {
    static_assert((NW & (NW - 1)) == 0, "a power of two of warps");
    double a[NW];
#pragma unroll
    for (int i = 0; i < NW; ++i) a[i] = src[i * step];
#pragma unroll
    for (int h = NW / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int i = 0; i < h; ++i) a[i] += a[i + h];
    return a[0] + 0.0;
}

// one batch from a narrow-row stage into registers (rows packed at n4 groups; lanes beyond the row or rows beyond the
// matrix read zeros); `full` = every lane's groups exist and the batch is complete: no bounds logic
template <class Raw, int NV, int LPR, int RB>
__device__ __forceinline__ void load_row_batch(Raw (&x)[RB][NV], const Raw* t4, int rows, int n4, bool full, int sub,
                                               int slot) {
    constexpr int RPW = 32 / LPR;
    if (full) {
#pragma unroll
        for (int r8 = 0; r8 < RB; ++r8)
#pragma unroll
            for (int k2 = 0; k2 < NV; ++k2) x[r8][k2] = t4[(r8 * RPW + slot) * (NV * LPR) + sub + k2 * LPR];
    } else {
#pragma unroll
        for (int r8 = 0; r8 < RB; ++r8) {
            const int r = r8 * RPW + slot;
#pragma unroll
            for (int k2 = 0; k2 < NV; ++k2) {
                const int idx = sub + k2 * LPR;
                x[r8][k2] = (r < rows && idx < n4) ? t4[r * n4 + idx] : Raw{};
            }
        }
    }
}

template <class E, int NV, int LPR, int RB, int NW, bool PREDICT>
__global__ void __launch_bounds__(NW * 32, 1) k_stream_rows(const StreamParams p) {
    constexpr int EPG = E::EPG;
    constexpr int RPW = 32 / LPR;                  // rows a warp touches with one load instruction
    constexpr int RPB = RB * RPW;                  // rows per batch
    constexpr int LOG_LPR = Log2<LPR>::value;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = LOG_LPR - LOG_RB;        // duplicate lanes per row after the reduction = 2^SHIFT
    static_assert(SHIFT >= 0, "rows per batch slot must not exceed lanes per row");
    static_assert(NW * kMaxDepth * 8 + 16 <= kHeaderBytes, "header too small");
    constexpr unsigned FULL = 0xffffffffu;

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                       // [NW][kMaxDepth]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    unsigned char* data = smem + kHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth;
    const int n = p.n, n4 = n / EPG;                   // n4 = 16-byte groups per row
    const uint32_t row_bytes = static_cast<uint32_t>(n) * E::BYTES;
    // rows of any length: a batch need not start on a 16-byte boundary; its copy then starts up to 12 bytes early
    constexpr uint32_t kSlack = E::EPG == 1 ? 16u : 0u;
    const uint32_t stage_stride = (static_cast<uint32_t>(RPB) * row_bytes + kSlack + 127u) & ~127u;
    unsigned char* my_stages = data + static_cast<size_t>(warp) * D * stage_stride;
    uint64_t* my_bars = bars + warp * kMaxDepth;

    // batches of this warp: g_i = (i*grid + cta)*NW + warp < num_batches, i in [0, cnt)
    const long long B = p.num_batches;
    const long long Bw = B > warp ? (B - warp + NW - 1) / NW : 0;     // CTA-level slots that contain a batch for this warp
    const int cnt = Bw > blockIdx.x ? static_cast<int>((Bw - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) mbar_init(&my_bars[d], 1);
        fence_mbar_init();
    }
    __syncthreads();

    const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
    const long long stride_rows = static_cast<long long>(gridDim.x) * NW * RPB;       // rows between this warp's batches
    long long row0 = (static_cast<long long>(blockIdx.x) * NW + warp) * RPB;          // first row of the current batch
    // (re)fills stage d with the batch that starts at row r0; called by lane 0 only
    auto issue = [&](long long r0, int d) {
        const long long left = p.m - r0;
        const uint32_t rows = left < RPB ? static_cast<uint32_t>(left) : RPB;
        const uint32_t xbytes = rows * row_bytes;
        unsigned char* dst = my_stages + static_cast<size_t>(d) * stage_stride;
        const unsigned char* src = static_cast<const unsigned char*>(p.X) + static_cast<size_t>(r0) * row_bytes;
        if constexpr (E::EPG == 1) {
            // rows of any length, X aligned to its element size: neither the start nor the size of a batch need be a multiple of 16
            // bytes.  The batch lands at dst + off, off = its address mod 16.  The bulk copy covers the 16-byte-aligned span
            // that starts at or up to 12 bytes before the batch (bytes of the row before it) and ends at or before its last
            // byte; for the very first batch of a matrix that is itself not 16-byte aligned it starts at the first boundary
            // inside the batch instead.  The few elements left over at either end are moved by this lane with plain loads
            // and stores.  Nothing outside [X, X + m*n) is read.
            const uint32_t off = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src)) & 15u;
            const uint32_t span = off + xbytes;                                   // stage bytes [off, span) hold the batch
            const uint32_t lo = (r0 == 0 && off != 0u) ? 16u : 0u;                // first stage byte the bulk copy writes
            const uint32_t bulk = span > lo ? (span - lo) & ~15u : 0u;
            if (bulk != 0u) {
                mbar_arrive_expect_tx(&my_bars[d], bulk);
                bulk_copy_g2s(dst + lo, src - off + lo, bulk, &my_bars[d], r0 < p.keep_rows ? pol_keep : pol_stream);
            } else {
                mbar_arrive(&my_bars[d]);
            }
            using Raw = typename E::Raw;                                          // one element
            for (uint32_t o = off; o < lo && o < span; o += E::BYTES)             // head (first batch of an unaligned matrix only)
                *reinterpret_cast<Raw*>(dst + o) = *reinterpret_cast<const Raw*>(src - off + o);
            for (uint32_t o = lo + bulk; o < span; o += E::BYTES)                 // tail
                *reinterpret_cast<Raw*>(dst + o) = *reinterpret_cast<const Raw*>(src - off + o);
        } else {
            mbar_arrive_expect_tx(&my_bars[d], xbytes);
            bulk_copy_g2s(dst, src, xbytes, &my_bars[d], r0 < p.keep_rows ? pol_keep : pol_stream);
        }
    };

    typename E::template Lane<NV> lm;              // this lane's slice of w and its fp32 accumulators
    double dacc[NV][EPG];
    float se = 0.f, sl = 0.f;
    double dse = 0.0, dsl = 0.0;
    lm.zero();
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
        for (int c = 0; c < EPG; ++c) dacc[k][c] = 0.0;
    const int sub = lane & (LPR - 1), slot = lane >> LOG_LPR;
    const int myr = ((sub >> SHIFT) & (RB - 1)) * RPW + slot;     // the row of a batch whose logit ends up on this lane
    const bool owner = (sub & ((1 << SHIFT) - 1)) == 0;           // one lane per row does the bookkeeping

    if (lane == 0) {
        const int pre = cnt < D ? cnt : D;
        for (int d = 0; d < pre; ++d) issue(row0 + d * stride_rows, d);
    }
    __syncwarp();                                  // orders the plain stores a ragged tail may have needed before the warp's reads
    float y_next = 0.f;                            // y of this lane's row in the next batch, loaded one batch ahead
    if constexpr (!PREDICT) {
        if (cnt > 0 && row0 + myr < p.m) y_next = __ldg(p.y + row0 + myr);
    }
    // X and y are inputs that no kernel of this library writes, so the first stages are already on their way; the
    // parameters (and the stop flag) come from the kernel before this one: wait for it only now.
    grid_dependency_release();
    grid_dependency_wait();
    if (p.stop != nullptr && *reinterpret_cast<const volatile int*>(p.stop) != 0) {
        // a stopping rule was met by an earlier iteration: let the copies just issued land, then leave
        if (lane == 0) {
            const int pre = cnt < D ? cnt : D;
            for (int d = 0; d < pre; ++d) mbar_wait_drain(&my_bars[d], 0u);
        }
        __syncwarp();
        return;
    }
    lm.template load_w<WSource::GlobalL2>(p.w, sub, LPR, n4);   // through L2: the kernel before this one may just have written them
    const float bval = __ldcg(p.b);
    const bool full_cols = n4 == NV * LPR;         // every lane's column groups exist
    const bool labels_word_aligned = PREDICT && (reinterpret_cast<uintptr_t>(p.labels) & 3u) == 0 && RPB % 4 == 0;
    int issued = cnt < D ? cnt : D;                // warp-uniform count of batches whose copies were issued
    int done = 0;                                  // batches whose stage wait has succeeded
    int since_flush = 0;
    int d = 0;
    uint32_t phase = 0;

    for (int i = 0; i < cnt; ++i) {
        bool ok = mbar_wait_bounded(&my_bars[d], phase, abort_flag);
        ok = __all_sync(FULL, ok);
        if (!ok) break;
        done = i + 1;
        if constexpr (E::EPG == 1) __syncwarp();   // lane 0 may have completed this stage with plain stores

        const long long left = p.m - row0;
        const int rows = left < RPB ? static_cast<int>(left) : RPB;
        using Raw = typename E::Raw;
        // (rows of any length: the batch sits at its address mod 16 within the stage)
        const uint32_t off = E::EPG == 1 ? static_cast<uint32_t>((reinterpret_cast<uintptr_t>(p.X) + row0 * row_bytes) & 15u) : 0u;
        const Raw* t4 = reinterpret_cast<const Raw*>(my_stages + static_cast<size_t>(d) * stage_stride + off);
        Raw x[RB][NV];
        load_row_batch<Raw, NV, LPR, RB>(x, t4, rows, n4, full_cols && rows == RPB, sub, slot);
        const bool myvalid = myr < rows;
        const float yv = y_next;
        if constexpr (!PREDICT) {
            const long long rn = row0 + stride_rows + myr;
            y_next = (i + 1 < cnt && rn < p.m) ? __ldg(p.y + rn) : 0.f;
        }
        // the batch now lives in registers: re-arm this stage with the batch `depth` steps ahead
        __syncwarp();
        if (i + D < cnt) {
            if (lane == 0) {
                fence_proxy_async_smem();
                issue(row0 + D * stride_rows, d);
            }
            issued = i + D + 1;
        }
        if (++d == D) { d = 0; phase ^= 1u; }

        const float z = batch_dot<E, NV, LPR, RB>(x, lm, lane) + bval;

        if constexpr (PREDICT) {
            // one bit per lane, then RPB/4 lanes each assemble and store four labels as one 32-bit word
            const unsigned hit = __ballot_sync(FULL, owner && myvalid && z >= p.cut);
            if (rows == RPB && labels_word_aligned) {
                if (lane < RPB / 4) {
                    unsigned word = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int r = 4 * lane + q;                                   // row of the batch
                        const int src = (r % RPW) * LPR + ((r / RPW) << SHIFT);       // the owner lane of that row
                        word |= ((hit >> src) & 1u) << (8 * q);
                    }
                    *reinterpret_cast<unsigned*>(p.labels + row0 + 4 * lane) = word;
                }
            } else if (owner && myvalid) {
                p.labels[row0 + myr] = z >= p.cut ? 1 : 0;
            }
        } else {
            float e, L;
            logistic_terms(z, yv, e, L);
            if (!myvalid) { e = 0.f; L = 0.f; }
            if (owner) { se += e; sl += L; }
            batch_accumulate<E, NV, LPR, RB>(x, e, lm);
            if (++since_flush == kFlushBatches) {
                since_flush = 0;
                fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
            }
        }
        row0 += stride_rows;
    }

    if (done < cnt) {
        // a bounded wait expired: report it, then let this warp's copies still in flight land (bounded again)
        // before the CTA retires and its shared memory is handed to another CTA
        if (lane == 0) {
            atomicExch(p.status, kStatusTimeout);
            for (int i = done; i < issued; ++i) mbar_wait_drain(&my_bars[i % D], static_cast<uint32_t>(i / D) & 1u);
        }
        __syncwarp();
    }
    if constexpr (!PREDICT) {
        fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);

        // ---------------- fixed-order combine of the CTA's warps ----------------
        __syncthreads();                               // all stages are idle: reuse them as the combine buffer
        double* red = reinterpret_cast<double*>(data); // [NW][n] column sums, then [NW] sum err, [NW] sum loss
        double* red_e = red + static_cast<size_t>(NW) * n;
        double* red_l = red_e + NW;
        // row slots of one warp that own the same columns: add in slot order
#pragma unroll
        for (int k2 = 0; k2 < NV; ++k2) {
#pragma unroll
            for (int c = 0; c < EPG; ++c) {
                const double t = slot_order_sum<LPR>(dacc[k2][c], sub);
                const int idx = sub + k2 * LPR;
                if (slot == 0 && idx < n4) red[static_cast<size_t>(warp) * n + idx * EPG + c] = t;
            }
        }
#pragma unroll
        for (int msk = 16; msk >= 1; msk >>= 1) {
            dse += __shfl_xor_sync(FULL, dse, msk);
            dsl += __shfl_xor_sync(FULL, dsl, msk);
        }
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }
        __syncthreads();
        double* out = p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
        for (int c = threadIdx.x; c < n + 2; c += blockDim.x) {
            out[c] = c < n ? warp_tree_sum<NW>(red + c, static_cast<size_t>(n)) : warp_tree_sum<NW>(c == n ? red_e : red_l, 1);
        }
    }
}

}  // namespace lrgd
