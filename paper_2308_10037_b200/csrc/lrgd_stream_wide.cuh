// Fused single-pass streaming kernel for wide rows of ANY length in a matrix aligned only to its element size
// (fp32: 513 <= n <= 8192 with n % 4 != 0 or X not 16-byte aligned; bfloat16 likewise with n % 8 / 2-byte alignment),
// and for every row of 8193..16384 elements (one row per batch).
// E is ElemF32Any or ElemBF16Any: the unit a lane owns is a single element.
//
// Such rows cannot be cut into aligned 16-byte groups, so neither a tensor map nor per-warp boxes can describe a
// warp's slice of them.  What stays true is that RB consecutive rows of a row-major matrix are ONE contiguous byte range.
// So the stages here belong to the whole CTA: a stage holds a batch of RB full rows, fetched by one thread with one 1-D
// bulk copy of the 16-byte-aligned span around the batch (the few bytes the span misses at either end are moved with
// plain loads, as in the narrow-row kernel for rows of any length; nothing outside X is read), and the NW warps of
// the CTA split every row by columns: warp w owns elements [w*CW, (w+1)*CW), lane l of it the elements l, l+32, ...
// Per batch every warp waits for the stage, moves its slice of the RB rows into registers (32-bit shared loads,
// consecutive lanes read consecutive words), forms its partial dot products, and the partials meet in a double-buffered
// shared array behind one __syncthreads -- the same exchange as in k_stream_split, so z = x.w + b has the same bits in
// every warp (model equation, Section II-A).  After that barrier every warp has its slice in registers, so the stage is
// re-armed for the batch `depth` steps ahead.  err, the loss term (warp 0) and acc[c] += x[r][c] * err[r] follow on the
// registers (Eq. 1; Algorithm 7; Algorithm 1's err.X).  Each column belongs to one lane of one warp: the CTA's partial
// row needs no cross-warp combine.  Batch g belongs to CTA g mod grid: a static map, bit-reproducible results.
//
// All warps wait on the same mbarrier of a stage.  They take every batch and meet at the per-batch barrier, so no warp
// is ever more than one batch ahead of another and the one-bit phase parity stays unambiguous for depth >= 2; with a
// single stage the re-arm follows the barrier after which nobody waits on the old phase any more.
#pragma once
#include "lrgd_common.cuh"
#include "lrgd_stream_rows.cuh"
#include "lrgd_stream_split.cuh"

namespace lrgd {

struct WideParams {
    const void* X;            // fp32 or bfloat16 [m][n], row-major, aligned to its element size
    const float* y;
    long long m;
    int n;
    const float* w;
    const float* b;
    double* partial;          // [grid][n+2]
    unsigned char* labels;    // predict mode
    float cut;
    int* status;
    const int* stop;          // nullable: non-zero makes the launch a no-op
    int depth;                // stages per CTA (1..kMaxDepth)
    int cw;                   // elements per warp slice
    long long num_batches;    // ceil(m / RB)
    long long keep_rows;      // rows [0, keep_rows) are fetched with an L2 evict-last hint, the rest evict-first
};

template <class E, int NV, int RB, int NW, bool PREDICT>
__global__ void __launch_bounds__(NW * 32, 1) k_stream_wide(const WideParams p) {
    static_assert(E::EPG == 1, "element-wise storage types only");
    using Raw = typename E::Raw;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = 5 - LOG_RB;              // log2 of the lanes holding the same row after the reduction
    constexpr int DUP = 1 << SHIFT;
    constexpr int PER_DUP = NW >= DUP ? NW / DUP : 1;   // partial logits each of those lanes adds up (with one row per batch
                                                        // there are more such lanes than warps: the first NW take one each)
    constexpr unsigned FULL = 0xffffffffu;
    // Slices of more than 16 elements per lane (rows beyond 8192 elements, one row per batch) leave no registers for fp64
    // copies of the accumulators: the fp32 sums are then added straight into the CTA's own fp64 partial row in global memory
    // (each column belongs to one lane, so the read-modify-write needs no ordering), once per 64 rows.
    constexpr bool FLUSH_GLOBAL = NV > 16;
    static_assert(NW % DUP == 0 || DUP % NW == 0, "warps must split evenly over the duplicate lanes");
    static_assert(kMaxDepth * 8 + 16 <= kSplitZOffset, "header too small");
    static_assert(kSplitZOffset + 2 * NW * RB * 4 <= kSplitHeaderBytes, "header too small");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                       // [kMaxDepth], one per CTA-wide stage
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + kMaxDepth);
    float* zpart = reinterpret_cast<float*>(smem + kSplitZOffset);            // [2][NW][RB]
    unsigned char* stages = smem + kSplitHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth, CW = p.cw;
    const int n = p.n;
    const int c0 = warp * CW;                                                 // first element of this warp's slice
    const int mycw = n - c0 < CW ? (n - c0 > 0 ? n - c0 : 0) : CW;            // elements of the slice inside the row
    const uint32_t row_bytes = static_cast<uint32_t>(n) * E::BYTES;
    const uint32_t stage_stride = (static_cast<uint32_t>(RB) * row_bytes + 16u + 127u) & ~127u;   // 16 bytes of slack for the span

    const long long B = p.num_batches;
    const int cnt = B > blockIdx.x ? static_cast<int>((B - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;   // CTA-uniform

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int d = 0; d < D; ++d) mbar_init(&bars[d], 1);
        fence_mbar_init();
    }
    __syncthreads();

    const long long stride_rows = static_cast<long long>(gridDim.x) * RB;     // rows between this CTA's batches
    long long row0 = static_cast<long long>(blockIdx.x) * RB;                 // first row of the current batch
    // (re)fills stage d with the batch that starts at row r0; called by thread 0 only.  The batch lands at its address
    // mod 16 within the stage; the bulk copy covers the aligned span, the elements it misses are moved by plain loads.
    auto issue = [&](long long r0, int d) {
        const long long left = p.m - r0;
        const uint32_t rows = left < RB ? static_cast<uint32_t>(left) : RB;
        const uint32_t xbytes = rows * row_bytes;
        unsigned char* dst = stages + static_cast<size_t>(d) * stage_stride;
        const unsigned char* src = static_cast<const unsigned char*>(p.X) + static_cast<size_t>(r0) * row_bytes;
        const uint32_t off = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src)) & 15u;
        const uint32_t span = off + xbytes;                                   // stage bytes [off, span) hold the batch
        const uint32_t lo = (r0 == 0 && off != 0u) ? 16u : 0u;                // nothing in front of the matrix may be read
        const uint32_t bulk = span > lo ? (span - lo) & ~15u : 0u;
        // the plain stores come first: the arrive below releases them to the warps that acquire the phase
        for (uint32_t o = off; o < lo && o < span; o += E::BYTES)             // head (first batch of an unaligned matrix only)
            *reinterpret_cast<Raw*>(dst + o) = *reinterpret_cast<const Raw*>(src - off + o);
        for (uint32_t o = lo + bulk; o < span; o += E::BYTES)                 // tail
            *reinterpret_cast<Raw*>(dst + o) = *reinterpret_cast<const Raw*>(src - off + o);
        if (bulk != 0u) {
            mbar_arrive_expect_tx(&bars[d], bulk);
            bulk_copy_g2s(dst + lo, src - off + lo, bulk, &bars[d], r0 < p.keep_rows ? l2_policy_evict_last() : l2_policy_evict_first());
        } else {
            mbar_arrive(&bars[d]);
        }
    };

    typename E::template Lane<NV> lm;              // this lane's elements of w (c0 + lane + 32k) and its fp32 accumulators
    double dacc[FLUSH_GLOBAL ? 1 : NV][1];
    float se = 0.f, sl = 0.f;
    double dse = 0.0, dsl = 0.0;
    lm.zero();
#pragma unroll
    for (int k = 0; k < (FLUSH_GLOBAL ? 1 : NV); ++k) dacc[k][0] = 0.0;
    double* const out_row = PREDICT ? nullptr : p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
    // adds this lane's fp32 sums to its columns of the CTA's partial row and clears them
    auto flush_global = [&]() {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int loc = lane + 32 * k;
            if (loc < mycw) out_row[c0 + loc] += static_cast<double>(lm.acc[k]);
            lm.acc[k] = 0.f;
        }
        dse += se; dsl += sl; se = 0.f; sl = 0.f;
    };
    const int myr = (lane >> SHIFT) & (RB - 1);    // the row of a batch whose logit ends up on this lane
    const int dup = lane & (DUP - 1);              // which of the lanes sharing that row this one is
    const bool owner = dup == 0;
    const bool labels_word_aligned = PREDICT && RB % 4 == 0 && (reinterpret_cast<uintptr_t>(p.labels) & 3u) == 0;

    int issued = cnt < D ? cnt : D;                // CTA-uniform: batches whose copies were issued
    if (threadIdx.x == 0)
        for (int d = 0; d < issued; ++d) issue(row0 + d * stride_rows, d);
    int done = 0;
    bool aborted = false;
    int since_flush = 0;
    int d = 0;
    uint32_t phase = 0;
    float y_next = 0.f;
    if constexpr (!PREDICT) {
        if (cnt > 0 && row0 + myr < p.m) y_next = __ldg(p.y + row0 + myr);
    }
    // X and y are inputs that no kernel of this library writes, so the first stages are already on their way; the
    // parameters (and the stop flag) come from the kernel before this one: wait for it only now.
    grid_dependency_release();
    grid_dependency_wait();
    if (p.stop != nullptr && *reinterpret_cast<const volatile int*>(p.stop) != 0) {
        // a stopping rule was met by an earlier iteration: let the copies just issued land, then leave
        if (threadIdx.x == 0)
            for (int d2 = 0; d2 < issued; ++d2) mbar_wait_drain(&bars[d2], 0u);
        __syncthreads();
        return;
    }
    lm.template load_w<WSource::GlobalL2>(p.w, c0 + lane, 32, c0 + mycw);    // through L2: the kernel before this one may just have written them
    const float bval = __ldcg(p.b);
    if constexpr (FLUSH_GLOBAL && !PREDICT) {
        // the row is accumulated into: start it at zero (only this lane ever touches these columns of it)
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int loc = lane + 32 * k;
            if (loc < mycw) out_row[c0 + loc] = 0.0;
        }
    }

    for (int i = 0; i < cnt; ++i) {
        const bool myvalid = row0 + myr < p.m;
        const float yv = y_next;
        if constexpr (!PREDICT) {
            const long long rn = row0 + stride_rows + myr;
            y_next = (i + 1 < cnt && rn < p.m) ? __ldg(p.y + rn) : 0.f;
        }

        Raw x[RB][NV];
        bool have = false;
        if (!aborted) {
            bool ok = mbar_wait_bounded(&bars[d], phase, abort_flag);
            ok = __all_sync(FULL, ok);
            if (!ok) {
                aborted = true;
            } else {
                done = i + 1;
                have = true;
                const long long left = p.m - row0;
                const int rows = left < RB ? static_cast<int>(left) : RB;
                const uint32_t off = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(p.X) + static_cast<size_t>(row0) * row_bytes) & 15u);
                const unsigned char* base = stages + static_cast<size_t>(d) * stage_stride + off;
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const Raw* row = reinterpret_cast<const Raw*>(base + static_cast<size_t>(r) * row_bytes) + c0;
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        const int loc = lane + 32 * k;
                        x[r][k] = (r < rows && loc < mycw) ? row[loc] : Raw{};
                    }
                }
            }
        }
        if (!have) {
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int k = 0; k < NV; ++k) x[r][k] = Raw{};
        }

        const float zpartial = batch_dot<E, NV, 32, RB>(x, lm, lane);
        float* zp = zpart + (i & 1) * (NW * RB);
        if (owner) zp[warp * RB + myr] = zpartial;
        __syncthreads();
        // every warp has moved its slice of stage d into registers: re-arm it with the batch `depth` steps ahead
        if (have) {                                // (CTA-uniform unless a wait expired, and then nothing is issued any more)
            if (i + D < cnt && !*abort_flag) {
                if (threadIdx.x == 0) {
                    fence_proxy_async_smem();
                    issue(row0 + D * stride_rows, d);
                }
                issued = i + D + 1;
            }
            if (++d == D) { d = 0; phase ^= 1u; }
        }
        // the lanes that share a row add PER_DUP partials each (warp order), then a butterfly: one fixed order, same in every warp
        float zs = 0.f;
#pragma unroll
        for (int j = 0; j < PER_DUP; ++j)
            if (NW >= DUP || dup < NW) zs += zp[(dup * PER_DUP + j) * RB + myr];
#pragma unroll
        for (int msk = DUP / 2; msk >= 1; msk >>= 1) zs += __shfl_xor_sync(FULL, zs, msk);
        const float z = zs + bval;

        if constexpr (PREDICT) {
            if (warp == 0) {
                const unsigned hit = __ballot_sync(FULL, owner && myvalid && z >= p.cut);
                if (row0 + RB <= p.m && labels_word_aligned) {
                    if (lane < RB / 4) {
                        unsigned word = 0;
#pragma unroll
                        for (int q = 0; q < 4; ++q) word |= ((hit >> ((4 * lane + q) << SHIFT)) & 1u) << (8 * q);
                        *reinterpret_cast<unsigned*>(p.labels + row0 + 4 * lane) = word;
                    }
                } else if (owner && myvalid) {
                    p.labels[row0 + myr] = z >= p.cut ? 1 : 0;
                }
            }
        } else {
            float e;
            if (warp == 0) {                       // warp-uniform: the loss term is needed once per row
                float L;
                logistic_terms(z, yv, e, L);
                if (owner && myvalid) { se += e; sl += L; }
            } else {
                e = logistic_err(z, yv);
            }
            if (!myvalid) e = 0.f;
            batch_accumulate<E, NV, 32, RB>(x, e, lm);
            if constexpr (FLUSH_GLOBAL) {
                if (++since_flush == 64 / RB) {
                    since_flush = 0;
                    flush_global();
                }
            } else {
                if (++since_flush == 2 * kFlushBatches) {
                    since_flush = 0;
                    fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
                }
            }
        }
        row0 += stride_rows;
    }

    if (*abort_flag) {
        // report, then let the copies still in flight land (bounded again) before the CTA retires
        __syncthreads();
        if (threadIdx.x == 0) {
            atomicExch(p.status, kStatusTimeout);
            for (int i = done; i < issued; ++i) mbar_wait_drain(&bars[i % D], static_cast<uint32_t>(i / D) & 1u);
        }
        __syncthreads();
    }
    if constexpr (!PREDICT) {
        double* out = out_row;
        if constexpr (FLUSH_GLOBAL) {
            flush_global();
        } else {
            fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int loc = lane + 32 * k;
                if (loc < mycw) out[c0 + loc] = dacc[k][0];
            }
        }
        if (warp == 0) {
#pragma unroll
            for (int msk = 16; msk >= 1; msk >>= 1) {
                dse += __shfl_xor_sync(FULL, dse, msk);
                dsl += __shfl_xor_sync(FULL, dsl, msk);
            }
            if (lane == 0) { out[n] = dse; out[n + 1] = dsl; }
        }
    }
}

}  // namespace lrgd
