// Fused single-pass streaming kernel for wide rows (more 16-byte groups per row than the narrow-row kernel takes, up
// to 1024: 512 < n <= 4096 fp32 columns or 512 < n <= 8192 bfloat16 columns; the row a whole number of groups, X
// 16-byte aligned).  E is the storage type of X (ElemF32 / ElemBF16).
//
// A row no longer fits one warp's registers, so the 16 warps of a CTA split every row by columns: warp w owns
// the contiguous slice of CW = ceil(n/4/16) 16-byte column groups starting at w*CW.  The CTA walks batches of RB
// rows (batch g belongs to CTA g mod grid).  As in the narrow-row kernel each warp runs its own asynchronous
// pipeline with `depth` private stages completing on its own mbarriers; a stage is one RB-row by CW-group box of X,
// fetched by the warp's elected lane with ONE tiled TMA copy (cp.async.bulk.tensor.2d through a tensor map of X,
// delivered to this CTA only).  Rows past m and columns past n arrive as zeros, so the loads need no bounds logic.
// Per batch:
//   1. every warp moves its box into registers (conflict-free 128-bit shared loads), re-arms the stage, and forms
//      its partial dot products (lane FMAs + transposing shuffle reduction);
//   2. the partials meet in a double-buffered shared array, one __syncthreads per batch; every warp then adds the 16
//      partials of each row in one fixed order, so all warps hold bit-identical z = x.w + b  (model equation, II-A);
//   3. err is formed by every warp, the loss term only by warp 0                            (Eq. 1, Algorithm 7);
//   4. acc[c] += x[r][c] * err[r] on the registers loaded in step 1                        (Algorithm 1's err.X).
// Each column belongs to exactly one lane of one warp, so the CTA's partial row needs no cross-warp combine.
// A warp whose bounded wait expires raises the CTA's abort flag; it (and then every other warp) keeps taking part in
// the per-batch barrier without touching its stages, so the CTA still retires, with the status word set.
#pragma once
#include <cuda.h>

#include "lrgd_common.cuh"
#include "lrgd_stream_rows.cuh"

namespace lrgd {

constexpr int kSplitHeaderBytes = 4096;   // mbarriers [NW][kMaxDepth], abort flag, partial logits [2][NW][RB] (RB up to 16)
constexpr int kSplitZOffset = 1024;

struct SplitParams {
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
    int depth;                // stages per warp
    int cw;                   // 16-byte column groups per warp slice (the tensor map's box is cw groups by RB rows)
    int x_per_group;          // tensor-map elements per 16-byte group: 4 (32-bit words) or 2 (64-bit words)
    long long num_batches;    // ceil(m / RB)
    long long keep_rows;      // rows [0, keep_rows) are fetched with an L2 evict-last hint, the rest evict-first
};

template <class E, int NV, int RB, int NW, bool PREDICT>
__global__ void __launch_bounds__(NW * 32, 1) k_stream_split(const __grid_constant__ CUtensorMap tmap, const SplitParams p) {
    constexpr int EPG = E::EPG;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = 5 - LOG_RB;              // log2 of the lanes holding the same row after the reduction
    constexpr int DUP = 1 << SHIFT;
    constexpr int PER_DUP = NW / DUP;              // partial logits each of those lanes adds up
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(NW % DUP == 0, "warps must split evenly over the duplicate lanes");
    static_assert(NW * kMaxDepth * 8 + 16 <= kSplitZOffset, "header too small");
    static_assert(kSplitZOffset + 2 * NW * RB * 4 <= kSplitHeaderBytes, "header too small");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    float* zpart = reinterpret_cast<float*>(smem + kSplitZOffset);            // [2][NW][RB]
    unsigned char* data = smem + kSplitHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth, CW = p.cw;
    const int n = p.n, n4 = n / EPG;                                          // 16-byte groups per row
    const int c0 = warp * CW;                                                 // first column group of this warp's slice
    const int mycw = n4 - c0 < CW ? (n4 - c0 > 0 ? n4 - c0 : 0) : CW;         // column groups of the slice inside the matrix
    const uint32_t box_bytes = static_cast<uint32_t>(CW) * 16u * RB;          // one stage = one box, rows packed densely
    const uint32_t stage_stride = (box_bytes + 127u) & ~127u;
    unsigned char* my_stages = data + static_cast<size_t>(warp) * D * stage_stride;
    uint64_t* my_bars = bars + warp * kMaxDepth;

    const long long B = p.num_batches;
    const int cnt = B > blockIdx.x ? static_cast<int>((B - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;   // CTA-uniform

    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) mbar_init(&my_bars[d], 1);
        fence_mbar_init();
    }
    __syncthreads();

    const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
    const int stride_rows = static_cast<int>(gridDim.x) * RB;                 // rows between this CTA's batches (m < 2^31 here)
    int row0 = static_cast<int>(blockIdx.x) * RB;                             // first row of the current batch
    auto issue = [&](int r0, int d) {              // lane 0 of a warp with mycw > 0
        mbar_arrive_expect_tx(&my_bars[d], box_bytes);
        bulk_tensor_2d_g2s(my_stages + static_cast<size_t>(d) * stage_stride, &tmap, c0 * p.x_per_group, r0, &my_bars[d],
                           r0 < p.keep_rows ? pol_keep : pol_stream);
    };

    typename E::template Lane<NV> lm;              // this lane's slice of w (groups c0 + lane + 32k) and its fp32 accumulators
    double dacc[NV][EPG];
    float se = 0.f, sl = 0.f;
    double dse = 0.0, dsl = 0.0;
    lm.zero();
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
        for (int c = 0; c < EPG; ++c) dacc[k][c] = 0.0;
    const int myr = (lane >> SHIFT) & (RB - 1);    // the row of a batch whose logit ends up on this lane
    const int dup = lane & (DUP - 1);              // which of the lanes sharing that row this one is
    const bool owner = dup == 0;
    const bool full_cw = CW == 32 * NV;            // every lane's column groups lie inside the box
    const bool labels_word_aligned = PREDICT && RB % 4 == 0 && (reinterpret_cast<uintptr_t>(p.labels) & 3u) == 0;

    const bool active = mycw > 0;
    if (active && lane == 0) {
        const int pre = cnt < D ? cnt : D;
        for (int d = 0; d < pre; ++d) issue(row0 + d * stride_rows, d);
    }
    int issued = active ? (cnt < D ? cnt : D) : 0;
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
        if (lane == 0) {
            for (int d2 = 0; d2 < issued; ++d2) mbar_wait_drain(&my_bars[d2], 0u);
        }
        __syncwarp();
        return;
    }
    lm.template load_w<WSource::GlobalL2>(p.w, c0 + lane, 32, c0 + mycw);    // through L2: the kernel before this one may just have written them
    const float bval = __ldcg(p.b);

    for (int i = 0; i < cnt; ++i) {
        const bool myvalid = row0 + myr < p.m;
        const float yv = y_next;
        if constexpr (!PREDICT) {
            const long long rn = static_cast<long long>(row0) + stride_rows + myr;
            y_next = (i + 1 < cnt && rn < p.m) ? __ldg(p.y + rn) : 0.f;
        }

        uint4 x[RB][NV];
        bool have = false;
        if (active && !aborted) {
            bool ok = mbar_wait_bounded(&my_bars[d], phase, abort_flag);
            ok = __all_sync(FULL, ok);
            if (!ok) {
                aborted = true;
            } else {
                done = i + 1;
                have = true;
                const uint4* t4 = reinterpret_cast<const uint4*>(my_stages + static_cast<size_t>(d) * stage_stride);
                if (full_cw) {
#pragma unroll
                    for (int r = 0; r < RB; ++r)
#pragma unroll
                        for (int k = 0; k < NV; ++k) x[r][k] = t4[r * (32 * NV) + lane + 32 * k];
                } else {
#pragma unroll
                    for (int r = 0; r < RB; ++r)
#pragma unroll
                        for (int k = 0; k < NV; ++k) {
                            const int loc = lane + 32 * k;
                            x[r][k] = loc < CW ? t4[r * CW + loc] : make_uint4(0u, 0u, 0u, 0u);
                        }
                }
                __syncwarp();
                if (i + D < cnt) {
                    if (lane == 0) {
                        fence_proxy_async_smem();
                        issue(row0 + D * stride_rows, d);
                    }
                    issued = i + D + 1;
                }
                if (++d == D) { d = 0; phase ^= 1u; }
            }
        }
        if (!have) {
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int k = 0; k < NV; ++k) x[r][k] = make_uint4(0u, 0u, 0u, 0u);
        }

        const float zpartial = batch_dot<E, NV, 32, RB>(x, lm, lane);
        float* zp = zpart + (i & 1) * (NW * RB);
        if (owner) zp[warp * RB + myr] = zpartial;
        __syncthreads();
        // the lanes that share a row add PER_DUP partials each (warp order), then a butterfly: one fixed order, same in every warp
        float zs = 0.f;
#pragma unroll
        for (int j = 0; j < PER_DUP; ++j) zs += zp[(dup * PER_DUP + j) * RB + myr];
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
            if (++since_flush == 2 * kFlushBatches) {
                since_flush = 0;
                fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
            }
        }
        row0 += stride_rows;
    }

    if (aborted) {
        // report, then let this warp's copies still in flight land (bounded again) before the CTA retires
        if (lane == 0) {
            atomicExch(p.status, kStatusTimeout);
            for (int i = done; i < issued; ++i) mbar_wait_drain(&my_bars[i % D], static_cast<uint32_t>(i / D) & 1u);
        }
        __syncwarp();
    }
    if constexpr (!PREDICT) {
        double* out = p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
        fold_into_fp64<E, NV>(lm, dacc, se, sl, dse, dsl);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int loc = lane + 32 * k;
            if (loc < mycw) {
                const int col = EPG * (c0 + loc);
#pragma unroll
                for (int c = 0; c < EPG; ++c) out[col + c] = dacc[k][c];
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
