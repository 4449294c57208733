// Fused single-pass streaming kernel for wide rows (512 < n <= 4096, n % 4 == 0, X 16-byte aligned).
//
// A row no longer fits one warp's registers, so the 16 warps of a CTA split every row by columns: warp w owns
// the contiguous slice of CW = ceil(n/4/16) 16-byte column groups starting at w*CW.  The CTA walks batches of RB
// rows (batch g belongs to CTA g mod grid).  As in the narrow-row kernel each warp runs its own asynchronous
// pipeline with `depth` private stages, filled by its elected lane with one 1-D bulk copy per row (the slice of
// a row is contiguous, slices of consecutive rows are n*4 bytes apart), completing on the warp's own mbarriers.
// Per batch:
//   1. every warp moves its slice of the RB rows into registers (conflict-free 128-bit shared loads), re-arms the
//      stage, and forms its partial dot products (lane FMAs + transposing shuffle reduction);
//   2. the partials meet in a double-buffered shared array, one __syncthreads per batch; every warp then adds the
//      16 partials of each row in warp order, so all warps hold bit-identical z = x.w + b  (model equation, II-A);
//   3. p, err and the loss term are formed (redundantly per warp, counted once by warp 0)   (Eq. 1, Algorithm 7);
//   4. acc[c] += x[r][c] * err[r] on the registers loaded in step 1                        (Algorithm 1's err.X).
// Each column belongs to exactly one lane of one warp, so the CTA's partial row needs no cross-warp combine.
// A warp whose bounded wait expires raises the CTA's abort flag; it (and then every other warp) keeps taking part in
// the per-batch barrier without touching its stages, so the CTA still retires, with the status word set.
#pragma once
#include "lrgd_common.cuh"
#include "lrgd_stream_rows.cuh"

namespace lrgd {

constexpr int kSplitHeaderBytes = 2048;   // mbarriers [NW][kMaxDepth], abort flag, partial logits [2][NW][RB]
constexpr int kSplitZOffset = 1024;

struct SplitParams {
    const float* X;
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
    int cw;                   // 16-byte column groups per warp slice
    long long num_batches;    // ceil(m / RB)
};

template <int NV, int RB, int NW, bool PREDICT>
__global__ void __launch_bounds__(NW * 32, 1) k_stream_split(const SplitParams p) {
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = 5 - LOG_RB;              // lanes holding the same row after the reduction = 2^SHIFT
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(NW * kMaxDepth * 8 + 16 <= kSplitZOffset, "header too small");
    static_assert(kSplitZOffset + 2 * NW * RB * 4 <= kSplitHeaderBytes, "header too small");

    if (p.stop != nullptr && *reinterpret_cast<const volatile int*>(p.stop) != 0) return;   // a stopping rule was met by an earlier iteration
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    float* zpart = reinterpret_cast<float*>(smem + kSplitZOffset);            // [2][NW][RB]
    unsigned char* data = smem + kSplitHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth, CW = p.cw;
    const int n = p.n, n4 = n >> 2;
    const int c0 = warp * CW;                                                 // first column group of this warp's slice
    const int mycw = n4 - c0 < CW ? (n4 - c0 > 0 ? n4 - c0 : 0) : CW;         // column groups in the slice (0: idle warp)
    const uint32_t row_stride = (static_cast<uint32_t>(CW) * 16u + 127u) & ~127u;
    const uint32_t stage_stride = RB * row_stride;
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

    const uint64_t pol = l2_policy_evict_first();
    auto issue = [&](int i, int d) {               // lane 0 only, mycw > 0
        const long long row0 = (static_cast<long long>(i) * gridDim.x + blockIdx.x) * RB;
        const long long left = p.m - row0;
        const int rows = left < RB ? static_cast<int>(left) : RB;
        unsigned char* dst = my_stages + static_cast<size_t>(d) * stage_stride;
        const uint32_t bytes = static_cast<uint32_t>(mycw) * 16u;
        mbar_arrive_expect_tx(&my_bars[d], bytes * rows);
        const float* src = p.X + row0 * n + c0 * 4;
        for (int r = 0; r < rows; ++r) bulk_copy_g2s(dst + r * row_stride, src + static_cast<long long>(r) * n, bytes, &my_bars[d], pol);
    };

    float4 acc[NV];
    double dacc[NV][4];
    float se = 0.f, sl = 0.f;
    double dse = 0.0, dsl = 0.0;
    float4 wv[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        dacc[k][0] = dacc[k][1] = dacc[k][2] = dacc[k][3] = 0.0;
        const int loc = lane + 32 * k;
        const int idx = c0 + loc;
        wv[k] = loc < mycw ? make_float4(__ldg(p.w + 4 * idx), __ldg(p.w + 4 * idx + 1), __ldg(p.w + 4 * idx + 2),
                                         __ldg(p.w + 4 * idx + 3))
                           : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const float bval = __ldg(p.b);
    const int myr = (lane >> SHIFT) & (RB - 1);    // the row of a batch whose logit ends up on this lane
    const bool owner = (lane & ((1 << SHIFT) - 1)) == 0;

    const bool active = mycw > 0;
    if (active && lane == 0) {
        const int pre = cnt < D ? cnt : D;
        for (int d = 0; d < pre; ++d) issue(d, d);
    }
    int issued = active ? (cnt < D ? cnt : D) : 0;
    int done = 0;
    bool aborted = false;
    int since_flush = 0;
    int d = 0;
    uint32_t phase = 0;

    for (int i = 0; i < cnt; ++i) {
        const long long row0 = (static_cast<long long>(i) * gridDim.x + blockIdx.x) * RB;
        const long long left = p.m - row0;
        const int rows = left < RB ? static_cast<int>(left) : RB;
        const bool myvalid = myr < rows;
        float yv = 0.f;
        if constexpr (!PREDICT) {
            if (myvalid) yv = __ldg(p.y + row0 + myr);
        }

        float4 x[RB][NV];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int k = 0; k < NV; ++k) x[r][k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (active && !aborted) {
            bool ok = mbar_wait_bounded(&my_bars[d], phase, abort_flag);
            ok = __all_sync(FULL, ok);
            if (!ok) {
                aborted = true;
            } else {
                done = i + 1;
                const unsigned char* stage = my_stages + static_cast<size_t>(d) * stage_stride;
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const float4* t4 = reinterpret_cast<const float4*>(stage + r * row_stride);
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        const int loc = lane + 32 * k;
                        if (r < rows && loc < mycw) x[r][k] = t4[loc];
                    }
                }
                __syncwarp();
                if (i + D < cnt) {
                    if (lane == 0) {
                        fence_proxy_async_smem();
                        issue(i + D, d);
                    }
                    issued = i + D + 1;
                }
                if (++d == D) { d = 0; phase ^= 1u; }
            }
        }

        float v[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            float dot = 0.f;
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                dot = fmaf(x[r][k].x, wv[k].x, dot);
                dot = fmaf(x[r][k].y, wv[k].y, dot);
                dot = fmaf(x[r][k].z, wv[k].z, dot);
                dot = fmaf(x[r][k].w, wv[k].w, dot);
            }
            v[r] = dot;
        }
        lane_reduce<RB, 16, RB>(v, lane);
        float* zp = zpart + (i & 1) * (NW * RB);
        if (owner) zp[warp * RB + myr] = v[0];
        __syncthreads();
        float z = bval;
#pragma unroll
        for (int wi = 0; wi < NW; ++wi) z += zp[wi * RB + myr];

        if constexpr (PREDICT) {
            if (warp == 0 && owner && myvalid) p.labels[row0 + myr] = z >= p.cut ? 1 : 0;
        } else {
            float e, L;
            logistic_terms(z, yv, e, L);
            if (!myvalid) { e = 0.f; L = 0.f; }
            if (warp == 0 && owner) { se += e; sl += L; }
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                const float er = __shfl_sync(FULL, e, r << SHIFT);
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    acc[k].x = fmaf(x[r][k].x, er, acc[k].x);
                    acc[k].y = fmaf(x[r][k].y, er, acc[k].y);
                    acc[k].z = fmaf(x[r][k].z, er, acc[k].z);
                    acc[k].w = fmaf(x[r][k].w, er, acc[k].w);
                }
            }
            if (++since_flush == 2 * kFlushBatches) {
                since_flush = 0;
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    dacc[k][0] += acc[k].x; dacc[k][1] += acc[k].y;
                    dacc[k][2] += acc[k].z; dacc[k][3] += acc[k].w;
                    acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                dse += se; dsl += sl; se = 0.f; sl = 0.f;
            }
        }
    }

    if (aborted) {
        // report, then let this warp's copies still in flight land (bounded again) before the CTA retires
        if (lane == 0) {
            atomicExch(p.status, kStatusTimeout);
            for (int i = done; i < issued; ++i) mbar_wait_bounded(&my_bars[i % D], static_cast<uint32_t>(i / D) & 1u, abort_flag);
        }
        __syncwarp();
    }
    if constexpr (!PREDICT) {
        double* out = p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int loc = lane + 32 * k;
            if (loc < mycw) {
                const int col = 4 * (c0 + loc);
                out[col + 0] = dacc[k][0] + acc[k].x;
                out[col + 1] = dacc[k][1] + acc[k].y;
                out[col + 2] = dacc[k][2] + acc[k].z;
                out[col + 3] = dacc[k][3] + acc[k].w;
            }
        }
        if (warp == 0) {
            dse += se; dsl += sl;
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
