// Fused single-pass streaming kernel for rows of up to 512 columns (n % 4 == 0, X 16-byte aligned).
//
// One CTA = NW consumer warps + 1 producer warp.  The producer's elected lane stages contiguous row
// tiles of X (and the matching slice of y) into a ring of shared-memory stages with 1-D bulk
// asynchronous copies that complete on mbarriers.  A consumer warp takes one batch of rows at a time
// from a stage straight into registers (one conflict-free 128-bit shared load per element group),
// releases the stage, and then, from those registers only:
//   z = x.w + b      lane-local FMAs, then a transposing shuffle reduction that leaves each row's sum
//                    on a distinct lane group                      (model equation, Section II-A)
//   p, err, loss     one row per lane                              (Eq. 1; Algorithm 7; log-likelihood)
//   X^T err          acc[c] += x[r][c] * err[r] on the same registers (Algorithm 1's err.X)
// so X is read from HBM once and from shared memory once per pass.  Per-lane fp32 accumulators are
// folded into fp64 every kFlushBatches batches; at the end the CTA combines its warps in a fixed
// order and writes one row of partial sums [n columns | sum err | sum loss] in fp64.
//
// Row -> (CTA, warp, lane) assignment is static (tile t belongs to CTA t mod grid; batch q of a CTA
// belongs to warp q mod NW), so results are bit-reproducible.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kMaxStages = 8;
constexpr int kHeaderBytes = 256;      // full[8], empty[8] mbarriers, abort flag
constexpr int kFlushBatches = 4;

struct StreamParams {
    const float* X;
    const float* y;
    long long m;
    int n;
    const float* w;
    const float* b;
    double* partial;          // [grid][n+2]           (loss/grad mode)
    unsigned char* labels;    // [m]                   (predict mode)
    float cut;                // predict: logit(thr)
    int* status;              // device status word
    int bpt;                  // batches per tile
    int stages;               // ring depth (<= kMaxStages)
    int stage_y;              // 1: y slices are staged with the tile (y 16-byte aligned)
    long long num_tiles;
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

template <int NV, int LPR, int RB, int NW, bool PREDICT>
__global__ void __launch_bounds__((NW + 1) * 32, 1) k_stream_rows(const StreamParams p) {
    constexpr int RPW = 32 / LPR;                  // rows a warp touches with one load instruction
    constexpr int RPB = RB * RPW;                  // rows per batch
    constexpr int LOG_LPR = Log2<LPR>::value;
    constexpr int LOG_RB = Log2<RB>::value;
    constexpr int SHIFT = LOG_LPR - LOG_RB;        // duplicate lanes per row after the reduction = 2^SHIFT
    static_assert(SHIFT >= 0, "rows per batch slot must not exceed lanes per row");
    constexpr unsigned FULL = 0xffffffffu;

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty_bar = full_bar + kMaxStages;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kMaxStages);
    volatile int* issued_tiles = abort_flag + 1;   // tiles whose copies the producer has issued
    unsigned char* data = smem + kHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages, bpt = p.bpt;
    const int R = bpt * RPB;
    const int n = p.n, n4 = n >> 2;
    const uint32_t tile_stride = (static_cast<uint32_t>(R) * n * 4u + 127u) & ~127u;
    float* ystage = reinterpret_cast<float*>(data + static_cast<size_t>(S) * tile_stride);
    const long long T = p.num_tiles;
    // tiles of this CTA: blockIdx.x + k*gridDim.x, k in [0, K); the host keeps K*bpt below 2^31
    const int K = (T > blockIdx.x) ? static_cast<int>((T - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], bpt);
        }
        *abort_flag = 0;
        *issued_tiles = 0;
        fence_mbar_init();
    }
    __syncthreads();

    // per-lane state of a consumer (unused by the producer warp)
    float4 acc[NV];
    double dacc[NV][4];
    float se = 0.f, sl = 0.f;
    double dse = 0.0, dsl = 0.0;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        dacc[k][0] = dacc[k][1] = dacc[k][2] = dacc[k][3] = 0.0;
    }
    const int sub = lane & (LPR - 1), slot = lane >> LOG_LPR;

    if (warp == NW) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t pol = l2_policy_evict_first();
            int s = 0;
            uint32_t phase = 0;                    // parity of the stage's current fill
            for (int k = 0; k < K; ++k) {
                if (k >= S) {
                    if (!mbar_wait_bounded(&empty_bar[s], phase ^ 1u, abort_flag)) break;   // previous fill released
                } else if (*abort_flag) {
                    break;
                }
                const long long row0 = (blockIdx.x + static_cast<long long>(k) * gridDim.x) * R;
                const long long left = p.m - row0;
                const int rows = left < R ? static_cast<int>(left) : R;
                const uint32_t xbytes = static_cast<uint32_t>(rows) * n * 4u;
                const bool with_y = !PREDICT && p.stage_y && rows == R;
                mbar_arrive_expect_tx(&full_bar[s], xbytes + (with_y ? R * 4u : 0u));
                bulk_copy_g2s(data + static_cast<size_t>(s) * tile_stride, p.X + row0 * n, xbytes, &full_bar[s], pol);
                if (with_y) bulk_copy_g2s(ystage + static_cast<size_t>(s) * R, p.y + row0, R * 4u, &full_bar[s], pol);
                *issued_tiles = k + 1;
                if (++s == S) { s = 0; phase ^= 1u; }
            }
        }
    } else {
        // ---------------- consumers ----------------
        float4 wv[NV];                             // this lane's slice of w (w needs no 16-byte alignment)
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int idx = sub + k * LPR;
            wv[k] = idx < n4 ? make_float4(__ldg(p.w + 4 * idx), __ldg(p.w + 4 * idx + 1), __ldg(p.w + 4 * idx + 2),
                                           __ldg(p.w + 4 * idx + 3))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const float bval = __ldg(p.b);
        const int my_row_in_batch = ((sub >> SHIFT) & (RB - 1)) * RPW + slot;   // the row whose logit ends up on this lane
        const bool owner = (sub & ((1 << SHIFT) - 1)) == 0;                      // one lane per row does the bookkeeping
        int since_flush = 0;
        // batch q of this CTA (q = warp, warp+NW, ...) is batch j of the CTA's k-th tile; advance (k, j, stage,
        // phase) incrementally so the loop carries no division
        const int dk = NW / bpt, dj = NW % bpt;
        int k = warp / bpt, j = warp % bpt;
        int s = k % S;
        uint32_t phase = static_cast<uint32_t>(k / S) & 1u;

        for (; k < K;) {
            const long long row0 = (blockIdx.x + static_cast<long long>(k) * gridDim.x) * R;
            const long long left = p.m - row0;
            const int rows = left < R ? static_cast<int>(left) : R;

            bool ok = mbar_wait_bounded(&full_bar[s], phase, abort_flag);
            ok = __all_sync(FULL, ok);
            if (!ok) break;

            const float4* t4 = reinterpret_cast<const float4*>(data + static_cast<size_t>(s) * tile_stride);
            const int brow0 = j * RPB;
            float4 x[RB][NV];
#pragma unroll
            for (int i = 0; i < RB; ++i) {
                const int r = brow0 + i * RPW + slot;
#pragma unroll
                for (int k2 = 0; k2 < NV; ++k2) {
                    const int idx = sub + k2 * LPR;
                    x[i][k2] = (r < rows && idx < n4) ? t4[r * n4 + idx] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            const int myr = brow0 + my_row_in_batch;
            const bool myvalid = myr < rows;
            float yv = 0.f;
            if constexpr (!PREDICT) {
                if (myvalid) yv = (p.stage_y && rows == R) ? ystage[static_cast<size_t>(s) * R + myr] : __ldg(p.y + row0 + myr);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);      // the stage may be refilled; the batch lives in registers now

            float v[RB];
#pragma unroll
            for (int i = 0; i < RB; ++i) {
                float d = 0.f;
#pragma unroll
                for (int k2 = 0; k2 < NV; ++k2) {
                    d = fmaf(x[i][k2].x, wv[k2].x, d);
                    d = fmaf(x[i][k2].y, wv[k2].y, d);
                    d = fmaf(x[i][k2].z, wv[k2].z, d);
                    d = fmaf(x[i][k2].w, wv[k2].w, d);
                }
                v[i] = d;
            }
            lane_reduce<RB, LPR / 2, RB>(v, lane);
            const float z = v[0] + bval;

            if constexpr (PREDICT) {
                if (owner && myvalid) p.labels[row0 + myr] = z >= p.cut ? 1 : 0;
            } else {
                float e, L;
                logistic_terms(z, yv, e, L);
                if (!myvalid) { e = 0.f; L = 0.f; }
                if (owner) { se += e; sl += L; }
#pragma unroll
                for (int i = 0; i < RB; ++i) {
                    const float ei = __shfl_sync(FULL, e, i << SHIFT, LPR);
#pragma unroll
                    for (int k2 = 0; k2 < NV; ++k2) {
                        acc[k2].x = fmaf(x[i][k2].x, ei, acc[k2].x);
                        acc[k2].y = fmaf(x[i][k2].y, ei, acc[k2].y);
                        acc[k2].z = fmaf(x[i][k2].z, ei, acc[k2].z);
                        acc[k2].w = fmaf(x[i][k2].w, ei, acc[k2].w);
                    }
                }
                if (++since_flush == kFlushBatches) {
                    since_flush = 0;
#pragma unroll
                    for (int k2 = 0; k2 < NV; ++k2) {
                        dacc[k2][0] += acc[k2].x; dacc[k2][1] += acc[k2].y;
                        dacc[k2][2] += acc[k2].z; dacc[k2][3] += acc[k2].w;
                        acc[k2] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    dse += se; dsl += sl; se = 0.f; sl = 0.f;
                }
            }
            // next batch of this warp
            int adv = dk;
            j += dj;
            if (j >= bpt) { j -= bpt; ++adv; }
            k += adv;
            s += adv;
            while (s >= S) { s -= S; phase ^= 1u; }
        }
#pragma unroll
        for (int k2 = 0; k2 < NV; ++k2) {
            dacc[k2][0] += acc[k2].x; dacc[k2][1] += acc[k2].y;
            dacc[k2][2] += acc[k2].z; dacc[k2][3] += acc[k2].w;
        }
        dse += se; dsl += sl;
    }

    __syncthreads();                               // every issued tile has been consumed, unless a wait gave up
    if (*abort_flag) {
        // a bounded wait expired: report it, and let the copies still in flight land (bounded) before the CTA retires
        if (threadIdx.x == 0) {
            atomicExch(p.status, kStatusTimeout);
            const int issued = *issued_tiles;
            for (int k = issued > S ? issued - S : 0; k < issued; ++k)
                mbar_wait_bounded(&full_bar[k % S], static_cast<uint32_t>(k / S) & 1u, abort_flag);
        }
        __syncthreads();
    }
    if constexpr (PREDICT) return;

    // ---------------- fixed-order combine of the CTA's warps ----------------
    double* red = reinterpret_cast<double*>(data); // [NW][n] column sums, then [NW] sum err, [NW] sum loss
    double* red_e = red + static_cast<size_t>(NW) * n;
    double* red_l = red_e + NW;
    if (warp < NW) {
        // row slots of one warp that own the same columns: add in slot order
#pragma unroll
        for (int k2 = 0; k2 < NV; ++k2) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                double t = 0.0;
#pragma unroll
                for (int sidx = 0; sidx < RPW; ++sidx) t += __shfl_sync(FULL, dacc[k2][c], sub + sidx * LPR);
                const int idx = sub + k2 * LPR;
                if (slot == 0 && idx < n4) red[static_cast<size_t>(warp) * n + idx * 4 + c] = t;
            }
        }
#pragma unroll
        for (int msk = 16; msk >= 1; msk >>= 1) {
            dse += __shfl_xor_sync(FULL, dse, msk);
            dsl += __shfl_xor_sync(FULL, dsl, msk);
        }
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }
    }
    __syncthreads();
    double* out = p.partial + static_cast<size_t>(blockIdx.x) * (n + 2);
    for (int c = threadIdx.x; c < n + 2; c += blockDim.x) {
        double t = 0.0;
        if (c < n) {
            for (int wi = 0; wi < NW; ++wi) t += red[static_cast<size_t>(wi) * n + c];
        } else {
            const double* src = (c == n) ? red_e : red_l;
            for (int wi = 0; wi < NW; ++wi) t += src[wi];
        }
        out[c] = t;
    }
}

}  // namespace lrgd
