// C-ABI layer: argument validation, launch planning, workspace, and the iteration loop.
// The declarations and their contracts are in include/lrgd.h.
#include "../../include/lrgd.h"

#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <utility>
#include <vector>

#include "lrgd_convert.cuh"
#include "lrgd_fit_cluster.cuh"
#include "lrgd_fit_rows.cuh"
#include "lrgd_generic.cuh"
#include "lrgd_reduce.cuh"
#include "lrgd_score.cuh"
#include "lrgd_stream_rows.cuh"
#include "lrgd_stream_split.cuh"
#include "lrgd_stream_wide.cuh"

using namespace lrgd;

namespace {

#ifndef LRGD_NW
#define LRGD_NW 16
#endif
constexpr int kNW = LRGD_NW;                   // warps per CTA of the staged kernels (512 threads, one CTA per SM)
constexpr int kStageBudgetBytes = 208 * 1024;  // shared memory the warps' stages may take (227 KB per CTA on sm_100)
constexpr int kMaxGridPerSm = 8;               // widest launch any variant uses, in CTAs per SM
constexpr int kMaxProfiled = 4096;
constexpr int kMaxDynamicSmem = 232448;         // opt-in dynamic shared memory per CTA on sm_100
constexpr int64_t kMaxRows = int64_t(1) << 40;
constexpr int kWideAnyMaxCols = 16384;          // widest row of the CTA-wide staged kernel for rows of any length

struct RowShape { int nv, lpr, rb; int nw = kNW; };    // nw = warps per CTA

// Which instantiation of the narrow-row kernel covers ng 16-byte column groups per row.  The shapes whose threads hold
// more than a 512-thread CTA's 128 registers run with eight warps per CTA (255 registers): fp32 rows of 17..32 groups
// (68..128 columns) with 16-row batches -- the per-batch work (the logistic terms, the reduction, the stage bookkeeping) is
// then shared by twice the rows, which is what these issue-bound rows need --, fp32 rows of 65..96 and 129..256 groups and
// bfloat16 rows of 33..128 groups (a thread holds its 32 columns of a row slice, their weights and accumulators).  The
// bytes in flight per SM stay the same.
bool row_shape_for(int ng, bool bf16, RowShape* s) {
    if (ng <= 2) *s = {1, 2, 2};                              // 4 or 8 fp32 (8 or 16 bfloat16) columns: two lanes per row
    else if (ng <= 4) *s = {1, 4, 4};                        // 12 or 16 (24 or 32)
    else if (ng <= 8) *s = {1, 8, 8};
    else if (ng <= 16) *s = {1, 16, 8};
    else if (ng <= 32 && !bf16) *s = {1, 32, 16, 8};        // 68..128 fp32 columns: eight warps, sixteen rows
    else if (ng <= 32) *s = {1, 32, 8};
    else if (ng <= 48 && !bf16) *s = {3, 16, 2};            // 132..192 fp32 columns: sixteen lanes per row, three groups each
    else if (ng <= 64 && !bf16) *s = {2, 32, 4};
    else if (ng <= 64 && bf16) *s = {2, 32, 8, 8};          // 264..512 bfloat16 columns: eight warps, eight rows (no spills)
    else if (ng <= 96 && !bf16) *s = {3, 32, 4, 8};         // 260..384 fp32 columns: three groups per lane (with four, a quarter
                                                            // to a half of a lane's slots would be dead work)
    else if (ng <= 128 && !bf16) *s = {4, 32, 4, 8};        // 388..512 fp32 columns: eight warps, four rows (4..8 KB batches)
    else if (ng <= 96 && bf16) *s = {3, 32, 2, 8};          // 520..768 bfloat16 columns
    else if (ng <= 128 && bf16) *s = {4, 32, 2, 8};         // 776..1024 bfloat16 columns: eight warps, as below
    else if (ng <= 160 && !bf16) *s = {5, 32, 2, 8};        // 516..640 fp32 columns: no more groups per lane than the row needs
    else if (ng <= 192 && !bf16) *s = {6, 32, 2, 8};        // 644..768
    else if (ng <= 224 && !bf16) *s = {7, 32, 2, 8};        // 772..896
    else if (ng <= 256 && !bf16) *s = {8, 32, 2, 8};
    else return false;
    return true;
}

// Narrow rows whose length is not a whole number of 16-byte groups, or whose matrix is not 16-byte aligned: a lane owns
// single elements (nv of them per row).
bool any_row_shape_for(int n, RowShape* s) {
    if (n <= 2) *s = {1, 2, 2};                             // one or two columns: two lanes per row (32 rows per batch either way)
    else if (n <= 4) *s = {1, 4, 4};
    else if (n <= 8) *s = {1, 8, 8};
    else if (n <= 16) *s = {1, 16, 16};
    else if (n <= 32) *s = {1, 32, 32};
    else if (n <= 64) *s = {2, 32, 16};
    else if (n <= 128) *s = {4, 32, 8};
    else if (n <= 256) *s = {8, 32, 4};
    else if (n <= 512) *s = {16, 32, 2};
    else return false;                                      // wider rows of any length: the CTA-wide staged kernel (variant 4)
    return true;
}

// bf16: X holds bfloat16 (2-byte) elements instead of fp32; a 16-byte group is then 8 columns instead of 4.
// Cluster sizes of the single-cluster fit, largest first (sixteen needs the non-portable opt-in).
constexpr int kClusterSizes[] = {16, 8};

// A narrow-row problem of `slots` CTA-loads of batches (nw batches each) whose rows all fit the shared memory of one
// thread-block cluster of C <= sms CTAs, every CTA busy, is PLANNED on C CTAs -- for every entry point, so that all of
// them divide the rows the same way and give the same bits as the single-cluster fit (k_fit_cluster), which is what
// lr_fit then runs.  Returns C, or 0 if the problem is not of that kind.
int cluster_size_for(int64_t slots, int nw, int64_t stage_stride, int32_t n, int32_t sms) {
    for (const int C : kClusterSizes) {
        if (C > sms || slots < C) continue;
        const int64_t per_warp = (slots + C - 1) / C;                          // stages per warp: all its batches at once
        if (per_warp > kMaxDepth) continue;
        if (kHeaderBytes + nw * per_warp * stage_stride + fit_tail_bytes(n) + 2LL * C * (n + 2) * 8 + 16 > kMaxDynamicSmem) continue;
        return C;
    }
    return 0;
}

int make_plan(int64_t m, int32_t n, bool aligned16, int32_t sms, lr_plan* P, bool bf16 = false) {
    if (!P) return LR_ERR_NULL;
    if (m < 1 || m > kMaxRows || n < 1 || sms < 1) return LR_ERR_SHAPE;
    std::memset(P, 0, sizeof(*P));
    const int epg = bf16 ? 8 : 4, eb = bf16 ? 2 : 4;
    RowShape rs;
    const bool grouped = aligned16 && n % epg == 0 && row_shape_for(n / epg, bf16, &rs);
    // rows of up to 512 columns that cannot be cut into aligned 16-byte groups (length not a whole number of groups, or X
    // aligned to its element size only)
    const bool any_len = !grouped && any_row_shape_for(n, &rs);
    if (grouped || any_len) {
        const int rpb = rs.rb * (32 / rs.lpr);                                  // rows per batch = rows per stage
        const int64_t B = (m + rpb - 1) / rpb;                                  // batches
        const int64_t slots = (B + rs.nw - 1) / rs.nw;                              // CTA-level groups of nw batches
        const int64_t stage_stride = (int64_t(rpb) * n * eb + (any_len ? 16 : 0) + 127) & ~int64_t(127);   // as the kernel lays it out
        const int cluster = grouped ? cluster_size_for(slots, rs.nw, stage_stride, n, sms) : 0;
        const int grid = cluster ? cluster : int(std::min<int64_t>(slots, sms));
        const int64_t per_warp = (slots + grid - 1) / grid;                     // most batches any warp handles
        int D = int(std::min<int64_t>(kMaxDepth, kStageBudgetBytes / (rs.nw * stage_stride)));
        D = int(std::min<int64_t>(D, per_warp));
        if (D < 1) D = 1;
        const int64_t combine = int64_t(rs.nw) * n * 8 + 2 * rs.nw * 8;
        P->variant = grouped ? 0 : 3;
        P->lanes_per_row = rs.lpr;
        P->vec_per_lane = rs.nv;
        P->rows_per_batch = rpb;
        P->tile_rows = rpb;
        P->stages = D;
        P->grid = grid;
        P->threads = rs.nw * 32;
        P->smem_bytes = int(kHeaderBytes + std::max<int64_t>(int64_t(rs.nw) * D * stage_stride, combine));
        if (per_warp >= (int64_t(1) << 31)) return LR_ERR_SHAPE;
        return LR_OK;
    }
    // (fp32 rows of 4100..6144 columns are the exception: slices of 65..96 groups per warp leave the row-split kernel with two
    // rows per batch and half-empty lanes, 3.7-5.1 TB/s, where the CTA-wide stages of variant 4 below reach 4.7-5.9)
    const bool split_weak = !bf16 && n / epg > 1024 && n / epg <= 1536;
    if (aligned16 && n % epg == 0 && n / epg <= kNW * (bf16 ? 64 : 128) && !split_weak && m < (int64_t(1) << 31) - 65536) {   // TMA coordinates are int32
        // wide rows: the warps of a CTA split each row by columns
        // bfloat16 rows are split across eight warps instead of sixteen: wider slices, and 255 registers per thread, which
        // batches of 16 (one group per lane), 8 (two groups) or 4 rows (four groups: 4104..8192 columns) need
        const int nw = bf16 ? 8 : kNW;
        const int cw = (n / epg + nw - 1) / nw;                                 // 16-byte column groups per warp slice
        const int nv = cw > 64 ? 4 : (cw > 32 ? 2 : 1);            // fp32 rows of 4100..8192 columns: four groups per lane, two rows
        // Rows per batch.  All warps of a CTA meet once per batch, so a batch must carry enough bytes to cover that
        // round trip: slices of up to 24 groups per warp take 16 rows at a time and slices of 33..48 groups 8 rows, where 8
        // and 4 left the pass latency-bound (1028 columns: 3.6 TB/s, 2052: 4.2 TB/s); wider slices would leave room for
        // one stage only.
        const int rb = nv == 4 ? (nw == 8 ? 4 : 2) : nv == 2 ? (nw == 8 || (cw <= 48 && !bf16) ? 8 : 4)  // (the 16-warp bfloat16 kernels would spill
                               : (nw == 8 || (cw <= 24 && !bf16) ? 16 : 8);          //  registers with the larger batches)
        const int64_t B = (m + rb - 1) / rb;
        const int grid = int(std::min<int64_t>(B, sms));
        const int64_t per_cta = (B + grid - 1) / grid;
        const int64_t stage_stride = (int64_t(cw) * 16 * rb + 127) & ~int64_t(127);   // one densely packed box per stage
        int D = int(std::min<int64_t>(kMaxDepth, kStageBudgetBytes / (nw * stage_stride)));
        D = int(std::min<int64_t>(D, per_cta));
        if (D < 1) D = 1;
        P->variant = 1;
        P->lanes_per_row = nw * 32;
        P->vec_per_lane = nv;
        P->rows_per_batch = rb;
        P->tile_rows = rb;
        P->stages = D;
        P->grid = grid;
        P->threads = nw * 32;
        P->smem_bytes = int(kSplitHeaderBytes + int64_t(nw) * D * stage_stride);
        if (per_cta >= (int64_t(1) << 31)) return LR_ERR_SHAPE;
        return LR_OK;
    }
    if (n > 512 && n <= kWideAnyMaxCols) {
        // wide rows of any length, matrix aligned to its element size: the warps of a CTA split each row by columns and the
        // stages, whole batches of contiguous rows, belong to the CTA.  A lane holds NV elements of each of RB rows (32 in
        // all); a batch is at most ~64 KB so that two to four of them are in flight.
        // rows of up to 1024 elements are split over eight warps (slices of 65..128 elements: three or four per lane, sixteen
        // rows per batch in 255 registers), wider ones over sixteen
        const int nw = n <= 1024 ? 8 : kNW;
        const int cw = (n + nw - 1) / nw;                                       // elements per warp slice
        // elements per lane and row: the smallest of 2, 3, 4, 6, 8, 12, 16 that covers the slice (a lane's slots beyond the
        // slice are dead work, so the steps are kept fine); rows per batch: as many as the registers hold (32 or 48 elements
        // of a batch per lane), because all warps meet once per batch
        // (rows beyond 8192 elements: one row per batch, 24 or 32 elements of it per lane; aligned rows of that width
        // land here too, since the row-split kernel's tensor-map boxes end at 8192 columns)
        static const int kNv[9] = {2, 3, 4, 6, 8, 12, 16, 24, 32}, kRb[9] = {16, 16, 8, 8, 4, 4, 2, 1, 1};
        int pick = 0;
        while (pick < 8 && kNv[pick] * 32 < cw) ++pick;
        const int nv = kNv[pick], rb = nw == 8 ? 16 : kRb[pick];
        const int64_t B = (m + rb - 1) / rb;
        const int grid = int(std::min<int64_t>(B, sms));
        const int64_t per_cta = (B + grid - 1) / grid;
        const int64_t stage_stride = (int64_t(rb) * n * eb + 16 + 127) & ~int64_t(127);
        int D = int(std::min<int64_t>(kMaxDepth, (kStageBudgetBytes + 12 * 1024) / stage_stride));
        D = int(std::min<int64_t>(D, per_cta));
        if (D < 1) D = 1;
        P->variant = 4;
        P->lanes_per_row = nw * 32;
        P->vec_per_lane = nv;
        P->rows_per_batch = rb;
        P->tile_rows = rb;
        P->stages = D;
        P->grid = grid;
        P->threads = nw * 32;
        P->smem_bytes = int(kSplitHeaderBytes + int64_t(D) * stage_stride);
        if (per_cta >= (int64_t(1) << 31)) return LR_ERR_SHAPE;
        return LR_OK;
    }
    // rows per chunk: 64, halved down to 8 while the chunks would not give every SM a few CTAs
    int gen_rows = kGenRows;
    while (gen_rows > 8 && (m + gen_rows - 1) / gen_rows < int64_t(sms) * kMaxGridPerSm) gen_rows /= 2;
    const int64_t nchunks = (m + gen_rows - 1) / gen_rows;
    P->variant = 2;
    P->lanes_per_row = 32;
    P->vec_per_lane = 0;
    P->rows_per_batch = 1;
    P->tile_rows = gen_rows;
    P->stages = 0;
    P->grid = int(std::min<int64_t>(nchunks, int64_t(sms) * kMaxGridPerSm));
    P->threads = kGenThreads;
    P->smem_bytes = 0;
    return LR_OK;
}

}  // namespace

struct lr_ctx {
    int device = 0;
    int sm_count = 0;
    int n_max = 0;
    double* d_partial = nullptr;
    int* d_status = nullptr;
    TolState* d_tol = nullptr;                      // stopping-rule state of lr_fit_tol
    double* d_gbuf = nullptr;                       // [n_max+1] gradient entries for the norm
    TolState* h_tol = nullptr;                      // pinned host mirror
    int* h_words = nullptr;                         // pinned: [0] status word before a blocking call, [1] after it, [2] abort word of a persistent launch
    float* d_vel = nullptr;                         // [n_max+1] velocity of lr_fit_opt when the caller passes none
    double* d_oscr = nullptr;                       // [n_max+2] scratch of the optimiser reduction
    unsigned int* d_oticket = nullptr;
    unsigned int* d_gbar = nullptr;                 // persistent fit kernel: [0] grid-barrier counter, [1] abort flag of the launch
                                                    // (one such pair per rank when several ranks run as one launch)
    FitParams* d_rank_params = nullptr;             // [kMaxWorld] parameters of the ranks of lr_fit_sharded_local
    int sm_limit = 0;                               // > 0: plans use at most this many SMs (lr_set_sm_limit)
    int cluster_mode = -1;                          // single-cluster fit kernel for tiny problems: -1 the library chooses, 0 never
    bool coop = false;                              // device supports cooperative launches
    int persistent_mode = -1;                       // single-launch fit kernel: -1 the library chooses, 0 never, 1 whenever the shape allows
    bool overlap = true;                            // consecutive kernels of one call are launched as programmatic dependents
    int64_t l2_keep_bytes = -1;                     // leading bytes of X fetched with an evict-last hint; -1 = per-kernel default
    int64_t l2_bytes = 0;                           // size of the device's L2
    // buffers of the host-pointer entry points (grown on demand)
    void* d_hX = nullptr; size_t hX_bytes = 0;
    void* d_hy = nullptr; size_t hy_bytes = 0;
    void* d_hw = nullptr; size_t hw_bytes = 0;      // w[n] | b | loss_hist
    void* d_hl = nullptr; size_t hl_bytes = 0;      // labels
    void* d_hXh = nullptr; size_t hXh_bytes = 0;    // bfloat16 copy of X (lr_fit_host_bf16, lr_predict_host_bf16)
    cudaStream_t hstream = nullptr;
    // profiling
    bool prof = false;
    std::vector<cudaEvent_t> ev;                    // pairs: start, stop
    int prof_used = 0;
    int64_t launches = 0;
    int last_cuda = 0;
    // guard regions: every device workspace that kernels index by a computed offset sits between two of them
    std::vector<unsigned char*> guard_bases;        // allocation bases; the user range starts kGuardBytes in
    std::vector<size_t> guard_sizes;                // user bytes, rounded up to kGuardBytes
};

namespace {

// Guard regions around the context's device workspaces (per-CTA partial rows, gradient buffer, velocity, optimiser scratch):
// kGuardBytes of a fixed pattern before and after each, written once at creation.  No kernel of the library has any
// business there, so a changed byte (lr_check_guards) means an index ran out of its array.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardPattern = 0xA5;

template <class T>
cudaError_t guarded_alloc(lr_ctx* c, T** user, size_t bytes) {
    const size_t body = (bytes + kGuardBytes - 1) / kGuardBytes * kGuardBytes;
    unsigned char* base = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&base), body + 2 * kGuardBytes);
    if (e != cudaSuccess) return e;
    c->guard_bases.push_back(base);
    c->guard_sizes.push_back(body);
    e = cudaMemset(base, kGuardPattern, kGuardBytes);
    if (e == cudaSuccess) e = cudaMemset(base + kGuardBytes + body, kGuardPattern, kGuardBytes);
    *user = reinterpret_cast<T*>(base + kGuardBytes);
    return e;
}

// A named range around a whole library call, visible on a profiler's timeline (costs nothing when no tool is attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(lr_ctx* c) {
        if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; }
        cudaError_t e = cudaSetDevice(c->device);
        if (e != cudaSuccess) { c->last_cuda = int(e); ok = false; }
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

#define LR_CK(ctx, call)                                 \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) {                        \
            (ctx)->last_cuda = int(e__);                 \
            return LR_ERR_CUDA;                          \
        }                                                \
    } while (0)

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// SMs the launch plans of this context may use (lr_set_sm_limit)
int plan_sms(const lr_ctx* ctx) { return ctx->sm_limit > 0 ? std::min(ctx->sm_limit, ctx->sm_count) : ctx->sm_count; }

// Launches `kern`; with `dependent` set, as a programmatic dependent launch: the kernel may start while the kernel
// before it in the stream is still draining, and synchronises with it on the device (grid_dependency_wait).
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool dependent,
                          Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = dependent ? attr : nullptr;
    cfg.numAttrs = dependent ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, args...);
    if (dependent && (e == cudaErrorNotSupported || e == cudaErrorInvalidValue)) {
        // a driver or stream that does not take the attribute: the ordinary launch computes the same thing
        cudaGetLastError();
        cfg.attrs = nullptr;
        cfg.numAttrs = 0;
        e = cudaLaunchKernelEx(&cfg, kern, args...);
    }
    return e;
}

// Raises a kernel's dynamic shared-memory limit to `smem` on the current device, once: the limit is remembered per
// kernel instantiation (Tag) and device, so that the thousands of launches of a fit do not repeat the runtime call.
template <class Tag>
cudaError_t ensure_dynamic_smem(const void* kern, int smem) {
    constexpr int kDevices = 64;
    static int have[kDevices] = {};
    static std::mutex mu;                          // contexts on different host threads may share an instantiation
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && dev < kDevices && have[dev] >= smem) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && dev >= 0 && dev < kDevices) have[dev] = smem;
    return e;
}
template <class E, int A, int B, int C, int D, bool F>
struct KernelTag {};

// One instantiation of the narrow-row kernels: storage type, groups per lane, lanes per row, rows per batch slot, warps.
template <class E, int NV, int LPR, int RB, int NW>
struct RowKernelShape {
    using Elem = E;
    static constexpr int nv = NV, lpr = LPR, rb = RB, nw = NW;
};

// Calls f(RowKernelShape<...>{}) for the instantiation a plan of variant 0 or 3 names; every shape the planner can
// produce is listed here once, and the two launchers below (single pass, persistent fit) share the list.
template <class F>
cudaError_t for_row_shape(const lr_plan& P, bool bf16, F&& f) {
    const int nw = P.threads / 32, lpr = P.lanes_per_row, nv = P.vec_per_lane, rb = P.rows_per_batch / (32 / lpr);
    auto is = [&](int a, int b, int c, int d) { return nv == a && lpr == b && rb == c && nw == d; };
#define LRGD_SHAPE(E, a, b, c, d) if (is(a, b, c, d)) return f(RowKernelShape<E, a, b, c, d>{});
    if (P.variant == 3) {                          // rows of any length: a lane owns single elements
        if (bf16) {
            LRGD_SHAPE(ElemBF16Any, 1, 2, 2, 16) LRGD_SHAPE(ElemBF16Any, 1, 4, 4, 16)
            LRGD_SHAPE(ElemBF16Any, 1, 8, 8, 16) LRGD_SHAPE(ElemBF16Any, 1, 16, 16, 16) LRGD_SHAPE(ElemBF16Any, 1, 32, 32, 16)
            LRGD_SHAPE(ElemBF16Any, 2, 32, 16, 16) LRGD_SHAPE(ElemBF16Any, 4, 32, 8, 16) LRGD_SHAPE(ElemBF16Any, 8, 32, 4, 16)
            LRGD_SHAPE(ElemBF16Any, 16, 32, 2, 16)
        } else {
            LRGD_SHAPE(ElemF32Any, 1, 2, 2, 16) LRGD_SHAPE(ElemF32Any, 1, 4, 4, 16)
            LRGD_SHAPE(ElemF32Any, 1, 8, 8, 16) LRGD_SHAPE(ElemF32Any, 1, 16, 16, 16) LRGD_SHAPE(ElemF32Any, 1, 32, 32, 16)
            LRGD_SHAPE(ElemF32Any, 2, 32, 16, 16) LRGD_SHAPE(ElemF32Any, 4, 32, 8, 16) LRGD_SHAPE(ElemF32Any, 8, 32, 4, 16)
            LRGD_SHAPE(ElemF32Any, 16, 32, 2, 16)
        }
    } else if (bf16) {
        LRGD_SHAPE(ElemBF16, 1, 2, 2, 16) LRGD_SHAPE(ElemBF16, 1, 4, 4, 16)
        LRGD_SHAPE(ElemBF16, 1, 8, 8, 16) LRGD_SHAPE(ElemBF16, 1, 16, 8, 16) LRGD_SHAPE(ElemBF16, 1, 32, 8, 16)
        LRGD_SHAPE(ElemBF16, 2, 32, 8, 8) LRGD_SHAPE(ElemBF16, 3, 32, 2, 8) LRGD_SHAPE(ElemBF16, 4, 32, 2, 8)
    } else {
        LRGD_SHAPE(ElemF32, 1, 2, 2, 16) LRGD_SHAPE(ElemF32, 1, 4, 4, 16)
        LRGD_SHAPE(ElemF32, 1, 8, 8, 16) LRGD_SHAPE(ElemF32, 1, 16, 8, 16) LRGD_SHAPE(ElemF32, 1, 32, 16, 8)
        LRGD_SHAPE(ElemF32, 3, 16, 2, 16) LRGD_SHAPE(ElemF32, 2, 32, 4, 16) LRGD_SHAPE(ElemF32, 3, 32, 4, 8) LRGD_SHAPE(ElemF32, 4, 32, 4, 8)
        LRGD_SHAPE(ElemF32, 5, 32, 2, 8) LRGD_SHAPE(ElemF32, 6, 32, 2, 8) LRGD_SHAPE(ElemF32, 7, 32, 2, 8) LRGD_SHAPE(ElemF32, 8, 32, 2, 8)
    }
#undef LRGD_SHAPE
    return cudaErrorInvalidValue;
}

template <bool PRED>
cudaError_t launch_rows(const lr_plan& P, const StreamParams& sp, cudaStream_t st, bool bf16 = false, bool dependent = false) {
    return for_row_shape(P, bf16, [&](auto shape) {
        using S = decltype(shape);
        auto kern = k_stream_rows<typename S::Elem, S::nv, S::lpr, S::rb, S::nw, PRED>;
        cudaError_t e = ensure_dynamic_smem<KernelTag<typename S::Elem, S::nv, S::lpr, S::rb, S::nw, PRED>>(
            reinterpret_cast<const void*>(kern), P.smem_bytes);
        if (e != cudaSuccess) return e;
        return launch_kernel(kern, dim3(P.grid), dim3(P.threads), size_t(P.smem_bytes), st, dependent, sp);
    });
}

// Tensor map of X for the wide-row kernel: [m][n] row-major, box = cw 16-byte groups by rb rows, zero fill outside.
// The copy moves bytes untouched, and a box may span at most 256 elements per dimension, so a bfloat16 matrix is
// described as 32-bit words (n/2 per row): the widest slice, 64 groups, is then 256 elements for either storage type.
// The encoder is a driver entry point, resolved at run time so that the library links against the runtime only.
bool split_words64(bool /*bf16*/, int cw) { return cw > 64; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t make_x_tensor_map(const void* X, bool bf16, int64_t m, int32_t n, int cw, int rb, CUtensorMap* out) {
    // resolved once per process; the initialisation of a function-local static is thread-safe
    struct Resolved { EncodeTiledFn fn = nullptr; cudaError_t err = cudaSuccess; };
    static const Resolved resolved = [] {
        Resolved r;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        r.err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (r.err == cudaSuccess && (q != cudaDriverEntryPointSuccess || !fn)) r.err = cudaErrorNotSupported;
        if (r.err == cudaSuccess) r.fn = reinterpret_cast<EncodeTiledFn>(fn);
        return r;
    }();
    if (resolved.err != cudaSuccess) return resolved.err;
    const EncodeTiledFn encode = resolved.fn;
    // (fp32 slices of more than 64 groups -- rows of more than 4096 columns -- are described as 64-bit words for the same reason)
    const bool wide64 = split_words64(bf16, cw);
    const cuuint64_t row_bytes = cuuint64_t(n) * (bf16 ? 2 : 4);
    const cuuint32_t wbytes = wide64 ? 8 : 4;
    const cuuint64_t dims[2] = {row_bytes / wbytes, cuuint64_t(m)};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {cuuint32_t(cw) * (16 / wbytes), cuuint32_t(rb)};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(out, wide64 ? CU_TENSOR_MAP_DATA_TYPE_UINT64 : bf16 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        const_cast<void*>(X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <class E, int NV, int RB, bool PRED, int NW = kNW>
cudaError_t launch_split_t(const lr_plan& P, const CUtensorMap& tm, const SplitParams& sp, cudaStream_t st, bool dependent) {
    auto kern = k_stream_split<E, NV, RB, NW, PRED>;
    cudaError_t e = ensure_dynamic_smem<KernelTag<E, NV, -1, RB, NW, PRED>>(reinterpret_cast<const void*>(kern), P.smem_bytes);
    if (e != cudaSuccess) return e;
    return launch_kernel(kern, dim3(P.grid), dim3(P.threads), size_t(P.smem_bytes), st, dependent, tm, sp);
}

template <bool PRED>
cudaError_t launch_split(const lr_plan& P, const void* X, const SplitParams& sp, cudaStream_t st, bool bf16 = false,
                         bool dependent = false) {
    CUtensorMap tm;
    cudaError_t e = make_x_tensor_map(X, bf16, sp.m, sp.n, sp.cw, P.rows_per_batch, &tm);
    if (e != cudaSuccess) return e;
    if (bf16) {
        // eight warps per CTA for every bfloat16 shape: 16, 8 or 4 rows per batch with one, two or four groups per lane
        if (P.threads != 256) return cudaErrorInvalidValue;
        if (P.vec_per_lane == 4) return launch_split_t<ElemBF16, 4, 4, PRED, 8>(P, tm, sp, st, dependent);
        if (P.vec_per_lane == 2) return launch_split_t<ElemBF16, 2, 8, PRED, 8>(P, tm, sp, st, dependent);
        return launch_split_t<ElemBF16, 1, 16, PRED, 8>(P, tm, sp, st, dependent);
    }
    if (P.vec_per_lane == 4) return launch_split_t<ElemF32, 4, 2, PRED>(P, tm, sp, st, dependent);
    if (P.vec_per_lane == 2 && P.rows_per_batch == 8) return launch_split_t<ElemF32, 2, 8, PRED>(P, tm, sp, st, dependent);
    if (P.vec_per_lane == 2) return launch_split_t<ElemF32, 2, 4, PRED>(P, tm, sp, st, dependent);
    if (P.rows_per_batch == 16) return launch_split_t<ElemF32, 1, 16, PRED>(P, tm, sp, st, dependent);
    return launch_split_t<ElemF32, 1, 8, PRED>(P, tm, sp, st, dependent);
}

template <class E, int NV, int RB, bool PRED, int NW = kNW>
cudaError_t launch_wide_t(const lr_plan& P, const WideParams& wp, cudaStream_t st, bool dependent) {
    auto kern = k_stream_wide<E, NV, RB, NW, PRED>;
    cudaError_t e = ensure_dynamic_smem<KernelTag<E, NV, -2, RB, NW, PRED>>(reinterpret_cast<const void*>(kern), P.smem_bytes);
    if (e != cudaSuccess) return e;
    return launch_kernel(kern, dim3(P.grid), dim3(P.threads), size_t(P.smem_bytes), st, dependent, wp);
}

template <bool PRED>
cudaError_t launch_wide(const lr_plan& P, const WideParams& wp, cudaStream_t st, bool bf16, bool dependent) {
#define LRGD_WIDE(E, nv, rb) if (P.vec_per_lane == nv && P.rows_per_batch == rb) return launch_wide_t<E, nv, rb, PRED>(P, wp, st, dependent);
    if (P.threads == 256) {                        // rows of 513..1024 elements: eight warps
        if (bf16) return P.vec_per_lane == 3 ? launch_wide_t<ElemBF16Any, 3, 16, PRED, 8>(P, wp, st, dependent)
                                             : launch_wide_t<ElemBF16Any, 4, 16, PRED, 8>(P, wp, st, dependent);
        return P.vec_per_lane == 3 ? launch_wide_t<ElemF32Any, 3, 16, PRED, 8>(P, wp, st, dependent)
                                   : launch_wide_t<ElemF32Any, 4, 16, PRED, 8>(P, wp, st, dependent);
    }
    if (bf16) {
        LRGD_WIDE(ElemBF16Any, 2, 16) LRGD_WIDE(ElemBF16Any, 3, 16) LRGD_WIDE(ElemBF16Any, 4, 8) LRGD_WIDE(ElemBF16Any, 6, 8)
        LRGD_WIDE(ElemBF16Any, 8, 4) LRGD_WIDE(ElemBF16Any, 12, 4) LRGD_WIDE(ElemBF16Any, 16, 2)
        LRGD_WIDE(ElemBF16Any, 24, 1) LRGD_WIDE(ElemBF16Any, 32, 1)
    } else {
        LRGD_WIDE(ElemF32Any, 2, 16) LRGD_WIDE(ElemF32Any, 3, 16) LRGD_WIDE(ElemF32Any, 4, 8) LRGD_WIDE(ElemF32Any, 6, 8)
        LRGD_WIDE(ElemF32Any, 8, 4) LRGD_WIDE(ElemF32Any, 12, 4) LRGD_WIDE(ElemF32Any, 16, 2)
        LRGD_WIDE(ElemF32Any, 24, 1) LRGD_WIDE(ElemF32Any, 32, 1)
    }
#undef LRGD_WIDE
    return cudaErrorInvalidValue;
}

// The persistent whole-fit kernel of a variant-0 plan; resident: every warp's share of X fits its stages, which are then
// filled once and kept for the whole fit.
cudaError_t launch_fit(const lr_plan& P, int smem, bool resident, FitParams& fp, cudaStream_t st, bool bf16 = false) {
    if (P.variant != 0) return cudaErrorInvalidValue;
    return for_row_shape(P, bf16, [&](auto shape) {
        using S = decltype(shape);
        if constexpr (S::Elem::EPG > 1) {
            const void* kern = resident ? reinterpret_cast<const void*>(k_fit_rows<typename S::Elem, S::nv, S::lpr, S::rb, S::nw, true>)
                                        : reinterpret_cast<const void*>(k_fit_rows<typename S::Elem, S::nv, S::lpr, S::rb, S::nw, false>);
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            void* args[] = {&fp};
            return cudaLaunchCooperativeKernel(kern, dim3(P.grid), dim3(P.threads), args, size_t(smem), st);
        } else {
            return cudaErrorInvalidValue;
        }
    });
}

// The same kernel with several ranks of a row-sharded fit as CTA groups of one cooperative launch (lr_fit_sharded_local).
// Built for two shapes only -- fp32 rows of up to 32 and of 132..256 columns -- which is what exercising the exchange needs.
cudaError_t launch_fit_ranks(const lr_plan& P, int smem, bool resident, const FitParams* d_ranks, int world, int ctas_per_rank,
                             cudaStream_t st) {
    if (P.variant != 0) return cudaErrorInvalidValue;
    return for_row_shape(P, false, [&](auto shape) {
        using S = decltype(shape);
        constexpr bool built = std::is_same<typename S::Elem, ElemF32>::value && S::nw == 16 &&
                               ((S::nv == 2 && S::lpr == 32 && S::rb == 4) || (S::nv == 1 && S::lpr == 8 && S::rb == 8));
        if constexpr (built) {
            const void* kern = resident ? reinterpret_cast<const void*>(k_fit_rows_ranks<ElemF32, S::nv, S::lpr, S::rb, S::nw, true>)
                                        : reinterpret_cast<const void*>(k_fit_rows_ranks<ElemF32, S::nv, S::lpr, S::rb, S::nw, false>);
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            void* args[] = {&d_ranks, &ctas_per_rank};
            return cudaLaunchCooperativeKernel(kern, dim3(world * ctas_per_rank), dim3(P.threads), args, size_t(smem), st);
        } else {
            return cudaErrorInvalidValue;
        }
    });
}

// Rows of X to fetch with the evict-last hint.  Defaults: three quarters of the L2 for the wide-row kernel (measured on
// 100k x 4096: 0.260 -> 0.231 ms per pass); a quarter of the L2 for the persistent narrow-row kernel -- the leading rows are
// every warp's first batches of an iteration, so the stream restarts from L2 after each grid barrier (measured per
// iteration with 0 / 32 / 64 MB kept: 1M x 100 62.2 / 60.7 / 60.4 us, 250k x 256 44.3 / 39.8 / 42.1, 125k x 256 25.2 / 22.8 /
// 24.6, 4M x 256 572.3 / - / 566.9); nothing for single narrow-row passes, which measure slower with any part kept.
int64_t keep_rows_for(const lr_ctx* ctx, int variant, int32_t n, bool bf16 = false, bool persistent = false) {
    int64_t bytes = ctx->l2_keep_bytes;
    if (bytes < 0) bytes = variant == 1 ? ctx->l2_bytes / 4 * 3 : (persistent ? ctx->l2_bytes / 4 : 0);
    return bytes / (int64_t(n) * (bf16 ? 2 : 4));
}

// Which form a multi-iteration fit on narrow rows takes.  Measured on B200 (us per iteration, persistent launch against
// two dependent-launched kernels): fp32 300 x 256 4.1 / 5.3, 1k x 256 4.7 / 6.1, 3k x 32 3.6 / 4.5, 10k x 32 4.6 / 4.7,
// 100k x 64 (26 MB, resident in shared memory) 6.7 / 11.5, 28k x 256 (29 MB, resident) 10.5 / 14.5, 32k x 256 12.2 / 15.0,
// 250k x 64 11.9 / 16.1, 125k x 256 24.7 / 26.9, 1M x 100 64.3 / 68.0, 4M x 256 577.9 / 584.4; bfloat16 4M x 256
// 328.5 / 328.6, 16M x 64 323.8 / 337.3.  With one grid barrier per iteration and the reduction done by every CTA for
// itself the persistent kernel is at least as fast everywhere, so it is the default wherever the shape allows it.
bool want_persistent(const lr_ctx* ctx, const lr_plan& P, bool bf16, int64_t m, int32_t n, int64_t iters) {
    (void)bf16; (void)m; (void)n;
    if (P.variant != 0 || !ctx->coop || ctx->prof || ctx->persistent_mode == 0) return false;
    if (iters * P.grid >= (int64_t(1) << 32)) return false;           // the grid-barrier counter is 32 bits
    return true;
}

// Shared-memory shape of the persistent kernel for a plan and a grid of G CTAs: stages per warp, whether every warp's
// share of X stays resident in them, and the dynamic shared memory of a CTA.
struct FitLayout { int depth; bool resident; int smem; };
FitLayout fit_layout(const lr_plan& P, bool bf16, int64_t m, int32_t n, int G) {
    const int nw = P.threads / 32;
    const int64_t stage_stride = (int64_t(P.rows_per_batch) * n * (bf16 ? 2 : 4) + 127) & ~int64_t(127);
    const int64_t tail = fit_tail_bytes(n);
    const int64_t room = kMaxDynamicSmem - kHeaderBytes - tail;
    const int64_t B = (m + P.rows_per_batch - 1) / P.rows_per_batch;
    const int64_t slots = (B + nw - 1) / nw;
    const int64_t per_warp = (slots + G - 1) / G;                              // most batches any warp handles per iteration
    FitLayout L;
    L.depth = int(std::max<int64_t>(1, std::min<int64_t>({int64_t(kMaxDepth), room / (nw * stage_stride), per_warp})));
    L.resident = per_warp <= L.depth;              // every warp's share of X fits its stages: filled once, kept for the fit
    L.smem = int(kHeaderBytes + int64_t(nw) * L.depth * stage_stride + tail);
    return L;
}

struct PersistentTol { TolState* state; double eps; float* gnorm_hist; };
struct PersistentShard {                           // row shards: this rank, the exchange buffers, the bound on waits for peers
    int rank, world; int64_t m_total; uint64_t epoch; uint64_t wait_ns; void* const* xbuf;
};

FitParams fit_params(lr_ctx* ctx, const lr_plan& P, bool bf16, const void* d_X, const float* d_y, int64_t m, int32_t n, float lr,
                     int32_t iters, float* d_w, float* d_b, float* d_loss_hist, int depth, const PersistentTol* tol,
                     const PersistentShard* shard) {
    FitParams fp{};
    fp.X = d_X; fp.y = d_y; fp.m = m; fp.n = n; fp.w = d_w; fp.b = d_b; fp.partial = ctx->d_partial;
    fp.loss_hist = d_loss_hist; fp.status = ctx->d_status; fp.gbar = ctx->d_gbar; fp.depth = depth;
    fp.num_batches = (m + P.rows_per_batch - 1) / P.rows_per_batch;
    fp.iters = iters; fp.lr = double(lr); fp.inv_m = 1.0 / double(shard ? shard->m_total : m);
    fp.keep_rows = keep_rows_for(ctx, 0, n, bf16, true);
    if (tol) { fp.tol = tol->state; fp.eps = tol->eps; fp.gnorm_hist = tol->gnorm_hist; }
    if (shard) {
        fp.rank = shard->rank; fp.world = shard->world; fp.epoch = shard->epoch; fp.wait_ns = shard->wait_ns;
        for (int r = 0; r < shard->world; ++r) fp.xbuf[r] = static_cast<unsigned char*>(shard->xbuf[r]);
    }
    return fp;
}

// Whether a plan is one that make_plan put on a cluster's worth of CTAs (see cluster_size_for): returns the cluster size with
// the layout and the dynamic shared memory of k_fit_cluster, or 0.
int cluster_plan(const lr_plan& P, bool bf16, int64_t m, int32_t n, FitLayout* L, int* smem) {
    if (P.variant != 0) return 0;
    const int nw = P.threads / 32;
    const int64_t stage_stride = (int64_t(P.rows_per_batch) * n * (bf16 ? 2 : 4) + 127) & ~int64_t(127);
    const int64_t B = (m + P.rows_per_batch - 1) / P.rows_per_batch;
    const int C = cluster_size_for((B + nw - 1) / nw, nw, stage_stride, n, P.grid);   // (C <= grid rules out larger clusters than planned)
    if (C == 0 || C != P.grid) return 0;
    *L = fit_layout(P, bf16, m, n, C);
    *smem = cluster_fit_smem(n, nw, L->depth, int(stage_stride), C);
    return L->resident ? C : 0;
}

// Problems whose X fits the shared memory of one thread-block cluster: the whole fit without leaving the cluster (see
// k_fit_cluster).  Returns cudaErrorNotSupported when the problem or the device does not allow it (the caller then takes
// the grid-wide persistent kernel, which gives the same bits on the same plan).
cudaError_t launch_cluster_fit(lr_ctx* ctx, const lr_plan& P, bool bf16, const void* d_X, const float* d_y, int64_t m, int32_t n,
                               float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist, const PersistentTol* tol,
                               cudaStream_t st) {
    if (ctx->cluster_mode == 0 || ctx->persistent_mode != -1) return cudaErrorNotSupported;
    FitLayout L;
    int smem = 0;
    const int C = cluster_plan(P, bf16, m, n, &L, &smem);
    if (C == 0) return cudaErrorNotSupported;
    if (cudaMemsetAsync(ctx->d_gbar, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) {   // [1]: the launch's abort word
        cudaGetLastError();
        return cudaErrorNotSupported;
    }
    const cudaError_t e = for_row_shape(P, bf16, [&](auto shape) {
        using S = decltype(shape);
        if constexpr (S::Elem::EPG > 1) {
            auto kern = k_fit_cluster<typename S::Elem, S::nv, S::lpr, S::rb, S::nw>;
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess && C > 8) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess) return e;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(C);
            cfg.blockDim = dim3(P.threads);
            cfg.dynamicSmemBytes = size_t(smem);
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = unsigned(C);
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            e = cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg);
            if (e != cudaSuccess) return e;
            if (clusters < 1) return cudaErrorNotSupported;   // a cluster of this size cannot be resident here
            ClusterFitParams cp{};
            cp.X = d_X; cp.y = d_y; cp.m = m; cp.n = n; cp.w = d_w; cp.b = d_b; cp.loss_hist = d_loss_hist;
            cp.status = ctx->d_status; cp.depth = L.depth;
            cp.num_batches = (m + P.rows_per_batch - 1) / P.rows_per_batch;
            cp.iters = iters; cp.lr = double(lr); cp.inv_m = 1.0 / double(m);
            cp.abort_word = ctx->d_gbar + 1;
            if (tol) { cp.tol = tol->state; cp.eps = tol->eps; cp.gnorm_hist = tol->gnorm_hist; }
            return cudaLaunchKernelEx(&cfg, kern, cp);
        } else {
            return cudaErrorNotSupported;
        }
    });
    if (e == cudaSuccess) { ctx->launches += 1; return cudaSuccess; }
    cudaGetLastError();
    return cudaErrorNotSupported;
}

// Enqueues the persistent kernel for a whole fit (fixed count, or with the stopping rule when `tol` is given, or as one
// rank of a row-sharded fit when `shard` is given).  Returns cudaErrorCooperativeLaunchTooLarge when the CTAs cannot all
// be resident (the caller then iterates with two kernels), any other error as it comes.
cudaError_t launch_persistent_fit(lr_ctx* ctx, const lr_plan& P, bool bf16, const void* d_X, const float* d_y, int64_t m,
                                  int32_t n, float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist,
                                  const PersistentTol* tol, cudaStream_t st, const PersistentShard* shard = nullptr) {
    const FitLayout L = fit_layout(P, bf16, m, n, P.grid);
    FitParams fp = fit_params(ctx, P, bf16, d_X, d_y, m, n, lr, iters, d_w, d_b, d_loss_hist, L.depth, tol, shard);
    cudaError_t e = cudaMemsetAsync(ctx->d_gbar, 0, 2 * sizeof(unsigned int), st);   // barrier counter and abort flag
    if (e != cudaSuccess) return e;
    e = launch_fit(P, L.smem, L.resident, fp, st, bf16);
    if (e == cudaSuccess) ctx->launches += 1;
    return e;
}

struct Pass {
    const void* X; const float* y; int64_t m; int32_t n; const float* w; const float* b;
    const int* stop = nullptr;                      // device flag that turns the launch into a no-op once set
    bool bf16 = false;                              // X holds bfloat16 elements instead of fp32
    bool dependent = false;                         // the kernel before this one in the stream is this library's own reduction:
                                                    // launch as its programmatic dependent (X is staged while it drains)
};

struct TolArgs {                                    // tolerance mode of the reduction
    TolState* state; double* gbuf; double eps; float* gnorm_out;
};

// Enqueues the streaming kernel for one pass (loss/grad partials, or labels when `labels` is set).
int launch_stream_pass(lr_ctx* ctx, const lr_plan& P, const Pass& a, uint8_t* labels, float cut, cudaStream_t st) {
    const bool predict = labels != nullptr;
    const bool timed = ctx->prof && ctx->prof_used < kMaxProfiled;
    const bool dep = a.dependent && ctx->overlap && !ctx->prof;      // event records between launches would split the pair
    if (timed) {
        while (int(ctx->ev.size()) < 2 * (ctx->prof_used + 1)) {
            cudaEvent_t e;
            LR_CK(ctx, cudaEventCreate(&e));
            ctx->ev.push_back(e);
        }
        LR_CK(ctx, cudaEventRecord(ctx->ev[2 * ctx->prof_used], st));
    }
    cudaError_t e;
    if (P.variant == 0 || P.variant == 3) {
        StreamParams sp{};
        sp.X = a.X; sp.y = a.y; sp.m = a.m; sp.n = a.n; sp.w = a.w; sp.b = a.b;
        sp.partial = ctx->d_partial; sp.labels = labels; sp.cut = cut; sp.status = ctx->d_status; sp.stop = a.stop;
        sp.depth = P.stages;
        sp.num_batches = (a.m + P.rows_per_batch - 1) / P.rows_per_batch;
        sp.keep_rows = keep_rows_for(ctx, 0, a.n, a.bf16);
        e = predict ? launch_rows<true>(P, sp, st, a.bf16, dep) : launch_rows<false>(P, sp, st, a.bf16, dep);
    } else if (P.variant == 1) {
        SplitParams sp{};
        sp.y = a.y; sp.m = a.m; sp.n = a.n; sp.w = a.w; sp.b = a.b;
        sp.partial = ctx->d_partial; sp.labels = labels; sp.cut = cut; sp.status = ctx->d_status; sp.stop = a.stop;
        sp.depth = P.stages;
        sp.cw = (a.n / (a.bf16 ? 8 : 4) + P.threads / 32 - 1) / (P.threads / 32);      // groups per warp slice, as planned
        sp.x_per_group = split_words64(a.bf16, sp.cw) ? 2 : 4;
        sp.num_batches = (a.m + P.rows_per_batch - 1) / P.rows_per_batch;
        sp.keep_rows = keep_rows_for(ctx, 1, a.n, a.bf16);
        e = predict ? launch_split<true>(P, a.X, sp, st, a.bf16, dep) : launch_split<false>(P, a.X, sp, st, a.bf16, dep);
    } else if (P.variant == 4) {
        WideParams wp{};
        wp.X = a.X; wp.y = a.y; wp.m = a.m; wp.n = a.n; wp.w = a.w; wp.b = a.b;
        wp.partial = ctx->d_partial; wp.labels = labels; wp.cut = cut; wp.status = ctx->d_status; wp.stop = a.stop;
        wp.depth = P.stages;
        wp.cw = (a.n + P.threads / 32 - 1) / (P.threads / 32);
        wp.num_batches = (a.m + P.rows_per_batch - 1) / P.rows_per_batch;
        wp.keep_rows = keep_rows_for(ctx, 1, a.n, a.bf16);
        e = predict ? launch_wide<true>(P, wp, st, a.bf16, dep) : launch_wide<false>(P, wp, st, a.bf16, dep);
    } else {
        GenericParams gp{};
        gp.X = a.X; gp.y = a.y; gp.m = a.m; gp.n = a.n; gp.w = a.w; gp.b = a.b;
        gp.partial = ctx->d_partial; gp.labels = labels; gp.cut = cut; gp.stop = a.stop; gp.rows = P.tile_rows;
        const dim3 g(P.grid), t(P.threads);
        if (a.bf16) e = predict ? launch_kernel(k_generic<ElemBF16, true>, g, t, 0, st, dep, gp)
                                : launch_kernel(k_generic<ElemBF16, false>, g, t, 0, st, dep, gp);
        else e = predict ? launch_kernel(k_generic<ElemF32, true>, g, t, 0, st, dep, gp)
                         : launch_kernel(k_generic<ElemF32, false>, g, t, 0, st, dep, gp);
    }
    LR_CK(ctx, e);
    ctx->launches += 1;
    if (timed) {
        LR_CK(ctx, cudaEventRecord(ctx->ev[2 * ctx->prof_used + 1], st));
        ctx->prof_used += 1;
    }
    return LR_OK;
}

int launch_reduce(lr_ctx* ctx, const double* partial, int G, int64_t m, int32_t n, double lr, bool update, float* w,
                  float* b, float* grad_w, float* grad_b, float* loss_out, double* raw_sums, cudaStream_t st,
                  const TolArgs* tol = nullptr) {
    ReduceParams rp{};
    rp.partial = partial; rp.G = G; rp.n = n; rp.inv_m = 1.0 / double(m); rp.lr = lr;
    rp.update = update ? 1 : 0; rp.w = w; rp.b = b; rp.grad_w = grad_w; rp.grad_b = grad_b; rp.loss_out = loss_out;
    rp.raw_sums = raw_sums;
    if (tol) { rp.tol = tol->state; rp.gbuf = tol->gbuf; rp.eps = tol->eps; rp.gnorm_out = tol->gnorm_out; }
    // always preceded in the stream by the pass that wrote `partial` (or, for lr_apply_sums, by whatever the caller ran:
    // the kernel waits for it on the device either way), so it is launched as that kernel's programmatic dependent
    LR_CK(ctx, launch_kernel(k_reduce_update, dim3((n + 2 + 31) / 32), dim3(32, kRedSlices), 0, st,
                             ctx->overlap && !ctx->prof, rp));
    ctx->launches += 1;
    return LR_OK;
}

int check_common(lr_ctx* ctx, const void* X, int64_t m, int32_t n, const void* w, const void* b, bool bf16 = false) {
    if (!ctx || !X || !w || !b) return LR_ERR_NULL;
    if (m < 1 || m > kMaxRows || n < 1 || n > ctx->n_max) return LR_ERR_SHAPE;
    if (!aligned(X, bf16 ? 2 : 4) || !aligned(w, 4) || !aligned(b, 4)) return LR_ERR_ALIGNMENT;
    return LR_OK;
}

int grow(lr_ctx* ctx, void** buf, size_t* have, size_t need) {
    if (*have >= need) return LR_OK;
    if (*buf) { LR_CK(ctx, cudaFree(*buf)); *buf = nullptr; *have = 0; }
    cudaError_t e = cudaMalloc(buf, need);
    if (e != cudaSuccess) { ctx->last_cuda = int(e); *buf = nullptr; return e == cudaErrorMemoryAllocation ? LR_ERR_NOMEM : LR_ERR_CUDA; }
    *have = need;
    return LR_OK;
}

int loss_grad_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, const float* d_w,
                   const float* d_b, float* d_loss, float* d_grad_w, float* d_grad_b, void* stream);
int fit_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
             float* d_w, float* d_b, float* d_loss_hist, void* stream);
int predict_impl(lr_ctx* ctx, const void* d_X, bool bf16, int64_t m, int32_t n, const float* d_w, const float* d_b, float thr,
                 uint8_t* d_labels, void* stream);

}  // namespace

extern "C" {

int lr_plan_query_bf16(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, lr_plan* out) {
    if (!out) return LR_ERR_NULL;
    return make_plan(m, n, x_aligned16 != 0, sm_count, out, true);
}

int lr_plan_query(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, lr_plan* out) {
    if (!out) return LR_ERR_NULL;
    return make_plan(m, n, x_aligned16 != 0, sm_count, out);
}

int lr_create(lr_ctx** out, int32_t device, int32_t n_max) {
    if (!out) return LR_ERR_NULL;
    *out = nullptr;
    if (n_max < 1) return LR_ERR_SHAPE;
    lr_ctx* c = new (std::nothrow) lr_ctx();
    if (!c) return LR_ERR_NOMEM;
    c->device = device;
    c->n_max = n_max;
    int prev = -1;
    cudaGetDevice(&prev);
    int rc = LR_OK;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) {
        const size_t bytes = size_t(c->sm_count) * kMaxGridPerSm * (size_t(n_max) + 2) * sizeof(double);
        e = guarded_alloc(c, &c->d_partial, bytes);
        if (e == cudaErrorMemoryAllocation) rc = LR_ERR_NOMEM;
    }
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&c->d_status), sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&c->d_tol), sizeof(TolState));
    if (e == cudaSuccess) e = cudaMemset(c->d_tol, 0, sizeof(TolState));
    if (e == cudaSuccess) e = guarded_alloc(c, &c->d_gbuf, (size_t(n_max) + 1) * sizeof(double));
    if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&c->h_tol), sizeof(TolState));
    if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&c->h_words), 4 * sizeof(int));
    if (e == cudaSuccess) e = guarded_alloc(c, &c->d_vel, (size_t(n_max) + 1) * sizeof(float));
    if (e == cudaSuccess) e = guarded_alloc(c, &c->d_oscr, (size_t(n_max) + 2) * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&c->d_oticket), sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(c->d_oticket, 0, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&c->d_gbar), 2 * kMaxWorld * sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&c->d_rank_params), kMaxWorld * sizeof(FitParams));
    if (e == cudaSuccess) {
        int l2 = 0;
        e = cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device);
        c->l2_bytes = l2;
    }
    if (e == cudaSuccess) {
        int coop = 0;
        e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device);
        c->coop = coop != 0;
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->hstream, cudaStreamNonBlocking);
    if (prev >= 0) cudaSetDevice(prev);
    if (e != cudaSuccess) {
        for (unsigned char* base : c->guard_bases) cudaFree(base);     // d_partial, d_gbuf, d_vel, d_oscr
        if (c->d_status) cudaFree(c->d_status);
        if (c->d_tol) cudaFree(c->d_tol);
        if (c->h_tol) cudaFreeHost(c->h_tol);
        if (c->h_words) cudaFreeHost(c->h_words);
        if (c->d_oticket) cudaFree(c->d_oticket);
        if (c->d_gbar) cudaFree(c->d_gbar);
        if (c->d_rank_params) cudaFree(c->d_rank_params);
        delete c;
        return rc != LR_OK ? rc : LR_ERR_CUDA;
    }
    *out = c;
    return LR_OK;
}

int lr_destroy(lr_ctx* ctx) {
    if (!ctx) return LR_OK;
    {
        DeviceGuard g(ctx);
        cudaDeviceSynchronize();
        for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
        if (ctx->hstream) cudaStreamDestroy(ctx->hstream);
        for (unsigned char* base : ctx->guard_bases) cudaFree(base);   // d_partial, d_gbuf, d_vel, d_oscr
        cudaFree(ctx->d_status);
        cudaFree(ctx->d_tol);
        if (ctx->h_tol) cudaFreeHost(ctx->h_tol);
        if (ctx->h_words) cudaFreeHost(ctx->h_words);
        cudaFree(ctx->d_oticket);
        cudaFree(ctx->d_gbar);
        cudaFree(ctx->d_rank_params);
        cudaFree(ctx->d_hX);
        cudaFree(ctx->d_hy);
        cudaFree(ctx->d_hw);
        cudaFree(ctx->d_hl);
        cudaFree(ctx->d_hXh);
    }
    delete ctx;
    return LR_OK;
}

int lr_loss_grad(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n, const float* d_w,
                 const float* d_b, float* d_loss, float* d_grad_w, float* d_grad_b, void* stream) {
    return loss_grad_impl(ctx, d_X, false, d_y, m, n, d_w, d_b, d_loss, d_grad_w, d_grad_b, stream);
}

int lr_loss_grad_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n, const float* d_w,
                      const float* d_b, float* d_loss, float* d_grad_w, float* d_grad_b, void* stream) {
    return loss_grad_impl(ctx, d_Xh, true, d_y, m, n, d_w, d_b, d_loss, d_grad_w, d_grad_b, stream);
}

int lr_fit(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
           float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    return fit_impl(ctx, d_X, false, d_y, m, n, lr, iters, d_w, d_b, d_loss_hist, stream);
}

int lr_fit_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
                float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    return fit_impl(ctx, d_Xh, true, d_y, m, n, lr, iters, d_w, d_b, d_loss_hist, stream);
}

int lr_predict(lr_ctx* ctx, const float* d_X, int64_t m, int32_t n, const float* d_w, const float* d_b, float thr,
               uint8_t* d_labels, void* stream) {
    return predict_impl(ctx, d_X, false, m, n, d_w, d_b, thr, d_labels, stream);
}

int lr_predict_bf16(lr_ctx* ctx, const uint16_t* d_Xh, int64_t m, int32_t n, const float* d_w, const float* d_b, float thr,
                    uint8_t* d_labels, void* stream) {
    return predict_impl(ctx, d_Xh, true, m, n, d_w, d_b, thr, d_labels, stream);
}

int lr_f1_counts(lr_ctx* ctx, const uint8_t* d_labels, const float* d_y, int64_t m, int64_t* d_counts, void* stream) {
    if (!ctx) return LR_ERR_NULL;
    if (m < 0 || m > kMaxRows) return LR_ERR_SHAPE;
    if (!d_counts || (m > 0 && (!d_labels || !d_y))) return LR_ERR_NULL;
    if (!aligned(d_counts, 8) || (m > 0 && !aligned(d_y, 4))) return LR_ERR_ALIGNMENT;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LR_CK(ctx, cudaMemsetAsync(d_counts, 0, 3 * sizeof(int64_t), st));
    if (m == 0) return LR_OK;
    const bool vec = aligned(d_labels, 16) && aligned(d_y, 16);
    const int64_t units = vec ? (m + 15) / 16 : m;
    const int grid = int(std::max<int64_t>(1, std::min<int64_t>((units + kScoreThreads - 1) / kScoreThreads, int64_t(ctx->sm_count) * 8)));
    k_confusion<<<grid, kScoreThreads, 0, st>>>(d_labels, d_y, m, reinterpret_cast<unsigned long long*>(d_counts), vec ? 1 : 0);
    LR_CK(ctx, cudaGetLastError());
    ctx->launches += 1;
    return LR_OK;
}

int lr_convert_bf16(lr_ctx* ctx, const float* d_X, int64_t count, uint16_t* d_Xh, void* stream) {
    if (!ctx) return LR_ERR_NULL;
    if (count < 0) return LR_ERR_SHAPE;
    if (count == 0) return LR_OK;                  // nothing to do; the pointers are not looked at
    if (!d_X || !d_Xh) return LR_ERR_NULL;
    if (!aligned(d_X, 4) || !aligned(d_Xh, 2)) return LR_ERR_ALIGNMENT;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    const bool vec = aligned(d_X, 16) && aligned(d_Xh, 8);
    const int64_t units = vec ? (count + 3) / 4 : count;
    const int grid = int(std::min<int64_t>((units + kConvertThreads - 1) / kConvertThreads, int64_t(ctx->sm_count) * 16));
    k_convert_bf16<<<grid, kConvertThreads, 0, static_cast<cudaStream_t>(stream)>>>(d_X, count, d_Xh, vec ? 1 : 0);
    LR_CK(ctx, cudaGetLastError());
    ctx->launches += 1;
    return LR_OK;
}

}  // extern "C"

namespace {

int loss_grad_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, const float* d_w,
                   const float* d_b, float* d_loss, float* d_grad_w, float* d_grad_b, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y || !d_loss || !d_grad_w || !d_grad_b) return LR_ERR_NULL;
    if (!aligned(d_y, 4) || !aligned(d_loss, 4) || !aligned(d_grad_w, 4) || !aligned(d_grad_b, 4)) return LR_ERR_ALIGNMENT;
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Pass pass{d_X, d_y, m, n, d_w, d_b};
    pass.bf16 = bf16;
    rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
    if (rc != LR_OK) return rc;
    return launch_reduce(ctx, ctx->d_partial, P.grid, m, n, 0.0, false, nullptr, nullptr, d_grad_w, d_grad_b, d_loss,
                         nullptr, st);
}

int fit_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
             float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y) return LR_ERR_NULL;
    if (iters < 0) return LR_ERR_SHAPE;
    if (!aligned(d_y, 4) || (d_loss_hist && !aligned(d_loss_hist, 4))) return LR_ERR_ALIGNMENT;
    if (!std::isfinite(lr)) return LR_ERR_VALUE;
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    if (iters == 0) return LR_OK;
    NvtxRange range(bf16 ? "lr_fit_bf16" : "lr_fit");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Narrow rows, several iterations: one cooperative launch runs the whole fit (same bits as the loop below).
    if (iters >= 2 && want_persistent(ctx, P, bf16, m, n, iters)) {
        if (launch_cluster_fit(ctx, P, bf16, d_X, d_y, m, n, lr, iters, d_w, d_b, d_loss_hist, nullptr, st) == cudaSuccess) return LR_OK;
        const cudaError_t le = launch_persistent_fit(ctx, P, bf16, d_X, d_y, m, n, lr, iters, d_w, d_b, d_loss_hist, nullptr, st);
        if (le == cudaSuccess) return LR_OK;
        if (le != cudaErrorCooperativeLaunchTooLarge) { ctx->last_cuda = int(le); return LR_ERR_CUDA; }
        cudaGetLastError();                        // the CTAs cannot all be resident here: use the two-kernel form below
    }
    Pass pass{d_X, d_y, m, n, d_w, d_b};
    pass.bf16 = bf16;
    for (int32_t t = 0; t < iters; ++t) {
        pass.dependent = t > 0;                    // follows this call's own reduction
        rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
        if (rc != LR_OK) return rc;
        rc = launch_reduce(ctx, ctx->d_partial, P.grid, m, n, double(lr), true, d_w, d_b, nullptr, nullptr,
                           d_loss_hist ? d_loss_hist + t : nullptr, nullptr, st);
        if (rc != LR_OK) return rc;
    }
    return LR_OK;
}

int predict_impl(lr_ctx* ctx, const void* d_X, bool bf16, int64_t m, int32_t n, const float* d_w, const float* d_b, float thr,
                 uint8_t* d_labels, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_labels) return LR_ERR_NULL;
    if (!(thr > 0.f && thr < 1.f)) return LR_ERR_VALUE;
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    const float cut = static_cast<float>(std::log(double(thr) / (1.0 - double(thr))));
    Pass pass{d_X, nullptr, m, n, d_w, d_b};
    pass.bf16 = bf16;
    return launch_stream_pass(ctx, P, pass, d_labels, cut, static_cast<cudaStream_t>(stream));
}

}  // namespace

extern "C" {

int lr_set_l2_keep(lr_ctx* ctx, int64_t bytes) {
    if (!ctx) return LR_ERR_NULL;
    if (bytes < -1) return LR_ERR_VALUE;
    ctx->l2_keep_bytes = bytes;
    return LR_OK;
}

int lr_set_overlap(lr_ctx* ctx, int32_t on) {
    if (!ctx) return LR_ERR_NULL;
    ctx->overlap = on != 0;
    return LR_OK;
}

int lr_set_persistent(lr_ctx* ctx, int32_t on) {
    if (!ctx) return LR_ERR_NULL;
    ctx->persistent_mode = on < 0 ? -1 : (on > 0 ? 1 : 0);
    return LR_OK;
}

int32_t lr_cluster_ctas(int64_t m, int32_t n, int32_t x_aligned16, int32_t sm_count, int32_t bf16) {
    lr_plan P;
    FitLayout L;
    int smem = 0;
    if (make_plan(m, n, x_aligned16 != 0, sm_count, &P, bf16 != 0) != LR_OK) return 0;
    return cluster_plan(P, bf16 != 0, m, n, &L, &smem);
}

int lr_set_cluster(lr_ctx* ctx, int32_t on) {
    if (!ctx) return LR_ERR_NULL;
    ctx->cluster_mode = on == 0 ? 0 : -1;
    return LR_OK;
}

}  // extern "C"

namespace {

int fit_tol_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, float lr, float eps,
                 int32_t max_iters, int32_t check_every, float* d_w, float* d_b, float* d_loss_hist, float* d_gnorm_hist,
                 int32_t* iters_done, float* grad_norm, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y || !iters_done || !grad_norm) return LR_ERR_NULL;
    if (max_iters < 0 || check_every < 1) return LR_ERR_SHAPE;
    if (!aligned(d_y, 4) || (d_loss_hist && !aligned(d_loss_hist, 4)) || (d_gnorm_hist && !aligned(d_gnorm_hist, 4)))
        return LR_ERR_ALIGNMENT;
    if (!std::isfinite(lr) || !(eps >= 0.f) || !std::isfinite(eps)) return LR_ERR_VALUE;
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    *iters_done = 0;
    *grad_norm = -1.f;
    if (max_iters == 0) return LR_OK;
    NvtxRange range(bf16 ? "lr_fit_tol_bf16" : "lr_fit_tol");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LR_CK(ctx, cudaMemsetAsync(ctx->d_tol, 0, sizeof(TolState), st));
    // the status word before this call's kernels, so that a give-up during the call can be told from an older, unread one
    LR_CK(ctx, cudaMemcpyAsync(&ctx->h_words[0], ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    // Narrow rows: one persistent launch that leaves its loop on the device as soon as the norm is small enough.
    if (want_persistent(ctx, P, bf16, m, n, max_iters)) {
        const PersistentTol pt{ctx->d_tol, double(eps), d_gnorm_hist};
        // (a problem that fits one thread-block cluster runs there; otherwise, or if the device refuses, the grid-wide kernel)
        cudaError_t le = launch_cluster_fit(ctx, P, bf16, d_X, d_y, m, n, lr, max_iters, d_w, d_b, d_loss_hist, &pt, st);
        if (le != cudaSuccess) le = launch_persistent_fit(ctx, P, bf16, d_X, d_y, m, n, lr, max_iters, d_w, d_b, d_loss_hist, &pt, st);
        if (le == cudaSuccess) {
            LR_CK(ctx, cudaMemcpyAsync(ctx->h_tol, ctx->d_tol, sizeof(TolState), cudaMemcpyDeviceToHost, st));
            LR_CK(ctx, cudaMemcpyAsync(&ctx->h_words[2], ctx->d_gbar + 1, sizeof(int), cudaMemcpyDeviceToHost, st));
            LR_CK(ctx, cudaStreamSynchronize(st));
            *iters_done = ctx->h_tol->iters_done;
            *grad_norm = static_cast<float>(ctx->h_tol->grad_norm);
            return ctx->h_words[2] != 0 ? LR_ERR_TIMEOUT : LR_OK;     // the launch's own abort flag: a bounded wait expired
        }
        if (le != cudaErrorCooperativeLaunchTooLarge) { ctx->last_cuda = int(le); return LR_ERR_CUDA; }
        cudaGetLastError();
    }
    const int* stop = &ctx->d_tol->stop;
    for (int32_t t = 0; t < max_iters;) {
        const int32_t chunk = std::min(check_every, max_iters - t);
        for (int32_t k = 0; k < chunk; ++k, ++t) {
            Pass pass{d_X, d_y, m, n, d_w, d_b};
            pass.stop = stop;
            pass.bf16 = bf16;
            pass.dependent = k > 0;                // within a chunk it follows this call's own reduction
            rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
            if (rc != LR_OK) return rc;
            TolArgs ta{ctx->d_tol, ctx->d_gbuf, double(eps), d_gnorm_hist ? d_gnorm_hist + t : nullptr};
            rc = launch_reduce(ctx, ctx->d_partial, P.grid, m, n, double(lr), true, d_w, d_b, nullptr, nullptr,
                               d_loss_hist ? d_loss_hist + t : nullptr, nullptr, st, &ta);
            if (rc != LR_OK) return rc;
        }
        LR_CK(ctx, cudaMemcpyAsync(ctx->h_tol, ctx->d_tol, sizeof(TolState), cudaMemcpyDeviceToHost, st));
        LR_CK(ctx, cudaMemcpyAsync(&ctx->h_words[1], ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
        LR_CK(ctx, cudaStreamSynchronize(st));
        if (ctx->h_words[1] != 0 && ctx->h_words[0] == 0) {           // a bounded wait expired in one of this call's kernels
            *iters_done = ctx->h_tol->iters_done;
            *grad_norm = static_cast<float>(ctx->h_tol->grad_norm);
            return LR_ERR_TIMEOUT;
        }
        if (ctx->h_tol->stop) break;
    }
    *iters_done = ctx->h_tol->iters_done;
    *grad_norm = static_cast<float>(ctx->h_tol->grad_norm);
    return LR_OK;
}

int fit_opt_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
                 const lr_opt* opt, float* d_w, float* d_b, float* d_velocity, float* d_loss_hist, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y || !opt) return LR_ERR_NULL;
    if (iters < 0) return LR_ERR_SHAPE;
    if (!aligned(d_y, 4) || (d_loss_hist && !aligned(d_loss_hist, 4)) || (d_velocity && !aligned(d_velocity, 4)))
        return LR_ERR_ALIGNMENT;
    if (!std::isfinite(lr) || !(opt->l2 >= 0.f) || !std::isfinite(opt->l2) || !(opt->momentum >= 0.f && opt->momentum < 1.f))
        return LR_ERR_VALUE;
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    if (iters == 0) return LR_OK;
    NvtxRange range(bf16 ? "lr_fit_opt_bf16" : "lr_fit_opt");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* vel = d_velocity;
    if (!vel) {
        vel = ctx->d_vel;
        LR_CK(ctx, cudaMemsetAsync(vel, 0, (size_t(n) + 1) * sizeof(float), st));
    }
    Pass pass{d_X, d_y, m, n, d_w, d_b};
    pass.bf16 = bf16;
    for (int32_t t = 0; t < iters; ++t) {
        pass.dependent = t > 0;                    // follows this call's own reduction
        rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
        if (rc != LR_OK) return rc;
        OptParams op{};
        op.partial = ctx->d_partial; op.G = P.grid; op.n = n; op.inv_m = 1.0 / double(m); op.lr = double(lr);
        op.l2 = double(opt->l2); op.mu = double(opt->momentum); op.nesterov = opt->nesterov ? 1 : 0;
        op.w = d_w; op.b = d_b; op.vel = vel; op.loss_out = d_loss_hist ? d_loss_hist + t : nullptr;
        op.scratch = ctx->d_oscr; op.ticket = ctx->d_oticket;
        LR_CK(ctx, launch_kernel(k_reduce_opt, dim3((n + 2 + 31) / 32), dim3(32, kRedSlices), 0, st,
                                 ctx->overlap && !ctx->prof, op));
        ctx->launches += 1;
    }
    return LR_OK;
}

int fit_sgd_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m, int32_t n, float lr, int64_t batch_rows,
                 int32_t steps, int64_t first_batch, float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    int rc = check_common(ctx, d_X, m, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y) return LR_ERR_NULL;
    if (steps < 0 || batch_rows < 1 || batch_rows > m || first_batch < 0) return LR_ERR_SHAPE;
    if (!aligned(d_y, 4) || (d_loss_hist && !aligned(d_loss_hist, 4))) return LR_ERR_ALIGNMENT;
    if (!std::isfinite(lr)) return LR_ERR_VALUE;
    if (steps == 0) return LR_OK;
    NvtxRange range(bf16 ? "lr_fit_sgd_bf16" : "lr_fit_sgd");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t nb = (m + batch_rows - 1) / batch_rows;
    for (int32_t s = 0; s < steps; ++s) {
        const int64_t k = (first_batch + s) % nb;
        const int64_t r0 = k * batch_rows;
        const int64_t rows = std::min(batch_rows, m - r0);
        const void* Xb = static_cast<const unsigned char*>(d_X) + size_t(r0) * n * (bf16 ? 2 : 4);
        lr_plan P;
        rc = make_plan(rows, n, aligned(Xb, 16), plan_sms(ctx), &P, bf16);
        if (rc != LR_OK) return rc;
        Pass pass{Xb, d_y + r0, rows, n, d_w, d_b};
        pass.bf16 = bf16;
        pass.dependent = s > 0;                    // follows this call's own reduction
        rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
        if (rc != LR_OK) return rc;
        rc = launch_reduce(ctx, ctx->d_partial, P.grid, rows, n, double(lr), true, d_w, d_b, nullptr, nullptr,
                           d_loss_hist ? d_loss_hist + s : nullptr, nullptr, st);
        if (rc != LR_OK) return rc;
    }
    return LR_OK;
}

int shard_sums_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m_local, int32_t n, const float* d_w,
                    const float* d_b, double* d_sums, void* stream) {
    int rc = check_common(ctx, d_X, m_local, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y || !d_sums) return LR_ERR_NULL;
    if (!aligned(d_y, 4) || !aligned(d_sums, 8)) return LR_ERR_ALIGNMENT;
    lr_plan P;
    rc = make_plan(m_local, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Pass pass{d_X, d_y, m_local, n, d_w, d_b};
    pass.bf16 = bf16;
    rc = launch_stream_pass(ctx, P, pass, nullptr, 0.f, st);
    if (rc != LR_OK) return rc;
    return launch_reduce(ctx, ctx->d_partial, P.grid, m_local, n, 0.0, false, nullptr, nullptr, nullptr, nullptr, nullptr,
                         d_sums, st);
}

// Host-pointer fits and predictions: copy in, run the device entry points on the context's own stream, copy out.
// store_bf16: X arrives as fp32 and is rounded to bfloat16 on the device right after the copy (lr_convert_bf16); the
// bfloat16 entry points then stream half the bytes per pass.
int stage_host_x(lr_ctx* ctx, const float* h_X, int64_t m, int32_t n, bool store_bf16, cudaStream_t st, const void** d_X) {
    const size_t xb = size_t(m) * n * 4;
    int rc;
    if ((rc = grow(ctx, &ctx->d_hX, &ctx->hX_bytes, xb)) != LR_OK) return rc;
    LR_CK(ctx, cudaMemcpyAsync(ctx->d_hX, h_X, xb, cudaMemcpyHostToDevice, st));
    *d_X = ctx->d_hX;
    if (store_bf16) {
        if ((rc = grow(ctx, &ctx->d_hXh, &ctx->hXh_bytes, xb / 2)) != LR_OK) return rc;
        rc = lr_convert_bf16(ctx, static_cast<const float*>(ctx->d_hX), m * n, static_cast<uint16_t*>(ctx->d_hXh), st);
        if (rc != LR_OK) return rc;
        *d_X = ctx->d_hXh;
    }
    return LR_OK;
}

int fit_host_impl(lr_ctx* ctx, const float* h_X, bool store_bf16, const float* h_y, int64_t m, int32_t n, float lr, int32_t iters,
                  float* h_w, float* h_b, float* h_loss_hist) {
    int rc = check_common(ctx, h_X, m, n, h_w, h_b);
    if (rc != LR_OK) return rc;
    if (!h_y) return LR_ERR_NULL;
    if (iters < 0) return LR_ERR_SHAPE;
    if (!std::isfinite(lr)) return LR_ERR_VALUE;
    NvtxRange range(store_bf16 ? "lr_fit_host_bf16" : "lr_fit_host");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    const size_t yb = size_t(m) * 4;
    const size_t wb = (size_t(n) + 1 + size_t(iters)) * 4;
    if ((rc = grow(ctx, &ctx->d_hy, &ctx->hy_bytes, yb)) != LR_OK) return rc;
    if ((rc = grow(ctx, &ctx->d_hw, &ctx->hw_bytes, wb)) != LR_OK) return rc;
    float* dy = static_cast<float*>(ctx->d_hy);
    float* dw = static_cast<float*>(ctx->d_hw);
    float* db = dw + n;
    float* dh = db + 1;
    cudaStream_t st = ctx->hstream;
    const void* dX = nullptr;
    if ((rc = stage_host_x(ctx, h_X, m, n, store_bf16, st, &dX)) != LR_OK) return rc;
    LR_CK(ctx, cudaMemcpyAsync(dy, h_y, yb, cudaMemcpyHostToDevice, st));
    LR_CK(ctx, cudaMemcpyAsync(dw, h_w, size_t(n) * 4, cudaMemcpyHostToDevice, st));
    LR_CK(ctx, cudaMemcpyAsync(db, h_b, 4, cudaMemcpyHostToDevice, st));
    rc = fit_impl(ctx, dX, store_bf16, dy, m, n, lr, iters, dw, db, h_loss_hist ? dh : nullptr, st);
    if (rc != LR_OK) return rc;
    LR_CK(ctx, cudaMemcpyAsync(h_w, dw, size_t(n) * 4, cudaMemcpyDeviceToHost, st));
    LR_CK(ctx, cudaMemcpyAsync(h_b, db, 4, cudaMemcpyDeviceToHost, st));
    if (h_loss_hist && iters > 0) LR_CK(ctx, cudaMemcpyAsync(h_loss_hist, dh, size_t(iters) * 4, cudaMemcpyDeviceToHost, st));
    LR_CK(ctx, cudaStreamSynchronize(st));
    return LR_OK;
}

int predict_host_impl(lr_ctx* ctx, const float* h_X, bool store_bf16, int64_t m, int32_t n, const float* h_w, const float* h_b,
                      float thr, uint8_t* h_labels) {
    int rc = check_common(ctx, h_X, m, n, h_w, h_b);
    if (rc != LR_OK) return rc;
    if (!h_labels) return LR_ERR_NULL;
    if (!(thr > 0.f && thr < 1.f)) return LR_ERR_VALUE;
    NvtxRange range(store_bf16 ? "lr_predict_host_bf16" : "lr_predict_host");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    if ((rc = grow(ctx, &ctx->d_hw, &ctx->hw_bytes, (size_t(n) + 1) * 4)) != LR_OK) return rc;
    if ((rc = grow(ctx, &ctx->d_hl, &ctx->hl_bytes, size_t(m))) != LR_OK) return rc;
    float* dw = static_cast<float*>(ctx->d_hw);
    float* db = dw + n;
    uint8_t* dl = static_cast<uint8_t*>(ctx->d_hl);
    cudaStream_t st = ctx->hstream;
    const void* dX = nullptr;
    if ((rc = stage_host_x(ctx, h_X, m, n, store_bf16, st, &dX)) != LR_OK) return rc;
    LR_CK(ctx, cudaMemcpyAsync(dw, h_w, size_t(n) * 4, cudaMemcpyHostToDevice, st));
    LR_CK(ctx, cudaMemcpyAsync(db, h_b, 4, cudaMemcpyHostToDevice, st));
    rc = predict_impl(ctx, dX, store_bf16, m, n, dw, db, thr, dl, st);
    if (rc != LR_OK) return rc;
    LR_CK(ctx, cudaMemcpyAsync(h_labels, dl, size_t(m), cudaMemcpyDeviceToHost, st));
    LR_CK(ctx, cudaStreamSynchronize(st));
    return LR_OK;
}

}  // namespace

extern "C" {

int lr_fit_tol(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n, float lr, float eps,
               int32_t max_iters, int32_t check_every, float* d_w, float* d_b, float* d_loss_hist, float* d_gnorm_hist,
               int32_t* iters_done, float* grad_norm, void* stream) {
    return fit_tol_impl(ctx, d_X, false, d_y, m, n, lr, eps, max_iters, check_every, d_w, d_b, d_loss_hist, d_gnorm_hist,
                        iters_done, grad_norm, stream);
}

int lr_fit_tol_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n, float lr, float eps,
                    int32_t max_iters, int32_t check_every, float* d_w, float* d_b, float* d_loss_hist, float* d_gnorm_hist,
                    int32_t* iters_done, float* grad_norm, void* stream) {
    return fit_tol_impl(ctx, d_Xh, true, d_y, m, n, lr, eps, max_iters, check_every, d_w, d_b, d_loss_hist, d_gnorm_hist,
                        iters_done, grad_norm, stream);
}

int lr_fit_opt(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
               const lr_opt* opt, float* d_w, float* d_b, float* d_velocity, float* d_loss_hist, void* stream) {
    return fit_opt_impl(ctx, d_X, false, d_y, m, n, lr, iters, opt, d_w, d_b, d_velocity, d_loss_hist, stream);
}

int lr_fit_opt_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n, float lr, int32_t iters,
                    const lr_opt* opt, float* d_w, float* d_b, float* d_velocity, float* d_loss_hist, void* stream) {
    return fit_opt_impl(ctx, d_Xh, true, d_y, m, n, lr, iters, opt, d_w, d_b, d_velocity, d_loss_hist, stream);
}

int lr_fit_sgd(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m, int32_t n, float lr, int64_t batch_rows,
               int32_t steps, int64_t first_batch, float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    return fit_sgd_impl(ctx, d_X, false, d_y, m, n, lr, batch_rows, steps, first_batch, d_w, d_b, d_loss_hist, stream);
}

int lr_fit_sgd_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m, int32_t n, float lr, int64_t batch_rows,
                    int32_t steps, int64_t first_batch, float* d_w, float* d_b, float* d_loss_hist, void* stream) {
    return fit_sgd_impl(ctx, d_Xh, true, d_y, m, n, lr, batch_rows, steps, first_batch, d_w, d_b, d_loss_hist, stream);
}

int lr_shard_sums(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m_local, int32_t n, const float* d_w,
                  const float* d_b, double* d_sums, void* stream) {
    return shard_sums_impl(ctx, d_X, false, d_y, m_local, n, d_w, d_b, d_sums, stream);
}

int lr_shard_sums_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m_local, int32_t n, const float* d_w,
                       const float* d_b, double* d_sums, void* stream) {
    return shard_sums_impl(ctx, d_Xh, true, d_y, m_local, n, d_w, d_b, d_sums, stream);
}

int lr_apply_sums(lr_ctx* ctx, const double* d_sums_all, int32_t parts, int64_t m_total, int32_t n, float lr, float* d_w,
                  float* d_b, float* d_loss, void* stream) {
    if (!ctx || !d_sums_all || !d_w || !d_b) return LR_ERR_NULL;
    if (parts < 1 || m_total < 1 || n < 1 || n > ctx->n_max) return LR_ERR_SHAPE;
    if (!aligned(d_sums_all, 8) || !aligned(d_w, 4) || !aligned(d_b, 4) || (d_loss && !aligned(d_loss, 4))) return LR_ERR_ALIGNMENT;
    if (!std::isfinite(lr)) return LR_ERR_VALUE;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    return launch_reduce(ctx, d_sums_all, parts, m_total, n, double(lr), true, d_w, d_b, nullptr, nullptr, d_loss, nullptr,
                         static_cast<cudaStream_t>(stream));
}

int lr_fit_host(lr_ctx* ctx, const float* h_X, const float* h_y, int64_t m, int32_t n, float lr, int32_t iters,
                float* h_w, float* h_b, float* h_loss_hist) {
    return fit_host_impl(ctx, h_X, false, h_y, m, n, lr, iters, h_w, h_b, h_loss_hist);
}

int lr_fit_host_bf16(lr_ctx* ctx, const float* h_X, const float* h_y, int64_t m, int32_t n, float lr, int32_t iters,
                     float* h_w, float* h_b, float* h_loss_hist) {
    return fit_host_impl(ctx, h_X, true, h_y, m, n, lr, iters, h_w, h_b, h_loss_hist);
}

int lr_predict_host(lr_ctx* ctx, const float* h_X, int64_t m, int32_t n, const float* h_w, const float* h_b, float thr,
                    uint8_t* h_labels) {
    return predict_host_impl(ctx, h_X, false, m, n, h_w, h_b, thr, h_labels);
}

int lr_predict_host_bf16(lr_ctx* ctx, const float* h_X, int64_t m, int32_t n, const float* h_w, const float* h_b, float thr,
                         uint8_t* h_labels) {
    return predict_host_impl(ctx, h_X, true, m, n, h_w, h_b, thr, h_labels);
}

int lr_profile_enable(lr_ctx* ctx, int32_t on) {
    if (!ctx) return LR_ERR_NULL;
    ctx->prof = on != 0;
    ctx->prof_used = 0;
    return LR_OK;
}

int lr_profile_read(lr_ctx* ctx, int32_t* launches, double* total_ms) {
    if (!ctx || !launches || !total_ms) return LR_ERR_NULL;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    double sum = 0.0;
    for (int i = 0; i < ctx->prof_used; ++i) {
        LR_CK(ctx, cudaEventSynchronize(ctx->ev[2 * i + 1]));
        float ms = 0.f;
        LR_CK(ctx, cudaEventElapsedTime(&ms, ctx->ev[2 * i], ctx->ev[2 * i + 1]));
        sum += ms;
    }
    *launches = ctx->prof_used;
    *total_ms = sum;
    ctx->prof_used = 0;
    return LR_OK;
}

int lr_launch_count(lr_ctx* ctx, int64_t* out) {
    if (!ctx || !out) return LR_ERR_NULL;
    *out = ctx->launches;
    return LR_OK;
}

int lr_last_device_status(lr_ctx* ctx, int32_t* out) {
    if (!ctx || !out) return LR_ERR_NULL;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    LR_CK(ctx, cudaDeviceSynchronize());
    int v = 0;
    LR_CK(ctx, cudaMemcpy(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    LR_CK(ctx, cudaMemset(ctx->d_status, 0, sizeof(int)));
    *out = v;
    return LR_OK;
}

int lr_check_guards(lr_ctx* ctx, int32_t* corrupted) {
    if (!ctx || !corrupted) return LR_ERR_NULL;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    LR_CK(ctx, cudaDeviceSynchronize());
    int bad = 0;
    unsigned char host[kGuardBytes];
    for (size_t i = 0; i < ctx->guard_bases.size(); ++i) {
        for (int side = 0; side < 2; ++side) {
            const unsigned char* src = ctx->guard_bases[i] + (side ? kGuardBytes + ctx->guard_sizes[i] : 0);
            LR_CK(ctx, cudaMemcpy(host, src, kGuardBytes, cudaMemcpyDeviceToHost));
            bool clean = true;
            for (size_t k = 0; k < kGuardBytes; ++k) clean = clean && host[k] == static_cast<unsigned char>(kGuardPattern);
            if (!clean) ++bad;
        }
    }
    *corrupted = bad;
    return LR_OK;
}

int lr_selftest_wait(lr_ctx* ctx, int32_t arm, int32_t limit_ms, void* stream) {
    if (!ctx) return LR_ERR_NULL;
    if (limit_ms < 1 || limit_ms > 1000) return LR_ERR_VALUE;
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    k_wait_probe<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status, 1000000ull * unsigned(limit_ms), arm ? 1 : 0);
    LR_CK(ctx, cudaGetLastError());
    ctx->launches += 1;
    return LR_OK;
}

int lr_last_cuda_error(lr_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

const char* lr_status_string(int code) {
    switch (code) {
        case LR_OK: return "ok";
        case LR_ERR_NULL: return "a required pointer is NULL";
        case LR_ERR_SHAPE: return "shape out of range (m, n, iters) or larger than the context allows";
        case LR_ERR_ALIGNMENT: return "a pointer is not aligned to its element size (4 bytes for float, 2 for bfloat16, 8 for double)";
        case LR_ERR_VALUE: return "value out of range (thr must be in (0,1), lr finite)";
        case LR_ERR_CUDA: return "a CUDA runtime call failed";
        case LR_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case LR_ERR_NOMEM: return "allocation failed";
        default: return "unknown status";
    }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------------
// Row-sharded fits with the exchange inside the persistent kernel.
// ------------------------------------------------------------------------------------------------------
namespace {

int fit_sharded_impl(lr_ctx* ctx, const void* d_X, bool bf16, const float* d_y, int64_t m_local, int64_t m_total, int32_t n,
                     float lr, int32_t iters, float* d_w, float* d_b, float* d_loss_hist, int32_t rank, int32_t world,
                     void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream) {
    int rc = check_common(ctx, d_X, m_local, n, d_w, d_b, bf16);
    if (rc != LR_OK) return rc;
    if (!d_y || !d_exchange) return LR_ERR_NULL;
    if (iters < 0 || world < 1 || world > kMaxWorld || rank < 0 || rank >= world || m_total < m_local || epoch < 0) return LR_ERR_SHAPE;
    if (wait_ms < 1 || wait_ms > 60000 || !std::isfinite(lr)) return LR_ERR_VALUE;
    for (int r = 0; r < world; ++r) {
        if (!d_exchange[r]) return LR_ERR_NULL;
        if (!aligned(d_exchange[r], 128)) return LR_ERR_ALIGNMENT;
    }
    if (!aligned(d_y, 4) || (d_loss_hist && !aligned(d_loss_hist, 4))) return LR_ERR_ALIGNMENT;
    lr_plan P;
    rc = make_plan(m_local, n, aligned(d_X, 16), plan_sms(ctx), &P, bf16);
    if (rc != LR_OK) return rc;
    if (P.variant != 0 || !ctx->coop || int64_t(iters) * P.grid >= (int64_t(1) << 32)) return LR_ERR_SHAPE;   // no persistent kernel for this shape
    if (iters == 0) return LR_OK;
    NvtxRange range("lr_fit_sharded");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    const PersistentShard shard{rank, world, m_total, uint64_t(epoch), uint64_t(wait_ms) * 1000000ull, d_exchange};
    const cudaError_t e = launch_persistent_fit(ctx, P, bf16, d_X, d_y, m_local, n, lr, iters, d_w, d_b, d_loss_hist, nullptr,
                                                static_cast<cudaStream_t>(stream), &shard);
    if (e != cudaSuccess) { ctx->last_cuda = int(e); cudaGetLastError(); return LR_ERR_CUDA; }
    return LR_OK;
}

}  // namespace

extern "C" {

int lr_exchange_bytes(int32_t world, int32_t n, int64_t* bytes) {
    if (!bytes) return LR_ERR_NULL;
    if (world < 1 || world > kMaxWorld || n < 1) return LR_ERR_SHAPE;
    *bytes = exchange_buffer_bytes(world, n);
    return LR_OK;
}

int lr_set_sm_limit(lr_ctx* ctx, int32_t sms) {
    if (!ctx) return LR_ERR_NULL;
    if (sms < 0) return LR_ERR_VALUE;
    ctx->sm_limit = sms;
    return LR_OK;
}

int lr_fit_sharded(lr_ctx* ctx, const float* d_X, const float* d_y, int64_t m_local, int64_t m_total, int32_t n, float lr,
                   int32_t iters, float* d_w, float* d_b, float* d_loss_hist, int32_t rank, int32_t world,
                   void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream) {
    return fit_sharded_impl(ctx, d_X, false, d_y, m_local, m_total, n, lr, iters, d_w, d_b, d_loss_hist, rank, world, d_exchange,
                            epoch, wait_ms, stream);
}

int lr_fit_sharded_bf16(lr_ctx* ctx, const uint16_t* d_Xh, const float* d_y, int64_t m_local, int64_t m_total, int32_t n, float lr,
                        int32_t iters, float* d_w, float* d_b, float* d_loss_hist, int32_t rank, int32_t world,
                        void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream) {
    return fit_sharded_impl(ctx, d_Xh, true, d_y, m_local, m_total, n, lr, iters, d_w, d_b, d_loss_hist, rank, world, d_exchange,
                            epoch, wait_ms, stream);
}

int lr_fit_sharded_local(lr_ctx* ctx, int32_t world, const float* const* d_X, const float* const* d_y, const int64_t* m_local,
                         int32_t n, float lr, int32_t iters, float* const* d_w, float* const* d_b, float* const* d_loss_hist,
                         void* const* d_exchange, int64_t epoch, int32_t wait_ms, void* stream) {
    if (!ctx || !d_X || !d_y || !m_local || !d_w || !d_b || !d_exchange) return LR_ERR_NULL;
    if (world < 2 || world > kMaxWorld || n < 1 || n > ctx->n_max || iters < 0 || epoch < 0) return LR_ERR_SHAPE;
    if (wait_ms < 1 || wait_ms > 60000 || !std::isfinite(lr)) return LR_ERR_VALUE;
    const int sms = plan_sms(ctx) / world;                                      // SMs (= CTAs) a rank may take
    if (sms < 1 || !ctx->coop) return LR_ERR_SHAPE;
    int64_t m_total = 0;
    lr_plan P{};
    int ctas = 0;
    for (int r = 0; r < world; ++r) {
        if (!d_X[r] || !d_y[r] || !d_w[r] || !d_b[r] || !d_exchange[r]) return LR_ERR_NULL;
        if (m_local[r] < 1 || m_local[r] > kMaxRows) return LR_ERR_SHAPE;
        if (!aligned(d_X[r], 16) || !aligned(d_y[r], 4) || !aligned(d_w[r], 4) || !aligned(d_b[r], 4) || !aligned(d_exchange[r], 128) ||
            (d_loss_hist && d_loss_hist[r] && !aligned(d_loss_hist[r], 4)))
            return LR_ERR_ALIGNMENT;
        lr_plan Pr;
        const int rc = make_plan(m_local[r], n, true, sms, &Pr);
        if (rc != LR_OK) return rc;
        if (Pr.variant != 0) return LR_ERR_SHAPE;
        if (r == 0) P = Pr;
        ctas = std::max(ctas, int(Pr.grid));
        m_total += m_local[r];
    }
    if (int64_t(iters) * ctas >= (int64_t(1) << 32)) return LR_ERR_SHAPE;
    if (size_t(world) * 2 * ctas * (size_t(n) + 2) > size_t(ctx->sm_count) * kMaxGridPerSm * (size_t(ctx->n_max) + 2)) return LR_ERR_SHAPE;
    if (iters == 0) return LR_OK;
    NvtxRange range("lr_fit_sharded_local");
    DeviceGuard g(ctx);
    if (!g.ok) return LR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // one shared-memory shape for all ranks: the deepest pipeline any of them wants; resident only if all of them are
    FitLayout L{1, true, 0};
    for (int r = 0; r < world; ++r) {
        const FitLayout Lr = fit_layout(P, false, m_local[r], n, ctas);
        L.depth = std::max(L.depth, Lr.depth);
        L.resident = L.resident && Lr.resident;
        L.smem = std::max(L.smem, Lr.smem);
    }
    std::vector<FitParams> h(static_cast<size_t>(world));
    for (int r = 0; r < world; ++r) {
        const PersistentShard shard{r, world, m_total, uint64_t(epoch), uint64_t(wait_ms) * 1000000ull, d_exchange};
        h[r] = fit_params(ctx, P, false, d_X[r], d_y[r], m_local[r], n, lr, iters, d_w[r], d_b[r],
                          d_loss_hist ? d_loss_hist[r] : nullptr, L.depth, nullptr, &shard);
        h[r].partial = ctx->d_partial + size_t(r) * 2 * ctas * (size_t(n) + 2);   // every rank its own partial rows ...
        h[r].gbar = ctx->d_gbar + 2 * r;                                         // ... and barrier words
        h[r].keep_rows = 0;
    }
    LR_CK(ctx, cudaMemsetAsync(ctx->d_gbar, 0, 2 * kMaxWorld * sizeof(unsigned int), st));
    LR_CK(ctx, cudaMemcpyAsync(ctx->d_rank_params, h.data(), sizeof(FitParams) * world, cudaMemcpyHostToDevice, st));
    LR_CK(ctx, cudaStreamSynchronize(st));          // the host copy of the parameters must outlive the (pageable) transfer
    lr_plan Pl = P;
    Pl.grid = ctas;
    const cudaError_t e = launch_fit_ranks(Pl, L.smem, L.resident, ctx->d_rank_params, world, ctas, st);
    if (e == cudaErrorInvalidValue) { cudaGetLastError(); return LR_ERR_SHAPE; }
    if (e != cudaSuccess) { ctx->last_cuda = int(e); cudaGetLastError(); return LR_ERR_CUDA; }
    ctx->launches += 1;
    return LR_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------------
// Allocation-free loss/gradient pass.  The per-CTA partial sums that lr_loss_grad keeps in a context's
// cudaMalloc'ed workspace live here in a fixed array inside the library's device image instead.
// ------------------------------------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxGrid = 256;                                    // CTAs
constexpr int kNoAllocRowDoubles = LR_NOALLOC_MAX_N + 2;                // one partial row: n columns, sum err, sum loss
constexpr size_t kNoAllocScratchDoubles = size_t(kNoAllocMaxGrid) * kNoAllocRowDoubles + 2;   // + status word slot

// 2 MiB + 16 B on every GPU that loads the library, for the life of the process.
static __device__ __align__(256) double g_noalloc_scratch[kNoAllocScratchDoubles];

constexpr int kNoAllocMaxDevices = 64;
struct NoAllocDevice {
    double* scratch = nullptr;      // device address of g_noalloc_scratch on this device (NOT the host-side symbol)
    int sm_count = 0;
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;

// First use on `device` (which must be current): resolve the symbol to its device address and cache it.
int noalloc_setup(int device, NoAllocDevice** out) {
    if (device < 0 || device >= kNoAllocMaxDevices) return LR_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& d = g_noalloc_dev[device];
    if (!d.scratch) {
        double* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch) != cudaSuccess || !ptr) return LR_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) return LR_ERR_CUDA;
        d.sm_count = sms;
        d.scratch = ptr;
    }
    *out = &d;
    return LR_OK;
}

}  // namespace

extern "C" int lr_loss_grad_noalloc(int32_t device, const float* d_X, const float* d_y, int64_t m, int32_t n,
                                    const float* d_w, const float* d_b, float* d_loss, float* d_grad_w, float* d_grad_b,
                                    int32_t* d_status, void* stream) {
    if (!d_X || !d_y || !d_w || !d_b || !d_loss || !d_grad_w || !d_grad_b) return LR_ERR_NULL;
    if (m < 1 || m > kMaxRows || n < 1) return LR_ERR_SHAPE;
    if (n > LR_NOALLOC_MAX_N) return LR_ERR_SHAPE;                      // the fixed scratch holds rows of at most this many columns
    if (!aligned(d_X, 4) || !aligned(d_y, 4) || !aligned(d_w, 4) || !aligned(d_b, 4) || !aligned(d_loss, 4) ||
        !aligned(d_grad_w, 4) || !aligned(d_grad_b, 4) || (d_status && !aligned(d_status, 4)))
        return LR_ERR_ALIGNMENT;
    int prev = -1;
    cudaGetDevice(&prev);
    if (cudaSetDevice(device) != cudaSuccess) return LR_ERR_CUDA;
    struct Restore { int p; ~Restore() { if (p >= 0) cudaSetDevice(p); } } restore{prev};

    NoAllocDevice* dev = nullptr;
    int rc = noalloc_setup(device, &dev);
    if (rc != LR_OK) return rc;
    // n <= LR_NOALLOC_MAX_N, so the plan is one of the narrow-row staged kernels (16-byte groups, or single elements for odd
    // lengths and 4-byte-aligned matrices) or, for such rows of more than 512 columns, the kernel with CTA-wide stages; the
    // grid never exceeds the SM count given here
    lr_plan P;
    rc = make_plan(m, n, aligned(d_X, 16), std::min(dev->sm_count, kNoAllocMaxGrid), &P);
    if (rc != LR_OK) return rc;
    if ((P.variant != 0 && P.variant != 3 && P.variant != 4) || P.grid > kNoAllocMaxGrid) return LR_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* partial = dev->scratch;
    int* status = d_status ? d_status : reinterpret_cast<int*>(dev->scratch + size_t(kNoAllocMaxGrid) * kNoAllocRowDoubles);
    // the array keeps whatever the previous call left: the status word must start at zero (the partial rows are
    // fully rewritten by the CTAs that the reduction reads)
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return LR_ERR_CUDA;
    cudaError_t e;
    if (P.variant == 4) {
        WideParams wp{};
        wp.X = d_X; wp.y = d_y; wp.m = m; wp.n = n; wp.w = d_w; wp.b = d_b;
        wp.partial = partial; wp.labels = nullptr; wp.cut = 0.f; wp.status = status;
        wp.depth = P.stages;
        wp.cw = (n + P.threads / 32 - 1) / (P.threads / 32);
        wp.num_batches = (m + P.rows_per_batch - 1) / P.rows_per_batch;
        e = launch_wide<false>(P, wp, st, false, false);
    } else {
        StreamParams sp{};
        sp.X = d_X; sp.y = d_y; sp.m = m; sp.n = n; sp.w = d_w; sp.b = d_b;
        sp.partial = partial; sp.labels = nullptr; sp.cut = 0.f; sp.status = status;
        sp.depth = P.stages;
        sp.num_batches = (m + P.rows_per_batch - 1) / P.rows_per_batch;
        e = launch_rows<false>(P, sp, st);
    }
    if (e != cudaSuccess) return LR_ERR_CUDA;
    ReduceParams rp{};
    rp.partial = partial; rp.G = P.grid; rp.n = n; rp.inv_m = 1.0 / double(m); rp.lr = 0.0; rp.update = 0;
    rp.w = nullptr; rp.b = nullptr; rp.grad_w = d_grad_w; rp.grad_b = d_grad_b; rp.loss_out = d_loss; rp.raw_sums = nullptr;
    k_reduce_update<<<(n + 2 + 31) / 32, dim3(32, kRedSlices), 0, st>>>(rp);
    if (cudaGetLastError() != cudaSuccess) return LR_ERR_CUDA;
    return LR_OK;
}
