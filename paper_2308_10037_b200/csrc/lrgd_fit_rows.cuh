// Persistent whole-fit kernel for rows of up to 512 columns: all `iters` gradient-descent iterations in ONE
// cooperative launch (one CTA per SM, co-resident), instead of two launches per iteration.
//
// Per iteration every CTA runs the same per-warp streaming pass as k_stream_rows (same static batch map, same
// arithmetic, same summation orders), writes its fp64 partial row, and meets the other CTAs at ONE grid barrier.  After
// it every CTA adds up all partial rows for itself -- the arithmetic of k_reduce_update, slice for slice, so every CTA
// gets the same bits -- and updates its own shared-memory copy of the parameters: there is no second barrier and no
// reload of the parameters through global memory.  The partial rows are double-buffered by iteration parity, so a CTA
// that is already writing the rows of iteration t+1 cannot disturb one that still reads those of iteration t (it
// cannot get to iteration t+2 before everybody has passed the barrier of t+1).  CTA 0 writes the loss history and, at
// the end, the parameters.  Results are bit-identical to the two-kernel path.
//
// What the single launch buys: no launch gaps, and the HBM stream never drains -- X does not depend on w, so each warp
// keeps re-arming its stages straight across the iteration boundary (the first batches of iteration t+1 are in flight
// while the CTAs reduce iteration t).  This matters for short passes (a 400 MB pass lasts ~60 us, of which launch,
// ramp-up and tail were ~20 %) and most for L2-resident problems.
//
// Resident form: when every warp's share of X fits its stages (a problem of up to ~28 MB on 148 SMs), the stages are
// filled once and kept for the whole fit; an iteration is then arithmetic on shared memory plus the boundary, with no
// copy, no re-arming and no mbarrier wait after the first pass.
//
// With a tolerance (lr_fit_tol) the kernel also forms ||grad||_2 after every update and all CTAs leave the loop together
// once it is <= eps: the stopping rule of Algorithm 7 with no host round trip and no wasted launch.
//
// Row shards on several GPUs (lr_fit_sharded): every rank runs this kernel on its own rows.  After the grid barrier CTA 0
// of a rank adds up the rank's partial rows, stores the n+2 sums into slot [t & 1][rank] of EVERY rank's exchange buffer
// (plain stores through peer mappings; no multicast, no bulk copies from or to a peer) and then publishes the step
// number in flag [rank] of every buffer with a system-scope release.  All CTAs of a rank wait (bounded) until the flags
// of all ranks in their own buffer show the step, add the `world` vectors in k_reduce_update's fixed order -- the order
// lr_apply_sums uses, so every rank gets the same bits -- and update their copy of the parameters.  The slots alternate
// with the parity of the step: a rank can only be one step ahead of the slowest one (it needs that rank's flag to go
// on), so the slot it overwrites has been read by everybody.
//
// Grid barrier: a monotonic counter in global memory; thread 0 of each CTA adds one and spins (bounded, 2 s) until the
// counter reaches grid * k.  A second word next to the counter is the run's abort flag: a CTA whose wait expires (here
// or on a stage) raises it, every other CTA sees it in its own wait, and all of them stop iterating, wait (bounded) for
// their own copies in flight and retire with LR_ERR_TIMEOUT in the context's status word.  Both words are cleared by the
// host before every launch, so a status left unread by an earlier call cannot end this one.
#pragma once
#include "lrgd_common.cuh"
#include "lrgd_reduce.cuh"
#include "lrgd_stream_rows.cuh"

namespace lrgd {

constexpr int kFitCombineCols = 128;           // columns combined per pass through the CTA's combine buffer
#ifndef LRGD_FIT_L2PF
#define LRGD_FIT_L2PF 4
#endif
constexpr int kFitL2Prefetch = LRGD_FIT_L2PF;   // batches per warp pulled into L2 ahead of the next iteration (beyond the staged ones)
constexpr int kFitMaxCols = 1024;              // widest row the persistent kernel takes
constexpr int kFitMaxWarps = 16;
// after the stages: combine buffer [warps][kFitCombineCols] fp64 (sized for 16 warps) and sum err / sum loss per warp, then
// the CTA's copy of the parameters (w[n], b) in fp32, then the reduced sums / gradient entries [n+2] in fp64
constexpr int kFitRedBytes = kFitMaxWarps * kFitCombineCols * 8 + 2 * kFitMaxWarps * 8;
__host__ __device__ constexpr int fit_param_bytes(int n) { return ((n + 1) * 4 + 15) / 16 * 16; }
__host__ __device__ constexpr int fit_tail_bytes(int n) { return (kFitRedBytes + fit_param_bytes(n) + (n + 2) * 8 + 127) / 128 * 128; }
constexpr int kFitRowChunk = 5;                // partial rows of one slice a thread has in flight (grids of up to 160 CTAs: the whole slice)
constexpr int kFitChunkPairs = 32;             // column pairs per chunk of the reduction: one per lane, 512 contiguous bytes per row
#ifndef LRGD_FIT_RED_INLINE
#define LRGD_FIT_RED_INLINE __noinline__       // out of line: the streaming loop of the caller then keeps all its registers
#endif
#ifndef LRGD_FIT_RED_CHUNKS
#define LRGD_FIT_RED_CHUNKS 2                  // 64-column chunks of the reduction in flight per round (where the registers allow)
#endif
static_assert(LRGD_FIT_RED_CHUNKS * kFitMaxWarps * 2 * kFitChunkPairs <= kFitMaxWarps * kFitCombineCols, "the reduction reuses the combine buffer");

constexpr int kMaxWorld = 32;                  // ranks of a row-sharded fit (one slice of the fixed summation tree each)
static_assert(kMaxWorld <= kRedSlices, "one reduction slice per rank");

struct FitParams {
    const void* X;             // fp32 or bfloat16 [m][n], row-major
    const float* y;
    long long m;
    int n;
    float* w;                  // [n] in/out
    float* b;                  // [1] in/out
    double* partial;           // [2][grid][n+2]: the per-CTA sums of even and odd iterations
    float* loss_hist;          // nullable [iters]
    int* status;               // device status word (sticky report; never read here)
    unsigned int* gbar;        // [0] grid-barrier counter, [1] abort flag of this launch; both zero at launch
    int depth;
    long long num_batches;
    long long keep_rows;       // rows [0, keep_rows) are fetched with an L2 evict-last hint, the rest evict-first
    int iters;
    double lr;
    double inv_m;
    // stopping rule (all null / zero for a fixed-count fit): as in k_reduce_update's tolerance mode
    TolState* tol;
    double eps;
    float* gnorm_hist;         // nullable [iters]
    // row shards (world == 0: a fit on one GPU, nothing below is used)
    int rank, world;
    unsigned long long epoch;  // steps exchanged through these buffers before this launch (the same on every rank)
    unsigned long long wait_ns;               // bound on each wait for the other ranks
    unsigned char* xbuf[kMaxWorld];           // exchange buffer of every rank as this rank addresses it; [rank] is its own
};

// Layout of one rank's exchange buffer: one 8-byte step flag per source rank, 128 bytes apart; then two slots
// (step parity) of `world` vectors of n+2 doubles, each vector padded to a multiple of 128 bytes.
__host__ __device__ constexpr long long exchange_vector_bytes(int n) { return ((n + 2) * 8LL + 127) / 128 * 128; }
__host__ __device__ constexpr long long exchange_flag_offset(int src) { return 128LL * src; }
__host__ __device__ constexpr long long exchange_slot_offset(int world, int n, int parity, int src) {
    return 128LL * world + (static_cast<long long>(parity) * world + src) * exchange_vector_bytes(n);
}
__host__ __device__ constexpr long long exchange_buffer_bytes(int world, int n) { return exchange_slot_offset(world, n, 2, 0); }

__device__ __forceinline__ unsigned long long ld_relaxed_sys_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// All threads of the CTA call this.  Returns false if the barrier gave up (or the CTA, or another one, had already
// given up).  Writes of the CTA before the call are visible to every CTA after it (release: fence, then the add; acquire:
// relaxed polling loads, then a fence; the CTA's other threads are ordered through the two __syncthreads).
__device__ __forceinline__ bool grid_barrier(unsigned int* gbar, unsigned int target, int* status, volatile int* cta_abort) {
    __syncthreads();
    if (threadIdx.x == 0) {
        if (*cta_abort) {
            atomicExch(gbar + 1, 1u);              // a stage wait of this CTA expired: tell the others
        } else {
            __threadfence();
            atomicAdd(gbar, 1u);
            if (ld_relaxed_u32(gbar) < target) {
                const unsigned long long t0 = global_timer_ns();
                for (;;) {
                    bool there = false;
#pragma unroll 1
                    for (int i = 0; i < 64 && !there; ++i) there = ld_relaxed_u32(gbar) >= target;
                    if (there) break;
                    const bool told = ld_relaxed_u32(gbar + 1) != 0u;
                    if (told || global_timer_ns() - t0 > kWaitLimitNs) {
                        if (!told) atomicExch(gbar + 1, 1u);
                        atomicExch(status, kStatusTimeout);
                        *cta_abort = 1;
                        break;
                    }
                }
            }
            __threadfence();                       // acquire side: the other CTAs' rows are read after this
        }
    }
    __syncthreads();
    return *cta_abort == 0;
}

// One column of up to 32 partial rows in k_reduce_update's order: a slice is a single row (an absent one counts as 0.0),
// then the fixed tree (s with s+16, then distance 8, 4, 2, 1).  `row_value(g)` yields the entry of row g; all of them are
// requested before the first addition.  NW only shapes the loop (slices i, i + NW, ... first: the tree levels of distance >= NW).
template <int NW, class F>
__device__ __forceinline__ double single_row_slices_sum(int G, F&& row_value) {
    constexpr int K = kRedSlices / NW;
    static_assert(K * NW == kRedSlices && (K & (K - 1)) == 0, "slices must split evenly");
    double a[NW];
    if (G <= NW) {
        // slices NW and up are absent: each would add +0.0 to a row entry, which leaves it as it is (an entry is never -0.0:
        // warp_tree_sum ends with + 0.0)
#pragma unroll
        for (int i = 0; i < NW; ++i) a[i] = i < G ? row_value(i) : 0.0;
    } else {
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            double r[K];
#pragma unroll
            for (int k = 0; k < K; ++k) r[k] = i + k * NW < G ? row_value(i + k * NW) : 0.0;
#pragma unroll
            for (int h = K / 2; h >= 1; h >>= 1)
#pragma unroll
                for (int k = 0; k < h; ++k) r[k] += r[k + h];
            a[i] = r[0];
        }
    }
#pragma unroll
    for (int h = NW / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int i = 0; i < h; ++i) a[i] += a[i + h];
    return a[0];
}

// Adds up the G partial rows [G][stride] column by column into sums[stride] (shared memory); called by all threads of a
// CTA, with the order of k_reduce_update so that the result has that kernel's bits: slice s = rows [s*per, (s+1)*per) in
// index order, then the 32 slice sums in the fixed tree (s with s+16, then distance 8, 4, 2, 1).
// Warp w owns the slices w, w + NW, w + 2 NW, ... -- the ones the first tree levels add to each other -- and a lane owns
// one pair of adjacent columns, so every load instruction of a warp reads 512 contiguous bytes of one partial row (all
// CTAs read the same rows at the same time: scattered 16-byte reads cost L2 eight times the requests).  The NW per-warp
// sums of a chunk of 64 columns meet in `buf` and one thread per column finishes the tree.  A thread has at most
// (32 / NW) * kFitRowChunk 16-byte loads in flight: few enough to live in the registers the streaming loop leaves free.
// Grids of up to 32 CTAs (small problems, where this call is most of the iteration): a slice is a single row and one
// thread per column holds all rows at once.
template <int NW>
__device__ LRGD_FIT_RED_INLINE void reduce_partial_rows(const double* pbuf, int G, int stride, double* buf, double* sums) {
    constexpr int K = kRedSlices / NW;             // slices per warp
    static_assert(K * NW == kRedSlices && (K & (K - 1)) == 0, "slices must split evenly over the warps");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per = (G + kRedSlices - 1) / kRedSlices;
    const int npairs = stride / 2;
    const double2 zero = make_double2(0.0, 0.0);
    if (per == 1) {
        // a slice is a single row: one thread per column holds all of them at once -- one round trip to L2 and a tree in
        // registers, no exchange through shared memory or shuffles (at 256 columns a butterfly per column pair took 2.5 us
        // more; a thread per PAIR of columns needs twice the registers, which the caller's streaming loop pays for)
        for (int col = threadIdx.x; col < stride; col += NW * 32)
            sums[col] = single_row_slices_sum<NW>(G, [&](int g) { return __ldcg(pbuf + static_cast<size_t>(g) * stride + col); });
        __syncthreads();
        return;
    }
    constexpr int CH = LRGD_FIT_RED_CHUNKS * K <= 4 ? LRGD_FIT_RED_CHUNKS : 1;   // chunks of 64 columns in flight (two with 16 warps)
    const int nchunks = (npairs + kFitChunkPairs - 1) / kFitChunkPairs;
    for (int c0 = 0; c0 < nchunks; c0 += CH) {
        double2 acc[CH][K];
#pragma unroll
        for (int u = 0; u < CH; ++u)
#pragma unroll
            for (int k = 0; k < K; ++k) acc[u][k] = zero;
        for (int r0 = 0; r0 < per; r0 += kFitRowChunk) {
            double2 v[CH][K][kFitRowChunk];
#pragma unroll
            for (int u = 0; u < CH; ++u) {
                const int q = (c0 + u) * kFitChunkPairs + lane;
                const bool live = q < npairs;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int first = (warp + k * NW) * per;               // slice warp + k NW
                    const int last = first + per < G ? first + per : G;
#pragma unroll
                    for (int r = 0; r < kFitRowChunk; ++r) {
                        const int g = first + r0 + r;
                        v[u][k][r] = (live && r0 + r < per && g < last)
                                         ? __ldcg(reinterpret_cast<const double2*>(pbuf + static_cast<size_t>(g) * stride) + q) : zero;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < CH; ++u)
#pragma unroll
                for (int k = 0; k < K; ++k)
#pragma unroll
                    for (int r = 0; r < kFitRowChunk; ++r) {               // (+0.0 where there is no row: changes nothing)
                        acc[u][k].x += v[u][k][r].x;
                        acc[u][k].y += v[u][k][r].y;
                    }
        }
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            // the tree levels inside this warp's slices: distance 16, 8, ... down to NW (in slices), i.e. K/2, ..., 1 here
#pragma unroll
            for (int h = K / 2; h >= 1; h >>= 1)
#pragma unroll
                for (int k = 0; k < h; ++k) { acc[u][k].x += acc[u][k + h].x; acc[u][k].y += acc[u][k + h].y; }
            reinterpret_cast<double2*>(buf)[(u * NW + warp) * kFitChunkPairs + lane] = acc[u][0];
        }
        __syncthreads();
        if (threadIdx.x < CH * 2 * kFitChunkPairs) {
            const int u = threadIdx.x / (2 * kFitChunkPairs), c = threadIdx.x % (2 * kFitChunkPairs);
            const int col = (c0 + u) * 2 * kFitChunkPairs + c;
            if (col < stride) {
                double t[NW];
#pragma unroll
                for (int i = 0; i < NW; ++i) t[i] = buf[(u * NW + i) * 2 * kFitChunkPairs + c];
#pragma unroll
                for (int h = NW / 2; h >= 1; h >>= 1)
#pragma unroll
                    for (int i = 0; i < h; ++i) t[i] = t[i] + t[i + h];
                sums[col] = t[0];
            }
        }
        __syncthreads();
    }
}

// The exchange of a row-sharded step, called by all threads of every CTA after the rank's grid barrier; leaves the global
// sums in sums[stride].  Returns false if a wait for another rank expired (the CTA's abort flag is then up).
template <int NW>
__device__ LRGD_FIT_RED_INLINE bool exchange_rank_sums(const FitParams& p, int cta, int G, int stride, int t, double* buf, double* sums,
                                                      volatile int* cta_abort) {
    const unsigned long long step = p.epoch + static_cast<unsigned long long>(t) + 1ull;
    const int parity = static_cast<int>(step & 1ull);
    if (cta == 0) {
        // this rank's sums, then one copy of them into every rank's buffer, then the flags
        reduce_partial_rows<NW>(p.partial + static_cast<size_t>(t & 1) * G * stride, G, stride, buf, sums);
        for (int r = 0; r < p.world; ++r) {
            double* dst = reinterpret_cast<double*>(p.xbuf[r] + exchange_slot_offset(p.world, p.n, parity, p.rank));
            for (int c = threadIdx.x; c < stride; c += NW * 32) dst[c] = sums[c];
        }
        __syncthreads();
        if (threadIdx.x < p.world) {
            __threadfence_system();                // the stores of the whole CTA (ordered by the barrier above) before the flag
            st_release_sys_u64(reinterpret_cast<unsigned long long*>(p.xbuf[threadIdx.x] + exchange_flag_offset(p.rank)), step);
        }
    }
    // wait for every rank's flag in this rank's own buffer
    if (threadIdx.x < p.world) {
        const unsigned long long* flag = reinterpret_cast<const unsigned long long*>(p.xbuf[p.rank] + exchange_flag_offset(threadIdx.x));
        if (ld_relaxed_sys_u64(flag) < step) {
            const unsigned long long t0 = global_timer_ns();
            for (;;) {
                bool there = false;
#pragma unroll 1
                for (int i = 0; i < 64 && !there; ++i) there = ld_relaxed_sys_u64(flag) >= step;
                if (there) break;
                if (*cta_abort || ld_relaxed_u32(p.gbar + 1) != 0u || global_timer_ns() - t0 > p.wait_ns) {
                    atomicExch(p.gbar + 1, 1u);
                    atomicExch(p.status, kStatusTimeout);
                    *cta_abort = 1;
                    break;
                }
            }
        }
        __threadfence_system();                    // acquire side: the other ranks' vectors are read after this
    }
    __syncthreads();
    if (*cta_abort) return false;
    // the `world` vectors in k_reduce_update's order for `world` rows: one row per slice, then the fixed tree
    const unsigned char* own = p.xbuf[p.rank];
    for (int c = threadIdx.x; c < stride; c += NW * 32) {
        double sl[kRedSlices];
#pragma unroll
        for (int r = 0; r < kRedSlices; ++r) {
            double v = 0.0;
            if (r < p.world) v += __ldcg(reinterpret_cast<const double*>(own + exchange_slot_offset(p.world, p.n, parity, r)) + c);
            sl[r] = v;
        }
        sums[c] = slice_tree_sum(sl);
    }
    __syncthreads();
    return true;
}

template <class E, int NV, int LPR, int RB, int NW, bool RESIDENT>
__device__ __forceinline__ void fit_rows_body(const FitParams& p, const int cta, const int G) {
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
    static_assert(NW <= kFitMaxWarps && kRedSlices % NW == 0, "tail layout and reduction are sized for up to 16 warps");
    static_assert(NV * LPR * EPG <= kFitMaxCols, "row wider than the parameter copy");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + NW * kMaxDepth);
    unsigned char* data = smem + kHeaderBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.depth;
    const int n = p.n, n4 = n / EPG;                   // n4 = 16-byte groups per row
    const int stride = n + 2;                          // doubles per partial row (even: n is a multiple of four)
    const uint32_t row_bytes = static_cast<uint32_t>(n) * E::BYTES;
    const uint32_t stage_stride = (static_cast<uint32_t>(RPB) * row_bytes + 127u) & ~127u;
    unsigned char* my_stages = data + static_cast<size_t>(warp) * D * stage_stride;
    unsigned char* tail = data + static_cast<size_t>(NW) * D * stage_stride;
    double* red = reinterpret_cast<double*>(tail);                     // [NW][kFitCombineCols]
    double* red_e = red + NW * kFitCombineCols;
    double* red_l = red_e + NW;
    float* w_s = reinterpret_cast<float*>(tail + kFitRedBytes);        // w[0..n), then b
    double* sum_s = reinterpret_cast<double*>(tail + kFitRedBytes + fit_param_bytes(n));   // [n+2]
    uint64_t* my_bars = bars + warp * kMaxDepth;

    const long long B = p.num_batches;
    const long long Bw = B > warp ? (B - warp + NW - 1) / NW : 0;
    const int cnt = Bw > cta ? static_cast<int>((Bw - cta + G - 1) / G) : 0;    // batches of this warp per iteration
    constexpr bool resident = RESIDENT;            // cnt <= D for every warp of the grid (the host checked)
    const int fill_iters = cnt > 0 ? (resident ? 1 : p.iters) : 0;   // the fit is cnt * fill_iters stage fills for this warp, iteration-major

    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) mbar_init(&my_bars[d], 1);
        fence_mbar_init();
    }
    // the CTA's own copy of the parameters
    for (int c = threadIdx.x; c <= n; c += NW * 32) w_s[c] = c < n ? __ldcg(p.w + c) : __ldcg(p.b);
    __syncthreads();

    const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
    const long long stride_rows = static_cast<long long>(G) * NW * RPB;
    const long long first_row = (static_cast<long long>(cta) * NW + warp) * RPB;
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
    // y of this lane's row in the first batch: the same in every iteration
    const float y_first = (cnt > 0 && first_row + myr < p.m) ? __ldg(p.y + first_row + myr) : 0.f;
    int d = 0;
    uint32_t phase = 0;
    unsigned int barrier_no = 0;
    bool alive = true;                             // CTA-uniform after every grid barrier

    for (int t = 0; t < p.iters && alive; ++t) {
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
        float y_next = y_first;
        const bool waits = !resident || t == 0;    // a resident stage is complete once and for all after the first pass

        for (int i = 0; i < cnt; ++i) {
            if (waits) {
                bool ok = mbar_wait_bounded(&my_bars[d], phase, abort_flag);
                ok = __all_sync(FULL, ok);
                if (!ok) break;                    // the CTA's abort flag is up; handled at the barrier
            }

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
            if constexpr (resident) {
                if (waits) --inflight;
                if (++d == cnt) d = 0;             // stage i holds batch i in every iteration
            } else {
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
            }

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

        // The grid barrier and the reduction below take longer than the staged batches of the next iteration last; keep
        // HBM busy meanwhile by pulling this warp's following batches of that iteration into L2.
        if (!resident && lane == 0 && t + 1 < p.iters) {
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
            for (int c = 0; c < EPG; ++c) dacc[k2][c] = slot_order_sum<LPR>(dacc[k2][c], sub);
#pragma unroll
        for (int msk = 16; msk >= 1; msk >>= 1) {
            dse += __shfl_xor_sync(FULL, dse, msk);
            dsl += __shfl_xor_sync(FULL, dsl, msk);
        }
        double* out = p.partial + (static_cast<size_t>(t & 1) * G + cta) * stride;
        if (lane == 0) { red_e[warp] = dse; red_l[warp] = dsl; }       // (the last reader of these was before the previous barrier)
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
            if (threadIdx.x < kFitCombineCols && c0 + threadIdx.x < n)
                out[c0 + threadIdx.x] = warp_tree_sum<NW>(red + threadIdx.x, kFitCombineCols);
            __syncthreads();
        }
        if (threadIdx.x < 2) out[n + threadIdx.x] = warp_tree_sum<NW>(threadIdx.x == 0 ? red_e : red_l, 1);

        barrier_no += 1;
        alive = grid_barrier(p.gbar, static_cast<unsigned int>(G) * barrier_no, p.status, abort_flag);
        if (!alive) break;

        // ---- reduction, by every CTA for itself (see reduce_partial_rows); with row shards on several GPUs the exchange ----
        if (p.world == 0) {
            reduce_partial_rows<NW>(p.partial + static_cast<size_t>(t & 1) * G * stride, G, stride, red, sum_s);
        } else {
            alive = exchange_rank_sums<NW>(p, cta, G, stride, t, red, sum_s, abort_flag);
            if (!alive) break;
        }

        // ---- update (the arithmetic of k_reduce_update), every CTA on its own copy; CTA 0 keeps the history ----
        for (int c = threadIdx.x; c < stride; c += NW * 32) {
            const double v = sum_s[c] * p.inv_m;
            if (c <= n) {
                w_s[c] = static_cast<float>(static_cast<double>(w_s[c]) - p.lr * v);
                sum_s[c] = v;                                           // gradient entry, for the norm below
            } else if (cta == 0 && p.loss_hist) {
                p.loss_hist[t] = static_cast<float>(v);
            }
        }
        __syncthreads();

        // ---- stopping rule (Algorithm 7): ||(grad_w, grad_b)||_2 of the update just applied, formed by every warp in the
        // same order as k_reduce_update's last block (lane-strided squares, xor tree), so all CTAs take the same decision ----
        if (p.tol != nullptr) {
            double q = 0.0;
            for (int c = lane; c <= n; c += 32) {
                const double v = sum_s[c];
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
            if (nrm <= p.eps) break;               // uniform over the whole grid: every warp computed the same nrm
        }
    }

    if (alive && *abort_flag == 0) {
        if (cta == 0)                              // every CTA holds the same parameters; one of them stores them
            for (int c = threadIdx.x; c <= n; c += NW * 32) {
                if (c < n) p.w[c] = w_s[c];
                else p.b[0] = w_s[n];
            }
    } else if (lane == 0) {
        atomicExch(p.status, kStatusTimeout);      // the parameters are left as they were at launch
        atomicExch(p.gbar + 1, 1u);
    }
    // Copies still in flight when the loop ends (a give-up, or an early stop with the next iteration already being
    // prefetched) must land before the CTA retires and its shared memory is handed to another CTA.
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

template <class E, int NV, int LPR, int RB, int NW, bool RESIDENT>
__global__ void __launch_bounds__(NW * 32, 1) k_fit_rows(const __grid_constant__ FitParams p) {
    // (__grid_constant__: the exchange takes the parameters by reference; without it the kernel would keep a copy of the
    // whole block in local memory and read its fields from there)
    fit_rows_body<E, NV, LPR, RB, NW, RESIDENT>(p, blockIdx.x, gridDim.x);
}

// Several ranks of a row-sharded fit as groups of CTAs of ONE cooperative launch on one GPU: CTAs
// [r * ctas_per_rank, (r + 1) * ctas_per_rank) play rank r with the parameters ranks[r] (its own rows, partial rows, barrier
// words and exchange buffer).  All CTAs are co-resident, so ranks that wait on one another cannot starve each other; the
// exchange runs exactly as it does between GPUs.  This is how the multi-rank path is exercised where only one GPU is there.
template <class E, int NV, int LPR, int RB, int NW, bool RESIDENT>
__global__ void __launch_bounds__(NW * 32, 1) k_fit_rows_ranks(const FitParams* ranks, int ctas_per_rank) {
    fit_rows_body<E, NV, LPR, RB, NW, RESIDENT>(ranks[blockIdx.x / ctas_per_rank], blockIdx.x % ctas_per_rank, ctas_per_rank);
}

}  // namespace lrgd
