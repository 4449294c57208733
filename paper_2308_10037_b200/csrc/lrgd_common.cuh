// Shared device helpers: mbarrier / bulk-async-copy wrappers (sm_90+ PTX, used here on sm_100a),
// bounded waits, and the per-row logistic terms.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lrgd {

constexpr int kStatusTimeout = -6;                 // LR_ERR_TIMEOUT
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait, then the kernel gives up
constexpr unsigned long long kDrainLimitNs = 500000000ull;   // 0.5 s per copy still in flight when a CTA winds down

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Orders this thread's earlier generic-proxy accesses to shared memory (and those it has synchronised with)
// before later asynchronous-proxy accesses (bulk copies) to the same locations.
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Waits for the phase with the given parity to complete, for at most limit_ns.  On expiry (or when another
// thread of the CTA has already given up) raises *abort_flag and returns false.
__device__ __forceinline__ bool mbar_wait_bounded_ns(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                     unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    return mbar_wait_bounded_ns(bar, parity, abort_flag, kWaitLimitNs);
}

// Wait used when a CTA winds down with copies of its own still in flight: it does not look at the abort flag (which
// is what ends the run), only at the clock, so that the copies really land before the shared memory is given up.
__device__ __forceinline__ bool mbar_wait_drain(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kDrainLimitNs) return false;
    }
}

// One warp waits on an mbarrier that is completed up front (arm != 0) or never (arm == 0), with the given limit; on
// expiry it sets the status word exactly as the streaming kernels do.  Used to exercise the give-up path on purpose.
__global__ void k_wait_probe(int* status, unsigned long long limit_ns, int arm) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (arm && threadIdx.x == 0) mbar_arrive(&bar);
    const bool ok = mbar_wait_bounded_ns(&bar, 0u, &abort_flag, limit_ns);
    if (!ok && threadIdx.x == 0) atomicExch(status, kStatusTimeout);
}

// Programmatic dependent launch (sm_90+).  A kernel launched with the programmatic-stream-serialization attribute may
// start as soon as every CTA of the kernel before it in the stream has called grid_dependency_release() (or exited);
// whatever it does before grid_dependency_wait() overlaps the tail of that kernel and must not touch anything that
// kernel (or any earlier one) writes.  grid_dependency_wait() returns once all earlier kernels have completed and their
// writes are visible.  Without the attribute both are no-ops and the launch is an ordinary one.
__device__ __forceinline__ void grid_dependency_release() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// 1-D bulk asynchronous copy global -> shared; completion is signalled on `bar` as transferred bytes.
// dst, src 16-byte aligned, bytes a non-zero multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Asks the memory system to bring [src, src+bytes) into L2 (no destination, no completion signal).
// src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes, uint64_t policy) {
    asm volatile("cp.async.bulk.prefetch.L2.global.L2::cache_hint [%0], %1, %2;" ::"l"(src), "r"(bytes), "l"(policy) : "memory");
}

// Tiled 2-D TMA copy global -> shared through a tensor map (single destination CTA): the box whose first element has
// coordinates (x, y) -- x along the contiguous dimension, x*4 bytes a multiple of 16 -- lands densely packed at dst
// (128-byte aligned); out-of-range elements are written as zeros and count towards the transferred bytes.
__device__ __forceinline__ void bulk_tensor_2d_g2s(void* dst, const void* tmap, int x, int y, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// err alone (same arithmetic as in logistic_terms, so the two agree bit for bit)
__device__ __forceinline__ float logistic_err(float z, float y) {
    const float t = expf(-fabsf(z));
    const float r = 1.0f / (1.0f + t);
    const float tr = t * r;
    const float p = z >= 0.0f ? r : tr;
    const float q = z >= 0.0f ? tr : r;
    return (y == 1.0f) ? -q : (p - y);
}

// Per-row logistic terms in fp32 from the logit z and the target y:
//   err  = sigmoid(z) - y            (Eq. 1; Algorithm 7's sigmoid followed by Substract(Y, res))
//   loss = max(z,0) + log1p(exp(-|z|)) - y*z  ( = -[y log p + (1-y) log(1-p)], finite for any z )
// For y exactly 1 the error is formed as -sigmoid(-z) so that it keeps full relative precision when p -> 1.
__device__ __forceinline__ void logistic_terms(float z, float y, float& err, float& loss) {
    const float t = expf(-fabsf(z));
    const float r = 1.0f / (1.0f + t);
    const float tr = t * r;
    const float p = z >= 0.0f ? r : tr;      // sigmoid(z)
    const float q = z >= 0.0f ? tr : r;      // sigmoid(-z) = 1 - p
    err = (y == 1.0f) ? -q : (p - y);
    loss = fmaxf(z, 0.0f) + log1pf(t) - y * z;
}

// Where a lane fetches its slice of w from: global memory through L2 (the kernel before this one may just have written
// it), or the CTA's own shared-memory copy (the persistent kernel keeps the current parameters there).
enum class WSource { GlobalL2, Shared };
template <WSource S>
__device__ __forceinline__ float load_param(const float* p) {
    if constexpr (S == WSource::GlobalL2) return __ldcg(p);
    else return *p;
}

// ---- per-lane arithmetic on 16-byte groups of X ----
// A lane owns NV groups of a row.  Lane<NV> keeps that lane's slice of w and its fp32 gradient accumulators in the form
// the storage type's arithmetic wants, and offers: load_w, zero, dot (this lane's part of x.w for one row), accumulate
// (acc += x * err for one row) and fold (acc added into fp64 partners and cleared).  Both storage types work on pairs
// of adjacent columns held in 64-bit registers, so that one packed instruction does two fp32 FMAs.

// Two fp32 values in one 64-bit register, and the packed fused multiply-add on such pairs (fma.rn.f32x2, sm_100):
// each half is an ordinary round-to-nearest fp32 FMA, so a pair of independent accumulators costs one instruction.
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// fp32 storage: four values per group; the group's (x, y) and (z, w) words are the two pairs of the packed FMAs, so
// the dot product runs as two chains (even and odd columns) that are added at the end.
template <int NV>
struct LaneF32 {
    static constexpr int EPG = 4;
    uint64_t wv[NV][2];
    uint64_t acc[NV][2];
    template <WSource S>
    __device__ __forceinline__ void load_w(const float* w, int first_group, int group_stride, int group_limit) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int idx = first_group + k * group_stride;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float lo = 0.f, hi = 0.f;
                if (idx < group_limit) {
                    lo = load_param<S>(w + 4 * idx + 2 * j);
                    hi = load_param<S>(w + 4 * idx + 2 * j + 1);
                }
                wv[k][j] = f32x2_pack(lo, hi);
            }
        }
    }
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int k = 0; k < NV; ++k) { acc[k][0] = 0ull; acc[k][1] = 0ull; }
    }
    static __device__ __forceinline__ uint64_t pair(uint32_t a, uint32_t b) {
        uint64_t r;
        asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
        return r;
    }
    __device__ __forceinline__ float dot(const uint4 (&xr)[NV]) const {
        uint64_t d = 0ull;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            d = f32x2_fma(pair(xr[k].x, xr[k].y), wv[k][0], d);
            d = f32x2_fma(pair(xr[k].z, xr[k].w), wv[k][1], d);
        }
        float even, odd;
        f32x2_unpack(d, even, odd);
        return even + odd;
    }
    __device__ __forceinline__ void accumulate(const uint4 (&xr)[NV], float er) {
        const uint64_t e2 = f32x2_pack(er, er);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            acc[k][0] = f32x2_fma(pair(xr[k].x, xr[k].y), e2, acc[k][0]);
            acc[k][1] = f32x2_fma(pair(xr[k].z, xr[k].w), e2, acc[k][1]);
        }
    }
    __device__ __forceinline__ void fold(double (&dacc)[NV][4]) {
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float lo, hi;
                f32x2_unpack(acc[k][j], lo, hi);
                dacc[k][2 * j] += lo;
                dacc[k][2 * j + 1] += hi;
                acc[k][j] = 0ull;
            }
    }
};

// bfloat16 storage: eight values per group, two per 32-bit word (element 2j in the low half).  bfloat16 is the upper
// half of a binary32 pattern, so widening is exact: low element = word << 16, high element = word & 0xffff0000.  The
// widened pair goes straight into a packed FMA against the matching pair of w (dot) or against (err, err)
// (accumulate).  The dot product therefore runs as two chains (even and odd columns) that are added at the end.
template <int NV>
struct LaneBF16 {
    static constexpr int EPG = 8;
    uint64_t wv[NV][4];                  // (w[8g + 2j], w[8g + 2j + 1])
    uint64_t acc[NV][4];                 // accumulators of the same column pairs
    static __device__ __forceinline__ uint64_t widen(uint32_t word) {
        return f32x2_pack(__uint_as_float(word << 16), __uint_as_float(word & 0xffff0000u));
    }
    template <WSource S>
    __device__ __forceinline__ void load_w(const float* w, int first_group, int group_stride, int group_limit) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int idx = first_group + k * group_stride;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float lo = 0.f, hi = 0.f;
                if (idx < group_limit) {
                    lo = load_param<S>(w + 8 * idx + 2 * j);
                    hi = load_param<S>(w + 8 * idx + 2 * j + 1);
                }
                wv[k][j] = f32x2_pack(lo, hi);
            }
        }
    }
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[k][j] = 0ull;
    }
    __device__ __forceinline__ float dot(const uint4 (&xr)[NV]) const {
        uint64_t d = 0ull;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            d = f32x2_fma(widen(xr[k].x), wv[k][0], d);
            d = f32x2_fma(widen(xr[k].y), wv[k][1], d);
            d = f32x2_fma(widen(xr[k].z), wv[k][2], d);
            d = f32x2_fma(widen(xr[k].w), wv[k][3], d);
        }
        float even, odd;
        f32x2_unpack(d, even, odd);
        return even + odd;
    }
    __device__ __forceinline__ void accumulate(const uint4 (&xr)[NV], float er) {
        const uint64_t e2 = f32x2_pack(er, er);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            acc[k][0] = f32x2_fma(widen(xr[k].x), e2, acc[k][0]);
            acc[k][1] = f32x2_fma(widen(xr[k].y), e2, acc[k][1]);
            acc[k][2] = f32x2_fma(widen(xr[k].z), e2, acc[k][2]);
            acc[k][3] = f32x2_fma(widen(xr[k].w), e2, acc[k][3]);
        }
    }
    __device__ __forceinline__ void fold(double (&dacc)[NV][8]) {
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float lo, hi;
                f32x2_unpack(acc[k][j], lo, hi);
                dacc[k][2 * j] += lo;
                dacc[k][2 * j + 1] += hi;
                acc[k][j] = 0ull;
            }
    }
};

// Rows of any length: the unit a lane owns is a single element, so a row needs no particular length.  Loads are one
// element wide (consecutive lanes read consecutive elements: conflict-free), arithmetic is scalar FMAs in ownership
// order.  Raw is the element as stored: a 32-bit word holding an fp32 value, or a 16-bit bfloat16 pattern.
__device__ __forceinline__ float widen_element(uint32_t v) { return __uint_as_float(v); }
__device__ __forceinline__ float widen_element(unsigned short v) { return __uint_as_float(static_cast<uint32_t>(v) << 16); }

template <class Raw, int NV>
struct LaneAny {
    static constexpr int EPG = 1;
    float wv[NV];
    float acc[NV];
    template <WSource S>
    __device__ __forceinline__ void load_w(const float* w, int first_group, int group_stride, int group_limit) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int idx = first_group + k * group_stride;
            wv[k] = idx < group_limit ? load_param<S>(w + idx) : 0.f;
        }
    }
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int k = 0; k < NV; ++k) acc[k] = 0.f;
    }
    __device__ __forceinline__ float dot(const Raw (&xr)[NV]) const {
        float d0 = 0.f, d1 = 0.f;                  // two chains: NV goes up to 16
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            if (k & 1) d1 = fmaf(widen_element(xr[k]), wv[k], d1);
            else d0 = fmaf(widen_element(xr[k]), wv[k], d0);
        }
        return d0 + d1;
    }
    __device__ __forceinline__ void accumulate(const Raw (&xr)[NV], float er) {
#pragma unroll
        for (int k = 0; k < NV; ++k) acc[k] = fmaf(widen_element(xr[k]), er, acc[k]);
    }
    __device__ __forceinline__ void fold(double (&dacc)[NV][1]) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            dacc[k][0] += acc[k];
            acc[k] = 0.f;
        }
    }
};

// Storage types of X.  A "group" is 16 bytes of a row -- the unit of every shared-memory load and of the column
// ownership of a lane: four fp32 values or eight bfloat16 values.  All arithmetic is fp32 for both.
struct ElemF32 {
    static constexpr int EPG = 4;        // elements per 16-byte group
    static constexpr int BYTES = 4;      // bytes per element
    using Raw = uint4;                   // a group as it sits in shared memory and registers
    template <int NV>
    using Lane = LaneF32<NV>;
    static __device__ __forceinline__ float load(const void* base, long long i) {
        return reinterpret_cast<const float*>(base)[i];
    }
};
struct ElemBF16 {
    static constexpr int EPG = 8;
    static constexpr int BYTES = 2;
    using Raw = uint4;
    template <int NV>
    using Lane = LaneBF16<NV>;
    static __device__ __forceinline__ float load(const void* base, long long i) {
        return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const unsigned short*>(base)[i]) << 16);
    }
};

// Rows that cannot be cut into aligned 16-byte groups (any length, matrix aligned to its element size only): the
// "group" degenerates to one element (see LaneAny).
struct ElemF32Any {
    static constexpr int EPG = 1;
    static constexpr int BYTES = 4;
    using Raw = uint32_t;
    template <int NV>
    using Lane = LaneAny<uint32_t, NV>;
    static __device__ __forceinline__ float load(const void* base, long long i) {
        return reinterpret_cast<const float*>(base)[i];
    }
};
struct ElemBF16Any {
    static constexpr int EPG = 1;
    static constexpr int BYTES = 2;
    using Raw = unsigned short;
    template <int NV>
    using Lane = LaneAny<unsigned short, NV>;
    static __device__ __forceinline__ float load(const void* base, long long i) {
        return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const unsigned short*>(base)[i]) << 16);
    }
};

template <int V>
struct Log2 {
    static constexpr int value = 1 + Log2<V / 2>::value;
};
template <>
struct Log2<1> {
    static constexpr int value = 0;
};

}  // namespace lrgd
