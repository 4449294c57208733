// fp32 -> bfloat16 conversion of a matrix (storage variant of X: half the bytes per pass; the paper does not discuss
// storage precision).  bfloat16 is the upper half of a binary32 pattern; rounding is to nearest with ties to even,
// done on the integer pattern: adding 0x7FFF plus the last kept bit carries into the kept half exactly when the
// discarded half is above one half, or equal to one half with an odd kept half.  The carry may run into the exponent,
// which is the correctly rounded result too (next binade, or infinity past the largest finite value).  NaN would be
// turned into infinity by that carry, so it is mapped to a quiet NaN of the same sign first.
#pragma once
#include "lrgd_common.cuh"

namespace lrgd {

constexpr int kConvertThreads = 256;

__device__ __forceinline__ unsigned short bf16_bits_rne(float x) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<unsigned short>((u >> 16) | 0x7fc0u);
    return static_cast<unsigned short>((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}

// vec != 0: src is 16-byte aligned and dst 8-byte aligned, so four elements move per load/store; the tail of a count
// that is not a multiple of four is done element by element by the thread that owns it.
__global__ void __launch_bounds__(kConvertThreads) k_convert_bf16(const float* __restrict__ src, long long count,
                                                                  unsigned short* __restrict__ dst, int vec) {
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    if (vec) {
        const long long quads = count >> 2;
        for (long long q = tid; q < quads; q += nthreads) {
            const float4 v = __ldcs(reinterpret_cast<const float4*>(src) + q);
            uint2 o;
            o.x = static_cast<uint32_t>(bf16_bits_rne(v.x)) | (static_cast<uint32_t>(bf16_bits_rne(v.y)) << 16);
            o.y = static_cast<uint32_t>(bf16_bits_rne(v.z)) | (static_cast<uint32_t>(bf16_bits_rne(v.w)) << 16);
            __stcs(reinterpret_cast<uint2*>(dst) + q, o);
        }
        for (long long i = (quads << 2) + tid; i < count; i += nthreads) dst[i] = bf16_bits_rne(src[i]);
    } else {
        for (long long i = tid; i < count; i += nthreads) dst[i] = bf16_bits_rne(src[i]);
    }
}

}  // namespace lrgd
