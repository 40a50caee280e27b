// Small device helpers shared by the translation units of libqtz: the (min, max, non-finite) block
// reduction of the range kernels, and the reader of weight codes in the API layouts.
#pragma once

#include <cfloat>
#include <stdint.h>

#include "qtz.h"

namespace qtz_dev {

constexpr int kReduceThreads = 256;   // block size of every kernel that calls block_reduce

struct Range {
    float lo, hi;
    unsigned bad;  // non-zero when a NaN or Inf was met
};

__device__ __forceinline__ void range_take(Range& r, float v)
{
    r.bad |= ((__float_as_uint(v) & 0x7f800000u) == 0x7f800000u);
    r.lo = fminf(r.lo, v);
    r.hi = fmaxf(r.hi, v);
}

// Folds the Range of every thread of a kReduceThreads block; the result is valid in thread 0.
__device__ __forceinline__ Range block_reduce(Range r)
{
    __shared__ float s_lo[kReduceThreads / 32], s_hi[kReduceThreads / 32];
    __shared__ unsigned s_bad[kReduceThreads / 32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        r.lo = fminf(r.lo, __shfl_xor_sync(0xffffffffu, r.lo, off));
        r.hi = fmaxf(r.hi, __shfl_xor_sync(0xffffffffu, r.hi, off));
        r.bad |= __shfl_xor_sync(0xffffffffu, r.bad, off);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        s_lo[warp] = r.lo;
        s_hi[warp] = r.hi;
        s_bad[warp] = r.bad;
    }
    __syncthreads();
    if (warp == 0) {
        r.lo = lane < kReduceThreads / 32 ? s_lo[lane] : FLT_MAX;
        r.hi = lane < kReduceThreads / 32 ? s_hi[lane] : -FLT_MAX;
        r.bad = lane < kReduceThreads / 32 ? s_bad[lane] : 0u;
#pragma unroll
        for (int off = 4; off > 0; off >>= 1) {
            r.lo = fminf(r.lo, __shfl_xor_sync(0xffffffffu, r.lo, off));
            r.hi = fmaxf(r.hi, __shfl_xor_sync(0xffffffffu, r.hi, off));
            r.bad |= __shfl_xor_sync(0xffffffffu, r.bad, off);
        }
    }
    return r;
}

// Weight code k of output channel `row` from the API layout, moved to int8: int8 stays, uint8 is
// shifted by -128 (its zero point moves with it), a 4-bit code (two per byte, even element in the
// low nibble) is sign-extended.
__device__ __forceinline__ int32_t load_code_s8(const void* w, int wkind, int64_t row, int64_t k, int64_t k_total)
{
    if (wkind == QTZ_W_S8_PER_CHANNEL_SYM) return static_cast<const int8_t*>(w)[row * k_total + k];
    if (wkind == QTZ_W_U8_PER_LAYER_ASYM) return static_cast<int32_t>(static_cast<const uint8_t*>(w)[row * k_total + k]) - 128;
    const uint32_t byte = static_cast<const uint8_t*>(w)[row * ((k_total + 1) >> 1) + (k >> 1)];
    const uint32_t nib = (k & 1) ? (byte >> 4) : (byte & 0xfu);
    return static_cast<int32_t>(nib << 28) >> 28;
}

}  // namespace qtz_dev
