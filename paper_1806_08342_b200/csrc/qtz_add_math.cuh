// Arithmetic of the element-wise add of two quantized tensors (Section 3.2.1), shared by the stand-alone
// add kernel and by the convolution epilogue that fuses a residual add.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace qtz_add {

struct AddRule {
    int32_t a_zp, a_mult, b_zp, b_mult, rshift, y_zp, act_min, act_max;
};

// d = (c << 16) | (sat_u8(a) << 8) | sat_u8(b)
__device__ __forceinline__ uint32_t pack_sat_u8(int32_t a, int32_t b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// (a m_a + b m_b + addend) >> r for one byte lane, relative to act_min and clamped to
// [0, act_max - act_min]; the zero points, the rounding constant and (z_y - act_min) 2^r are all
// inside `addend`.  |a m| < 2^39, so the shifted value fits 32 bits whenever r >= 10; smaller
// shifts take the 64-bit route.
template <int kShiftKind>  // 0: r >= 32, 1: 10 <= r < 32, 2: r < 10
__device__ __forceinline__ int32_t add1(uint32_t a, uint32_t b, const AddRule& r, int64_t addend, int32_t span)
{
    const int64_t v = static_cast<int64_t>(static_cast<uint64_t>(a) * static_cast<uint32_t>(r.a_mult)) +
                      static_cast<int64_t>(static_cast<uint64_t>(b) * static_cast<uint32_t>(r.b_mult)) + addend;
    if (kShiftKind == 0) return __vimin_s32_relu(static_cast<int32_t>(v >> 32) >> (r.rshift - 32), span);
    if (kShiftKind == 1)
        return __vimin_s32_relu(static_cast<int32_t>(__funnelshift_r(static_cast<uint32_t>(v), static_cast<uint32_t>(v >> 32), r.rshift)), span);
    const int64_t s = v >> r.rshift;
    return static_cast<int32_t>(min(max(s, static_cast<int64_t>(0)), static_cast<int64_t>(span)));
}

template <int kShiftKind>
__device__ __forceinline__ uint32_t add4(uint32_t a, uint32_t b, const AddRule& r, int64_t addend, int32_t span, uint32_t lo4)
{
    const int32_t y0 = add1<kShiftKind>(a & 0xff, b & 0xff, r, addend, span);
    const int32_t y1 = add1<kShiftKind>((a >> 8) & 0xff, (b >> 8) & 0xff, r, addend, span);
    const int32_t y2 = add1<kShiftKind>((a >> 16) & 0xff, (b >> 16) & 0xff, r, addend, span);
    const int32_t y3 = add1<kShiftKind>(a >> 24, b >> 24, r, addend, span);
    return pack_sat_u8(y1, y0, pack_sat_u8(y3, y2, 0u)) + lo4;
}

// The same for shifts 16 <= r <= 38 without 64-bit multiplies.  With m = mh 2^16 + ml (both halves below 2^16):
//   a m_a + b m_b + addend = (a mah + b mbh + Ah) 2^16 + (a mal + b mbl + Al),  addend = Ah 2^16 + Al, 0 <= Al < 2^16,
// every bracket fits 32 bits (a, b < 2^8; |addend| < 2^47), and since floor(floor(x / 2^16) / 2^(r-16)) =
// floor(x / 2^r) the result is ((hi + Ah + (lo >> 16)) >> (r - 16)) exactly.  Each bracket is one dp2a on the
// byte pair (a, b) against the 16-bit pair (m_a half, m_b half).
struct AddSplit {
    uint32_t mh, ml;     // (mah | mbh << 16), (mal | mbl << 16)
    int32_t ah;          // addend >> 16 (arithmetic)
    uint32_t al;         // addend & 0xffff
    int32_t sh, span;    // r - 16, act_max - act_min
};

__device__ __forceinline__ uint32_t dp2a_lo(uint32_t m16x2, uint32_t bytes, uint32_t c)
{
    uint32_t d;
    asm("dp2a.lo.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(m16x2), "r"(bytes), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t dp2a_hi(uint32_t m16x2, uint32_t bytes, uint32_t c)
{
    uint32_t d;
    asm("dp2a.hi.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(m16x2), "r"(bytes), "r"(c));
    return d;
}

__device__ __forceinline__ int32_t add_split1(uint32_t hi, uint32_t lo, const AddSplit& q)
{
    return __vimin_s32_relu((static_cast<int32_t>(hi) + q.ah + static_cast<int32_t>(lo >> 16)) >> q.sh, q.span);
}

__device__ __forceinline__ uint32_t add_split4(uint32_t a, uint32_t b, const AddSplit& q, uint32_t lo4)
{
    const uint32_t p01 = __byte_perm(a, b, 0x5140), p23 = __byte_perm(a, b, 0x7362);   // (a0,b0,a1,b1), (a2,b2,a3,b3)
    const int32_t y0 = add_split1(dp2a_lo(q.mh, p01, 0u), dp2a_lo(q.ml, p01, q.al), q);
    const int32_t y1 = add_split1(dp2a_hi(q.mh, p01, 0u), dp2a_hi(q.ml, p01, q.al), q);
    const int32_t y2 = add_split1(dp2a_lo(q.mh, p23, 0u), dp2a_lo(q.ml, p23, q.al), q);
    const int32_t y3 = add_split1(dp2a_hi(q.mh, p23, 0u), dp2a_hi(q.ml, p23, q.al), q);
    return pack_sat_u8(y1, y0, pack_sat_u8(y3, y2, 0u)) + lo4;
}


// The 64-bit addend of y - act_min = (a m_a + b m_b + addend) >> r: rounding constant, output offset and both zero points.
__host__ __device__ inline int64_t add_addend(const AddRule& r)
{
    return (static_cast<int64_t>(1) << (r.rshift - 1)) + static_cast<int64_t>(r.y_zp - r.act_min) * (static_cast<int64_t>(1) << r.rshift) -
           static_cast<int64_t>(r.a_zp) * r.a_mult - static_cast<int64_t>(r.b_zp) * r.b_mult;
}

__host__ __device__ inline AddSplit make_split(const AddRule& r)
{
    const int64_t addend = add_addend(r);
    AddSplit q;
    q.mh = (static_cast<uint32_t>(r.a_mult) >> 16) | (static_cast<uint32_t>(r.b_mult) & 0xffff0000u);
    q.ml = (static_cast<uint32_t>(r.a_mult) & 0xffffu) | (static_cast<uint32_t>(r.b_mult) << 16);
    q.ah = static_cast<int32_t>(addend >> 16);
    q.al = static_cast<uint32_t>(addend) & 0xffffu;
    q.sh = r.rshift - 16;
    q.span = r.act_max - r.act_min;
    return q;
}

}  // namespace qtz_add
