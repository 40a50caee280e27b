// Device arithmetic of the 3x3 depthwise convolution (Eq. 5-6 with K = 9, then the requantisation of Section 2.3's
// integer pipeline), shared by the stand-alone depthwise kernel and by the fused depthwise -> pointwise kernel: a
// thread owns 4 channels x 2 adjacent output columns, keeps three byte-transposed input rows in registers and
// spends three dp4a per output.
#pragma once
#include <cstdint>

namespace qtz_dw {

// Requantisation forms (template parameter kMode).
constexpr int kModeGeneral = 0;   // any right shift, 64-bit arithmetic throughout
constexpr int kModeFast = 1;      // right shifts 32..53: one 64-bit multiply-add, then a shift of the high word
constexpr int kModeRaw = 2;       // int32 accumulators out, no requantisation
constexpr int kNumModes = 3;


__device__ __forceinline__ int32_t dp4a_us(uint32_t a, uint32_t b, int32_t c)
{
    int32_t d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// d = (c << 16) | (sat_u8(a) << 8) | sat_u8(b)
__device__ __forceinline__ uint32_t pack_sat_u8(int32_t a, int32_t b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// 4x4 byte transpose: a_j holds 4 channels of pixel j; t[ch] receives 4 pixels of channel ch.
__device__ __forceinline__ void transpose4(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t* t)
{
    const uint32_t lo01 = __byte_perm(a0, a1, 0x5140), hi01 = __byte_perm(a0, a1, 0x7362);
    const uint32_t lo23 = __byte_perm(a2, a3, 0x5140), hi23 = __byte_perm(a2, a3, 0x7362);
    t[0] = __byte_perm(lo01, lo23, 0x5410);
    t[1] = __byte_perm(lo01, lo23, 0x7632);
    t[2] = __byte_perm(hi01, hi23, 0x5410);
    t[3] = __byte_perm(hi01, hi23, 0x7632);
}

// One input row as the two output columns of a thread see it, 4 channels.
//   stride 1: t[ch] = pixels (w0-1, w0, w0+1, w0+2): column w0 reads bytes 0..2, column w0+1 bytes 1..3
//   stride 2: t[ch] = inputs (2w0, .., 2w0+3): column w0+1 reads bytes 1..3;
//             l[ch] = inputs (2w0-1, 2w0, 2w0+1, -): column w0 reads bytes 0..2
template <int kStride>
struct RowState {
    uint32_t t[4];
    uint32_t l[kStride == 2 ? 4 : 1];
};

// Pixel offsets of a thread's window inside a tile row (multiples of the pixel pitch).
struct WinOffsets {
    uint32_t o1, o2, o3, o4;
};

// Reads the thread's window of one tile row from shared memory.  `cell` is the shared-memory
// address of the first window pixel of that row (4 channels of the thread).
template <int kStride>
__device__ __forceinline__ void load_row(uint32_t cell, const WinOffsets& o, RowState<kStride>& r)
{
    const uint32_t p0 = lds_u32(cell), p1 = lds_u32(cell + o.o1), p2 = lds_u32(cell + o.o2), p3 = lds_u32(cell + o.o3);
    if (kStride == 1) {
        transpose4(p0, p1, p2, p3, r.t);
    } else {
        const uint32_t p4 = lds_u32(cell + o.o4);
        transpose4(p1, p2, p3, p4, r.t);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) r.l[ch] = __byte_perm(p0, r.t[ch], 0x6540 | ch);
    }
}

// Per-thread constants of its four channels.
template <int kMode>
struct ChanConst {
    uint32_t wa[3][4];                              // per filter row: bytes (k0,k1,k2,0)
    uint32_t wb[3][4];                              // per filter row: bytes (0,k0,k1,k2)
    int32_t m[4];
    int32_t sh[4];                                  // kModeGeneral: r;  kModeFast: r - 32
    int64_t add[kMode == kModeFast ? 4 : 1];        // 2^(r-1) + ((z_y - act_min) << r) + base * m
    int32_t base[kMode == kModeFast ? 1 : 4];       // bias - z_x sum(w) + 9 z_x z_w (kModeFast folds it into `add`)
    uint32_t lo4;                                   // act_min in every byte
    int32_t span;                                   // act_max - act_min
    int32_t off;                                    // z_y - act_min
    int32_t zw;
};

// The nine taps of one output row for the thread's two columns: filter row i applied to input row i.
template <int kStride, bool kAsym, int kMode>
__device__ __forceinline__ void mac3(const RowState<kStride>& r0, const RowState<kStride>& r1, const RowState<kStride>& r2,
                                     const ChanConst<kMode>& k, int32_t (&acc)[2][4])
{
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        const uint32_t f0 = kStride == 1 ? r0.t[ch] : r0.l[kStride == 2 ? ch : 0];
        const uint32_t f1 = kStride == 1 ? r1.t[ch] : r1.l[kStride == 2 ? ch : 0];
        const uint32_t f2 = kStride == 1 ? r2.t[ch] : r2.l[kStride == 2 ? ch : 0];
        const int32_t init = kMode == kModeFast ? 0 : k.base[kMode == kModeFast ? 0 : ch];
        acc[0][ch] = dp4a_us(f2, k.wa[2][ch], dp4a_us(f1, k.wa[1][ch], dp4a_us(f0, k.wa[0][ch], init)));
        acc[1][ch] = dp4a_us(r2.t[ch], k.wb[2][ch], dp4a_us(r1.t[ch], k.wb[1][ch], dp4a_us(r0.t[ch], k.wb[0][ch], init)));
        if (kAsym) {   // uint8 weights: subtract z_w times the sum of the window
            const int32_t s0 = dp4a_us(f2, 0x00010101u, dp4a_us(f1, 0x00010101u, dp4a_us(f0, 0x00010101u, 0)));
            const int32_t s1 = dp4a_us(r2.t[ch], 0x01010100u, dp4a_us(r1.t[ch], 0x01010100u, dp4a_us(r0.t[ch], 0x01010100u, 0)));
            acc[0][ch] -= k.zw * s0;
            acc[1][ch] -= k.zw * s1;
        }
    }
}

// Requantises 4 channels of one pixel and returns them as one packed word.  The clamp is done
// relative to act_min: max(min(y - act_min, span), 0) is a single instruction, act_min is added
// back to all four bytes at once.  Without kClamp (act_min = 0, act_max = 255) the saturating
// pack is the clamp.
template <int kMode, bool kClamp>
__device__ __forceinline__ uint32_t requant_pixel(const int32_t (&v)[4], const ChanConst<kMode>& k)
{
    int32_t y[4];
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        if (kMode == kModeFast) {          // floor((v m + addend) / 2^r) = hi32(v m + addend) >> (r - 32)
            const int64_t p = static_cast<int64_t>(v[ch]) * k.m[ch] + k.add[kMode == kModeFast ? ch : 0];
            y[ch] = static_cast<int32_t>(p >> 32) >> k.sh[ch];
            if (kClamp) y[ch] = __vimin_s32_relu(y[ch], k.span);
        } else {
            const int64_t p = static_cast<int64_t>(v[ch]) * k.m[ch] + (static_cast<int64_t>(1) << (k.sh[ch] - 1));
            const int64_t s = (p >> k.sh[ch]) + k.off;
            y[ch] = static_cast<int32_t>(min(max(s, static_cast<int64_t>(0)), static_cast<int64_t>(k.span)));
        }
    }
    const uint32_t o = pack_sat_u8(y[1], y[0], pack_sat_u8(y[3], y[2], 0u));
    return (kClamp || kMode == kModeGeneral) ? o + k.lo4 : o;
}

}  // namespace qtz_dw
