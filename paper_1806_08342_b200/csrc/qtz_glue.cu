// Integer glue operations of a quantized network (Section 3.2.1): element-wise add with
// rescale and fused clamp, max pooling, global average pooling.  All HBM-bound; each
// thread moves 16 bytes per operand.
#include <algorithm>

#include "qtz_internal.cuh"

namespace {

constexpr int kThreads = 256;

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

// y = clamp(z_y + (((a - z_a) m_a + (b - z_b) m_b + 2^(r-1)) >> r)).  All constants fold into one
// 64-bit addend: 2^(r-1) + (z_y - act_min) 2^r - z_a m_a - z_b m_b (|.| < 2^62 for r <= 53).
template <int kShiftKind>
__global__ void __launch_bounds__(kThreads)
add_u8_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ b, int64_t bytes, AddRule r,
              uint8_t* __restrict__ y)
{
    const int64_t addend = (static_cast<int64_t>(1) << (r.rshift - 1)) +
                           static_cast<int64_t>(r.y_zp - r.act_min) * (static_cast<int64_t>(1) << r.rshift) -
                           static_cast<int64_t>(r.a_zp) * r.a_mult - static_cast<int64_t>(r.b_zp) * r.b_mult;
    const uint32_t lo4 = 0x01010101u * static_cast<uint32_t>(r.act_min);
    const int32_t span = r.act_max - r.act_min;
    const int64_t groups = bytes >> 4;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g >= groups) return;
    const uint4 va = __ldcs(reinterpret_cast<const uint4*>(a) + g);
    const uint4 vb = __ldcs(reinterpret_cast<const uint4*>(b) + g);
    uint4 o;
    if (kShiftKind == 3) {
        AddSplit q;
        q.mh = (static_cast<uint32_t>(r.a_mult) >> 16) | (static_cast<uint32_t>(r.b_mult) & 0xffff0000u);
        q.ml = (static_cast<uint32_t>(r.a_mult) & 0xffffu) | (static_cast<uint32_t>(r.b_mult) << 16);
        q.ah = static_cast<int32_t>(addend >> 16);
        q.al = static_cast<uint32_t>(addend) & 0xffffu;
        q.sh = r.rshift - 16;
        q.span = span;
        o.x = add_split4(va.x, vb.x, q, lo4); o.y = add_split4(va.y, vb.y, q, lo4);
        o.z = add_split4(va.z, vb.z, q, lo4); o.w = add_split4(va.w, vb.w, q, lo4);
        reinterpret_cast<uint4*>(y)[g] = o;
        return;
    }
    o.x = add4<kShiftKind == 3 ? 0 : kShiftKind>(va.x, vb.x, r, addend, span, lo4); o.y = add4<kShiftKind == 3 ? 0 : kShiftKind>(va.y, vb.y, r, addend, span, lo4);
    o.z = add4<kShiftKind == 3 ? 0 : kShiftKind>(va.z, vb.z, r, addend, span, lo4);
    o.w = add4<kShiftKind == 3 ? 0 : kShiftKind>(va.w, vb.w, r, addend, span, lo4);
    reinterpret_cast<uint4*>(y)[g] = o;
}

// One thread per (output pixel, 16-channel group).
__global__ void __launch_bounds__(kThreads)
maxpool_u8_kernel(const uint8_t* __restrict__ x, uint8_t* __restrict__ y, int batch, int hh, int ww, int pitch,
                  int k, int stride, int pad, int oh_n, int ow_n)
{
    const int groups = pitch >> 4;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    const int64_t total = static_cast<int64_t>(batch) * oh_n * ow_n * groups;
    if (t >= total) return;
    const int g = static_cast<int>(t % groups);
    int64_t p = t / groups;
    const int ow = static_cast<int>(p % ow_n); p /= ow_n;
    const int oh = static_cast<int>(p % oh_n);
    const int b = static_cast<int>(p / oh_n);
    uint4 m = make_uint4(0, 0, 0, 0);
    for (int i = 0; i < k; ++i) {
        const int ih = oh * stride - pad + i;
        if (ih < 0 || ih >= hh) continue;
        for (int j = 0; j < k; ++j) {
            const int iw = ow * stride - pad + j;
            if (iw < 0 || iw >= ww) continue;
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + ((static_cast<int64_t>(b) * hh + ih) * ww + iw) * pitch) + g);
            m.x = __vmaxu4(m.x, v.x); m.y = __vmaxu4(m.y, v.y); m.z = __vmaxu4(m.z, v.z); m.w = __vmaxu4(m.w, v.w);
        }
    }
    reinterpret_cast<uint4*>(y + ((static_cast<int64_t>(b) * oh_n + oh) * ow_n + ow) * pitch)[g] = m;
}

// One thread per (image, 4-channel group); sums hw pixels, then one requantisation.
__global__ void __launch_bounds__(kThreads)
global_avgpool_u8_kernel(const uint8_t* __restrict__ x, int32_t x_zp, uint8_t* __restrict__ y, int32_t y_zp,
                         int32_t mult, int32_t rshift, int batch, int hw, int pitch)
{
    const int groups = pitch >> 2;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (t >= static_cast<int64_t>(batch) * groups) return;
    const int g = static_cast<int>(t % groups), b = static_cast<int>(t / groups);
    int32_t s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    const uint8_t* base = x + static_cast<int64_t>(b) * hw * pitch + 4 * g;
    for (int p = 0; p < hw; ++p) {
        const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(base + static_cast<int64_t>(p) * pitch));
        s0 += v & 0xff; s1 += (v >> 8) & 0xff; s2 += (v >> 16) & 0xff; s3 += v >> 24;
    }
    const int64_t rnd = static_cast<int64_t>(1) << (rshift - 1);
    const int32_t off = hw * x_zp;
    auto rq = [&](int32_t s) -> uint32_t {
        const int64_t v = static_cast<int64_t>(s - off) * mult + rnd;
        const int64_t r = static_cast<int64_t>(y_zp) + (v >> rshift);
        return static_cast<uint32_t>(r < 0 ? 0 : (r > 255 ? 255 : r));
    };
    reinterpret_cast<uint32_t*>(y + static_cast<int64_t>(b) * pitch)[g] = rq(s0) | (rq(s1) << 8) | (rq(s2) << 16) | (rq(s3) << 24);
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

}  // namespace

extern "C" qtz_status qtz_add_u8(qtz_handle h, const uint8_t* a_dev, int32_t a_zp, int32_t a_mult,
                                 const uint8_t* b_dev, int32_t b_zp, int32_t b_mult, int32_t rshift, uint8_t* y_dev,
                                 int32_t y_zp, int32_t act_min, int32_t act_max, int64_t pixels, int32_t c,
                                 int32_t c_pitch, void* stream)
{
    if (!h || !a_dev || !b_dev || !y_dev || pixels <= 0 || c <= 0 || c_pitch < c) return QTZ_ERR_INVALID_ARG;
    if (a_mult < 0 || b_mult < 0 || act_min < 0 || act_max > 255 || act_min > act_max) return QTZ_ERR_INVALID_ARG;
    if (y_zp < 0 || y_zp > 255 || a_zp < 0 || a_zp > 255 || b_zp < 0 || b_zp > 255) return QTZ_ERR_INVALID_ARG;
    if (rshift < 1 || rshift > 53) return QTZ_ERR_UNSUPPORTED;
    if ((c_pitch & 15) || !qtz_aligned16(a_dev) || !qtz_aligned16(b_dev) || !qtz_aligned16(y_dev)) return QTZ_ERR_MISALIGNED;
    const int64_t bytes = pixels * c_pitch;
    const AddRule r{a_zp, a_mult, b_zp, b_mult, rshift, y_zp, act_min, act_max};
    const unsigned blocks = static_cast<unsigned>(ceil_div(bytes >> 4, kThreads));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (rshift >= 16 && rshift <= 38)
        add_u8_kernel<3><<<blocks, kThreads, 0, st>>>(a_dev, b_dev, bytes, r, y_dev);
    else if (rshift >= 32)
        add_u8_kernel<0><<<blocks, kThreads, 0, st>>>(a_dev, b_dev, bytes, r, y_dev);
    else if (rshift >= 10)
        add_u8_kernel<1><<<blocks, kThreads, 0, st>>>(a_dev, b_dev, bytes, r, y_dev);
    else
        add_u8_kernel<2><<<blocks, kThreads, 0, st>>>(a_dev, b_dev, bytes, r, y_dev);
    QTZ_LAUNCH_CHECK(h, "add_u8_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_maxpool_u8(qtz_handle h, const uint8_t* x_dev, uint8_t* y_dev, int32_t batch, int32_t hh,
                                     int32_t ww, int32_t c, int32_t c_pitch, int32_t k, int32_t stride, int32_t pad,
                                     void* stream)
{
    if (!h || !x_dev || !y_dev || batch <= 0 || hh <= 0 || ww <= 0 || c <= 0 || c_pitch < c || k <= 0 || stride <= 0 ||
        pad < 0 || pad >= k)
        return QTZ_ERR_INVALID_ARG;
    if ((c_pitch & 15) || !qtz_aligned16(x_dev) || !qtz_aligned16(y_dev)) return QTZ_ERR_MISALIGNED;
    const int oh_n = (hh + 2 * pad - k) / stride + 1, ow_n = (ww + 2 * pad - k) / stride + 1;
    if (oh_n <= 0 || ow_n <= 0) return QTZ_ERR_INVALID_ARG;
    const int64_t total = static_cast<int64_t>(batch) * oh_n * ow_n * (c_pitch >> 4);
    maxpool_u8_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        x_dev, y_dev, batch, hh, ww, c_pitch, k, stride, pad, oh_n, ow_n);
    QTZ_LAUNCH_CHECK(h, "maxpool_u8_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_global_avgpool_u8(qtz_handle h, const uint8_t* x_dev, int32_t x_zp, uint8_t* y_dev,
                                            int32_t y_zp, int32_t mult, int32_t rshift, int32_t batch, int32_t hw,
                                            int32_t c, int32_t c_pitch, void* stream)
{
    if (!h || !x_dev || !y_dev || batch <= 0 || hw <= 0 || c <= 0 || c_pitch < c || mult < 0) return QTZ_ERR_INVALID_ARG;
    if (rshift < 1 || rshift > 62 || x_zp < 0 || x_zp > 255 || y_zp < 0 || y_zp > 255) return QTZ_ERR_INVALID_ARG;
    if (hw > (1 << 22)) return QTZ_ERR_OVERFLOW;
    if ((c_pitch & 15) || !qtz_aligned16(x_dev) || !qtz_aligned16(y_dev)) return QTZ_ERR_MISALIGNED;
    const int64_t total = static_cast<int64_t>(batch) * (c_pitch >> 2);
    global_avgpool_u8_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        x_dev, x_zp, y_dev, y_zp, mult, rshift, batch, hw, c_pitch);
    QTZ_LAUNCH_CHECK(h, "global_avgpool_u8_kernel");
    return QTZ_OK;
}
