// Integer glue operations of a quantized network (Section 3.2.1): element-wise add with
// rescale and fused clamp, max pooling, global average pooling.  All HBM-bound; each
// thread moves 16 bytes per operand.
#include <algorithm>

#include "qtz_add_math.cuh"
#include "qtz_internal.cuh"

namespace {

constexpr int kThreads = 256;

using namespace qtz_add;

// y = clamp(z_y + (((a - z_a) m_a + (b - z_b) m_b + 2^(r-1)) >> r)).  All constants fold into one
// 64-bit addend: 2^(r-1) + (z_y - act_min) 2^r - z_a m_a - z_b m_b (|.| < 2^62 for r <= 53).
template <int kShiftKind>
__global__ void __launch_bounds__(kThreads)
add_u8_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ b, int64_t bytes, AddRule r,
              uint8_t* __restrict__ y)
{
    const int64_t addend = add_addend(r);
    const uint32_t lo4 = 0x01010101u * static_cast<uint32_t>(r.act_min);
    const int32_t span = r.act_max - r.act_min;
    const int64_t groups = bytes >> 4;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g >= groups) return;
    const uint4 va = __ldcs(reinterpret_cast<const uint4*>(a) + g);
    const uint4 vb = __ldcs(reinterpret_cast<const uint4*>(b) + g);
    uint4 o;
    if (kShiftKind == 3) {
        const AddSplit q = make_split(r);
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
// kK > 0: the window size, known at compile time, so that all its loads are in flight together (out-of-image
// taps read as 0, the neutral element of max over unsigned codes); kK = 0: any window.
template <int kK>
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
    if (kK > 0) {
        uint4 v[kK > 0 ? kK * kK : 1];
#pragma unroll
        for (int i = 0; i < kK; ++i)
#pragma unroll
            for (int j = 0; j < kK; ++j) {
                const int ih = oh * stride - pad + i, iw = ow * stride - pad + j;
                const bool in = ih >= 0 && ih < hh && iw >= 0 && iw < ww;
                v[i * kK + j] = in ? __ldg(reinterpret_cast<const uint4*>(x + ((static_cast<int64_t>(b) * hh + ih) * ww + iw) * pitch) + g)
                                   : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
        for (int q = 0; q < kK * kK; ++q) {
            m.x = __vmaxu4(m.x, v[q].x); m.y = __vmaxu4(m.y, v[q].y); m.z = __vmaxu4(m.z, v[q].z); m.w = __vmaxu4(m.w, v[q].w);
        }
    } else {
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
    // Eight loads in flight at a time; the four byte lanes are summed two to a register (16 bits each hold up to 256
    // pixels of 255) and unpacked once per 256 pixels.
    for (int p0 = 0; p0 < hw; p0 += 256) {
        const int p1 = min(hw, p0 + 256);
        uint32_t even = 0, odd = 0;
        int p = p0;
        for (; p + 8 <= p1; p += 8) {
            uint32_t v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = __ldg(reinterpret_cast<const uint32_t*>(base + static_cast<int64_t>(p + i) * pitch));
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                even += v[i] & 0x00ff00ffu;
                odd += (v[i] >> 8) & 0x00ff00ffu;
            }
        }
        for (; p < p1; ++p) {
            const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(base + static_cast<int64_t>(p) * pitch));
            even += v & 0x00ff00ffu;
            odd += (v >> 8) & 0x00ff00ffu;
        }
        s0 += even & 0xffff; s2 += even >> 16; s1 += odd & 0xffff; s3 += odd >> 16;
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
    const unsigned blocks = static_cast<unsigned>(ceil_div(total, kThreads));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (k == 3)
        maxpool_u8_kernel<3><<<blocks, kThreads, 0, st>>>(x_dev, y_dev, batch, hh, ww, c_pitch, k, stride, pad, oh_n, ow_n);
    else if (k == 2)
        maxpool_u8_kernel<2><<<blocks, kThreads, 0, st>>>(x_dev, y_dev, batch, hh, ww, c_pitch, k, stride, pad, oh_n, ow_n);
    else
        maxpool_u8_kernel<0><<<blocks, kThreads, 0, st>>>(x_dev, y_dev, batch, hh, ww, c_pitch, k, stride, pad, oh_n, ow_n);
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

// ---- 4-bit activation storage (Section 3.2.4) ---------------------------------------------------
namespace {

constexpr int kPackThreads = 256;

// One thread per packed byte (generic) or per four packed bytes (rows 4-byte aligned on both sides).
__global__ void __launch_bounds__(kPackThreads)
pack_u4_kernel(const uint8_t* __restrict__ x, int64_t pixels, int c, int x_pitch, uint8_t* __restrict__ y, int y_pitch, int fast)
{
    const int bytes = (c + 1) >> 1;
    const int per_row = fast ? (bytes + 3) >> 2 : bytes;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kPackThreads + threadIdx.x;
    if (t >= pixels * per_row) return;
    const int64_t p = t / per_row;
    const int j = static_cast<int>(t - p * per_row);
    const uint8_t* row = x + p * x_pitch;
    uint8_t* out = y + p * y_pitch;
    if (fast && 8 * j + 8 <= c) {          // eight codes in, four bytes out
        const uint2 v = *reinterpret_cast<const uint2*>(row + 8 * j);
        const uint32_t lo = v.x & 0x0f0f0f0fu, hi = v.y & 0x0f0f0f0fu;
        // bytes (a0 a1 a2 a3) -> (a0 | a1 << 4), (a2 | a3 << 4)
        const uint32_t l2 = (lo | (lo >> 4)) & 0x00ff00ffu, h2 = (hi | (hi >> 4)) & 0x00ff00ffu;
        const uint32_t l = (l2 | (l2 >> 8)) & 0xffffu, hh = (h2 | (h2 >> 8)) & 0xffffu;
        *reinterpret_cast<uint32_t*>(out + 4 * j) = l | (hh << 16);
        return;
    }
    const int first = fast ? 4 * j : j, last = fast ? min(4 * j + 4, bytes) : j + 1;
    for (int b = first; b < last; ++b) {
        const uint32_t lo = row[2 * b] & 0xfu, hi = 2 * b + 1 < c ? (row[2 * b + 1] & 0xfu) : 0u;
        out[b] = static_cast<uint8_t>(lo | (hi << 4));
    }
}

__global__ void __launch_bounds__(kPackThreads)
unpack_u4_kernel(const uint8_t* __restrict__ x, int64_t pixels, int c, int x_pitch, uint8_t* __restrict__ y, int y_pitch, int fast)
{
    const int bytes = (c + 1) >> 1;
    const int per_row = fast ? (bytes + 3) >> 2 : bytes;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kPackThreads + threadIdx.x;
    if (t >= pixels * per_row) return;
    const int64_t p = t / per_row;
    const int j = static_cast<int>(t - p * per_row);
    const uint8_t* row = x + p * x_pitch;
    uint8_t* out = y + p * y_pitch;
    if (fast && 8 * j + 8 <= c) {          // four bytes in, eight codes out
        const uint32_t v = *reinterpret_cast<const uint32_t*>(row + 4 * j);
        const uint32_t even = v & 0x0f0f0f0fu, odd = (v >> 4) & 0x0f0f0f0fu;       // codes 0,2,4,6 and 1,3,5,7
        uint2 o;
        o.x = __byte_perm(even, odd, 0x5140);                                       // c0 c1 c2 c3
        o.y = __byte_perm(even, odd, 0x7362);                                       // c4 c5 c6 c7
        *reinterpret_cast<uint2*>(out + 8 * j) = o;
        return;
    }
    const int first = fast ? 4 * j : j, last = fast ? min(4 * j + 4, bytes) : j + 1;
    for (int b = first; b < last; ++b) {
        const uint32_t v = row[b];
        out[2 * b] = static_cast<uint8_t>(v & 0xfu);
        if (2 * b + 1 < c) out[2 * b + 1] = static_cast<uint8_t>(v >> 4);
    }
}

qtz_status pack_args_ok(qtz_handle h, const void* x, const void* y, int64_t pixels, int32_t c, int32_t wide_pitch, int32_t packed_pitch)
{
    if (!h || !x || !y || pixels <= 0 || c <= 0 || wide_pitch < c || packed_pitch < (c + 1) / 2) return QTZ_ERR_INVALID_ARG;
    if (pixels > (INT64_MAX / 4) / (c + 8)) return QTZ_ERR_INVALID_ARG;
    return QTZ_OK;
}

}  // namespace

extern "C" qtz_status qtz_pack_u4(qtz_handle h, const uint8_t* x_dev, int64_t pixels, int32_t c, int32_t x_pitch,
                                  uint8_t* y_dev, int32_t y_pitch, void* stream)
{
    qtz_status s = pack_args_ok(h, x_dev, y_dev, pixels, c, x_pitch, y_pitch);
    if (s != QTZ_OK) return s;
    const int fast = ((reinterpret_cast<uintptr_t>(x_dev) & 7u) == 0 && (x_pitch & 7) == 0 &&
                      (reinterpret_cast<uintptr_t>(y_dev) & 3u) == 0 && (y_pitch & 3) == 0) ? 1 : 0;
    const int bytes = (c + 1) >> 1;
    const int64_t work = pixels * (fast ? (bytes + 3) >> 2 : bytes);
    pack_u4_kernel<<<static_cast<unsigned>((work + kPackThreads - 1) / kPackThreads), kPackThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        x_dev, pixels, c, x_pitch, y_dev, y_pitch, fast);
    QTZ_LAUNCH_CHECK(h, "pack_u4_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_unpack_u4(qtz_handle h, const uint8_t* x_dev, int64_t pixels, int32_t c, int32_t x_pitch,
                                    uint8_t* y_dev, int32_t y_pitch, void* stream)
{
    qtz_status s = pack_args_ok(h, x_dev, y_dev, pixels, c, y_pitch, x_pitch);
    if (s != QTZ_OK) return s;
    const int fast = ((reinterpret_cast<uintptr_t>(x_dev) & 3u) == 0 && (x_pitch & 3) == 0 &&
                      (reinterpret_cast<uintptr_t>(y_dev) & 7u) == 0 && (y_pitch & 7) == 0) ? 1 : 0;
    const int bytes = (c + 1) >> 1;
    const int64_t work = pixels * (fast ? (bytes + 3) >> 2 : bytes);
    unpack_u4_kernel<<<static_cast<unsigned>((work + kPackThreads - 1) / kPackThreads), kPackThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        x_dev, pixels, c, x_pitch, y_dev, y_pitch, fast);
    QTZ_LAUNCH_CHECK(h, "unpack_u4_kernel");
    return QTZ_OK;
}
