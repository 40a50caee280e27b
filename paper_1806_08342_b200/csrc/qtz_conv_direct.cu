// CUDA-core convolution kernel of libqtz for geometries the other paths do not take.
//
//  * direct_conv_kernel: any kh x kw / stride / pad / channel count.  It serves the layers
//    the tensor-core path does not take (3-channel stem convolutions, odd geometries).  The
//    zero-point terms follow the expansion of Eq. 5-6: the raw u8 x s8 dot products are
//    corrected by -z_x sum(w) - z_w sum(x) + K z_x z_w per output.  Out-of-image taps are
//    staged as the code z_x (real zero, Section 2.1), so every output sees all K taps.
#include <algorithm>

#include "qtz_plan.cuh"

namespace {

__device__ __forceinline__ int32_t dp4a_us(uint32_t a, uint32_t b, int32_t c)
{
    int32_t d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// y = clamp(z_y + ((acc m + 2^(r-1)) >> r)): one 64-bit multiply-add, one shift.
__device__ __forceinline__ uint32_t requant_u8(int32_t acc, int32_t m, int32_t r, int32_t zy, int32_t lo, int32_t hi)
{
    const int64_t v = static_cast<int64_t>(acc) * m + (static_cast<int64_t>(1) << (r - 1));
    const int64_t y = (v >> r) + zy;
    return static_cast<uint32_t>(min(max(y, static_cast<int64_t>(lo)), static_cast<int64_t>(hi)));
}

struct DirectArgs {
    const uint8_t* x;
    const int8_t* w;
    const int32_t* bias;
    const int32_t* wsum;
    const int32_t* mult;
    const int32_t* rshift;
    void* y;
    int64_t pixels;
    int h, w_, c, xp, n, yp, kh, kw, stride, pad, oh, ow, k_total, k_padded;
    int zx, zw, zy, act_min, act_max, raw_out;
};

constexpr int kTilePx = 64, kTileN = 64, kChunk = 256, kRow = kChunk + 16, kDirectThreads = 256;

__global__ void __launch_bounds__(kDirectThreads)
direct_conv_kernel(const DirectArgs a)
{
    __shared__ __align__(16) uint8_t xs[kTilePx * kRow];
    __shared__ __align__(16) int8_t ws[kTileN * kRow];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t p0 = static_cast<int64_t>(blockIdx.x) * kTilePx;
    const int n0 = blockIdx.y * kTileN;

    int32_t acc[4][4];
    int32_t rowsum[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

    for (int k0 = 0; k0 < a.k_padded; k0 += kChunk) {
        const int span = min(kChunk, a.k_padded - k0);  // multiple of 16
        // activation window bytes: (pixel, k) -> (tap, channel) -> input byte or the code z_x
        for (int idx = tid; idx < kTilePx * span; idx += kDirectThreads) {
            const int p = idx / span, kk = idx - p * span, k = k0 + kk;
            const int64_t pix = p0 + p;
            uint8_t v = 0;
            if (pix < a.pixels && k < a.k_total) {
                const int tap = k / a.c, ch = k - tap * a.c;
                const int i = tap / a.kw, j = tap - i * a.kw;
                const int ow = static_cast<int>(pix % a.ow);
                const int64_t q = pix / a.ow;
                const int oh = static_cast<int>(q % a.oh);
                const int64_t b = q / a.oh;
                const int ih = oh * a.stride - a.pad + i, iw = ow * a.stride - a.pad + j;
                v = (ih >= 0 && ih < a.h && iw >= 0 && iw < a.w_)
                        ? a.x[((b * a.h + ih) * a.w_ + iw) * a.xp + ch]
                        : static_cast<uint8_t>(a.zx);
            }
            xs[p * kRow + kk] = v;
        }
        for (int idx = tid; idx < kTileN * (span >> 4); idx += kDirectThreads) {
            const int r = idx / (span >> 4), v = idx - r * (span >> 4);
            const int4 wv = *reinterpret_cast<const int4*>(a.w + static_cast<int64_t>(n0 + r) * a.k_padded + k0 + 16 * v);
            *reinterpret_cast<int4*>(ws + r * kRow + 16 * v) = wv;
        }
        __syncthreads();
        for (int kk = 0; kk < span; kk += 16) {
            uint4 xv[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const uint4*>(xs + (4 * ty + i) * kRow + kk);
#pragma unroll
            for (int j = 0; j < 4; ++j) wv[j] = *reinterpret_cast<const uint4*>(ws + (4 * tx + j) * kRow + kk);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[i][j] = dp4a_us(xv[i].x, wv[j].x, acc[i][j]);
                    acc[i][j] = dp4a_us(xv[i].y, wv[j].y, acc[i][j]);
                    acc[i][j] = dp4a_us(xv[i].z, wv[j].z, acc[i][j]);
                    acc[i][j] = dp4a_us(xv[i].w, wv[j].w, acc[i][j]);
                }
                if (a.zw != 0) {
                    rowsum[i] = dp4a_us(xv[i].x, 0x01010101u, rowsum[i]);
                    rowsum[i] = dp4a_us(xv[i].y, 0x01010101u, rowsum[i]);
                    rowsum[i] = dp4a_us(xv[i].z, 0x01010101u, rowsum[i]);
                    rowsum[i] = dp4a_us(xv[i].w, 0x01010101u, rowsum[i]);
                }
            }
        }
        __syncthreads();
    }

    // epilogue: cross terms of Eq. 5-6, bias, requantise, clamp, store 4 channels per pixel
    const int nb = n0 + 4 * tx;
    if (nb >= a.n) return;
    int32_t corr[4], m[4], r[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int nn = min(nb + j, a.n - 1);
        corr[j] = a.bias[nn] - a.zx * a.wsum[nn] + a.k_total * a.zx * a.zw;
        m[j] = a.raw_out ? 0 : a.mult[nn];
        r[j] = a.raw_out ? 1 : a.rshift[nn];
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t pix = p0 + 4 * ty + i;
        if (pix >= a.pixels) continue;
        int32_t full[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) full[j] = acc[i][j] + corr[j] - a.zw * rowsum[i];
        if (a.raw_out) {
            int32_t* out = static_cast<int32_t*>(a.y) + pix * a.n;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (nb + j < a.n) out[nb + j] = full[j];
        } else {
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                word |= requant_u8(full[j], m[j], r[j], a.zy, a.act_min, a.act_max) << (8 * j);
            *reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(a.y) + pix * a.yp + nb) = word;
        }
    }
}

}  // namespace

qtz_status qtz_direct_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, void* y, int32_t y_zp, int32_t act_min,
                             int32_t act_max, cudaStream_t st)
{
    const qtz_conv_desc& d = p->d;
    DirectArgs a{};
    a.x = x; a.w = p->w_direct; a.bias = p->bias; a.wsum = p->wsum; a.mult = p->mult; a.rshift = p->rshift; a.y = y;
    a.pixels = static_cast<int64_t>(d.batch) * p->oh * p->ow;
    a.h = d.h; a.w_ = d.w; a.c = d.c; a.xp = d.c_pitch_in; a.n = d.n; a.yp = d.c_pitch_out;
    a.kh = d.kh; a.kw = d.kw; a.stride = d.stride; a.pad = d.pad; a.oh = p->oh; a.ow = p->ow;
    a.k_total = p->k_total; a.k_padded = p->k_padded;
    a.zx = x_zp; a.zw = p->w_zp_signed; a.zy = y_zp; a.act_min = act_min; a.act_max = act_max;
    a.raw_out = d.outkind == QTZ_OUT_S32_RAW;
    const int64_t px_tiles = (a.pixels + kTilePx - 1) / kTilePx;
    if (px_tiles > 0x7fffffff) return QTZ_ERR_UNSUPPORTED;
    dim3 grid(static_cast<unsigned>(px_tiles), static_cast<unsigned>(p->n_padded / kTileN));
    if (p->ev_start) QTZ_CUDA(p->h, cudaEventRecord(p->ev_start, st));
    direct_conv_kernel<<<grid, kDirectThreads, 0, st>>>(a);
    QTZ_LAUNCH_CHECK(p->h, "direct_conv_kernel");
    if (p->ev_stop) QTZ_CUDA(p->h, cudaEventRecord(p->ev_stop, st));
    return QTZ_OK;
}
