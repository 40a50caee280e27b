// Quantizer utilities around the convolution path: simulated quantization (Section 2.4), the
// signal-to-quantization-noise ratio of Appendix A, the moving average of activation ranges
// over batches (Section 2.5, host arithmetic) and the rescale of a uint8 tensor to another
// quantizer (what a concatenation needs, Section 3.2.1).  The device kernels are HBM-bound
// streams with 16-byte accesses where the view allows.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "qtz_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kSqnrChunksMax = 1024;

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------------------------
// SimQuant: Eq. 1-2 followed by Eq. 3, with the quantizer's fp32 steps (one IEEE division,
// round-half-even, clamp) and the de-quantizer's single fp32 multiply.
// ------------------------------------------------------------------------------------
struct SimRule {
    float scale, tlo, thi;  // clamp bounds already shifted by -z
};

__device__ __forceinline__ float sim1(float x, const SimRule& q)
{
    float t = rintf(__fdiv_rn(x, q.scale));
    t = fminf(fmaxf(t, q.tlo), q.thi);
    // (q - z) as an integer and back: the value is t itself, but a negative zero becomes +0 as it
    // does when the code is formed and the zero point subtracted again
    return __fmul_rn(static_cast<float>(static_cast<int32_t>(t)), q.scale);
}

__device__ __forceinline__ float4 sim4(const float4& v, const SimRule& q)
{
    return make_float4(sim1(v.x, q), sim1(v.y, q), sim1(v.z, q), sim1(v.w, q));
}

// Per-layer: 16 values per thread, four 16-byte loads and stores.  Needs 16-byte aligned pointers.
__global__ void __launch_bounds__(kThreads)
simquant_flat_kernel(const float* __restrict__ x, int64_t n, SimRule q, float* __restrict__ y)
{
    const int64_t groups = n >> 4;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g < groups) {
        const float4* xv = reinterpret_cast<const float4*>(x) + 4 * g;
        float4* yv = reinterpret_cast<float4*>(y) + 4 * g;
        const float4 a = __ldcs(xv), b = __ldcs(xv + 1), c = __ldcs(xv + 2), d = __ldcs(xv + 3);
        __stcs(yv, sim4(a, q));
        __stcs(yv + 1, sim4(b, q));
        __stcs(yv + 2, sim4(c, q));
        __stcs(yv + 3, sim4(d, q));
    } else if (g == groups) {
        for (int64_t i = groups << 4; i < n; ++i) y[i] = sim1(x[i], q);
    }
}

// Any view: one value per thread, the rule fetched per axis index.
__global__ void __launch_bounds__(kThreads)
simquant_axis_kernel(const float* __restrict__ x, int64_t total, int64_t axis_len, int64_t inner,
                     const SimRule* __restrict__ rules, float* __restrict__ y)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    y[i] = sim1(x[i], rules[(i / inner) % axis_len]);
}

// ------------------------------------------------------------------------------------
// SQNR: per axis index, sum w^2 and sum (w - w_hat)^2 in fp64.  Block (chunk, a) reduces its
// share of slice a in a fixed order and leaves one pair in `partial`; a second kernel adds the
// chunks of each slice in order, so the result does not depend on scheduling.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
sqnr_partial_kernel(const float* __restrict__ w, const float* __restrict__ w_hat, int64_t outer, int64_t axis_len,
                    int64_t inner, double* __restrict__ partial)
{
    const int64_t a = blockIdx.y;
    const int64_t count = outer * inner;
    double signal = 0.0, noise = 0.0;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; j < count;
         j += static_cast<int64_t>(gridDim.x) * kThreads) {
        int64_t idx = j;
        if (axis_len > 1) {
            const int64_t o = j / inner, i = j - o * inner;
            idx = (o * axis_len + a) * inner + i;
        }
        const double v = static_cast<double>(__ldg(w + idx));
        const double e = v - static_cast<double>(__ldg(w_hat + idx));
        signal = __dadd_rn(signal, __dmul_rn(v, v));
        noise = __dadd_rn(noise, __dmul_rn(e, e));
    }
    __shared__ double s_sig[kThreads / 32], s_noi[kThreads / 32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        signal += __shfl_xor_sync(0xffffffffu, signal, off);
        noise += __shfl_xor_sync(0xffffffffu, noise, off);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        s_sig[warp] = signal;
        s_noi[warp] = noise;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0, n = 0.0;
        for (int k = 0; k < kThreads / 32; ++k) {
            s += s_sig[k];
            n += s_noi[k];
        }
        partial[(a * gridDim.x + blockIdx.x) * 2 + 0] = s;
        partial[(a * gridDim.x + blockIdx.x) * 2 + 1] = n;
    }
}

__global__ void __launch_bounds__(kThreads)
sqnr_finish_kernel(const double* __restrict__ partial, int64_t axis_len, int chunks, double* __restrict__ out)
{
    const int64_t a = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (a >= axis_len) return;
    double s = 0.0, n = 0.0;
    for (int k = 0; k < chunks; ++k) {
        s += partial[(a * chunks + k) * 2 + 0];
        n += partial[(a * chunks + k) * 2 + 1];
    }
    out[2 * a + 0] = s;
    out[2 * a + 1] = n;
}

// ------------------------------------------------------------------------------------
// Rescale to another quantizer: y = clamp(z_y + ((x - z_x) m + 2^(r-1)) >> r), one rounding.
// ------------------------------------------------------------------------------------
struct RescaleArgs {
    int32_t zx, m, r, zy, act_min, act_max;
};

__device__ __forceinline__ uint32_t rescale1(uint32_t code, const RescaleArgs& q)
{
    const int64_t v = static_cast<int64_t>(static_cast<int32_t>(code) - q.zx) * q.m + (static_cast<int64_t>(1) << (q.r - 1));
    const int64_t y = (v >> q.r) + q.zy;
    return static_cast<uint32_t>(min(max(y, static_cast<int64_t>(q.act_min)), static_cast<int64_t>(q.act_max)));
}

// One 32-bit word (four channels) per thread; needs 4-byte aligned rows on both sides.
__global__ void __launch_bounds__(kThreads)
rescale_word_kernel(const uint8_t* __restrict__ x, int64_t pixels, int32_t words, int32_t x_pitch, RescaleArgs q,
                    uint8_t* __restrict__ y, int32_t y_pitch)
{
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (t >= pixels * words) return;
    const int64_t p = t / words;
    const int32_t k = static_cast<int32_t>(t - p * words);
    const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(x + p * x_pitch) + k);
    const uint32_t o = rescale1(v & 0xffu, q) | (rescale1((v >> 8) & 0xffu, q) << 8) | (rescale1((v >> 16) & 0xffu, q) << 16) |
                       (rescale1(v >> 24, q) << 24);
    reinterpret_cast<uint32_t*>(y + p * y_pitch)[k] = o;
}

__global__ void __launch_bounds__(kThreads)
rescale_byte_kernel(const uint8_t* __restrict__ x, int64_t pixels, int32_t c, int32_t x_pitch, RescaleArgs q,
                    uint8_t* __restrict__ y, int32_t y_pitch)
{
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (t >= pixels * c) return;
    const int64_t p = t / c;
    const int32_t ch = static_cast<int32_t>(t - p * c);
    y[p * y_pitch + ch] = static_cast<uint8_t>(rescale1(x[p * x_pitch + ch], q));
}

qtz_status check_view(const void* a, const void* b, int64_t outer, int64_t axis_len, int64_t inner)
{
    if (!a || !b || outer <= 0 || axis_len <= 0 || inner <= 0) return QTZ_ERR_INVALID_ARG;
    if (outer > (INT64_MAX / axis_len) / inner) return QTZ_ERR_INVALID_ARG;
    return QTZ_OK;
}

}  // namespace

extern "C" qtz_status qtz_simquant(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len, int64_t inner,
                                   const qtz_qparams* params_host, int32_t code_dtype, int32_t restrict_range,
                                   float* y_dev, void* stream)
{
    if (!h || !params_host) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(x_dev, y_dev, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    int32_t qmin, qmax;
    if (!qtz_code_range(code_dtype, restrict_range, &qmin, &qmax)) return QTZ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(y_dev)) & 3u) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t total = outer * axis_len * inner;
    std::vector<SimRule> rules(static_cast<size_t>(axis_len));
    for (int64_t a = 0; a < axis_len; ++a) {
        const qtz_qparams& p = params_host[a];
        if (!(p.scale > 0.f)) return QTZ_ERR_INVALID_ARG;
        rules[a] = SimRule{p.scale, static_cast<float>(qmin - p.zero_point), static_cast<float>(qmax - p.zero_point)};
    }
    if (axis_len == 1 && qtz_aligned16(x_dev) && qtz_aligned16(y_dev)) {
        const int64_t groups = (total >> 4) + 1;
        simquant_flat_kernel<<<static_cast<unsigned>(ceil_div(groups, kThreads)), kThreads, 0, st>>>(x_dev, total, rules[0], y_dev);
        QTZ_LAUNCH_CHECK(h, "simquant_flat_kernel");
        return QTZ_OK;
    }
    const size_t bytes = sizeof(SimRule) * rules.size();
    s = qtz_ensure_params(h, bytes);
    if (s != QTZ_OK) return s;
    QTZ_CUDA(h, cudaMemcpyAsync(h->params_dev, rules.data(), bytes, cudaMemcpyHostToDevice, st));
    simquant_axis_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, st>>>(
        x_dev, total, axis_len, inner, static_cast<const SimRule*>(h->params_dev), y_dev);
    QTZ_LAUNCH_CHECK(h, "simquant_axis_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_sqnr(qtz_handle h, const float* w_dev, const float* w_hat_dev, int64_t outer, int64_t axis_len,
                               int64_t inner, double* sqnr_db_host, void* stream)
{
    if (!h || !sqnr_db_host) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(w_dev, w_hat_dev, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    if ((reinterpret_cast<uintptr_t>(w_dev) | reinterpret_cast<uintptr_t>(w_hat_dev)) & 3u) return QTZ_ERR_MISALIGNED;
    if (axis_len > 65535) return QTZ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t count = outer * inner;
    const int chunks = static_cast<int>(std::min<int64_t>(kSqnrChunksMax, std::max<int64_t>(1, ceil_div(count, kThreads * 8))));
    // layout of the handle's reduction scratch: [axis_len][2] results, then [axis_len][chunks][2] partials
    const size_t result_bytes = sizeof(double) * 2 * static_cast<size_t>(axis_len);
    s = qtz_ensure_reduce(h, result_bytes * (1 + static_cast<size_t>(chunks)));
    if (s != QTZ_OK) return s;
    double* result = reinterpret_cast<double*>(h->reduce_dev);
    double* partial = result + 2 * axis_len;
    sqnr_partial_kernel<<<dim3(static_cast<unsigned>(chunks), static_cast<unsigned>(axis_len)), kThreads, 0, st>>>(
        w_dev, w_hat_dev, outer, axis_len, inner, partial);
    QTZ_LAUNCH_CHECK(h, "sqnr_partial_kernel");
    sqnr_finish_kernel<<<static_cast<unsigned>(ceil_div(axis_len, kThreads)), kThreads, 0, st>>>(partial, axis_len, chunks, result);
    QTZ_LAUNCH_CHECK(h, "sqnr_finish_kernel");
    QTZ_CUDA(h, cudaMemcpyAsync(h->reduce_host, result, result_bytes, cudaMemcpyDeviceToHost, st));
    QTZ_CUDA(h, cudaStreamSynchronize(st));
    const double* r = reinterpret_cast<const double*>(h->reduce_host);
    for (int64_t a = 0; a < axis_len; ++a)
        sqnr_db_host[a] = r[2 * a + 1] == 0.0 ? INFINITY : 10.0 * std::log10(r[2 * a] / r[2 * a + 1]);
    return QTZ_OK;
}

extern "C" qtz_status qtz_ema_update(double* state_lo_host, double* state_hi_host, const float* batch_lo_host,
                                     const float* batch_hi_host, int64_t n, double decay, int32_t* initialised)
{
    if (!state_lo_host || !state_hi_host || !batch_lo_host || !batch_hi_host || !initialised || n <= 0)
        return QTZ_ERR_INVALID_ARG;
    if (!(decay >= 0.0 && decay < 1.0)) return QTZ_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i)
        if (!std::isfinite(batch_lo_host[i]) || !std::isfinite(batch_hi_host[i])) return QTZ_ERR_NONFINITE;
    const double keep = decay, take = 1.0 - decay;
    for (int64_t i = 0; i < n; ++i) {
        const double lo = static_cast<double>(batch_lo_host[i]), hi = static_cast<double>(batch_hi_host[i]);
        if (*initialised == 0) {
            state_lo_host[i] = lo;
            state_hi_host[i] = hi;
        } else {
            // two roundings per term, as written: no fused multiply-add on the host either
            volatile double a = keep * state_lo_host[i], b = take * lo, c = keep * state_hi_host[i], d = take * hi;
            state_lo_host[i] = a + b;
            state_hi_host[i] = c + d;
        }
    }
    *initialised = 1;
    return QTZ_OK;
}

extern "C" qtz_status qtz_rescale_u8(qtz_handle h, const uint8_t* x_dev, int32_t x_zp, int32_t mult, int32_t rshift,
                                     uint8_t* y_dev, int32_t y_zp, int32_t act_min, int32_t act_max, int64_t pixels,
                                     int32_t c, int32_t x_pitch, int32_t y_pitch, void* stream)
{
    if (!h || !x_dev || !y_dev || pixels <= 0 || c <= 0 || x_pitch < c || y_pitch < c) return QTZ_ERR_INVALID_ARG;
    if (rshift < 1 || rshift > 62 || mult < 0 || act_min < 0 || act_max > 255 || act_min > act_max) return QTZ_ERR_INVALID_ARG;
    if (x_zp < 0 || x_zp > 255 || y_zp < 0 || y_zp > 255) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const RescaleArgs q{x_zp, mult, rshift, y_zp, act_min, act_max};
    const bool words = ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(y_dev) |
                         static_cast<uintptr_t>(x_pitch) | static_cast<uintptr_t>(y_pitch) | static_cast<uintptr_t>(c)) & 3u) == 0;
    if (words) {
        const int64_t work = pixels * (c >> 2);
        rescale_word_kernel<<<static_cast<unsigned>(ceil_div(work, kThreads)), kThreads, 0, st>>>(x_dev, pixels, c >> 2, x_pitch, q,
                                                                                                y_dev, y_pitch);
        QTZ_LAUNCH_CHECK(h, "rescale_word_kernel");
    } else {
        const int64_t work = pixels * c;
        rescale_byte_kernel<<<static_cast<unsigned>(ceil_div(work, kThreads)), kThreads, 0, st>>>(x_dev, pixels, c, x_pitch, q, y_dev,
                                                                                                y_pitch);
        QTZ_LAUNCH_CHECK(h, "rescale_byte_kernel");
    }
    return QTZ_OK;
}
