// HBM-bound element-wise kernels of libqtz: min/max range reduction (Section 2.5),
// quantize (Eq. 1-2, 7-11), dequantize (Eq. 3), batch-norm folding (Eq. 20-21) and bias
// quantization.  All of them stream their operands once with 16-byte accesses.
#include <algorithm>
#include <cfloat>
#include <cstring>
#include <vector>

#include "qtz_device_util.cuh"
#include "qtz_internal.cuh"

namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------
// min / max reduction
// ------------------------------------------------------------------------------------
using qtz_dev::Range;
using qtz_dev::range_take;
using qtz_dev::block_reduce;
static_assert(kThreads == qtz_dev::kReduceThreads, "block_reduce assumes this block size");

// Per-layer reduction, first pass: every block streams a grid-strided share of the tensor
// with 16-byte loads and leaves one (lo, hi, bad) triple in `partial`.
__global__ void __launch_bounds__(kThreads)
minmax_flat_kernel(const float* __restrict__ x, int64_t n, float* __restrict__ partial)
{
    Range r{FLT_MAX, -FLT_MAX, 0u};
    // elements before the first 16-byte boundary, then whole float4s, then the tail
    const int64_t misalign = static_cast<int64_t>((4 - ((reinterpret_cast<uintptr_t>(x) >> 2) & 3)) & 3);
    const int64_t head = misalign < n ? misalign : n;
    const int64_t nvec = (n - head) >> 2;
    const float4* xv = reinterpret_cast<const float4*>(x + head);
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        float4 a = __ldg(xv + i), b = __ldg(xv + i + stride), c = __ldg(xv + i + 2 * stride),
               d = __ldg(xv + i + 3 * stride);
        range_take(r, a.x); range_take(r, a.y); range_take(r, a.z); range_take(r, a.w);
        range_take(r, b.x); range_take(r, b.y); range_take(r, b.z); range_take(r, b.w);
        range_take(r, c.x); range_take(r, c.y); range_take(r, c.z); range_take(r, c.w);
        range_take(r, d.x); range_take(r, d.y); range_take(r, d.z); range_take(r, d.w);
    }
    for (; i < nvec; i += stride) {
        float4 a = __ldg(xv + i);
        range_take(r, a.x); range_take(r, a.y); range_take(r, a.z); range_take(r, a.w);
    }
    if (blockIdx.x == 0) {
        const int64_t tail0 = head + (nvec << 2);
        for (int64_t j = threadIdx.x; j < head; j += kThreads) range_take(r, x[j]);
        for (int64_t j = tail0 + threadIdx.x; j < n; j += kThreads) range_take(r, x[j]);
    }
    r = block_reduce(r);
    if (threadIdx.x == 0) {
        partial[3 * blockIdx.x + 0] = r.lo;
        partial[3 * blockIdx.x + 1] = r.hi;
        partial[3 * blockIdx.x + 2] = __uint_as_float(r.bad);
    }
}

// Second pass: one block folds the partial triples into out[0..2].
__global__ void __launch_bounds__(kThreads)
minmax_finish_kernel(const float* __restrict__ partial, int count, float* __restrict__ out)
{
    Range r{FLT_MAX, -FLT_MAX, 0u};
    for (int i = threadIdx.x; i < count; i += kThreads) {
        r.lo = fminf(r.lo, partial[3 * i]);
        r.hi = fmaxf(r.hi, partial[3 * i + 1]);
        r.bad |= __float_as_uint(partial[3 * i + 2]);
    }
    r = block_reduce(r);
    if (threadIdx.x == 0) {
        out[0] = r.lo;
        out[1] = r.hi;
        out[2] = __uint_as_float(r.bad);
    }
}

// Per-channel reduction: block a reduces the slice x[:, a, :] of the [outer][axis][inner] view.
__global__ void __launch_bounds__(kThreads)
minmax_axis_kernel(const float* __restrict__ x, int64_t outer, int64_t axis_len, int64_t inner,
                   float* __restrict__ out)
{
    const int64_t a = blockIdx.x;
    Range r{FLT_MAX, -FLT_MAX, 0u};
    const int64_t count = outer * inner;
    for (int64_t j = threadIdx.x; j < count; j += kThreads) {
        const int64_t o = j / inner, i = j - o * inner;
        range_take(r, __ldg(x + (o * axis_len + a) * inner + i));
    }
    r = block_reduce(r);
    if (threadIdx.x == 0) {
        out[3 * a + 0] = r.lo;
        out[3 * a + 1] = r.hi;
        out[3 * a + 2] = __uint_as_float(r.bad);
    }
}

// ------------------------------------------------------------------------------------
// quantize
// ------------------------------------------------------------------------------------
struct QuantRule {
    float scale, tlo, thi;  // clamp bounds already shifted by -z
    int32_t zp;
};

// Eq. 1-2: one IEEE division, round-half-even, clamp, add the zero point.
__device__ __forceinline__ int32_t quant1(float x, const QuantRule& q)
{
    float t = rintf(__fdiv_rn(x, q.scale));
    t = fminf(fmaxf(t, q.tlo), q.thi);
    return static_cast<int32_t>(t) + q.zp;
}

__device__ __forceinline__ uint32_t quant4(const float4& v, const QuantRule& q)
{
    return (static_cast<uint32_t>(quant1(v.x, q)) & 0xffu) | ((static_cast<uint32_t>(quant1(v.y, q)) & 0xffu) << 8) |
           ((static_cast<uint32_t>(quant1(v.z, q)) & 0xffu) << 16) | (static_cast<uint32_t>(quant1(v.w, q)) << 24);
}

// Per-layer, byte output (uint8 or int8 share the low byte): 16 values per thread,
// 4 x 16-byte loads and one 16-byte store.  Needs both pointers 16-byte aligned.
__global__ void __launch_bounds__(kThreads)
quantize_flat_kernel(const float* __restrict__ x, int64_t n, QuantRule q, uint8_t* __restrict__ out)
{
    const int64_t groups = n >> 4;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g < groups) {
        const float4* xv = reinterpret_cast<const float4*>(x) + 4 * g;
        const float4 a = __ldcs(xv), b = __ldcs(xv + 1), c = __ldcs(xv + 2), d = __ldcs(xv + 3);
        uint4 o;
        o.x = quant4(a, q); o.y = quant4(b, q); o.z = quant4(c, q); o.w = quant4(d, q);
        reinterpret_cast<uint4*>(out)[g] = o;
    } else if (g == groups) {
        for (int64_t i = groups << 4; i < n; ++i) out[i] = static_cast<uint8_t>(quant1(x[i], q));
    }
}

// Per-layer, 16-bit output (uint16 or int16 share the low half word): 8 values per thread,
// 2 x 16-byte loads and one 16-byte store.  Needs both pointers 16-byte aligned.
__global__ void __launch_bounds__(kThreads)
quantize_flat16_kernel(const float* __restrict__ x, int64_t n, QuantRule q, uint16_t* __restrict__ out)
{
    const int64_t groups = n >> 3;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g < groups) {
        const float4* xv = reinterpret_cast<const float4*>(x) + 2 * g;
        const float4 a = __ldcs(xv), b = __ldcs(xv + 1);
        auto two = [&](float lo, float hi) {
            return (static_cast<uint32_t>(quant1(lo, q)) & 0xffffu) | (static_cast<uint32_t>(quant1(hi, q)) << 16);
        };
        uint4 o;
        o.x = two(a.x, a.y); o.y = two(a.z, a.w); o.z = two(b.x, b.y); o.w = two(b.z, b.w);
        reinterpret_cast<uint4*>(out)[g] = o;
    } else if (g == groups) {
        for (int64_t i = groups << 3; i < n; ++i) out[i] = static_cast<uint16_t>(quant1(x[i], q));
    }
}

// Any view, 16-bit output: one value per thread.
__global__ void __launch_bounds__(kThreads)
quantize_axis16_kernel(const float* __restrict__ x, int64_t total, int64_t axis_len, int64_t inner,
                       const QuantRule* __restrict__ rules, uint16_t* __restrict__ out)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    const int64_t a = (i / inner) % axis_len;
    out[i] = static_cast<uint16_t>(quant1(x[i], rules[a]));
}

// Any view, byte output: one value per thread, the rule fetched per axis index.
__global__ void __launch_bounds__(kThreads)
quantize_axis_kernel(const float* __restrict__ x, int64_t total, int64_t axis_len, int64_t inner,
                     const QuantRule* __restrict__ rules, uint8_t* __restrict__ out)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    const int64_t a = (i / inner) % axis_len;
    out[i] = static_cast<uint8_t>(quant1(x[i], rules[a]));
}

// 4-bit output: one byte (two codes of the same run) per thread.  run_len is the length of
// the innermost run; run_axis_stride tells how the axis index follows from the element index.
__global__ void __launch_bounds__(kThreads)
quantize_s4_kernel(const float* __restrict__ x, int64_t runs, int64_t run_len, int64_t axis_len,
                   int64_t inner, const QuantRule* __restrict__ rules, uint8_t* __restrict__ out)
{
    const int64_t bytes_per_run = (run_len + 1) >> 1;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (t >= runs * bytes_per_run) return;
    const int64_t run = t / bytes_per_run, j = t - run * bytes_per_run;
    const int64_t e0 = run * run_len + 2 * j;
    const int64_t a0 = (e0 / inner) % axis_len;
    uint32_t lo = static_cast<uint32_t>(quant1(x[e0], rules[a0])) & 0xfu, hi = 0;
    if (2 * j + 1 < run_len) {
        const int64_t a1 = ((e0 + 1) / inner) % axis_len;
        hi = static_cast<uint32_t>(quant1(x[e0 + 1], rules[a1])) & 0xfu;
    }
    out[t] = static_cast<uint8_t>(lo | (hi << 4));
}

// ------------------------------------------------------------------------------------
// dequantize (Eq. 3)
// ------------------------------------------------------------------------------------
struct DequantRule {
    float scale;
    int32_t zp;
};

template <bool kSigned>
__device__ __forceinline__ float4 dequant4(uint32_t w, const DequantRule& q)
{
    int32_t a, b, c, d;
    if (kSigned) {
        a = static_cast<int8_t>(w); b = static_cast<int8_t>(w >> 8);
        c = static_cast<int8_t>(w >> 16); d = static_cast<int8_t>(w >> 24);
    } else {
        a = w & 0xff; b = (w >> 8) & 0xff; c = (w >> 16) & 0xff; d = w >> 24;
    }
    return make_float4(__fmul_rn(static_cast<float>(a - q.zp), q.scale), __fmul_rn(static_cast<float>(b - q.zp), q.scale),
                       __fmul_rn(static_cast<float>(c - q.zp), q.scale), __fmul_rn(static_cast<float>(d - q.zp), q.scale));
}

template <bool kSigned>
__global__ void __launch_bounds__(kThreads)
dequantize_flat_kernel(const uint8_t* __restrict__ q, int64_t n, DequantRule rule, float* __restrict__ x)
{
    const int64_t groups = n >> 4;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g < groups) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(q) + g);
        float4* xv = reinterpret_cast<float4*>(x) + 4 * g;
        __stcs(xv, dequant4<kSigned>(v.x, rule));
        __stcs(xv + 1, dequant4<kSigned>(v.y, rule));
        __stcs(xv + 2, dequant4<kSigned>(v.z, rule));
        __stcs(xv + 3, dequant4<kSigned>(v.w, rule));
    } else if (g == groups) {
        for (int64_t i = groups << 4; i < n; ++i) {
            const int32_t c = kSigned ? static_cast<int32_t>(static_cast<int8_t>(q[i])) : static_cast<int32_t>(q[i]);
            x[i] = __fmul_rn(static_cast<float>(c - rule.zp), rule.scale);
        }
    }
}

// Per-layer 16-bit codes: 8 values per thread (one 16-byte load, two 16-byte stores).
template <bool kSigned>
__global__ void __launch_bounds__(kThreads)
dequantize_flat16_kernel(const uint16_t* __restrict__ q, int64_t n, DequantRule rule, float* __restrict__ x)
{
    const int64_t groups = n >> 3;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    auto one = [&](uint32_t half) {
        const int32_t c = kSigned ? static_cast<int32_t>(static_cast<int16_t>(half)) : static_cast<int32_t>(half & 0xffffu);
        return __fmul_rn(static_cast<float>(c - rule.zp), rule.scale);
    };
    if (g < groups) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(q) + g);
        float4* xv = reinterpret_cast<float4*>(x) + 2 * g;
        __stcs(xv, make_float4(one(v.x), one(v.x >> 16), one(v.y), one(v.y >> 16)));
        __stcs(xv + 1, make_float4(one(v.z), one(v.z >> 16), one(v.w), one(v.w >> 16)));
    } else if (g == groups) {
        for (int64_t i = groups << 3; i < n; ++i) x[i] = one(q[i]);
    }
}

// Any view and any code type: one value per thread.
__global__ void __launch_bounds__(kThreads)
dequantize_axis_kernel(const void* __restrict__ q, int32_t dtype, int64_t total, int64_t axis_len,
                       int64_t inner, int64_t run_len, const DequantRule* __restrict__ rules,
                       float* __restrict__ x)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    const DequantRule r = rules[(i / inner) % axis_len];
    int32_t code;
    if (dtype == QTZ_U8) {
        code = static_cast<const uint8_t*>(q)[i];
    } else if (dtype == QTZ_S8) {
        code = static_cast<const int8_t*>(q)[i];
    } else if (dtype == QTZ_S32) {
        code = static_cast<const int32_t*>(q)[i];
    } else if (dtype == QTZ_U16) {
        code = static_cast<const uint16_t*>(q)[i];
    } else if (dtype == QTZ_S16) {
        code = static_cast<const int16_t*>(q)[i];
    } else {  // packed 4-bit: locate the byte inside the element's run
        const int64_t run = i / run_len, e = i - run * run_len;
        const uint32_t byte = static_cast<const uint8_t*>(q)[run * ((run_len + 1) >> 1) + (e >> 1)];
        const uint32_t nib = (e & 1) ? (byte >> 4) : (byte & 0xfu);
        code = dtype == QTZ_U4_PACKED ? static_cast<int32_t>(nib) : static_cast<int32_t>(nib << 28) >> 28;
    }
    x[i] = __fmul_rn(static_cast<float>(code - r.zp), r.scale);
}

// ------------------------------------------------------------------------------------
// batch-norm folding (Eq. 20-21) and bias quantization
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
fold_bn_weights_kernel(const float* __restrict__ w, const float* __restrict__ gamma,
                       const float* __restrict__ var, float eps, int64_t k, float* __restrict__ w_inf)
{
    const int64_t row = blockIdx.y;
    const double sigma = sqrt(__dadd_rn(static_cast<double>(var[row]), static_cast<double>(eps)));
    const double g = static_cast<double>(gamma[row]);
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < k;
         i += static_cast<int64_t>(gridDim.x) * kThreads) {
        const double num = __dmul_rn(g, static_cast<double>(w[row * k + i]));
        w_inf[row * k + i] = static_cast<float>(__ddiv_rn(num, sigma));
    }
}

__global__ void __launch_bounds__(kThreads)
fold_bn_bias_kernel(const float* __restrict__ conv_bias, const float* __restrict__ gamma,
                    const float* __restrict__ beta, const float* __restrict__ mean,
                    const float* __restrict__ var, float eps, int64_t n, float* __restrict__ bias_inf)
{
    const int64_t c = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (c >= n) return;
    const double sigma = sqrt(__dadd_rn(static_cast<double>(var[c]), static_cast<double>(eps)));
    const double b = conv_bias ? static_cast<double>(conv_bias[c]) : 0.0;
    const double centred = __dsub_rn(b, static_cast<double>(mean[c]));
    const double q = __ddiv_rn(__dmul_rn(static_cast<double>(gamma[c]), centred), sigma);
    bias_inf[c] = static_cast<float>(__dadd_rn(static_cast<double>(beta[c]), q));
}

__global__ void __launch_bounds__(kThreads)
quantize_bias_kernel(const float* __restrict__ bias, int64_t n, float x_scale,
                     const float* __restrict__ w_scale, int per_layer, int32_t* __restrict__ out)
{
    const int64_t c = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (c >= n) return;
    const double s = __dmul_rn(static_cast<double>(x_scale), static_cast<double>(w_scale[per_layer ? 0 : c]));
    double r = rint(__ddiv_rn(static_cast<double>(bias[c]), s));
    r = fmin(fmax(r, -2147483648.0), 2147483647.0);
    out[c] = static_cast<int32_t>(r);
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

qtz_status check_view(const void* a, const void* b, int64_t outer, int64_t axis_len, int64_t inner)
{
    if (!a || !b || outer <= 0 || axis_len <= 0 || inner <= 0) return QTZ_ERR_INVALID_ARG;
    if (outer > (INT64_MAX / axis_len) / inner) return QTZ_ERR_INVALID_ARG;
    return QTZ_OK;
}

}  // namespace

// Device part of calibration: leaves axis_len (lo, hi, bad) triples in h->reduce_dev.
static qtz_status launch_minmax(qtz_ctx* h, const float* x_dev, int64_t outer, int64_t axis_len,
                                int64_t inner, cudaStream_t st)
{
    const int64_t total = outer * axis_len * inner;
    if (axis_len == 1) {
        const int blocks = static_cast<int>(std::min<int64_t>(static_cast<int64_t>(h->num_sms) * 8,
                                                              std::max<int64_t>(1, ceil_div(total, kThreads * 16))));
        qtz_status s = qtz_ensure_reduce(h, sizeof(float) * 3 * (static_cast<size_t>(blocks) + 1));
        if (s != QTZ_OK) return s;
        float* partial = h->reduce_dev + 3;
        minmax_flat_kernel<<<blocks, kThreads, 0, st>>>(x_dev, total, partial);
        QTZ_LAUNCH_CHECK(h, "minmax_flat_kernel");
        minmax_finish_kernel<<<1, kThreads, 0, st>>>(partial, blocks, h->reduce_dev);
        QTZ_LAUNCH_CHECK(h, "minmax_finish_kernel");
    } else {
        if (axis_len > (1 << 30)) return QTZ_ERR_INVALID_ARG;
        qtz_status s = qtz_ensure_reduce(h, sizeof(float) * 3 * static_cast<size_t>(axis_len));
        if (s != QTZ_OK) return s;
        minmax_axis_kernel<<<static_cast<unsigned>(axis_len), kThreads, 0, st>>>(x_dev, outer, axis_len, inner,
                                                                                  h->reduce_dev);
        QTZ_LAUNCH_CHECK(h, "minmax_axis_kernel");
    }
    return QTZ_OK;
}

extern "C" qtz_status qtz_minmax(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len, int64_t inner,
                                 float* lo_host, float* hi_host, void* stream)
{
    if (!h || !hi_host) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(x_dev, lo_host, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    if (reinterpret_cast<uintptr_t>(x_dev) & 3u) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = launch_minmax(h, x_dev, outer, axis_len, inner, st);
    if (s != QTZ_OK) return s;
    const size_t bytes = sizeof(float) * 3 * static_cast<size_t>(axis_len);
    QTZ_CUDA(h, cudaMemcpyAsync(h->reduce_host, h->reduce_dev, bytes, cudaMemcpyDeviceToHost, st));
    QTZ_CUDA(h, cudaStreamSynchronize(st));
    for (int64_t a = 0; a < axis_len; ++a) {
        const float* t = h->reduce_host + 3 * a;
        uint32_t bad;
        memcpy(&bad, t + 2, sizeof(bad));
        if (bad) return QTZ_ERR_NONFINITE;
        lo_host[a] = t[0];
        hi_host[a] = t[1];
    }
    return QTZ_OK;
}

// ---- streaming range estimation (Section 2.5: moving average of per-batch min and max) ----------
namespace {

// Device-resident state of qtz_range_accumulate: the averaged (lo, hi) per axis index in fp64 and a header.
struct RangeHeader {
    int32_t batches;      // batches folded in so far (0: the next batch initialises the state)
    int32_t nonfinite;    // a batch held NaN or Inf: it was skipped and qtz_range_finish reports it
    int32_t pad[2];
};

__host__ __device__ inline double* range_lo(void* state) { return reinterpret_cast<double*>(static_cast<char*>(state) + sizeof(RangeHeader)); }

// One block: first agrees on whether this batch is usable at all (any non-finite value skips the whole
// batch, as the host rule does), then state <- decay * state + (1 - decay) * batch, each product and the sum
// rounded separately (no fused multiply-add), so that the host rule gives the same bits.
__global__ void __launch_bounds__(kThreads)
range_ema_kernel(const float* __restrict__ triples, int64_t axis_len, double keep, double take, void* state)
{
    RangeHeader* hdr = static_cast<RangeHeader*>(state);
    double* lo = range_lo(state);
    double* hi = lo + axis_len;
    int bad = 0;
    for (int64_t a = threadIdx.x; a < axis_len; a += kThreads) bad |= __float_as_uint(triples[3 * a + 2]) != 0u;
    bad = __syncthreads_or(bad);
    if (bad) {
        if (threadIdx.x == 0) hdr->nonfinite = 1;
        return;
    }
    const bool first = hdr->batches == 0;
    for (int64_t a = threadIdx.x; a < axis_len; a += kThreads) {
        const double blo = static_cast<double>(triples[3 * a]), bhi = static_cast<double>(triples[3 * a + 1]);
        lo[a] = first ? blo : __dadd_rn(__dmul_rn(keep, lo[a]), __dmul_rn(take, blo));
        hi[a] = first ? bhi : __dadd_rn(__dmul_rn(keep, hi[a]), __dmul_rn(take, bhi));
    }
    __syncthreads();
    if (threadIdx.x == 0) hdr->batches += 1;
}

}  // namespace

extern "C" int64_t qtz_range_state_bytes(int64_t axis_len)
{
    if (axis_len <= 0 || axis_len > (1 << 30)) return 0;
    return static_cast<int64_t>(sizeof(RangeHeader)) + 2 * static_cast<int64_t>(sizeof(double)) * axis_len;
}

extern "C" qtz_status qtz_range_reset(qtz_handle h, void* state_dev, int64_t axis_len, void* stream)
{
    if (!h || !state_dev || qtz_range_state_bytes(axis_len) == 0) return QTZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(state_dev) & 7u) return QTZ_ERR_MISALIGNED;
    QTZ_CUDA(h, cudaMemsetAsync(state_dev, 0, static_cast<size_t>(qtz_range_state_bytes(axis_len)), static_cast<cudaStream_t>(stream)));
    return QTZ_OK;
}

extern "C" qtz_status qtz_range_accumulate(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len, int64_t inner,
                                           double decay, void* state_dev, void* stream)
{
    if (!h) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(x_dev, state_dev, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    if (!(decay >= 0.0 && decay < 1.0) || qtz_range_state_bytes(axis_len) == 0) return QTZ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x_dev) & 3u) || (reinterpret_cast<uintptr_t>(state_dev) & 7u)) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = launch_minmax(h, x_dev, outer, axis_len, inner, st);
    if (s != QTZ_OK) return s;
    range_ema_kernel<<<1, kThreads, 0, st>>>(h->reduce_dev, axis_len, decay, 1.0 - decay, state_dev);
    QTZ_LAUNCH_CHECK(h, "range_ema_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_range_finish(qtz_handle h, const void* state_dev, int64_t axis_len, int32_t bits, int32_t symmetric,
                                       float* lo_host, float* hi_host, qtz_qparams* params_host, int32_t* batches_host,
                                       void* stream)
{
    if (!h || !state_dev || qtz_range_state_bytes(axis_len) == 0) return QTZ_ERR_INVALID_ARG;
    if (params_host && (bits < 2 || bits > 16)) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = static_cast<size_t>(qtz_range_state_bytes(axis_len));
    std::vector<char> host(bytes);
    QTZ_CUDA(h, cudaMemcpyAsync(host.data(), state_dev, bytes, cudaMemcpyDeviceToHost, st));
    QTZ_CUDA(h, cudaStreamSynchronize(st));
    const RangeHeader* hdr = reinterpret_cast<const RangeHeader*>(host.data());
    if (batches_host) *batches_host = hdr->batches;
    if (hdr->nonfinite) return QTZ_ERR_NONFINITE;
    if (hdr->batches == 0) return QTZ_ERR_INVALID_ARG;       // nothing was accumulated
    const double* lo = range_lo(host.data());
    const double* hi = lo + axis_len;
    for (int64_t a = 0; a < axis_len; ++a) {
        const float flo = static_cast<float>(lo[a]), fhi = static_cast<float>(hi[a]);
        if (lo_host) lo_host[a] = flo;
        if (hi_host) hi_host[a] = fhi;
        if (params_host) {
            const qtz_status s = symmetric ? qtz_host_symmetric_params(flo, fhi, bits, params_host + a)
                                           : qtz_host_affine_params(flo, fhi, bits, params_host + a);
            if (s != QTZ_OK) return s;
        }
    }
    return QTZ_OK;
}

extern "C" qtz_status qtz_calibrate_minmax(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len,
                                           int64_t inner, int32_t bits, int32_t symmetric,
                                           qtz_qparams* out_host, void* stream)
{
    if (!h) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(x_dev, out_host, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    if (bits < 2 || bits > 16) return QTZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_dev) & 3u) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = launch_minmax(h, x_dev, outer, axis_len, inner, st);
    if (s != QTZ_OK) return s;
    const size_t bytes = sizeof(float) * 3 * static_cast<size_t>(axis_len);
    QTZ_CUDA(h, cudaMemcpyAsync(h->reduce_host, h->reduce_dev, bytes, cudaMemcpyDeviceToHost, st));
    QTZ_CUDA(h, cudaStreamSynchronize(st));
    for (int64_t a = 0; a < axis_len; ++a) {
        const float* t = h->reduce_host + 3 * a;
        uint32_t bad;
        memcpy(&bad, t + 2, sizeof(bad));
        if (bad) return QTZ_ERR_NONFINITE;
        s = symmetric ? qtz_host_symmetric_params(t[0], t[1], bits, out_host + a)
                      : qtz_host_affine_params(t[0], t[1], bits, out_host + a);
        if (s != QTZ_OK) return s;
    }
    return QTZ_OK;
}

extern "C" qtz_status qtz_quantize_tensor(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len,
                                          int64_t inner, const qtz_qparams* params_host, int32_t out_dtype,
                                          int32_t restrict_range, void* q_dev, void* stream)
{
    if (!h || !params_host) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(x_dev, q_dev, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    int32_t qmin, qmax;
    if (!qtz_code_range(out_dtype, restrict_range, &qmin, &qmax)) return QTZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_dev) & 3u) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t total = outer * axis_len * inner;

    std::vector<QuantRule> rules(static_cast<size_t>(axis_len));
    for (int64_t a = 0; a < axis_len; ++a) {
        const qtz_qparams& p = params_host[a];
        if (!(p.scale > 0.f)) return QTZ_ERR_INVALID_ARG;
        rules[a] = QuantRule{p.scale, static_cast<float>(qmin - p.zero_point),
                             static_cast<float>(qmax - p.zero_point), p.zero_point};
    }
    const bool packed4 = out_dtype == QTZ_S4_PACKED || out_dtype == QTZ_U4_PACKED;
    const bool wide = out_dtype == QTZ_U16 || out_dtype == QTZ_S16;
    if (wide && (reinterpret_cast<uintptr_t>(q_dev) & 1u)) return QTZ_ERR_MISALIGNED;
    if (axis_len == 1 && wide && qtz_aligned16(x_dev) && qtz_aligned16(q_dev)) {
        const int64_t groups = (total >> 3) + 1;
        quantize_flat16_kernel<<<static_cast<unsigned>(ceil_div(groups, kThreads)), kThreads, 0, st>>>(
            x_dev, total, rules[0], static_cast<uint16_t*>(q_dev));
        QTZ_LAUNCH_CHECK(h, "quantize_flat16_kernel");
        return QTZ_OK;
    }
    if (axis_len == 1 && !packed4 && !wide && qtz_aligned16(x_dev) && qtz_aligned16(q_dev)) {
        const int64_t groups = (total >> 4) + 1;
        quantize_flat_kernel<<<static_cast<unsigned>(ceil_div(groups, kThreads)), kThreads, 0, st>>>(
            x_dev, total, rules[0], static_cast<uint8_t*>(q_dev));
        QTZ_LAUNCH_CHECK(h, "quantize_flat_kernel");
        return QTZ_OK;
    }
    const size_t bytes = sizeof(QuantRule) * rules.size();
    s = qtz_ensure_params(h, bytes);
    if (s != QTZ_OK) return s;
    QTZ_CUDA(h, cudaMemcpyAsync(h->params_dev, rules.data(), bytes, cudaMemcpyHostToDevice, st));
    const QuantRule* rules_dev = static_cast<const QuantRule*>(h->params_dev);
    if (packed4) {
        const int64_t run_len = inner > 1 ? inner : axis_len;
        const int64_t runs = total / run_len;
        const int64_t work = runs * ((run_len + 1) >> 1);
        quantize_s4_kernel<<<static_cast<unsigned>(ceil_div(work, kThreads)), kThreads, 0, st>>>(
            x_dev, runs, run_len, axis_len, inner, rules_dev, static_cast<uint8_t*>(q_dev));
        QTZ_LAUNCH_CHECK(h, "quantize_s4_kernel");
    } else if (wide) {
        quantize_axis16_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, st>>>(
            x_dev, total, axis_len, inner, rules_dev, static_cast<uint16_t*>(q_dev));
        QTZ_LAUNCH_CHECK(h, "quantize_axis16_kernel");
    } else {
        quantize_axis_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, st>>>(
            x_dev, total, axis_len, inner, rules_dev, static_cast<uint8_t*>(q_dev));
        QTZ_LAUNCH_CHECK(h, "quantize_axis_kernel");
    }
    // The staging vector dies with this call; pageable-source async copies have been
    // staged by the runtime before cudaMemcpyAsync returned.
    return QTZ_OK;
}

extern "C" qtz_status qtz_dequantize(qtz_handle h, const void* q_dev, int32_t in_dtype, int64_t outer,
                                     int64_t axis_len, int64_t inner, const qtz_qparams* params_host,
                                     float* x_dev, void* stream)
{
    if (!h || !params_host) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_view(q_dev, x_dev, outer, axis_len, inner);
    if (s != QTZ_OK) return s;
    if (in_dtype < QTZ_U8 || in_dtype > QTZ_S16) return QTZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_dev) & 3u) return QTZ_ERR_MISALIGNED;
    const bool wide = in_dtype == QTZ_U16 || in_dtype == QTZ_S16;
    if (wide && (reinterpret_cast<uintptr_t>(q_dev) & 1u)) return QTZ_ERR_MISALIGNED;
    if (in_dtype == QTZ_S32 && (reinterpret_cast<uintptr_t>(q_dev) & 3u)) return QTZ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t total = outer * axis_len * inner;
    std::vector<DequantRule> rules(static_cast<size_t>(axis_len));
    for (int64_t a = 0; a < axis_len; ++a) {
        if (in_dtype == QTZ_S32 && params_host[a].zero_point != 0) return QTZ_ERR_INVALID_ARG;
        rules[a] = DequantRule{params_host[a].scale, params_host[a].zero_point};
    }
    if (axis_len == 1 && (in_dtype == QTZ_U8 || in_dtype == QTZ_S8) && qtz_aligned16(q_dev) && qtz_aligned16(x_dev)) {
        const int64_t groups = (total >> 4) + 1;
        const unsigned blocks = static_cast<unsigned>(ceil_div(groups, kThreads));
        if (in_dtype == QTZ_S8)
            dequantize_flat_kernel<true><<<blocks, kThreads, 0, st>>>(static_cast<const uint8_t*>(q_dev), total, rules[0], x_dev);
        else
            dequantize_flat_kernel<false><<<blocks, kThreads, 0, st>>>(static_cast<const uint8_t*>(q_dev), total, rules[0], x_dev);
        QTZ_LAUNCH_CHECK(h, "dequantize_flat_kernel");
        return QTZ_OK;
    }
    if (axis_len == 1 && wide && qtz_aligned16(q_dev) && qtz_aligned16(x_dev)) {
        const int64_t groups = (total >> 3) + 1;
        const unsigned blocks = static_cast<unsigned>(ceil_div(groups, kThreads));
        if (in_dtype == QTZ_S16)
            dequantize_flat16_kernel<true><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(q_dev), total, rules[0], x_dev);
        else
            dequantize_flat16_kernel<false><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(q_dev), total, rules[0], x_dev);
        QTZ_LAUNCH_CHECK(h, "dequantize_flat16_kernel");
        return QTZ_OK;
    }
    const size_t bytes = sizeof(DequantRule) * rules.size();
    s = qtz_ensure_params(h, bytes);
    if (s != QTZ_OK) return s;
    QTZ_CUDA(h, cudaMemcpyAsync(h->params_dev, rules.data(), bytes, cudaMemcpyHostToDevice, st));
    const int64_t run_len = inner > 1 ? inner : axis_len;
    dequantize_axis_kernel<<<static_cast<unsigned>(ceil_div(total, kThreads)), kThreads, 0, st>>>(
        q_dev, in_dtype, total, axis_len, inner, run_len, static_cast<const DequantRule*>(h->params_dev), x_dev);
    QTZ_LAUNCH_CHECK(h, "dequantize_axis_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_fold_batchnorm(qtz_handle h, const float* w_dev, const float* conv_bias_dev,
                                         const float* gamma_dev, const float* beta_dev, const float* mean_dev,
                                         const float* var_dev, float eps, int64_t n, int64_t k,
                                         float* w_inf_dev, float* bias_inf_dev, void* stream)
{
    if (!h || !w_dev || !gamma_dev || !beta_dev || !mean_dev || !var_dev || !w_inf_dev || !bias_inf_dev)
        return QTZ_ERR_INVALID_ARG;
    if (n <= 0 || k <= 0 || n > 65535 || !(eps >= 0.f)) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(static_cast<unsigned>(std::min<int64_t>(ceil_div(k, kThreads), 64)), static_cast<unsigned>(n));
    fold_bn_weights_kernel<<<grid, kThreads, 0, st>>>(w_dev, gamma_dev, var_dev, eps, k, w_inf_dev);
    QTZ_LAUNCH_CHECK(h, "fold_bn_weights_kernel");
    fold_bn_bias_kernel<<<static_cast<unsigned>(ceil_div(n, kThreads)), kThreads, 0, st>>>(
        conv_bias_dev, gamma_dev, beta_dev, mean_dev, var_dev, eps, n, bias_inf_dev);
    QTZ_LAUNCH_CHECK(h, "fold_bn_bias_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_quantize_bias(qtz_handle h, const float* bias_dev, int64_t n, float x_scale,
                                        const qtz_qparams* w_params_host, int32_t per_layer,
                                        int32_t* bias_q_dev, void* stream)
{
    if (!h || !bias_dev || !w_params_host || !bias_q_dev || n <= 0 || !(x_scale > 0.f)) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t count = per_layer ? 1 : n;
    std::vector<float> scales(static_cast<size_t>(count));
    for (int64_t c = 0; c < count; ++c) {
        if (!(w_params_host[c].scale > 0.f)) return QTZ_ERR_INVALID_ARG;
        scales[c] = w_params_host[c].scale;
    }
    qtz_status s = qtz_ensure_params(h, sizeof(float) * scales.size());
    if (s != QTZ_OK) return s;
    QTZ_CUDA(h, cudaMemcpyAsync(h->params_dev, scales.data(), sizeof(float) * scales.size(), cudaMemcpyHostToDevice, st));
    quantize_bias_kernel<<<static_cast<unsigned>(ceil_div(n, kThreads)), kThreads, 0, st>>>(
        bias_dev, n, x_scale, static_cast<const float*>(h->params_dev), per_layer ? 1 : 0, bias_q_dev);
    QTZ_LAUNCH_CHECK(h, "quantize_bias_kernel");
    return QTZ_OK;
}
