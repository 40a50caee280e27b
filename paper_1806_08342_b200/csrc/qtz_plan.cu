// Per-layer preparation (weights are constant at inference, Section 2.1) and dispatch of
// the convolution entry points.
#include <algorithm>
#include <cstdlib>
#include <new>
#include <vector>

#include "qtz_device_util.cuh"
#include "qtz_plan.cuh"

namespace {

constexpr int kThreads = 256;

using qtz_dev::load_code_s8;

__global__ void __launch_bounds__(kThreads)
prepack_direct_kernel(const void* __restrict__ w, int wkind, int n, int k_total, int n_padded, int k_padded,
                      int8_t* __restrict__ out)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= static_cast<int64_t>(n_padded) * k_padded) return;
    const int64_t row = i / k_padded, k = i - row * k_padded;
    out[i] = (row < n && k < k_total) ? static_cast<int8_t>(load_code_s8(w, wkind, row, k, k_total)) : 0;
}

// wsum[row] = sum over the whole receptive field of the int8 codes.
__global__ void __launch_bounds__(kThreads)
weight_sum_kernel(const int8_t* __restrict__ w, int k_padded, int32_t* __restrict__ wsum)
{
    __shared__ int32_t part[kThreads / 32];
    const int row = blockIdx.x;
    int32_t s = 0;
    for (int k = threadIdx.x; k < k_padded; k += kThreads) s += w[static_cast<int64_t>(row) * k_padded + k];
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t t = 0;
        for (int i = 0; i < kThreads / 32; ++i) t += part[i];
        wsum[row] = t;
    }
}

// Depthwise weights [3][3][c] -> per filter row and channel one word (k0, k1, k2, 0) of int8 codes,
// plus the sum of the nine codes; channels beyond c are zero.
__global__ void __launch_bounds__(kThreads)
prepack_depthwise_kernel(const void* __restrict__ w, int wkind, int c, int pitch, uint32_t* __restrict__ taps,
                         int32_t* __restrict__ wsum)
{
    const int ch = blockIdx.x * kThreads + threadIdx.x;
    if (ch >= pitch) return;
    int32_t total = 0;
    for (int i = 0; i < 3; ++i) {
        uint32_t word = 0;
        for (int j = 0; j < 3; ++j) {
            const int32_t code = ch < c ? load_code_s8(w, wkind, 3 * i + j, ch, c) : 0;
            word |= (static_cast<uint32_t>(code) & 0xffu) << (8 * j);
            total += code;
        }
        taps[i * pitch + ch] = word;
    }
    wsum[ch] = total;
}

__global__ void fill_i32_kernel(int32_t* p, int n, int32_t v)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

qtz_status validate_desc(const qtz_conv_desc& d, int depthwise)
{
    if (d.batch <= 0 || d.h <= 0 || d.w <= 0 || d.c <= 0 || d.n <= 0 || d.kh <= 0 || d.kw <= 0 || d.stride <= 0 ||
        d.pad < 0 || d.c_pitch_in < d.c)
        return QTZ_ERR_INVALID_ARG;
    if (d.wkind < QTZ_W_S8_PER_CHANNEL_SYM || d.wkind > QTZ_W_S4_PACKED_PER_CHANNEL_SYM) return QTZ_ERR_INVALID_ARG;
    if (d.outkind != QTZ_OUT_U8 && d.outkind != QTZ_OUT_S32_RAW) return QTZ_ERR_INVALID_ARG;
    // (image tensors of up to 8 channels may come at a pixel pitch of 4 or 8 bytes: the stem paths repack them anyway)
    const bool narrow_image = !depthwise && (d.c_pitch_in == 4 || d.c_pitch_in == 8) && !(d.kh == 1 && d.kw == 1);
    if ((d.c_pitch_in & 15) && !narrow_image) return QTZ_ERR_MISALIGNED;
    if (d.outkind == QTZ_OUT_U8) {
        if (d.c_pitch_out < d.n) return QTZ_ERR_INVALID_ARG;
        if (d.c_pitch_out & 15) return QTZ_ERR_MISALIGNED;
    }
    if (d.h + 2 * d.pad < d.kh || d.w + 2 * d.pad < d.kw) return QTZ_ERR_INVALID_ARG;
    if (d.kh > 64 || d.kw > 64 || d.pad >= d.kh || d.pad >= d.kw) return QTZ_ERR_INVALID_ARG;
    const int64_t k = depthwise ? static_cast<int64_t>(d.kh) * d.kw : static_cast<int64_t>(d.kh) * d.kw * d.c;
    if (k > 32768) return QTZ_ERR_OVERFLOW;
    if (depthwise) {
        if (d.n != d.c) return QTZ_ERR_INVALID_ARG;
        if (d.kh != 3 || d.kw != 3 || d.pad != 1 || (d.stride != 1 && d.stride != 2))
            return QTZ_ERR_UNSUPPORTED;
    }
    return QTZ_OK;
}

}  // namespace

extern "C" qtz_status qtz_conv_destroy(qtz_conv_plan p)
{
    if (!p) return QTZ_ERR_INVALID_ARG;
    // cudaFree waits for the work that may still use a buffer before it releases it, so no
    // device-wide synchronisation is needed here
    qtz_device_guard guard(p->device);
    qtz_tc_release(p);
    qtz_depthwise_release(p);
    cudaFree(p->w_direct);
    cudaFree(p->dw_taps);
    cudaFree(p->dw_wsum);
    cudaFree(p->bias);
    cudaFree(p->wsum);
    cudaFree(p->mult);
    cudaFree(p->rshift);
    cudaFree(p->x_gather);
    (void)cudaGetLastError();
    delete p;
    return QTZ_OK;
}

extern "C" qtz_status qtz_conv_set_profile_events(qtz_conv_plan p, void* start_event, void* stop_event)
{
    if (!p || ((start_event == nullptr) != (stop_event == nullptr))) return QTZ_ERR_INVALID_ARG;
    p->ev_start = static_cast<cudaEvent_t>(start_event);
    p->ev_stop = static_cast<cudaEvent_t>(stop_event);
    return QTZ_OK;
}

extern "C" const char* qtz_conv_plan_kernel(qtz_conv_plan p)
{
    if (!p) return "";
    return p->family == QTZ_K_TCGEN05 ? "tcgen05" : (p->family == QTZ_K_DEPTHWISE ? "depthwise" : "direct");
}

extern "C" const char* qtz_conv_plan_detail(qtz_conv_plan p)
{
    if (!p) return "";
    if (p->detail.empty()) return qtz_conv_plan_kernel(p);
    return p->detail.c_str();
}

extern "C" qtz_status qtz_conv_create(qtz_handle h, const qtz_conv_desc* desc, int32_t depthwise, const void* w_q_dev,
                                      const int32_t* bias_q_dev, const int32_t* w_zero_point_host,
                                      const int32_t* mult_host, const int32_t* rshift_host, qtz_conv_plan* out,
                                      void* stream)
{
    if (!h || !desc || !w_q_dev || !out) return QTZ_ERR_INVALID_ARG;
    *out = nullptr;
    qtz_status s = validate_desc(*desc, depthwise);
    if (s != QTZ_OK) return s;
    const qtz_conv_desc& d = *desc;
    const bool raw = d.outkind == QTZ_OUT_S32_RAW;
    if (!raw && (!mult_host || !rshift_host)) return QTZ_ERR_INVALID_ARG;
    if (d.wkind == QTZ_W_U8_PER_LAYER_ASYM && !w_zero_point_host) return QTZ_ERR_INVALID_ARG;
    if (d.wkind != QTZ_W_U8_PER_LAYER_ASYM && w_zero_point_host && *w_zero_point_host != 0) return QTZ_ERR_INVALID_ARG;
    if (w_zero_point_host && (*w_zero_point_host < 0 || *w_zero_point_host > 255)) return QTZ_ERR_INVALID_ARG;
    if (!raw)
        for (int i = 0; i < d.n; ++i)
            if (mult_host[i] < 0 || rshift_host[i] < 1 || rshift_host[i] > 62) return QTZ_ERR_INVALID_ARG;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    qtz_device_guard guard(h->device);       // the caller's current device is restored on every return path
    qtz_plan* p = new (std::nothrow) qtz_plan();
    if (!p) return QTZ_ERR_INVALID_ARG;
    p->h = h;
    p->device = h->device;
    p->d = d;
    p->depthwise = depthwise ? 1 : 0;
    p->oh = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
    p->ow = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
    p->k_total = depthwise ? d.kh * d.kw : d.kh * d.kw * d.c;
    p->w_zp_signed = d.wkind == QTZ_W_U8_PER_LAYER_ASYM ? *w_zero_point_host - 128 : 0;
    if (!raw)
        for (int i = 0; i < d.n; ++i) {
            p->rshift_min = std::min(p->rshift_min, rshift_host[i]);
            p->rshift_max = std::max(p->rshift_max, rshift_host[i]);
        }

#define PLAN_CUDA(expr)                                        \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) {                               \
            qtz_cuda_fail(h, _e, #expr);                       \
            qtz_conv_destroy(p);                               \
            return QTZ_ERR_CUDA;                               \
        }                                                      \
    } while (0)

    const size_t nb = sizeof(int32_t) * static_cast<size_t>(d.n);
    const int n_alloc = d.n + 16;  // room for whole 16-byte channel groups past the last channel
    const size_t nb_alloc = sizeof(int32_t) * static_cast<size_t>(n_alloc);
    PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->bias), nb_alloc));
    PLAN_CUDA(cudaMemsetAsync(p->bias, 0, nb_alloc, st));
    if (bias_q_dev) PLAN_CUDA(cudaMemcpyAsync(p->bias, bias_q_dev, nb, cudaMemcpyDeviceToDevice, st));
    // Largest accumulator any input can produce: |acc| <= K 255 wmax + |bias|.  Beyond int32 the layer is refused
    // (the accumulator of Eq. 4 is 32 bits wide); when even the requantised value stays inside 32 bits for every
    // channel, the epilogue may narrow before it clamps.
    std::vector<int32_t> bias_host(static_cast<size_t>(d.n), 0);
    if (bias_q_dev) {
        PLAN_CUDA(cudaMemcpyAsync(bias_host.data(), bias_q_dev, nb, cudaMemcpyDeviceToHost, st));
        PLAN_CUDA(cudaStreamSynchronize(st));
    }
    const int64_t wmax = d.wkind == QTZ_W_S4_PACKED_PER_CHANNEL_SYM ? 8 : (d.wkind == QTZ_W_S8_PER_CHANNEL_SYM ? 128 : 255);
    for (int i = 0; i < d.n; ++i) {
        const int64_t bound = static_cast<int64_t>(p->k_total) * 255 * wmax + std::llabs(static_cast<long long>(bias_host[i]));
        if (bound > 2147483647LL) {
            qtz_conv_destroy(p);
            return QTZ_ERR_OVERFLOW;
        }
    }
    if (!raw) {
        p->narrow_ok = true;
        for (int i = 0; i < d.n; ++i) {
            const int64_t bound = static_cast<int64_t>(p->k_total) * 255 * wmax + std::llabs(static_cast<long long>(bias_host[i]));
            const unsigned __int128 scaled = (static_cast<unsigned __int128>(bound) * static_cast<uint32_t>(mult_host[i])) >> rshift_host[i];
            if (scaled > static_cast<unsigned __int128>(0x7fffffff - 1024)) p->narrow_ok = false;
        }
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->mult), nb_alloc));
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->rshift), nb_alloc));
        PLAN_CUDA(cudaMemsetAsync(p->mult, 0, nb_alloc, st));
        fill_i32_kernel<<<(n_alloc + 255) / 256, 256, 0, st>>>(p->rshift, n_alloc, 40);
        PLAN_CUDA(cudaGetLastError());
        PLAN_CUDA(cudaMemcpyAsync(p->mult, mult_host, nb, cudaMemcpyHostToDevice, st));
        PLAN_CUDA(cudaMemcpyAsync(p->rshift, rshift_host, nb, cudaMemcpyHostToDevice, st));
    }

    if (depthwise) {
        p->family = QTZ_K_DEPTHWISE;
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->dw_taps), sizeof(uint32_t) * 3 * d.c_pitch_in));
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->dw_wsum), sizeof(int32_t) * d.c_pitch_in));
        prepack_depthwise_kernel<<<(d.c_pitch_in + kThreads - 1) / kThreads, kThreads, 0, st>>>(
            w_q_dev, d.wkind, d.c, d.c_pitch_in, p->dw_taps, p->dw_wsum);
        PLAN_CUDA(cudaGetLastError());
        s = qtz_depthwise_prepare(p);
        if (s != QTZ_OK) {
            qtz_conv_destroy(p);
            return s;
        }
    } else if (qtz_tc_supported(d)) {
        p->family = QTZ_K_TCGEN05;
        s = qtz_tc_prepare(p, w_q_dev, st);
        if (s != QTZ_OK) {
            qtz_conv_destroy(p);
            return s;
        }
    } else {
        if (d.c_pitch_in & 15) {                     // the direct path reads whole 16-byte channel groups
            qtz_conv_destroy(p);
            return QTZ_ERR_MISALIGNED;
        }
        p->family = QTZ_K_DIRECT;
        p->k_padded = (p->k_total + 15) & ~15;
        p->n_padded = (d.n + 63) & ~63;
        const int64_t elems = static_cast<int64_t>(p->n_padded) * p->k_padded;
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->w_direct), static_cast<size_t>(elems)));
        PLAN_CUDA(cudaMalloc(reinterpret_cast<void**>(&p->wsum), sizeof(int32_t) * p->n_padded));
        prepack_direct_kernel<<<static_cast<unsigned>((elems + kThreads - 1) / kThreads), kThreads, 0, st>>>(
            w_q_dev, d.wkind, d.n, p->k_total, p->n_padded, p->k_padded, p->w_direct);
        PLAN_CUDA(cudaGetLastError());
        weight_sum_kernel<<<p->n_padded, kThreads, 0, st>>>(p->w_direct, p->k_padded, p->wsum);
        PLAN_CUDA(cudaGetLastError());
    }
#undef PLAN_CUDA
    *out = p;
    return QTZ_OK;
}

static qtz_status check_run_args(qtz_conv_plan p, const void* x, const void* y, int32_t x_zp, int32_t y_zp,
                                 int32_t act_min, int32_t act_max)
{
    if (!p || !x || !y) return QTZ_ERR_INVALID_ARG;
    if (x_zp < 0 || x_zp > 255) return QTZ_ERR_INVALID_ARG;
    if (p->d.outkind == QTZ_OUT_U8) {
        if (y_zp < 0 || y_zp > 255 || act_min < 0 || act_max > 255 || act_min > act_max) return QTZ_ERR_INVALID_ARG;
    }
    if (!qtz_aligned16(x) || !qtz_aligned16(y)) return QTZ_ERR_MISALIGNED;
    return QTZ_OK;
}

extern "C" qtz_status qtz_conv2d_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point, void* y_dev,
                                    int32_t y_zero_point, int32_t act_min, int32_t act_max, void* stream)
{
    qtz_status s = check_run_args(p, x_dev, y_dev, x_zero_point, y_zero_point, act_min, act_max);
    if (s != QTZ_OK) return s;
    if (p->depthwise) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    qtz_device_guard guard(p->device);
    if (p->family == QTZ_K_TCGEN05)
        return qtz_tc_launch(p, x_dev, x_zero_point, y_dev, y_zero_point, act_min, act_max, st);
    return qtz_direct_launch(p, x_dev, x_zero_point, y_dev, y_zero_point, act_min, act_max, st);
}

extern "C" qtz_status qtz_conv2d_add_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point, const qtz_residual* r,
                                        const uint8_t* s_dev, void* y_dev, int32_t y_zero_point, int32_t act_min,
                                        int32_t act_max, void* stream)
{
    qtz_status s = check_run_args(p, x_dev, y_dev, x_zero_point, y_zero_point, act_min, act_max);
    if (s != QTZ_OK) return s;
    if (!r || !s_dev || p->depthwise) return QTZ_ERR_INVALID_ARG;
    if (!qtz_aligned16(s_dev)) return QTZ_ERR_MISALIGNED;
    if (r->t_zero_point < 0 || r->t_zero_point > 255 || r->s_zero_point < 0 || r->s_zero_point > 255 || r->t_act_min < 0 ||
        r->t_act_max > 255 || r->t_act_min > r->t_act_max || r->t_mult < 0 || r->s_mult < 0)
        return QTZ_ERR_INVALID_ARG;
    if (r->rshift < 1 || r->rshift > 53) return QTZ_ERR_UNSUPPORTED;
    if (p->family != QTZ_K_TCGEN05 || p->d.outkind != QTZ_OUT_U8) return QTZ_ERR_UNSUPPORTED;
    qtz_device_guard guard(p->device);
    return qtz_tc_launch(p, x_dev, x_zero_point, y_dev, y_zero_point, act_min, act_max, static_cast<cudaStream_t>(stream), r, s_dev);
}

extern "C" qtz_status qtz_conv2d_dw_pw_u8(qtz_conv_plan dw, qtz_conv_plan pw, const uint8_t* x_dev, int32_t x_zero_point,
                                          int32_t mid_zero_point, int32_t mid_act_min, int32_t mid_act_max, void* y_dev,
                                          int32_t y_zero_point, int32_t act_min, int32_t act_max, void* stream)
{
    if (!dw) return QTZ_ERR_INVALID_ARG;
    qtz_status s = check_run_args(pw, x_dev, y_dev, x_zero_point, y_zero_point, act_min, act_max);
    if (s != QTZ_OK) return s;
    if (!dw->depthwise || pw->depthwise || dw->h != pw->h || dw->device != pw->device) return QTZ_ERR_INVALID_ARG;
    if (mid_zero_point < 0 || mid_zero_point > 255 || mid_act_min < 0 || mid_act_max > 255 || mid_act_min > mid_act_max)
        return QTZ_ERR_INVALID_ARG;
    if (pw->family != QTZ_K_TCGEN05 || dw->family != QTZ_K_DEPTHWISE) return QTZ_ERR_UNSUPPORTED;
    qtz_device_guard guard(pw->device);
    return qtz_tc_launch_dw_pw(dw, pw, x_dev, x_zero_point, mid_zero_point, mid_act_min, mid_act_max, y_dev, y_zero_point,
                               act_min, act_max, static_cast<cudaStream_t>(stream));
}

extern "C" qtz_status qtz_depthwise_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point, void* y_dev,
                                       int32_t y_zero_point, int32_t act_min, int32_t act_max, void* stream)
{
    qtz_status s = check_run_args(p, x_dev, y_dev, x_zero_point, y_zero_point, act_min, act_max);
    if (s != QTZ_OK) return s;
    if (!p->depthwise) return QTZ_ERR_INVALID_ARG;
    qtz_device_guard guard(p->device);
    return qtz_depthwise_launch(p, x_dev, x_zero_point, static_cast<uint8_t*>(y_dev), y_zero_point, act_min, act_max,
                                static_cast<cudaStream_t>(stream));
}
