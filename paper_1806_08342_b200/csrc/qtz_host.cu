// Handle management and the host-side scalar rules of libqtz: quantizer parameters
// from a range (Section 2.1-2.2), fixed-point multipliers, activation clamp ranges.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "qtz_internal.cuh"

extern "C" const char* qtz_status_string(qtz_status s)
{
    switch (s) {
        case QTZ_OK: return "ok";
        case QTZ_ERR_INVALID_ARG: return "invalid argument";
        case QTZ_ERR_MISALIGNED: return "pointer or pitch not aligned as the call requires";
        case QTZ_ERR_UNSUPPORTED: return "unsupported configuration";
        case QTZ_ERR_OVERFLOW: return "reduction too long for int32 accumulation";
        case QTZ_ERR_NONFINITE: return "non-finite value in calibration data";
        case QTZ_ERR_CUDA: return "CUDA error";
        case QTZ_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case QTZ_ERR_NO_DEVICE: return "no usable CUDA device";
        case QTZ_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this non-allocating call";
        default: return "unknown status";
    }
}

extern "C" qtz_status qtz_create(qtz_handle* out, int device)
{
    if (!out) return QTZ_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return QTZ_ERR_NO_DEVICE;
    }
    qtz_ctx* h = new (std::nothrow) qtz_ctx();
    if (!h) return QTZ_ERR_INVALID_ARG;
    h->device = device;
    if (const char* v = std::getenv("QTZ_NO_PAIRS")) h->no_pairs = v[0] == '1';
    if (const char* v = std::getenv("QTZ_SINGLE_ROW_STEMS")) h->single_row_stems = v[0] == '1';
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaMalloc(&h->status_dev, 2 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(h->status_dev, 0, 2 * sizeof(int32_t));
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete h;
        return QTZ_ERR_NO_DEVICE;
    }
    qtz_status s = qtz_ensure_params(h, 64 * 1024);
    if (s == QTZ_OK) s = qtz_ensure_reduce(h, 64 * 1024);
    if (s != QTZ_OK) {
        qtz_destroy(h);
        return s;
    }
    *out = h;
    return QTZ_OK;
}

extern "C" qtz_status qtz_destroy(qtz_handle h)
{
    if (!h) return QTZ_ERR_INVALID_ARG;
    cudaSetDevice(h->device);
    cudaDeviceSynchronize();
    if (h->params_dev) cudaFree(h->params_dev);
    if (h->reduce_dev) cudaFree(h->reduce_dev);
    if (h->status_dev) cudaFree(h->status_dev);
    if (h->reduce_host) cudaFreeHost(h->reduce_host);
    (void)cudaGetLastError();
    delete h;
    return QTZ_OK;
}

extern "C" const char* qtz_last_error(qtz_handle h) { return h ? h->last_error.c_str() : ""; }

extern "C" qtz_status qtz_last_device_status(qtz_handle h, int32_t* site_id, void* stream)
{
    if (!h) return QTZ_ERR_INVALID_ARG;
    int32_t host[2] = {0, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    QTZ_CUDA(h, cudaMemcpyAsync(host, h->status_dev, sizeof(host), cudaMemcpyDeviceToHost, st));
    QTZ_CUDA(h, cudaStreamSynchronize(st));
    if (site_id) *site_id = host[1];
    if (host[0] != 0) {
        QTZ_CUDA(h, cudaMemsetAsync(h->status_dev, 0, sizeof(host), st));
        return QTZ_ERR_DEVICE_TIMEOUT;
    }
    return QTZ_OK;
}

qtz_status qtz_ensure_params(qtz_ctx* h, size_t bytes)
{
    if (bytes <= h->params_bytes) return QTZ_OK;
    if (h->params_dev) QTZ_CUDA(h, cudaFree(h->params_dev));
    h->params_dev = nullptr;
    h->params_bytes = 0;
    QTZ_CUDA(h, cudaMalloc(&h->params_dev, bytes));
    h->params_bytes = bytes;
    return QTZ_OK;
}

qtz_status qtz_ensure_reduce(qtz_ctx* h, size_t bytes)
{
    if (bytes > h->reduce_bytes) {
        if (h->reduce_dev) QTZ_CUDA(h, cudaFree(h->reduce_dev));
        h->reduce_dev = nullptr;
        h->reduce_bytes = 0;
        QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&h->reduce_dev), bytes));
        h->reduce_bytes = bytes;
    }
    if (bytes > h->reduce_host_bytes) {
        if (h->reduce_host) QTZ_CUDA(h, cudaFreeHost(h->reduce_host));
        h->reduce_host = nullptr;
        h->reduce_host_bytes = 0;
        QTZ_CUDA(h, cudaMallocHost(reinterpret_cast<void**>(&h->reduce_host), bytes));
        h->reduce_host_bytes = bytes;
    }
    return QTZ_OK;
}

// Section 2.1.  The real range is widened to hold 0, split into 2^bits - 1 steps, and the
// zero point is the (integer) code that real 0 falls on.
qtz_status qtz_host_affine_params(float lo, float hi, int bits, qtz_qparams* q)
{
    if (!q || bits < 2 || bits > 16) return QTZ_ERR_INVALID_ARG;
    if (!std::isfinite(lo) || !std::isfinite(hi)) return QTZ_ERR_NONFINITE;
    if (hi < lo) return QTZ_ERR_INVALID_ARG;
    const double levels = static_cast<double>((1 << bits) - 1);
    const double rmin = lo < 0.f ? static_cast<double>(lo) : 0.0;
    const double rmax = hi > 0.f ? static_cast<double>(hi) : 0.0;
    float step = static_cast<float>((rmax - rmin) / levels);
    double zp = 0.0;
    if (rmax > rmin && step > 0.f && std::isfinite(step)) {
        zp = std::nearbyint(-rmin / static_cast<double>(step));
        zp = std::fmin(std::fmax(zp, 0.0), levels);
    } else {
        step = 1.0f;  // all-zero tensor
    }
    q->scale = step;
    q->zero_point = static_cast<int32_t>(zp);
    q->min_nudged = static_cast<float>(-q->zero_point) * step;
    q->max_nudged = static_cast<float>(static_cast<int32_t>(levels) - q->zero_point) * step;
    return QTZ_OK;
}

// Section 2.2: zero point fixed at 0, the largest magnitude maps to the top positive code.
qtz_status qtz_host_symmetric_params(float lo, float hi, int bits, qtz_qparams* q)
{
    if (!q || bits < 2 || bits > 16) return QTZ_ERR_INVALID_ARG;
    if (!std::isfinite(lo) || !std::isfinite(hi)) return QTZ_ERR_NONFINITE;
    const int top = (1 << (bits - 1)) - 1;
    const float amax = std::fmax(std::fabs(lo), std::fabs(hi));
    float step = static_cast<float>(static_cast<double>(amax) / top);
    if (!(amax > 0.f) || !(step > 0.f) || !std::isfinite(step)) step = 1.0f;
    q->scale = step;
    q->zero_point = 0;
    q->min_nudged = static_cast<float>(-top) * step;
    q->max_nudged = static_cast<float>(top) * step;
    return QTZ_OK;
}

extern "C" qtz_status qtz_params_from_range(float lo, float hi, int32_t bits, int32_t symmetric,
                                            qtz_qparams* out_host)
{
    return symmetric ? qtz_host_symmetric_params(lo, hi, bits, out_host)
                     : qtz_host_affine_params(lo, hi, bits, out_host);
}

bool qtz_code_range(int32_t dtype, int32_t restrict_range, int32_t* qmin, int32_t* qmax)
{
    switch (dtype) {
        case QTZ_U8: *qmin = 0; *qmax = restrict_range ? 254 : 255; return true;
        case QTZ_S8: *qmin = restrict_range ? -127 : -128; *qmax = 127; return true;
        case QTZ_S4_PACKED: *qmin = restrict_range ? -7 : -8; *qmax = 7; return true;
        case QTZ_U4_PACKED: *qmin = 0; *qmax = restrict_range ? 14 : 15; return true;
        case QTZ_U16: *qmin = 0; *qmax = restrict_range ? 65534 : 65535; return true;
        case QTZ_S16: *qmin = restrict_range ? -32767 : -32768; *qmax = 32767; return true;
        default: return false;
    }
}

// M = mantissa * 2^exponent with mantissa in [0.5, 1): keep 31 bits of the mantissa.
extern "C" qtz_status qtz_quantize_multiplier(double real_multiplier, int32_t* mult, int32_t* rshift)
{
    if (!mult || !rshift || !(real_multiplier >= 0.0) || !std::isfinite(real_multiplier))
        return QTZ_ERR_INVALID_ARG;
    if (real_multiplier == 0.0) {
        *mult = 0;
        *rshift = 1;
        return QTZ_OK;
    }
    int exponent = 0;
    const double mantissa = std::frexp(real_multiplier, &exponent);
    long long fixed = std::llrint(std::ldexp(mantissa, 31));
    if (fixed >= (1LL << 31)) {  // mantissa rounded up to 1.0
        fixed >>= 1;
        ++exponent;
    }
    const int shift = 31 - exponent;
    if (shift < 1 || shift > 62) return QTZ_ERR_UNSUPPORTED;
    *mult = static_cast<int32_t>(fixed);
    *rshift = shift;
    return QTZ_OK;
}

extern "C" qtz_status qtz_activation_range_bits(int32_t kind, float y_scale, int32_t y_zero_point, int32_t bits,
                                                int32_t* act_min, int32_t* act_max)
{
    if (!act_min || !act_max || bits < 2 || bits > 8) return QTZ_ERR_INVALID_ARG;
    const int32_t top_code = (1 << bits) - 1;
    switch (kind) {
        case 0: *act_min = 0; *act_max = top_code; return QTZ_OK;
        case 1: *act_min = y_zero_point; *act_max = top_code; return QTZ_OK;
        case 2: {
            if (!(y_scale > 0.f)) return QTZ_ERR_INVALID_ARG;
            const double top = y_zero_point + std::nearbyint(6.0 / static_cast<double>(y_scale));
            *act_min = y_zero_point;
            *act_max = top < static_cast<double>(top_code) ? static_cast<int32_t>(top) : top_code;
            return QTZ_OK;
        }
        default: return QTZ_ERR_INVALID_ARG;
    }
}

extern "C" qtz_status qtz_activation_range(int32_t kind, float y_scale, int32_t y_zero_point,
                                           int32_t* act_min, int32_t* act_max)
{
    return qtz_activation_range_bits(kind, y_scale, y_zero_point, 8, act_min, act_max);
}

extern "C" qtz_status qtz_add_params(float a_scale, float b_scale, float y_scale, int32_t* a_mult,
                                     int32_t* b_mult, int32_t* rshift)
{
    if (!a_mult || !b_mult || !rshift || !(y_scale > 0.f) || !(a_scale > 0.f) || !(b_scale > 0.f))
        return QTZ_ERR_INVALID_ARG;
    const double ra = static_cast<double>(a_scale) / y_scale;
    const double rb = static_cast<double>(b_scale) / y_scale;
    const bool a_is_big = ra >= rb;
    int32_t big = 0, sh = 0;
    qtz_status s = qtz_quantize_multiplier(a_is_big ? ra : rb, &big, &sh);
    if (s != QTZ_OK) return s;
    const double small = std::nearbyint(std::ldexp(a_is_big ? rb : ra, sh));
    if (small > 2147483647.0) return QTZ_ERR_UNSUPPORTED;
    *a_mult = a_is_big ? big : static_cast<int32_t>(small);
    *b_mult = a_is_big ? static_cast<int32_t>(small) : big;
    *rshift = sh;
    return QTZ_OK;
}

// ---- range rules for the tensors between the layers of a network (Sections 2.5, 3.1.2, 3.2.1) ----

extern "C" qtz_status qtz_range_after_activation(float lo, float hi, int32_t kind, float* lo_out, float* hi_out)
{
    if (!lo_out || !hi_out || kind < 0 || kind > 2) return QTZ_ERR_INVALID_ARG;
    if (!std::isfinite(lo) || !std::isfinite(hi)) return QTZ_ERR_NONFINITE;
    if (hi < lo) return QTZ_ERR_INVALID_ARG;
    if (kind != 0) {                       // ReLU and ReLU6 are monotone: the range goes through them end by end
        lo = std::fmax(lo, 0.0f);
        hi = std::fmax(hi, 0.0f);
    }
    if (kind == 2) {
        lo = std::fmin(lo, 6.0f);
        hi = std::fmin(hi, 6.0f);
    }
    *lo_out = lo;
    *hi_out = hi;
    return QTZ_OK;
}

extern "C" qtz_status qtz_add_output_range(const qtz_qparams* a, const qtz_qparams* b, int32_t kind, float* lo_out,
                                           float* hi_out)
{
    if (!a || !b) return QTZ_ERR_INVALID_ARG;
    // interval sum of what the two inputs can represent, in fp32
    return qtz_range_after_activation(a->min_nudged + b->min_nudged, a->max_nudged + b->max_nudged, kind, lo_out, hi_out);
}

extern "C" qtz_status qtz_accumulator_scales(float x_scale, const qtz_qparams* w_params_host, int64_t n,
                                             qtz_qparams* acc_params_host)
{
    if (!w_params_host || !acc_params_host || n <= 0 || !(x_scale > 0.f)) return QTZ_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {
        acc_params_host[i].scale = x_scale * w_params_host[i].scale;     // one fp32 product
        acc_params_host[i].zero_point = 0;
        acc_params_host[i].min_nudged = 0.f;
        acc_params_host[i].max_nudged = 0.f;
    }
    return QTZ_OK;
}

extern "C" qtz_status qtz_requant_multipliers(float x_scale, const qtz_qparams* w_params_host, int64_t n, float y_scale,
                                              int32_t* mult_host, int32_t* rshift_host)
{
    if (!w_params_host || !mult_host || !rshift_host || n <= 0 || !(x_scale > 0.f) || !(y_scale > 0.f))
        return QTZ_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {
        const double m = static_cast<double>(x_scale) * static_cast<double>(w_params_host[i].scale) / static_cast<double>(y_scale);
        const qtz_status s = qtz_quantize_multiplier(m, mult_host + i, rshift_host + i);
        if (s != QTZ_OK) return s;
    }
    return QTZ_OK;
}

extern "C" qtz_status qtz_avgpool_multiplier(int32_t hw, float x_scale, float y_scale, int32_t* mult, int32_t* rshift)
{
    if (hw <= 0 || !(x_scale > 0.f) || !(y_scale > 0.f)) return QTZ_ERR_INVALID_ARG;
    // identical quantizers in and out leave exactly 1 / hw
    const double m = x_scale == y_scale ? 1.0 / hw : static_cast<double>(x_scale) / (static_cast<double>(hw) * static_cast<double>(y_scale));
    return qtz_quantize_multiplier(m, mult, rshift);
}
