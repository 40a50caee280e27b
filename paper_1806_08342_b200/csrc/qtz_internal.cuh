// Internal definitions shared by the translation units of libqtz.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "qtz.h"

#define QTZ_NUM_SMS_DEFAULT 148

struct qtz_ctx {
    int device = 0;
    int num_sms = QTZ_NUM_SMS_DEFAULT;
    // Device scratch reused by consecutive calls (stream-ordered):
    //   params: per-axis quantizer parameters uploaded for quantize / dequantize
    //   reduce: block partials of the min/max reduction
    //   status: [0] device status word, [1] site id
    void* params_dev = nullptr;
    size_t params_bytes = 0;
    float* reduce_dev = nullptr;
    size_t reduce_bytes = 0;
    int32_t* status_dev = nullptr;
    float* reduce_host = nullptr;  // pinned
    size_t reduce_host_bytes = 0;
    bool no_pairs = false;                  // never run layers on CTA pairs (A/B comparisons; set by QTZ_NO_PAIRS=1)
    bool single_row_stems = false;          // row-window layers: one output row per tile (A/B comparisons; QTZ_SINGLE_ROW_STEMS=1)
    long long wait_budget = 2000000000LL;   // cycle budget of every bounded device-side wait (about one second)
    std::string last_error;
};

enum qtz_kernel_family { QTZ_K_DIRECT = 0, QTZ_K_TCGEN05 = 1, QTZ_K_DEPTHWISE = 2 };

// Device status sites (which bounded wait gave up).
enum { QTZ_SITE_TMA_FULL = 1, QTZ_SITE_SMEM_EMPTY = 2, QTZ_SITE_TMEM_FULL = 3,
       QTZ_SITE_TMEM_EMPTY = 4, QTZ_SITE_STORE = 5, QTZ_SITE_OUT_FULL = 6, QTZ_SITE_OUT_EMPTY = 7,
       QTZ_SITE_SELFTEST = 8, QTZ_SITE_PROBE = 9 };

inline qtz_status qtz_cuda_fail(qtz_ctx* h, cudaError_t e, const char* what)
{
    if (h) h->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError();
    return QTZ_ERR_CUDA;
}

#define QTZ_CUDA(h, expr)                                              \
    do {                                                               \
        cudaError_t _e = (expr);                                       \
        if (_e != cudaSuccess) return qtz_cuda_fail((h), _e, #expr);   \
    } while (0)

#define QTZ_LAUNCH_CHECK(h, name)                                      \
    do {                                                               \
        cudaError_t _e = cudaGetLastError();                           \
        if (_e != cudaSuccess) return qtz_cuda_fail((h), _e, name);    \
    } while (0)

// Makes `device` current for the lifetime of the object and puts the caller's device back afterwards.
struct qtz_device_guard {
    int prev = -1;
    bool switched = false;
    explicit qtz_device_guard(int device)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != device) switched = cudaSetDevice(device) == cudaSuccess;
    }
    ~qtz_device_guard()
    {
        if (switched) cudaSetDevice(prev);
    }
    qtz_device_guard(const qtz_device_guard&) = delete;
    qtz_device_guard& operator=(const qtz_device_guard&) = delete;
};

static inline bool qtz_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Grows a handle-owned device buffer (never shrinks).  Stream-ordered reuse is the
// caller's contract, so a plain free + malloc is enough.
qtz_status qtz_ensure_params(qtz_ctx* h, size_t bytes);
qtz_status qtz_ensure_reduce(qtz_ctx* h, size_t bytes);

// Host-side scalar rules (parameter derivation).
qtz_status qtz_host_affine_params(float lo, float hi, int bits, qtz_qparams* q);
qtz_status qtz_host_symmetric_params(float lo, float hi, int bits, qtz_qparams* q);
bool qtz_code_range(int32_t dtype, int32_t restrict_range, int32_t* qmin, int32_t* qmax);
