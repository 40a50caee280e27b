// A convolution plan: the layer's geometry plus everything prepared once per layer
// (re-laid weights, per-channel weight sums of the zero-point cross term, multipliers).
#pragma once

#include <cuda.h>

#include "qtz_internal.cuh"

struct qtz_tc_state;  // tensor-core path state (tensor maps, tile shape); see qtz_conv_tc.cu
struct qtz_dw_state;  // depthwise path state (tile shape, thread mapping); see qtz_depthwise.cu

struct qtz_plan {
    qtz_ctx* h = nullptr;
    int device = 0;
    qtz_conv_desc d{};
    int depthwise = 0;
    int family = QTZ_K_DIRECT;
    int oh = 0, ow = 0;
    int k_total = 0;      // kh*kw*c
    int k_padded = 0;     // row length of w_direct (multiple of 16)
    int n_padded = 0;     // rows of w_direct (multiple of 64)
    int rshift_max = 1;
    int rshift_min = 62;  // smallest per-channel right shift (selects the epilogue's requantise form)
    bool narrow_ok = false;  // every requantised value provably fits 32 bits before the clamp (any accumulator, any shift)
    int w_zp_signed = 0;  // weight zero point after moving codes to int8 (z_w - 128 for uint8 weights)

    int8_t* w_direct = nullptr;   // [n_padded][k_padded] int8, zero padded       (direct path)
    uint32_t* dw_taps = nullptr;  // [3][c_pitch_in]: per filter row and channel the int8 codes (k0,k1,k2,0)  (depthwise path)
    int32_t* dw_wsum = nullptr;   // [c_pitch_in]: sum of the nine int8 codes                                   (depthwise path)
    int32_t* bias = nullptr;      // [n + 16] (zeros when the layer has no bias); bias, mult, rshift are padded so that
                                  // 16-byte loads of a channel group never leave the array
    int32_t* wsum = nullptr;      // [classes][n] sum of int8 weight codes per border class
    int32_t* mult = nullptr;      // [n + 16], padded like bias (multiplier 0, shift 40 beyond n)
    int32_t* rshift = nullptr;    // [n + 16]
    uint8_t* x_gather = nullptr;  // strided 1x1 layers: the sub-sampled input, pitched NHWC
    qtz_tc_state* tc = nullptr;
    qtz_dw_state* dw = nullptr;
    cudaEvent_t ev_start = nullptr, ev_stop = nullptr;  // optional profiling hook
    std::string detail;                                 // how the most recent launch ran (qtz_conv_plan_detail)
};

// Direct (CUDA-core) path.
qtz_status qtz_direct_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, void* y, int32_t y_zp,
                             int32_t act_min, int32_t act_max, cudaStream_t st);
qtz_status qtz_depthwise_prepare(qtz_plan* p);
void qtz_depthwise_release(qtz_plan* p);
qtz_status qtz_depthwise_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, uint8_t* y, int32_t y_zp,
                                int32_t act_min, int32_t act_max, cudaStream_t st);

// Tensor-core (tcgen05) path.
bool qtz_tc_supported(const qtz_conv_desc& d);
qtz_status qtz_tc_prepare(qtz_plan* p, const void* w_q_dev, cudaStream_t st);
void qtz_tc_release(qtz_plan* p);
// res / s_dev: NULL, or the residual add fused into the epilogue and its second addend (qtz_conv2d_add_u8).
qtz_status qtz_tc_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, void* y, int32_t y_zp,
                         int32_t act_min, int32_t act_max, cudaStream_t st, const qtz_residual* res = nullptr,
                         const uint8_t* s_dev = nullptr);

// A 3x3 depthwise plan and the pointwise plan that follows it, in one kernel (the intermediate tensor, with zero point
// mid_zp and clamp [mid_min, mid_max], stays in shared memory).  QTZ_ERR_UNSUPPORTED when the pair cannot run that way.
qtz_status qtz_tc_launch_dw_pw(qtz_plan* dw, qtz_plan* pw, const uint8_t* x, int32_t x_zp, int32_t mid_zp, int32_t mid_min,
                               int32_t mid_max, void* y, int32_t y_zp, int32_t act_min, int32_t act_max, cudaStream_t st);

// Encodes a rank-2 or rank-4 uint8 tensor map (dims[0] contiguous).  swizzle_bytes: 0 (none), 32, 64 or 128.
bool qtz_encode_u8_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                       const uint32_t* box, int swizzle_bytes);
