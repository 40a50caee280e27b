/*
 * qtz_oracle_conv.c -- TEST INFRASTRUCTURE, not a product path (see qtz_oracle.c).
 *
 * Batch-norm folding, fixed-point multipliers, the quantized convolution in its
 * defining form (zero points subtracted before every multiply), depthwise
 * convolution, and the integer element-wise add / pooling the networks need.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "orc_common.h"

/* ------------------------------------------------------------------------- */
/* Eq. 20-21: W_inf = gamma W / sigma, Bias_inf = beta - gamma mu / sigma.    */
/* Readings: sigma = sqrt(var + eps) (the paper writes sigma only); a conv    */
/* bias b, when present, enters as beta + gamma (b - mu) / sigma; arithmetic  */
/* in float64, results rounded once to fp32.  W is [n][k] (one row per output */
/* channel).                                                                  */
/* ------------------------------------------------------------------------- */
int orc_fold_batchnorm(const float* w, const float* conv_bias, const float* gamma,
                       const float* beta, const float* mean, const float* var, float eps,
                       int64_t n, int64_t k, float* w_inf, float* bias_inf)
{
    if (n <= 0 || k <= 0) return ORC_ERR_INVALID;
    for (int64_t c = 0; c < n; ++c) {
        double sigma = sqrt((double)var[c] + (double)eps);
        double g = (double)gamma[c];
        for (int64_t i = 0; i < k; ++i)
            w_inf[c * k + i] = (float)((g * (double)w[c * k + i]) / sigma);
        double b = conv_bias ? (double)conv_bias[c] : 0.0;
        bias_inf[c] = (float)((double)beta[c] + (g * (b - (double)mean[c])) / sigma);
    }
    return ORC_OK;
}

/* Bias as an int32 with scale Delta_x * Delta_w[n] and zero point 0, so that it */
/* adds to the accumulator of Eq. 4 without rescaling (the paper's fixed-point   */
/* figure is missing; this is the reading taken).                                */
int orc_quantize_bias(const float* bias, int64_t n, float x_scale, const float* w_scale,
                      int32_t* bias_q)
{
    for (int64_t c = 0; c < n; ++c) {
        double s = (double)x_scale * (double)w_scale[c];
        double r = rint((double)bias[c] / s);
        if (isnan(r)) return ORC_ERR_NONFINITE;
        if (r > 2147483647.0) r = 2147483647.0;
        if (r < -2147483648.0) r = -2147483648.0;
        bias_q[c] = (int32_t)r;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Fixed-point form of a positive real multiplier M (the rescale              */
/* Delta_w Delta_x / Delta_y implied by Eq. 4; the paper defers the details   */
/* to its references, so this is a definition of this code base):             */
/*   M = f 2^e, f in [0.5,1);  m = round(f 2^31);  m == 2^31 -> m = 2^30, e+1 */
/*   r = 31 - e, 1 <= r <= 62;  M ~= m 2^-r.   M == 0 -> m = 0, r = 1.        */
/* ------------------------------------------------------------------------- */
int orc_quantize_multiplier(double real_multiplier, int32_t* mult, int32_t* rshift)
{
    if (!(real_multiplier >= 0.0) || !isfinite(real_multiplier)) return ORC_ERR_INVALID;
    if (real_multiplier == 0.0) {
        *mult = 0;
        *rshift = 1;
        return ORC_OK;
    }
    int e = 0;
    double f = frexp(real_multiplier, &e);
    int64_t m = (int64_t)rint(f * 2147483648.0);
    if (m == 2147483648LL) {
        m = 1073741824LL;
        e += 1;
    }
    int r = 31 - e;
    if (r < 1 || r > 62) return ORC_ERR_UNSUPPORTED;
    *mult = (int32_t)m;
    *rshift = r;
    return ORC_OK;
}

/* Clamp range of a fused activation in the quantized domain (Section 3.2.1:  */
/* the activation fuses into the producing op).  kind 0: none -> [0,255];     */
/* 1: ReLU -> [z_y,255]; 2: ReLU6 -> [z_y, min(255, z_y + round(6/Delta_y))]. */
int orc_activation_range(int kind, float y_scale, int32_t y_zero_point,
                         int32_t* act_min, int32_t* act_max)
{
    if (kind == 0) {
        *act_min = 0;
        *act_max = 255;
    } else if (kind == 1) {
        *act_min = y_zero_point;
        *act_max = 255;
    } else if (kind == 2) {
        double six = rint(6.0 / (double)y_scale);
        double hi = (double)y_zero_point + six;
        *act_min = y_zero_point;
        *act_max = hi > 255.0 ? 255 : (int32_t)hi;
    } else
        return ORC_ERR_INVALID;
    return ORC_OK;
}

int orc_requantize(const int32_t* acc, int64_t rows, int64_t n, const int32_t* mult,
                   const int32_t* rshift, int32_t y_zero_point, int32_t act_min,
                   int32_t act_max, int32_t* y)
{
    for (int64_t c = 0; c < n; ++c)
        if (rshift[c] < 1 || rshift[c] > 62 || mult[c] < 0) return ORC_ERR_INVALID;
    for (int64_t p = 0; p < rows; ++p)
        for (int64_t c = 0; c < n; ++c)
            y[p * n + c] = orc_requant1(acc[p * n + c], mult[c], rshift[c], y_zero_point,
                                    act_min, act_max);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Eq. 4, the defining form: each accumulator is                              */
/*   acc(b,oh,ow,n) = bias_q[n] + sum_{kh,kw,c} (x_Q - z_x)(w_Q[n] - z_w[n]), */
/* the zero points being subtracted BEFORE the multiply.  Taps that fall      */
/* outside the image contribute nothing: padding is real zero, which is the   */
/* code z_x (Section 2.1).  x is NHWC with channel pitch xp (bytes per pixel),*/
/* w is [n][kh][kw][c] (int32 codes), acc is [b][oh][ow][n] int32.            */
/* Accumulation in int64; a sum that leaves int32 is an error.                */
/* ------------------------------------------------------------------------- */
int orc_conv2d_acc(const uint8_t* x, int32_t batch, int32_t h, int32_t w_, int32_t c,
                   int32_t xp, int32_t z_x, const int32_t* wq, const int32_t* z_w,
                   const int32_t* bias_q, int32_t n, int32_t kh, int32_t kw,
                   int32_t stride, int32_t pad, int32_t* acc)
{
    if (batch <= 0 || h <= 0 || w_ <= 0 || c <= 0 || n <= 0 || kh <= 0 || kw <= 0 ||
        stride <= 0 || pad < 0 || xp < c)
        return ORC_ERR_INVALID;
    const int32_t oh_n = (h + 2 * pad - kh) / stride + 1;
    const int32_t ow_n = (w_ + 2 * pad - kw) / stride + 1;
    if (oh_n <= 0 || ow_n <= 0) return ORC_ERR_INVALID;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int32_t b = 0; b < batch; ++b)
        for (int32_t oh = 0; oh < oh_n; ++oh)
            for (int32_t ow = 0; ow < ow_n; ++ow)
                for (int32_t o = 0; o < n; ++o) {
                    int64_t s = bias_q ? bias_q[o] : 0;
                    const int32_t zw = z_w ? z_w[o] : 0;
                    for (int32_t i = 0; i < kh; ++i) {
                        const int32_t ih = oh * stride - pad + i;
                        if (ih < 0 || ih >= h) continue;
                        for (int32_t j = 0; j < kw; ++j) {
                            const int32_t iw = ow * stride - pad + j;
                            if (iw < 0 || iw >= w_) continue;
                            const uint8_t* xr = x + (((int64_t)b * h + ih) * w_ + iw) * xp;
                            const int32_t* wr = wq + (((int64_t)o * kh + i) * kw + j) * c;
                            for (int32_t ch = 0; ch < c; ++ch)
                                s += (int64_t)((int32_t)xr[ch] - z_x) * (int64_t)(wr[ch] - zw);
                        }
                    }
                    if (s > 2147483647LL || s < -2147483648LL) overflow = 1;
                    acc[(((int64_t)b * oh_n + oh) * ow_n + ow) * n + o] = (int32_t)s;
                }
    return overflow ? ORC_ERR_OVERFLOW : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Eq. 5-6, the expanded form, written out term by term so that the identity  */
/* with Eq. 4 can be tested:                                                  */
/*   raw conv(w_Q, x_Q) - z_w sum x_Q - z_x sum w_Q + K_valid z_x z_w.        */
/* Reading: the paper prints the constant as z_x z_w with no count; expanding */
/* Eq. 4 gives one z_x z_w per in-image tap and channel, K_valid of them.     */
/* Sums run over in-image taps only.                                          */
/* ------------------------------------------------------------------------- */
int orc_conv2d_acc_expanded(const uint8_t* x, int32_t batch, int32_t h, int32_t w_,
                            int32_t c, int32_t xp, int32_t z_x, const int32_t* wq,
                            const int32_t* z_w, const int32_t* bias_q, int32_t n,
                            int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                            int32_t* acc)
{
    const int32_t oh_n = (h + 2 * pad - kh) / stride + 1;
    const int32_t ow_n = (w_ + 2 * pad - kw) / stride + 1;
    if (oh_n <= 0 || ow_n <= 0) return ORC_ERR_INVALID;
    for (int32_t b = 0; b < batch; ++b)
        for (int32_t oh = 0; oh < oh_n; ++oh)
            for (int32_t ow = 0; ow < ow_n; ++ow)
                for (int32_t o = 0; o < n; ++o) {
                    int64_t raw = 0, sum_x = 0, sum_w = 0, k_valid = 0;
                    for (int32_t i = 0; i < kh; ++i)
                        for (int32_t j = 0; j < kw; ++j) {
                            const int32_t ih = oh * stride - pad + i, iw = ow * stride - pad + j;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w_) continue;
                            for (int32_t ch = 0; ch < c; ++ch) {
                                int64_t xv = x[(((int64_t)b * h + ih) * w_ + iw) * xp + ch];
                                int64_t wv = wq[(((int64_t)o * kh + i) * kw + j) * c + ch];
                                raw += xv * wv;
                                sum_x += xv;
                                sum_w += wv;
                                k_valid += 1;
                            }
                        }
                    const int64_t zw = z_w ? z_w[o] : 0;
                    int64_t s = raw - zw * sum_x - (int64_t)z_x * sum_w + k_valid * z_x * zw +
                                (bias_q ? bias_q[o] : 0);
                    acc[(((int64_t)b * oh_n + oh) * ow_n + ow) * n + o] = (int32_t)s;
                }
    return ORC_OK;
}
