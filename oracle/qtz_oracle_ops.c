/*
 * qtz_oracle_ops.c -- TEST INFRASTRUCTURE, not a product path (see qtz_oracle.c).
 *
 * Depthwise convolution and the integer glue operations of a quantized network:
 * element-wise add with rescale, max pooling, global average pooling.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#include "orc_common.h"

int orc_quantize_multiplier(double real_multiplier, int32_t* mult, int32_t* rshift);

/* ------------------------------------------------------------------------- */
/* Depthwise form of Eq. 4 (depth multiplier 1): the sum runs over (kh,kw)    */
/* only, each channel has its own kernel w[kh][kw][c] and zero point.         */
/*   acc(b,oh,ow,c) = bias_q[c] + sum_{kh,kw} (x_Q - z_x)(w_Q - z_w[c]).      */
/* x NHWC with pitch xp; acc [b][oh][ow][c].                                  */
/* ------------------------------------------------------------------------- */
int orc_depthwise_acc(const uint8_t* x, int32_t batch, int32_t h, int32_t w_, int32_t c,
                      int32_t xp, int32_t z_x, const int32_t* wq, const int32_t* z_w,
                      const int32_t* bias_q, int32_t kh, int32_t kw, int32_t stride,
                      int32_t pad, int32_t* acc)
{
    if (batch <= 0 || h <= 0 || w_ <= 0 || c <= 0 || kh <= 0 || kw <= 0 || stride <= 0 ||
        pad < 0 || xp < c)
        return ORC_ERR_INVALID;
    const int32_t oh_n = (h + 2 * pad - kh) / stride + 1;
    const int32_t ow_n = (w_ + 2 * pad - kw) / stride + 1;
    if (oh_n <= 0 || ow_n <= 0) return ORC_ERR_INVALID;
#pragma omp parallel for collapse(2) schedule(static)
    for (int32_t b = 0; b < batch; ++b)
        for (int32_t oh = 0; oh < oh_n; ++oh)
            for (int32_t ow = 0; ow < ow_n; ++ow)
                for (int32_t ch = 0; ch < c; ++ch) {
                    int64_t s = bias_q ? bias_q[ch] : 0;
                    const int32_t zw = z_w ? z_w[ch] : 0;
                    for (int32_t i = 0; i < kh; ++i)
                        for (int32_t j = 0; j < kw; ++j) {
                            const int32_t ih = oh * stride - pad + i, iw = ow * stride - pad + j;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w_) continue;
                            int32_t xv = x[(((int64_t)b * h + ih) * w_ + iw) * xp + ch];
                            int32_t wv = wq[((int64_t)i * kw + j) * c + ch];
                            s += (int64_t)(xv - z_x) * (int64_t)(wv - zw);
                        }
                    acc[(((int64_t)b * oh_n + oh) * ow_n + ow) * c + ch] = (int32_t)s;
                }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Section 3.2.1, element-wise add in fixed point: both inputs are rescaled   */
/* to the output scale before they are added (the figure that draws this is   */
/* missing from the text; reading taken):                                     */
/*   M_a = Delta_a/Delta_y, M_b = Delta_b/Delta_y; the larger one fixes the   */
/*   shift r through the normalised 31-bit form, the other is round(M 2^r);   */
/*   y = z_y + floor(((a-z_a) m_a + (b-z_b) m_b + 2^(r-1)) / 2^r), clamped.   */
/* The fused activation (no re-quantisation between add and ReLU) is the      */
/* clamp.                                                                     */
/* ------------------------------------------------------------------------- */
int orc_add_params(float a_scale, float b_scale, float y_scale, int32_t* m_a, int32_t* m_b,
                   int32_t* rshift)
{
    double Ma = (double)a_scale / (double)y_scale, Mb = (double)b_scale / (double)y_scale;
    int32_t m, r;
    int rc = orc_quantize_multiplier(Ma >= Mb ? Ma : Mb, &m, &r);
    if (rc != ORC_OK) return rc;
    double other = rint((Ma >= Mb ? Mb : Ma) * ldexp(1.0, r));
    if (other > 2147483647.0) return ORC_ERR_UNSUPPORTED;
    if (Ma >= Mb) {
        *m_a = m;
        *m_b = (int32_t)other;
    } else {
        *m_b = m;
        *m_a = (int32_t)other;
    }
    *rshift = r;
    return ORC_OK;
}

int orc_add_u8(const uint8_t* a, int32_t z_a, int32_t m_a, const uint8_t* b, int32_t z_b,
               int32_t m_b, int32_t rshift, int32_t z_y, int32_t act_min, int32_t act_max,
               int64_t pixels, int32_t c, int32_t pitch, uint8_t* y)
{
    if (rshift < 1 || rshift > 62 || pitch < c) return ORC_ERR_INVALID;
    for (int64_t p = 0; p < pixels; ++p)
        for (int32_t ch = 0; ch < c; ++ch) {
            int64_t i = p * pitch + ch;
            int64_t v = (int64_t)((int32_t)a[i] - z_a) * m_a + (int64_t)((int32_t)b[i] - z_b) * m_b;
            int64_t r = (int64_t)z_y + ((v + ((int64_t)1 << (rshift - 1))) >> rshift);
            if (r < act_min) r = act_min;
            if (r > act_max) r = act_max;
            y[i] = (uint8_t)r;
        }
    return ORC_OK;
}

/* Max pooling on codes.  The quantizer is monotone, so the maximum of the    */
/* codes is the code of the maximum; input and output share (Delta, z).       */
/* Taps outside the image are skipped.                                        */
int orc_maxpool_u8(const uint8_t* x, int32_t batch, int32_t h, int32_t w_, int32_t c,
                   int32_t xp, int32_t k, int32_t stride, int32_t pad, int32_t yp, uint8_t* y)
{
    const int32_t oh_n = (h + 2 * pad - k) / stride + 1, ow_n = (w_ + 2 * pad - k) / stride + 1;
    if (oh_n <= 0 || ow_n <= 0 || xp < c || yp < c) return ORC_ERR_INVALID;
    for (int32_t b = 0; b < batch; ++b)
        for (int32_t oh = 0; oh < oh_n; ++oh)
            for (int32_t ow = 0; ow < ow_n; ++ow)
                for (int32_t ch = 0; ch < c; ++ch) {
                    int32_t m = 0;
                    for (int32_t i = 0; i < k; ++i)
                        for (int32_t j = 0; j < k; ++j) {
                            const int32_t ih = oh * stride - pad + i, iw = ow * stride - pad + j;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w_) continue;
                            int32_t v = x[(((int64_t)b * h + ih) * w_ + iw) * xp + ch];
                            if (v > m) m = v;
                        }
                    y[(((int64_t)b * oh_n + oh) * ow_n + ow) * yp + ch] = (uint8_t)m;
                }
    return ORC_OK;
}

/* Global average pooling in integers: S = sum_{h,w} (x_Q - z_x), then one     */
/* requantisation with M = Delta_x / (HW Delta_y) supplied as (mult, rshift).  */
int orc_global_avgpool_u8(const uint8_t* x, int32_t z_x, int32_t batch, int32_t hw, int32_t c,
                          int32_t xp, int32_t mult, int32_t rshift, int32_t z_y, int32_t yp,
                          uint8_t* y)
{
    if (rshift < 1 || rshift > 62 || xp < c || yp < c) return ORC_ERR_INVALID;
    for (int32_t b = 0; b < batch; ++b)
        for (int32_t ch = 0; ch < c; ++ch) {
            int64_t s = 0;
            for (int32_t p = 0; p < hw; ++p) s += (int32_t)x[((int64_t)b * hw + p) * xp + ch] - z_x;
            y[(int64_t)b * yp + ch] = (uint8_t)orc_requant1(s, mult, rshift, z_y, 0, 255);
        }
    return ORC_OK;
}
