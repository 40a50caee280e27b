/*
 * qtz_oracle_sim.c -- TEST INFRASTRUCTURE, not a product path (see qtz_oracle.c).
 *
 * The quantizer utilities around the convolution path: simulated quantization
 * and the signal-to-quantization-noise ratio built on it, the moving average of
 * activation ranges over batches, and the rescale of a uint8 tensor to another
 * quantizer (what a concatenation needs).  Plain loops, fp64 where the paper
 * does not fix a precision.
 *
 * Parity pins (tests/test_oracle_sim.py): idempotence and the half-step error
 * bound of SimQuant, its float64 closed form away from ties, the textbook
 * 20 log10(2 (2^b - 1)) dB of a uniform signal, hand-computed SQNR values, the
 * closed form of an exponential average of a constant, exact rationals for the
 * rescale.  By-definition choices are listed beside each function.
 */
#include <math.h>
#include <stdint.h>

#include "orc_common.h"

typedef struct {
    float scale;
    int32_t zero_point;
    float min_nudged;
    float max_nudged;
} orc_qparams;

/* ------------------------------------------------------------------------- */
/* Section 2.4 (the SimQuant equations): a quantizer followed by a            */
/* de-quantizer.  The printed second line has the sign of z flipped and never */
/* removes z again; the reading taken is Eq. 3 applied to Eq. 1-2:            */
/*   x_out = (clamp(round(x / Delta) + z, qmin, qmax) - z) * Delta            */
/* with the same fp32 steps as the quantizer and the de-quantizer.            */
/* ------------------------------------------------------------------------- */
int orc_simquant(const float* x, int64_t outer, int64_t axis_len, int64_t inner,
                 const orc_qparams* p, int32_t qmin, int32_t qmax, float* y)
{
    if (outer <= 0 || axis_len <= 0 || inner <= 0 || qmin > qmax) return ORC_ERR_INVALID;
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t a = 0; a < axis_len; ++a) {
            const float delta = p[a].scale;
            const int32_t z = p[a].zero_point;
            const float tlo = (float)(qmin - z), thi = (float)(qmax - z);
            for (int64_t i = 0; i < inner; ++i) {
                int64_t idx = (o * axis_len + a) * inner + i;
                /* quantize (Eq. 1-2) */
                float t = x[idx] / delta;
                t = rintf(t);
                t = fminf(fmaxf(t, tlo), thi);
                int32_t q = (int32_t)t + z;
                /* de-quantize (Eq. 3) */
                y[idx] = (float)(q - z) * delta;
            }
        }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Appendix A: SQNR = 10 log10( sum W^2 / sum (W - SimQuant(W))^2 ), here per */
/* index of the middle axis of w[outer][axis_len][inner] (per output feature  */
/* map), or for the whole tensor with axis_len = 1.  fp64 sums in index       */
/* order.  Reading: no noise at all gives +infinity.                          */
/* ------------------------------------------------------------------------- */
int orc_sqnr(const float* w, const float* w_hat, int64_t outer, int64_t axis_len, int64_t inner,
             double* sqnr_db)
{
    if (outer <= 0 || axis_len <= 0 || inner <= 0) return ORC_ERR_INVALID;
    for (int64_t a = 0; a < axis_len; ++a) {
        double signal = 0.0, noise = 0.0;
        for (int64_t o = 0; o < outer; ++o)
            for (int64_t i = 0; i < inner; ++i) {
                int64_t idx = (o * axis_len + a) * inner + i;
                double v = (double)w[idx], e = (double)w[idx] - (double)w_hat[idx];
                signal += v * v;
                noise += e * e;
            }
        sqnr_db[a] = noise == 0.0 ? INFINITY : 10.0 * log10(signal / noise);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Section 2.5: activation ranges are the moving average of the per-batch     */
/* minimum and maximum.  The paper names no weighting; the reading taken is   */
/* the exponential average  s <- d s + (1 - d) v  (0 <= d < 1) in fp64, the   */
/* first batch initialising the state.                                        */
/* ------------------------------------------------------------------------- */
int orc_ema_update(double* state_lo, double* state_hi, const float* batch_lo, const float* batch_hi,
                   int64_t n, double decay, int32_t* initialised)
{
    if (n <= 0 || !(decay >= 0.0 && decay < 1.0)) return ORC_ERR_INVALID;
    for (int64_t i = 0; i < n; ++i) {
        if (!isfinite(batch_lo[i]) || !isfinite(batch_hi[i])) return ORC_ERR_NONFINITE;
        if (!*initialised) {
            state_lo[i] = (double)batch_lo[i];
            state_hi[i] = (double)batch_hi[i];
        } else {
            state_lo[i] = decay * state_lo[i] + (1.0 - decay) * (double)batch_lo[i];
            state_hi[i] = decay * state_hi[i] + (1.0 - decay) * (double)batch_hi[i];
        }
    }
    *initialised = 1;
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Section 3.2.1 (concatenation): the inputs of a concat must share the       */
/* output's quantizer, so each one is rescaled to it.  With M = Delta_x /     */
/* Delta_y = m 2^-r in the fixed-point form of this code base:                */
/*   y = clamp(z_y + floor(((x - z_x) m + 2^(r-1)) / 2^r))                    */
/* x is [pixels][c] with a pixel pitch, y likewise (a channel slice of the    */
/* concatenated tensor is y + offset with the pitch of the whole).            */
/* ------------------------------------------------------------------------- */
int orc_rescale_u8(const uint8_t* x, int64_t pixels, int32_t c, int32_t x_pitch, int32_t zx,
                   int32_t m, int32_t r, int32_t zy, int32_t act_min, int32_t act_max,
                   uint8_t* y, int32_t y_pitch)
{
    if (pixels <= 0 || c <= 0 || x_pitch < c || y_pitch < c || r < 1 || r > 62) return ORC_ERR_INVALID;
    if (act_min < 0 || act_max > 255 || act_min > act_max) return ORC_ERR_INVALID;
    for (int64_t p = 0; p < pixels; ++p)
        for (int32_t ch = 0; ch < c; ++ch)
            y[p * y_pitch + ch] =
                (uint8_t)orc_requant1((int64_t)x[p * x_pitch + ch] - zx, m, r, zy, act_min, act_max);
    return ORC_OK;
}
