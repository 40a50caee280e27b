/*
 * qtz_oracle.c -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, obviously-correct CPU statement of integer-only inference of a
 * quantized convolution layer under uniform affine quantization (Krishnamoorthi,
 * "Quantizing deep convolutional networks for efficient inference", 2018).
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no code with the CUDA library and must never be used to produce a
 * product result.
 *
 * Every function cites the passage of the paper it follows.  Where the paper is
 * silent (fixed-point requantisation, integer pooling, bias format) the reading
 * taken is written next to the code.
 *
 * Parity pins: every function here is pinned by tests that do not call it to
 * derive their expected values (closed forms, the paper's worked example, exact
 * rational arithmetic, float64 convolution of dequantised tensors, textbook
 * special cases).  The only by-definition choices ("parity unpinned" by the
 * paper itself) are the tie rules: round-half-to-even on the fp32 quotient in
 * the quantizer and round-half-up in the requantising shift.
 *
 * Build: gcc -O2 -std=c11 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "orc_common.h"

typedef struct {
    float scale;        /* Delta                                  */
    int32_t zero_point; /* z                                      */
    float min_nudged;   /* real value of the lowest code          */
    float max_nudged;   /* real value of the highest code         */
} orc_qparams;

/* ------------------------------------------------------------------------- */
/* Section 2.5: weights use their actual min and max; activations use the     */
/* min and max seen on a batch.  View: x[outer][axis_len][inner]; one (lo,hi) */
/* pair per index of the middle axis.                                         */
/* ------------------------------------------------------------------------- */
int orc_minmax(const float* x, int64_t outer, int64_t axis_len, int64_t inner,
               float* lo_out, float* hi_out)
{
    if (outer <= 0 || axis_len <= 0 || inner <= 0) return ORC_ERR_INVALID;
    int bad = 0;
    for (int64_t a = 0; a < axis_len; ++a) {
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t o = 0; o < outer; ++o)
            for (int64_t i = 0; i < inner; ++i) {
                float v = x[(o * axis_len + a) * inner + i];
                if (!isfinite(v)) bad = 1;
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
        lo_out[a] = lo;
        hi_out[a] = hi;
    }
    return bad ? ORC_ERR_NONFINITE : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Section 2.1: scale and zero-point of the affine quantizer.                 */
/*  - the range is relaxed to contain 0 (the (2.1,3.5) -> (0,3.5) example);   */
/*  - Delta = (max - min) / (N_levels - 1);                                   */
/*  - z is an integer so that real 0 is a code: z = round(-min / Delta),      */
/*    kept inside [0, N_levels-1];                                            */
/*  - the representable range moves to [(0-z)Delta, (L-z)Delta] ("nudging").  */
/* Reading where the paper is silent: an all-zero tensor gets Delta=1, z=0.   */
/* ------------------------------------------------------------------------- */
int orc_affine_params(float lo, float hi, int bits, orc_qparams* q)
{
    if (bits < 2 || bits > 16) return ORC_ERR_INVALID;   /* Section 7: 4, 8 and 16 bits */
    if (!isfinite(lo) || !isfinite(hi)) return ORC_ERR_NONFINITE;
    if (lo > hi) return ORC_ERR_INVALID;
    if (lo > 0.0f) lo = 0.0f;
    if (hi < 0.0f) hi = 0.0f;
    const int L = (1 << bits) - 1;
    float delta;
    int32_t z;
    double d64 = ((double)hi - (double)lo) / (double)L;
    delta = (float)d64;
    if (hi == lo || !(delta > 0.0f) || !isfinite(delta)) {
        delta = 1.0f;
        z = 0;
    } else {
        double zr = rint(-(double)lo / (double)delta);
        if (zr < 0.0) zr = 0.0;
        if (zr > (double)L) zr = (double)L;
        z = (int32_t)zr;
    }
    q->scale = delta;
    q->zero_point = z;
    q->min_nudged = (float)(0 - z) * delta;
    q->max_nudged = (float)(L - z) * delta;
    return ORC_OK;
}

/* Section 2.2: symmetric quantizer, z = 0, Delta = max|x| / (N_levels/2 - 1). */
/* All-zero channel: Delta = 1.                                                */
int orc_symmetric_params(float lo, float hi, int bits, orc_qparams* q)
{
    if (bits < 2 || bits > 16) return ORC_ERR_INVALID;   /* Section 7: 4, 8 and 16 bits */
    if (!isfinite(lo) || !isfinite(hi)) return ORC_ERR_NONFINITE;
    float a = fabsf(lo) > fabsf(hi) ? fabsf(lo) : fabsf(hi);
    const int P = (1 << (bits - 1)) - 1;
    float delta = (float)((double)a / (double)P);
    if (a == 0.0f || !(delta > 0.0f) || !isfinite(delta)) delta = 1.0f;
    q->scale = delta;
    q->zero_point = 0;
    q->min_nudged = (float)(-P) * delta;
    q->max_nudged = (float)(P)*delta;
    return ORC_OK;
}

/* min/max reduction followed by parameter derivation, one entry per axis index. */
int orc_calibrate_minmax(const float* x, int64_t outer, int64_t axis_len, int64_t inner,
                         int bits, int symmetric, orc_qparams* out)
{
    float* lo = (float*)malloc(sizeof(float) * (size_t)(axis_len > 0 ? axis_len : 1));
    float* hi = (float*)malloc(sizeof(float) * (size_t)(axis_len > 0 ? axis_len : 1));
    int rc = orc_minmax(x, outer, axis_len, inner, lo, hi);
    for (int64_t a = 0; rc == ORC_OK && a < axis_len; ++a)
        rc = symmetric ? orc_symmetric_params(lo[a], hi[a], bits, &out[a])
                       : orc_affine_params(lo[a], hi[a], bits, &out[a]);
    free(lo);
    free(hi);
    return rc;
}

/* Code range of a quantizer: Eq. 2 (affine, unsigned), Eq. 8 (signed           */
/* symmetric), Eq. 10 (signed symmetric with the restricted range).            */
int orc_code_range(int bits, int is_signed, int restrict_range, int32_t* qmin, int32_t* qmax)
{
    if (bits < 2 || bits > 16) return ORC_ERR_INVALID;   /* Section 7: 4, 8 and 16 bits */
    if (is_signed) {
        *qmax = (1 << (bits - 1)) - 1;
        *qmin = restrict_range ? -*qmax : -(1 << (bits - 1));
    } else {
        *qmin = 0;
        *qmax = (1 << bits) - 1 - (restrict_range ? 1 : 0);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Eq. 1-2 (and Eq. 7-11 with z = 0): x_int = round(x/Delta) + z, clamped to  */
/* the code range.  Readings: the quotient is one IEEE fp32 division, round() */
/* is round-half-to-even, the clamp is applied before z is added (the same    */
/* result, without integer overflow for huge |x|).  NaN maps to the lowest    */
/* code (fmaxf drops the NaN operand).  Codes are returned as int32.          */
/* ------------------------------------------------------------------------- */
int orc_quantize(const float* x, int64_t outer, int64_t axis_len, int64_t inner,
                 const orc_qparams* p, int32_t qmin, int32_t qmax, int32_t* q)
{
    if (outer <= 0 || axis_len <= 0 || inner <= 0 || qmin > qmax) return ORC_ERR_INVALID;
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t a = 0; a < axis_len; ++a) {
            const float delta = p[a].scale;
            const int32_t z = p[a].zero_point;
            const float tlo = (float)(qmin - z), thi = (float)(qmax - z);
            for (int64_t i = 0; i < inner; ++i) {
                int64_t idx = (o * axis_len + a) * inner + i;
                float t = x[idx] / delta;
                t = rintf(t);
                t = fminf(fmaxf(t, tlo), thi);
                q[idx] = (int32_t)t + z;
            }
        }
    return ORC_OK;
}

/* Eq. 3: x_float = (x_Q - z) * Delta, one fp32 multiply. */
int orc_dequantize(const int32_t* q, int64_t outer, int64_t axis_len, int64_t inner,
                   const orc_qparams* p, float* x)
{
    if (outer <= 0 || axis_len <= 0 || inner <= 0) return ORC_ERR_INVALID;
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t a = 0; a < axis_len; ++a)
            for (int64_t i = 0; i < inner; ++i) {
                int64_t idx = (o * axis_len + a) * inner + i;
                x[idx] = (float)(q[idx] - p[a].zero_point) * p[a].scale;
            }
    return ORC_OK;
}

/* 4-bit storage (Section 3.2.4 uses 4-bit weights; the paper gives no layout). */
/* Reading: two's-complement nibbles, element 2i in the low nibble of byte i,   */
/* element 2i+1 in the high nibble; an odd tail leaves the high nibble zero.    */
int orc_pack_s4(const int32_t* codes, int64_t rows, int64_t k, uint8_t* packed)
{
    int64_t kb = (k + 1) / 2;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < kb; ++j) {
            int32_t lo = codes[r * k + 2 * j];
            int32_t hi = (2 * j + 1 < k) ? codes[r * k + 2 * j + 1] : 0;
            if (lo < -8 || lo > 7 || hi < -8 || hi > 7) return ORC_ERR_INVALID;
            packed[r * kb + j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
        }
    return ORC_OK;
}

int orc_unpack_s4(const uint8_t* packed, int64_t rows, int64_t k, int32_t* codes)
{
    int64_t kb = (k + 1) / 2;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t i = 0; i < k; ++i) {
            uint8_t byte = packed[r * kb + i / 2];
            int32_t nib = (i & 1) ? (byte >> 4) : (byte & 0xF);
            codes[r * k + i] = nib >= 8 ? nib - 16 : nib;
        }
    return ORC_OK;
}
