/*
 * qtz.h -- C ABI of libqtz: integer-only inference of quantized convolution layers
 * under uniform affine quantization, for NVIDIA B200 (sm_100a).
 *
 * The operations follow R. Krishnamoorthi, "Quantizing deep convolutional networks
 * for efficient inference: A whitepaper" (2018); every entry point names the section
 * or equation that defines what it computes.
 *
 * Conventions
 *  - Every call returns a qtz_status: 0 on success, a negative code otherwise.  Nothing
 *    throws or aborts.  After QTZ_ERR_CUDA, qtz_last_error() describes the CUDA failure.
 *  - Pointers named *_dev are device pointers on the handle's device, *_host are host
 *    pointers.  The caller owns every buffer it passes.  The library owns only what
 *    qtz_create / qtz_conv_create return, until the matching destroy call.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *    enqueued on it and the call returns without waiting, except where stated.
 *  - Calls that share one handle or one plan must be issued in stream order on ONE stream
 *    at a time: the handle and the plans hold small device scratch buffers that
 *    consecutive calls reuse.
 *  - Activations are uint8, NHWC, with a channel pitch: pixel p, channel c lives at
 *    base[p * c_pitch + c].  Pitches are multiples of 16 and base pointers 16-byte
 *    aligned (else QTZ_ERR_MISALIGNED).  Bytes in [c, c_pitch) are never read as data;
 *    outputs leave them unspecified.  One exception: the INPUT of an image stem (a k x k
 *    convolution, k > 1, over at most 8 channels with kh*kw*c <= 1024) may have a pitch of 4 or
 *    8 bytes, so that a 3-channel image need not be stored at 16 bytes per pixel.
 *  - Tensors handed to calibrate / quantize / dequantize are viewed as
 *    x[outer][axis_len][inner] (row-major); one quantizer per index of the middle axis.
 *    axis_len == 1 is per-layer quantization (Section 2.6).
 */
#ifndef QTZ_H
#define QTZ_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define QTZ_API __attribute__((visibility("default")))
#else
#define QTZ_API
#endif

typedef int32_t qtz_status;
#define QTZ_OK 0
#define QTZ_ERR_INVALID_ARG (-1)    /* null pointer, non-positive size, bad enum            */
#define QTZ_ERR_MISALIGNED (-2)     /* pointer or pitch misaligned (16 bytes unless a call says otherwise) */
#define QTZ_ERR_UNSUPPORTED (-3)    /* well-formed request outside what is implemented      */
#define QTZ_ERR_OVERFLOW (-4)       /* reduction length too large for int32 accumulation    */
#define QTZ_ERR_NONFINITE (-5)      /* NaN or Inf met while calibrating                     */
#define QTZ_ERR_CUDA (-6)           /* a CUDA runtime/driver call failed                    */
#define QTZ_ERR_DEVICE_TIMEOUT (-7) /* a bounded device-side wait gave up                   */
#define QTZ_ERR_NO_DEVICE (-8)      /* no usable CUDA device                                */
#define QTZ_ERR_TOO_LARGE (-9)      /* size beyond the fixed capacity of a non-allocating call */

typedef struct qtz_ctx* qtz_handle;     /* library-owned, opaque */
typedef struct qtz_plan* qtz_conv_plan; /* library-owned: prepacked weights and tables */

/* Scale, zero point and the nudged real range of one quantizer (Section 2.1). */
typedef struct {
    float scale;        /* Delta */
    int32_t zero_point; /* z, an integer so that real 0.0 is exactly a code */
    float min_nudged;   /* real value of the lowest code,  (0 - z) * Delta  */
    float max_nudged;   /* real value of the highest code, (L - z) * Delta  */
} qtz_qparams;

typedef enum {
    QTZ_U8 = 0, QTZ_S8 = 1, QTZ_S4_PACKED = 2, QTZ_S32 = 3, QTZ_U4_PACKED = 4,
    QTZ_U16 = 5, QTZ_S16 = 6   /* 16-bit codes (Section 7: 4, 8 and 16 bits), stored as uint16_t / int16_t */
} qtz_dtype;

typedef enum {
    QTZ_W_S8_PER_CHANNEL_SYM = 0,       /* int8 codes, one scale per output channel, z_w = 0 */
    QTZ_W_U8_PER_LAYER_ASYM = 1,        /* uint8 codes, one (scale, z_w) for the layer       */
    QTZ_W_S4_PACKED_PER_CHANNEL_SYM = 2 /* 4-bit codes in [-8,7], two per byte, z_w = 0      */
} qtz_wkind;

typedef enum { QTZ_OUT_U8 = 0, QTZ_OUT_S32_RAW = 1 } qtz_outkind;

/* Geometry of one convolution.  Input NHWC [batch][h][w][c] with pitch c_pitch_in; output
 * [batch][oh][ow][n] with pitch c_pitch_out, oh = (h + 2 pad - kh)/stride + 1 (same for ow).
 * For a depthwise plan n must equal c.  With QTZ_OUT_S32_RAW the output is a dense int32
 * array [batch*oh*ow][n] and c_pitch_out is ignored.                                       */
typedef struct {
    int32_t batch, h, w, c, c_pitch_in;
    int32_t n, c_pitch_out;
    int32_t kh, kw, stride, pad;
    int32_t wkind;   /* qtz_wkind   */
    int32_t outkind; /* qtz_outkind */
} qtz_conv_desc;

/* ---- library ------------------------------------------------------------------------- */

/* Creates a handle bound to CUDA device `device` (allocates a few MB of device scratch).
 * Blocking.  QTZ_ERR_NO_DEVICE when the device cannot be used.
 * Two environment variables, read here, switch scheduling choices off for A/B timing (results are the
 * same either way): QTZ_NO_PAIRS=1 keeps large GEMM-like layers on single CTAs instead of CTA pairs;
 * QTZ_SINGLE_ROW_STEMS=1 keeps image stems at one output row per tile.                      */
QTZ_API qtz_status qtz_create(qtz_handle* out, int device);
QTZ_API qtz_status qtz_destroy(qtz_handle h);
QTZ_API const char* qtz_status_string(qtz_status s);
/* Text of the last CUDA error seen through this handle ("" if none).  Host only.          */
QTZ_API const char* qtz_last_error(qtz_handle h);
/* Status word written by device code whose bounded waits gave up: 0, or
 * QTZ_ERR_DEVICE_TIMEOUT with *site_id telling which wait.  Synchronises `stream`.        */
QTZ_API qtz_status qtz_last_device_status(qtz_handle h, int32_t* site_id, void* stream);

/* Cycle budget of every bounded device-side wait of later launches through this handle (default
 * 2e9, about one second of SM clocks; at least 1000).  When a wait runs out the kernel records
 * QTZ_ERR_DEVICE_TIMEOUT and returns; qtz_last_device_status reports it.                        */
QTZ_API qtz_status qtz_set_wait_budget(qtz_handle h, int64_t cycles);
/* Self-test of that mechanism: launches one small CTA that waits, for at most budget_cycles
 * (1 .. 1e8), on a barrier nothing ever signals.  The wait gives up by itself and the kernel
 * returns normally; afterwards qtz_last_device_status reports QTZ_ERR_DEVICE_TIMEOUT with site
 * id 8.  Asynchronous on `stream`.  Nothing faults, traps or hangs.                             */
QTZ_API qtz_status qtz_selftest_wait_timeout(qtz_handle h, int64_t budget_cycles, void* stream);
/* Measures the tensor cores alone for the contraction of Eq. 5 (first term): one CTA per SM issues
 * mmas_per_cta (>= 32, rounded down to a multiple of 32) tcgen05.mma kind::i8 instructions of
 * 128 x 256 x 32 (u8 x s8 -> s32) on operands that stay in shared memory, `launches` times back
 * to back.  Writes the achieved TOP/s (2 ops per multiply-accumulate) and, if ms_out is not NULL,
 * the elapsed milliseconds of the timed launches (CUDA events on `stream`).  BLOCKS.             */
QTZ_API qtz_status qtz_probe_int8_peak(qtz_handle h, int32_t mmas_per_cta, int32_t launches, double* tops_out,
                                       float* ms_out, void* stream);

/* Measures the CUDA cores' rate for the integer arithmetic of an output code, on register operands:
 * kind 0 three dp4a (the nine taps of a depthwise output); kind 1 one requantisation (32x32->64
 * multiply-add, shift of the high word, clamp: the y of Eq. 4's rescale); kind 2 both.  Writes outputs
 * per clock and SM (at the device's maximum SM clock) and, if not NULL, outputs per second.  BLOCKS. */
QTZ_API qtz_status qtz_probe_requant_rate(qtz_handle h, int32_t kind, double* outputs_per_clock_sm,
                                          double* outputs_per_second, void* stream);

/* ---- quantizer parameters (Sections 2.1, 2.2, 2.5, 2.6) ------------------------------- */

/* Range estimation by min/max (Section 2.5) followed by parameter derivation.
 * Affine (symmetric == 0, Section 2.1): the range is first relaxed to contain 0, then
 *   Delta = (max - min)/(2^bits - 1), z = round(-min/Delta) clamped to [0, 2^bits - 1], and
 *   the representable range is nudged to [(0-z)Delta, (2^bits-1-z)Delta].
 * Symmetric (Section 2.2): z = 0, Delta = max|x| / (2^(bits-1) - 1).
 * A tensor (or channel) that is all zero gets Delta = 1, z = 0.
 * Reads x_dev (fp32, device, outer*axis_len*inner values), writes axis_len entries to
 * out_host.  BLOCKS until `stream` has finished.  bits in [2,16].
 * Errors: QTZ_ERR_NONFINITE if any value is NaN/Inf (out_host is then unspecified).       */
QTZ_API qtz_status qtz_calibrate_minmax(qtz_handle h, const float* x_dev, int64_t outer,
                                int64_t axis_len, int64_t inner, int32_t bits,
                                int32_t symmetric, qtz_qparams* out_host, void* stream);

/* The range reduction alone (Section 2.5): min and max of each axis slice, written to
 * lo_host / hi_host (axis_len floats each).  BLOCKS until `stream` has finished.
 * QTZ_ERR_NONFINITE as above.  Lets a caller post-process a range (for instance clamp it to
 * [0,6] for a layer followed by ReLU6) before deriving parameters from it.                */
QTZ_API qtz_status qtz_minmax(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len,
                              int64_t inner, float* lo_host, float* hi_host, void* stream);

/* The per-layer range reduction for callers that must not allocate device memory -- for
 * instance a server that handed all of the GPU's memory to its own pool when it started, or a
 * latency-critical loop that cannot afford the device-wide synchronisation cudaMalloc/cudaFree
 * may bring.  (The paper has no counterpart to this call: it is a property of this library,
 * not of the method.  What it computes is the min/max of Section 2.5, exactly as qtz_minmax.)
 *   x_dev    `count` fp32 values on the CURRENT device (no handle is involved)
 *   out_dev  3 x 4 bytes on the device, written by the call: float lo, float hi, and a 32-bit
 *            word that is non-zero when a NaN or Inf was met (lo/hi are then unspecified)
 * Asynchronous on `stream`; nothing is copied to the host.
 * The block partials live in a fixed 48 KB array inside the library image, which every GPU that
 * loads the library keeps until the process exits.  Consequences:
 *   - count may not exceed qtz_minmax_static_max_count() (2^28 values); larger tensors are
 *     refused with QTZ_ERR_TOO_LARGE and nothing is launched;
 *   - all calls on a device share that array (it keeps the previous call's partials; none of
 *     them is read before the current call has rewritten it, so nothing needs clearing), and
 *     two calls whose kernels may overlap on the GPU -- different streams -- race on it: issue
 *     them in order on one stream, or synchronise in between;
 *   - the first call on each device looks the array's device address up
 *     (cudaGetSymbolAddress) and makes the CUDA runtime load this library's kernels and the
 *     array onto that device, which takes a little device memory once: make one small warm-up
 *     call per device early -- before a memory pool claims the rest of the GPU, and before
 *     starting any stream capture.  If that first call fails for lack of memory it returns
 *     QTZ_ERR_CUDA (there is no handle to ask for the error text).
 * x_dev and out_dev must be 4-byte aligned (QTZ_ERR_MISALIGNED otherwise; no 16-byte rule here).
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine.         */
QTZ_API qtz_status qtz_minmax_static(const float* x_dev, int64_t count, float* out_dev, void* stream);
QTZ_API int64_t qtz_minmax_static_max_count(void);

/* Streaming range estimation for activations (Section 2.5: "a moving average of the minimum and
 * maximum values across batches"; Section 3.1.2 calibrates on about 100 mini-batches).  The running
 * state lives on the device, so a calibration loop enqueues one call per batch and tensor and never
 * waits; one blocking read at the end turns the state into parameters.
 *   state_dev   qtz_range_state_bytes(axis_len) bytes of device memory, 8-byte aligned, owned by the
 *               caller; qtz_range_reset (or zero filling) starts a new average.
 *   accumulate  min/max of this batch per index of the middle axis (the view of
 *               qtz_calibrate_minmax), then state <- decay * state + (1 - decay) * batch in fp64
 *               (0 <= decay < 1; the first batch initialises the state) -- the arithmetic of
 *               qtz_ema_update, bit for bit.  A batch that holds NaN or Inf is skipped as a whole and
 *               remembered.  Asynchronous on `stream`.
 *   finish      BLOCKS once: copies the state to the host and writes, per axis index, the averaged
 *               range rounded to fp32 (lo_host / hi_host, may be NULL) and the parameters derived from
 *               it by the rules of qtz_params_from_range (params_host, may be NULL); *batches_host
 *               (may be NULL) receives the number of batches folded in.  QTZ_ERR_NONFINITE if a batch
 *               was skipped, QTZ_ERR_INVALID_ARG if nothing was accumulated.
 * Calls that share a handle share its scratch: keep them on one stream.                          */
QTZ_API int64_t qtz_range_state_bytes(int64_t axis_len);
QTZ_API qtz_status qtz_range_reset(qtz_handle h, void* state_dev, int64_t axis_len, void* stream);
QTZ_API qtz_status qtz_range_accumulate(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len,
                                        int64_t inner, double decay, void* state_dev, void* stream);
QTZ_API qtz_status qtz_range_finish(qtz_handle h, const void* state_dev, int64_t axis_len, int32_t bits,
                                    int32_t symmetric, float* lo_host, float* hi_host, qtz_qparams* params_host,
                                    int32_t* batches_host, void* stream);

/* Host-only: parameters from a known real range (same rules as above).                    */
QTZ_API qtz_status qtz_params_from_range(float lo, float hi, int32_t bits, int32_t symmetric,
                                 qtz_qparams* out_host);

/* ---- quantize / dequantize (Eq. 1-3, 7-11) --------------------------------------------- */

/* x_int = round(x / Delta) + z, clamped to the code range (Eq. 1-2; Eq. 7-11 with z = 0).
 * The quotient is one IEEE fp32 division and round() is round-half-to-even.  Code ranges:
 *   QTZ_U8 [0,255] (restrict_range: [0,254]); QTZ_S8 [-128,127] (restrict_range, Eq. 10:
 *   [-127,127]); QTZ_S4_PACKED [-8,7] (restrict_range: [-7,7]); QTZ_U4_PACKED [0,15]
 *   (restrict_range: [0,14]) -- 4-bit activations, Section 3.2.4; QTZ_U16 [0,65535] (restrict_range:
 *   [0,65534]) and QTZ_S16 [-32768,32767] (restrict_range: [-32767,32767]) -- the 16-bit precision of
 *   Section 7, two bytes per code, q_dev 2-byte aligned.  (fp32 holds every 16-bit code exactly; the
 *   quotient x / Delta is then good to 2^-8 of a step, so a value within that distance of a tie may
 *   round either way against exact arithmetic, never against these fp32 steps.)
 * NaN maps to the lowest code, +-Inf saturate.
 * params_host: axis_len entries, read before the call returns.
 * QTZ_S4_PACKED / QTZ_U4_PACKED: nibbles (two's complement / unsigned) packed along the innermost run of the view
 * (`inner`, or `axis_len` when inner == 1): element 2i in the low nibble and 2i+1 in the
 * high nibble of byte i; each run occupies (len+1)/2 bytes, an odd tail's high nibble is 0. */
QTZ_API qtz_status qtz_quantize_tensor(qtz_handle h, const float* x_dev, int64_t outer,
                               int64_t axis_len, int64_t inner, const qtz_qparams* params_host,
                               int32_t out_dtype, int32_t restrict_range, void* q_dev,
                               void* stream);

/* x = (q - z) * Delta with one fp32 multiply (Eq. 3; z = 0 for the symmetric quantizer).
 * in_dtype QTZ_S32 dequantizes int32 accumulators: zero_point must be 0 and `scale` holds
 * the product Delta_x * Delta_w[n] of Eq. 4.                                                */
QTZ_API qtz_status qtz_dequantize(qtz_handle h, const void* q_dev, int32_t in_dtype, int64_t outer,
                          int64_t axis_len, int64_t inner, const qtz_qparams* params_host,
                          float* x_dev, void* stream);

/* ---- simulated quantization, SQNR, range averaging, rescale ------------------------------ */

/* SimQuant (Section 2.4): a quantizer followed by a de-quantizer,
 *   y = (clamp(round(x / Delta) + z, qmin, qmax) - z) * Delta
 * with exactly the fp32 steps of qtz_quantize_tensor and qtz_dequantize (the paper prints the
 * formula with the sign of z flipped; this is Eq. 3 applied to Eq. 1-2).  fp32 in, fp32 out,
 * same view and parameter conventions; code_dtype (any qtz_dtype but QTZ_S32) and
 * restrict_range only select the code range [qmin, qmax].  y_dev may alias x_dev.           */
QTZ_API qtz_status qtz_simquant(qtz_handle h, const float* x_dev, int64_t outer, int64_t axis_len,
                                int64_t inner, const qtz_qparams* params_host, int32_t code_dtype,
                                int32_t restrict_range, float* y_dev, void* stream);

/* Signal-to-quantization-noise ratio (Appendix A),
 *   SQNR = 10 log10( sum w^2 / sum (w - w_hat)^2 )   in dB,
 * one value per index of the middle axis (per output feature map), or of the whole tensor with
 * axis_len == 1.  Sums are accumulated in fp64; no noise at all gives +infinity.  Writes axis_len
 * doubles to sqnr_db_host and BLOCKS until `stream` has finished.  axis_len <= 65535.        */
QTZ_API qtz_status qtz_sqnr(qtz_handle h, const float* w_dev, const float* w_hat_dev, int64_t outer,
                            int64_t axis_len, int64_t inner, double* sqnr_db_host, void* stream);

/* Host-only: the moving average of per-batch ranges that Section 2.5 prescribes for
 * activations.  The paper names no weighting; this is the exponential average
 *   state <- decay * state + (1 - decay) * batch      (0 <= decay < 1, fp64)
 * applied to n (lo, hi) pairs, e.g. the output of qtz_minmax.  While *initialised is 0 the batch
 * values are copied instead and the flag is set.  Feed (float)state to qtz_params_from_range.
 * Errors: QTZ_ERR_NONFINITE if a batch value is NaN/Inf (the state is then untouched).        */
QTZ_API qtz_status qtz_ema_update(double* state_lo_host, double* state_hi_host, const float* batch_lo_host,
                                  const float* batch_hi_host, int64_t n, double decay, int32_t* initialised);

/* A uint8 tensor re-expressed in another quantizer -- what the inputs of a concatenation need
 * so that they share the output's scale and zero point (Section 3.2.1):
 *   y = clamp(y_zp + floor(((x - x_zp) mult + 2^(rshift-1)) / 2^rshift), act_min, act_max)
 * with (mult, rshift) = qtz_quantize_multiplier(Delta_x / Delta_y).  x is [pixels][c] with pitch
 * x_pitch, y likewise with y_pitch; to fill a channel slice of a concatenated tensor pass
 * y_dev = base + channel offset and the pitch of the whole.  Pointers and pitches need no
 * particular alignment (rows that are 4-byte aligned on both sides take a faster path).     */
QTZ_API qtz_status qtz_rescale_u8(qtz_handle h, const uint8_t* x_dev, int32_t x_zp, int32_t mult, int32_t rshift,
                                  uint8_t* y_dev, int32_t y_zp, int32_t act_min, int32_t act_max, int64_t pixels,
                                  int32_t c, int32_t x_pitch, int32_t y_pitch, void* stream);

/* ---- activations at fewer than 8 bits (Section 3.2.4, Table 6: 4-bit activations) --------------- */

/* A convolution takes its activations as one code per byte; 4-bit codes (0..15) go through it
 * unchanged, with act_max <= 15 as the clamp of a 4-bit output.  For storage they pack two per
 * byte: element 2i of a pixel's channels in the low nibble of byte i, element 2i+1 in the high
 * nibble, an odd tail leaves the high nibble zero.
 *   qtz_pack_u4    x [pixels][c] one code per byte, pitch x_pitch -> y [pixels][(c+1)/2], pitch y_pitch;
 *                  only the low four bits of a code are kept.
 *   qtz_unpack_u4  the reverse; bytes of y beyond c in a pixel are left untouched.
 * No alignment rules (rows that are 4-byte aligned on both sides take a faster path).           */
QTZ_API qtz_status qtz_pack_u4(qtz_handle h, const uint8_t* x_dev, int64_t pixels, int32_t c, int32_t x_pitch,
                               uint8_t* y_dev, int32_t y_pitch, void* stream);
QTZ_API qtz_status qtz_unpack_u4(qtz_handle h, const uint8_t* x_dev, int64_t pixels, int32_t c, int32_t x_pitch,
                                 uint8_t* y_dev, int32_t y_pitch, void* stream);
/* qtz_activation_range for an output of `bits` bits (2..8): the top code is 2^bits - 1.          */
QTZ_API qtz_status qtz_activation_range_bits(int32_t kind, float y_scale, int32_t y_zero_point, int32_t bits,
                                             int32_t* act_min, int32_t* act_max);

/* ---- batch-norm folding (Eq. 20-21) ------------------------------------------------------ */

/* W_inf[n][:] = gamma[n] W[n][:] / sigma[n],  Bias_inf[n] = beta[n] + gamma[n] (b[n] - mu[n]) /
 * sigma[n], with sigma = sqrt(var + eps) and b = conv_bias (NULL means 0).  W is [n][k]
 * (OHWI flattened), arithmetic in fp64 rounded once to fp32.  w_inf_dev may alias w_dev.     */
QTZ_API qtz_status qtz_fold_batchnorm(qtz_handle h, const float* w_dev, const float* conv_bias_dev,
                              const float* gamma_dev, const float* beta_dev,
                              const float* mean_dev, const float* var_dev, float eps, int64_t n,
                              int64_t k, float* w_inf_dev, float* bias_inf_dev, void* stream);

/* bias_q[n] = sat_int32(round(bias[n] / (Delta_x * Delta_w[n]))): the bias in the scale of the
 * accumulator of Eq. 4, zero point 0.  w_params_host has n entries (or 1 if per_layer != 0).  */
QTZ_API qtz_status qtz_quantize_bias(qtz_handle h, const float* bias_dev, int64_t n, float x_scale,
                             const qtz_qparams* w_params_host, int32_t per_layer,
                             int32_t* bias_q_dev, void* stream);

/* ---- fixed-point rescale helpers (host only; implied by Eq. 4, defined by this library) ---- */

/* Real multiplier M >= 0 as m * 2^-rshift with 2^30 <= m < 2^31 and 1 <= rshift <= 62
 * (M = 0 gives m = 0, rshift = 1).  QTZ_ERR_UNSUPPORTED when M is too large or too small.      */
QTZ_API qtz_status qtz_quantize_multiplier(double real_multiplier, int32_t* mult, int32_t* rshift);
/* Clamp range of a fused activation in the quantized domain (Section 3.2.1: the activation
 * fuses into the producing op).  kind 0 none [0,255]; 1 ReLU [z_y,255];
 * 2 ReLU6 [z_y, min(255, z_y + round(6/Delta_y))].                                            */
QTZ_API qtz_status qtz_activation_range(int32_t kind, float y_scale, int32_t y_zero_point,
                                int32_t* act_min, int32_t* act_max);
/* Multipliers of the element-wise add (Section 3.2.1): the larger of Delta_a/Delta_y and
 * Delta_b/Delta_y fixes rshift through qtz_quantize_multiplier, the other is round(M 2^rshift). */
QTZ_API qtz_status qtz_add_params(float a_scale, float b_scale, float y_scale, int32_t* a_mult,
                          int32_t* b_mult, int32_t* rshift);

/* ---- range rules between the layers of a network (host only; Sections 2.5, 3.1.2, 3.2.1) ---- */

/* Range of a layer's output tensor from the min/max of its pre-activation values on calibration
 * data (Section 2.5: activations take the min/max seen on a batch) and the activation fused into
 * the layer (Section 3.2.1).  The quantized tensor is the one after the activation, and ReLU /
 * ReLU6 are monotone, so each end of the range goes through the activation: kind 0 [lo,hi];
 * 1 [max(lo,0), max(hi,0)]; 2 both ends also capped at 6.  Feed the result to
 * qtz_params_from_range.  QTZ_ERR_NONFINITE for NaN/Inf, QTZ_ERR_INVALID_ARG for hi < lo.       */
QTZ_API qtz_status qtz_range_after_activation(float lo, float hi, int32_t kind, float* lo_out, float* hi_out);
/* Range of an element-wise sum of two quantized tensors (Section 3.2.1): the interval sum of the
 * inputs' representable ranges (min_nudged + min_nudged, max_nudged + max_nudged, one fp32 add
 * each) -- a bound that needs no pass over data and cannot saturate -- followed by the fused
 * activation as in qtz_range_after_activation.                                                   */
QTZ_API qtz_status qtz_add_output_range(const qtz_qparams* a_host, const qtz_qparams* b_host, int32_t kind,
                                        float* lo_out, float* hi_out);
/* Scale of Eq. 4's accumulator per output channel: acc_params[i].scale = x_scale * w_params[i].scale
 * (one fp32 product), zero point 0 -- the parameters qtz_dequantize needs for QTZ_S32 input.     */
QTZ_API qtz_status qtz_accumulator_scales(float x_scale, const qtz_qparams* w_params_host, int64_t n,
                                          qtz_qparams* acc_params_host);
/* Fixed-point form of Delta_x Delta_w[i] / Delta_y (the rescale Eq. 4 implies) for n output
 * channels: the quotient is formed in fp64 and handed to qtz_quantize_multiplier.                 */
QTZ_API qtz_status qtz_requant_multipliers(float x_scale, const qtz_qparams* w_params_host, int64_t n, float y_scale,
                                           int32_t* mult_host, int32_t* rshift_host);
/* Fixed-point form of Delta_x / (hw Delta_y) for qtz_global_avgpool_u8 (exactly 1 / hw when the
 * two scales are equal).                                                                          */
QTZ_API qtz_status qtz_avgpool_multiplier(int32_t hw, float x_scale, float y_scale, int32_t* mult, int32_t* rshift);

/* ---- convolution (Eq. 4-6) -------------------------------------------------------------- */

/* One-time preparation of a layer ("the weights are constant at inference", Section 2.1):
 * copies and re-lays the weights for the kernels, and precomputes per output channel the
 * weight sums of the zero-point cross term of Eq. 5-6 (for padded 3x3 layers one sum per
 * border class, so that padding behaves as real zero, i.e. the code z_x).
 *   w_q_dev     OHWI codes [n][kh][kw][c] (depthwise: [kh][kw][c]); int8, uint8, or 4-bit
 *               packed along the flattened kh*kw*c run of each output channel (depthwise:
 *               along c), per desc->wkind.
 *   bias_q_dev  n int32 (scale Delta_x Delta_w[n]); NULL means no bias.
 *   w_zero_point_host  NULL, or 1 value (per-layer asymmetric weights).
 *   mult_host, rshift_host  n entries: fixed-point form of Delta_x Delta_w[n] / Delta_y
 *               (ignored, may be NULL, with QTZ_OUT_S32_RAW).
 * The caller may free or overwrite all inputs once `stream` has passed this call.
 * Errors: QTZ_ERR_OVERFLOW when kh*kw*c > 32768, or when kh*kw*c * 255 * max|w| + |bias_q[n]| (the
 * largest accumulator any input can produce) does not fit int32; QTZ_ERR_UNSUPPORTED for
 * depthwise layers other than 3x3 / pad 1 / stride 1 or 2.                                      */
QTZ_API qtz_status qtz_conv_create(qtz_handle h, const qtz_conv_desc* desc, int32_t depthwise,
                           const void* w_q_dev, const int32_t* bias_q_dev,
                           const int32_t* w_zero_point_host, const int32_t* mult_host,
                           const int32_t* rshift_host, qtz_conv_plan* out, void* stream);
QTZ_API qtz_status qtz_conv_destroy(qtz_conv_plan p);
/* Profiling hook: when both events (cudaEvent_t as void*) are non-NULL, every later
 * qtz_conv2d_u8 / qtz_depthwise_u8 call on this plan records them on the launch stream
 * immediately before and after its main kernel (pre-passes excluded, except the activation-sum
 * pre-pass of asymmetric-weight layers, beside which the main kernel runs).  NULL, NULL clears. */
QTZ_API qtz_status qtz_conv_set_profile_events(qtz_conv_plan p, void* start_event, void* stop_event);
/* Name of the kernel family a plan dispatches to ("tcgen05", "direct", "depthwise").           */
QTZ_API const char* qtz_conv_plan_kernel(qtz_conv_plan p);
/* How the plan's most recent launch ran, as text: the family, the layer form and where the weights
 * lived ("tcgen05 pointwise weights:int4-expanded-in-smem": packed 4-bit codes read from global
 * memory and expanded to int8 in shared memory -- the on-the-fly decompression Section 7 asks
 * hardware for; "weights:resident" / "weights:streamed": int8 codes).  Valid until the next launch
 * or destroy; before the first launch it is the family name.                                      */
QTZ_API const char* qtz_conv_plan_detail(qtz_conv_plan p);

/* Quantized convolution, evaluated through the expansion of Eq. 5-6:
 *   acc = conv(w_Q, x_Q) - z_w sum(x_Q) - z_x sum(w_Q) + K_valid z_x z_w + bias_q
 * which equals Eq. 4's conv(w_Q - z_w, x_Q - z_x) exactly; sums run over in-image taps and
 * K_valid counts them.  Then y = clamp(z_y + ((acc * mult[n] + 2^(rshift[n]-1)) >> rshift[n]),
 * act_min, act_max), 0 <= act_min <= act_max <= 255 (the fused ReLU/ReLU6 clamp).  With
 * QTZ_OUT_S32_RAW y_dev receives acc as int32 and y_zero_point / act_* are ignored.
 * x_dev / y_dev follow the plan's geometry; they must not overlap.                             */
QTZ_API qtz_status qtz_conv2d_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point,
                         void* y_dev, int32_t y_zero_point, int32_t act_min, int32_t act_max,
                         void* stream);
/* Convolution with the element-wise add that follows it fused into the epilogue (Section 3.2.1: "the
 * addition and the activation fuse"; Section 7 recommends aggressive operator fusion).  Computes exactly
 * what qtz_conv2d_u8 followed by qtz_add_u8 computes, without ever storing the intermediate tensor:
 *   t = clamp(t_zero_point + ((acc mult[n] + 2^(rshift[n]-1)) >> rshift[n]), t_act_min, t_act_max)
 *   y = clamp(z_y + (((t - t_zero_point) t_mult + (s - s_zero_point) s_mult + 2^(r-1)) >> r), act_min, act_max)
 * where acc is the accumulator of qtz_conv2d_u8, (t_zero_point, t_act_min, t_act_max) the quantizer and
 * clamp of the convolution's own output, s_dev the other addend (uint8, the geometry and pitch of the
 * output; it may be y_dev itself), and (t_mult, s_mult, r = rshift) come from qtz_add_params.
 * Both roundings of the two-step definition are kept, so results equal the unfused pair bit for bit.
 * Errors: QTZ_ERR_UNSUPPORTED when the plan does not run on the tensor-core path or its output kind is
 * not QTZ_OUT_U8 (run the two calls separately then), or when rshift > 53.                          */
typedef struct {
    int32_t t_zero_point, t_act_min, t_act_max; /* quantizer of the convolution's own output t        */
    int32_t t_mult;                             /* multiplier of (t - t_zero_point) in the add        */
    int32_t s_zero_point, s_mult;               /* zero point and multiplier of the other addend      */
    int32_t rshift;                             /* right shift of the add                             */
} qtz_residual;
QTZ_API qtz_status qtz_conv2d_add_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point,
                                     const qtz_residual* r_host, const uint8_t* s_dev, void* y_dev,
                                     int32_t y_zero_point, int32_t act_min, int32_t act_max, void* stream);
/* A depthwise-separable block in one kernel (Section 7 recommends fusing operators): the 3x3 depthwise
 * plan `dw` followed by the pointwise plan `pw`, whose input is the depthwise output.  Computes exactly
 * what qtz_depthwise_u8 (output zero point mid_zero_point, clamp [mid_act_min, mid_act_max]) followed by
 * qtz_conv2d_u8 (input zero point mid_zero_point) computes, bit for bit; the intermediate tensor is
 * produced chunk of channels by chunk of channels in shared memory, as the activation operand of the
 * tensor cores, and never stored.  x_dev follows the geometry of `dw`, y_dev that of `pw`.
 * Errors: QTZ_ERR_INVALID_ARG when the plans do not chain (channels, batch, extent); QTZ_ERR_UNSUPPORTED
 * when this pair cannot run fused -- run the two calls separately then.  Fused are: symmetric int8
 * weights on both layers, depthwise stride 1 or 2 with right shifts 32..53, a stride-1 pointwise layer on
 * the tensor-core path with at most 256 output channels whose 8-bit weights fit in shared memory
 * (channels x outputs <= 80 KB).                                                                    */
QTZ_API qtz_status qtz_conv2d_dw_pw_u8(qtz_conv_plan dw, qtz_conv_plan pw, const uint8_t* x_dev, int32_t x_zero_point,
                                       int32_t mid_zero_point, int32_t mid_act_min, int32_t mid_act_max, void* y_dev,
                                       int32_t y_zero_point, int32_t act_min, int32_t act_max, void* stream);

/* Depthwise form of the same (depth multiplier 1; Section 3.1.3 networks): the sum runs over
 * the kh x kw taps of one channel.  Plan must have been created with depthwise != 0.           */
QTZ_API qtz_status qtz_depthwise_u8(qtz_conv_plan p, const uint8_t* x_dev, int32_t x_zero_point,
                            void* y_dev, int32_t y_zero_point, int32_t act_min, int32_t act_max,
                            void* stream);

/* ---- integer glue ops of a quantized network (Section 3.2.1) -------------------------------- */

/* Element-wise add with both inputs rescaled to the output scale, fused clamp:
 *   y = clamp(z_y + (((a - z_a) a_mult + (b - z_b) b_mult + 2^(rshift-1)) >> rshift)).
 * a, b, y: `pixels` rows of c channels with the same pitch.                                     */
QTZ_API qtz_status qtz_add_u8(qtz_handle h, const uint8_t* a_dev, int32_t a_zp, int32_t a_mult,
                      const uint8_t* b_dev, int32_t b_zp, int32_t b_mult, int32_t rshift,
                      uint8_t* y_dev, int32_t y_zp, int32_t act_min, int32_t act_max,
                      int64_t pixels, int32_t c, int32_t c_pitch, void* stream);
/* k x k max pooling on codes (the quantizer is monotone, so input and output share (Delta, z));
 * out-of-image taps are skipped.                                                                */
QTZ_API qtz_status qtz_maxpool_u8(qtz_handle h, const uint8_t* x_dev, uint8_t* y_dev, int32_t batch,
                          int32_t hh, int32_t ww, int32_t c, int32_t c_pitch, int32_t k,
                          int32_t stride, int32_t pad, void* stream);
/* Global average pool: S = sum_{h,w}(x - z_x); y = clamp(z_y + ((S mult + 2^(rshift-1)) >> rshift),
 * 0, 255) with (mult, rshift) the fixed-point form of Delta_x / (hw Delta_y).  y: [batch][c_pitch]. */
QTZ_API qtz_status qtz_global_avgpool_u8(qtz_handle h, const uint8_t* x_dev, int32_t x_zp, uint8_t* y_dev,
                                 int32_t y_zp, int32_t mult, int32_t rshift, int32_t batch,
                                 int32_t hw, int32_t c, int32_t c_pitch, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QTZ_H */
