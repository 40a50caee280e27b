/*
 * qtz_oracle_net.c -- TEST INFRASTRUCTURE, not a product path (see qtz_oracle.c).
 *
 * Range rules of post-training quantization for the tensors between the layers of a
 * network (Section 3.1.2: activation ranges come from calibration data; Section 2.5:
 * min/max of what was observed; Section 3.2.1: activations fuse into the producing op).
 * The paper states these in words only; each reading is written next to the code.
 */
#include <math.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#include "orc_common.h"

typedef struct {
    float scale;
    int32_t zero_point;
    float min_nudged;
    float max_nudged;
} orc_qparams_net;

/* Range of a layer's output tensor, given the min/max of its pre-activation values on   */
/* the calibration batch (Section 2.5) and the activation fused into the layer (Section  */
/* 3.2.1).  The tensor that is quantized is the one AFTER the activation, so its range   */
/* is the observed range pushed through the activation, which is monotone:               */
/*   none  -> [lo, hi];  ReLU -> [max(lo,0), max(hi,0)];  ReLU6 -> both ends also <= 6.   */
int orc_range_after_activation(float lo, float hi, int32_t kind, float* lo_out, float* hi_out)
{
    if (!isfinite(lo) || !isfinite(hi)) return ORC_ERR_NONFINITE;
    if (lo > hi || kind < 0 || kind > 2) return ORC_ERR_INVALID;
    if (kind >= 1) {
        if (lo < 0.0f) lo = 0.0f;
        if (hi < 0.0f) hi = 0.0f;
    }
    if (kind == 2) {
        if (lo > 6.0f) lo = 6.0f;
        if (hi > 6.0f) hi = 6.0f;
    }
    *lo_out = lo;
    *hi_out = hi;
    return ORC_OK;
}

/* Range of an element-wise sum a + b of two quantized tensors (Section 3.2.1; the paper */
/* would observe it on calibration data, Section 2.5).  Reading taken: the interval sum   */
/* of the inputs' representable (nudged) ranges, formed in fp32 -- a bound that needs no  */
/* extra pass over data and can never saturate -- then the fused activation as above.     */
int orc_add_output_range(const orc_qparams_net* a, const orc_qparams_net* b, int32_t kind,
                         float* lo_out, float* hi_out)
{
    const float lo = a->min_nudged + b->min_nudged;
    const float hi = a->max_nudged + b->max_nudged;
    return orc_range_after_activation(lo, hi, kind, lo_out, hi_out);
}

/* Number of threads the oracle's OpenMP loops use from now on (timing runs report a   */
/* one-thread figure beside the all-cores one).  Returns the value in force.            */
int orc_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}
