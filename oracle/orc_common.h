/*
 * orc_common.h -- TEST INFRASTRUCTURE (see qtz_oracle.c).  Status codes and the
 * single requantisation step shared by the oracle's translation units.
 */
#ifndef ORC_COMMON_H
#define ORC_COMMON_H
#include <stdint.h>

#define ORC_OK 0
#define ORC_ERR_INVALID (-1)
#define ORC_ERR_NONFINITE (-2)
#define ORC_ERR_UNSUPPORTED (-3)
#define ORC_ERR_OVERFLOW (-4)

/* One requantisation: y = z_y + floor((acc m + 2^(r-1)) / 2^r), clamped.     */
/* A single rounding, ties toward +infinity.  (The rescale by                 */
/* Delta_w Delta_x / Delta_y is implied by Eq. 4; its fixed-point form is a   */
/* definition of this code base.)                                             */
static inline int32_t orc_requant1(int64_t acc, int32_t m, int32_t r, int32_t zy,
                                   int32_t act_min, int32_t act_max)
{
    int64_t v = acc * (int64_t)m;
    int64_t y = (int64_t)zy + ((v + ((int64_t)1 << (r - 1))) >> r);
    if (y < act_min) y = act_min;
    if (y > act_max) y = act_max;
    return (int32_t)y;
}
#endif
