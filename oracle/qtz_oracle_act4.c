/*
 * qtz_oracle_act4.c -- TEST INFRASTRUCTURE, not a product path (see qtz_oracle.c).
 *
 * Activations at fewer than 8 bits (Section 3.2.4 / Table 6 evaluates 4-bit activations;
 * Section 7 asks hardware for 4, 8 and 16 bit support).  The quantizer itself is Eq. 1-3 with
 * N_levels = 2^bits (orc_affine_params / orc_quantize already take the bit width); what is
 * added here is the storage of 4-bit unsigned codes and the clamp of a fused activation for
 * any width.
 */
#include <math.h>
#include <stdint.h>

#include "orc_common.h"

/* Unsigned 4-bit codes 0..15 of an activation tensor [rows][k], two per byte along k.   */
/* The paper gives no layout; reading taken (the one used for 4-bit weights): element 2i  */
/* in the low nibble of byte i, element 2i+1 in the high nibble, an odd tail leaves the    */
/* high nibble zero.  Rows of the packed tensor are pitch bytes apart.                     */
int orc_pack_u4(const uint8_t* codes, int64_t rows, int64_t k, int64_t code_pitch, uint8_t* packed,
                int64_t packed_pitch)
{
    if (rows <= 0 || k <= 0 || code_pitch < k || packed_pitch < (k + 1) / 2) return ORC_ERR_INVALID;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < (k + 1) / 2; ++j) {
            uint8_t lo = codes[r * code_pitch + 2 * j];
            uint8_t hi = (2 * j + 1 < k) ? codes[r * code_pitch + 2 * j + 1] : 0;
            if (lo > 15 || hi > 15) return ORC_ERR_INVALID;
            packed[r * packed_pitch + j] = (uint8_t)(lo | (hi << 4));
        }
    return ORC_OK;
}

int orc_unpack_u4(const uint8_t* packed, int64_t rows, int64_t k, int64_t packed_pitch, uint8_t* codes,
                  int64_t code_pitch)
{
    if (rows <= 0 || k <= 0 || code_pitch < k || packed_pitch < (k + 1) / 2) return ORC_ERR_INVALID;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t i = 0; i < k; ++i) {
            uint8_t byte = packed[r * packed_pitch + i / 2];
            codes[r * code_pitch + i] = (i & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 0xF);
        }
    return ORC_OK;
}

/* Clamp range of a fused activation when the output has `bits` bits (Section 3.2.1 with   */
/* L = 2^bits - 1 as the top code): none [0,L]; ReLU [z,L]; ReLU6 [z, min(L, z + round(6/Delta))]. */
int orc_activation_range_bits(int kind, float y_scale, int32_t y_zero_point, int bits,
                              int32_t* act_min, int32_t* act_max)
{
    if (bits < 2 || bits > 8 || kind < 0 || kind > 2) return ORC_ERR_INVALID;
    const int32_t L = (1 << bits) - 1;
    *act_min = kind == 0 ? 0 : y_zero_point;
    *act_max = L;
    if (kind == 2) {
        double top = (double)y_zero_point + rint(6.0 / (double)y_scale);
        if (top < (double)L) *act_max = (int32_t)top;
    }
    return ORC_OK;
}
