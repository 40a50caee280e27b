// Tensor-core (tcgen05) convolution path -- placeholder until the kernel lands.
#include "qtz_plan.cuh"

bool qtz_tc_supported(const qtz_conv_desc&) { return false; }
qtz_status qtz_tc_prepare(qtz_plan*, const void*, cudaStream_t) { return QTZ_ERR_UNSUPPORTED; }
void qtz_tc_release(qtz_plan*) {}
qtz_status qtz_tc_launch(qtz_plan*, const uint8_t*, int32_t, void*, int32_t, int32_t, int32_t, cudaStream_t)
{
    return QTZ_ERR_UNSUPPORTED;
}
