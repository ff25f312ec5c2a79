// Implicit-GEMM tensor-core conv2d kernels -- placeholder until the kernels land.
#include "conv.h"

namespace relay {

bool conv_tc_eligible(const ConvDims &) { return false; }
size_t conv_tc_fwd_workspace(const ConvDims &) { return 0; }
size_t conv_tc_grad_workspace(const ConvDims &) { return 0; }
relay_status_t launch_conv_fwd_tc(const ConvDims &, const void *, const void *, const void *, int32_t, int, void *, void *, cudaStream_t)
{
    return fail(RELAY_ERR_UNSUPPORTED, "tensor-core conv2d not built");
}
relay_status_t launch_conv_dx_tc(const ConvDims &, const void *, const void *, void *, void *, cudaStream_t)
{
    return fail(RELAY_ERR_UNSUPPORTED, "tensor-core conv2d not built");
}
relay_status_t launch_conv_dw_tc(const ConvDims &, const void *, const void *, void *, void *, cudaStream_t)
{
    return fail(RELAY_ERR_UNSUPPORTED, "tensor-core conv2d not built");
}

}  // namespace relay
