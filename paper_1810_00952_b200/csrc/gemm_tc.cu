// Tensor-core contraction kernel (tcgen05 + TMEM + TMA) -- placeholder until the kernel lands.
#include "gemm.h"

namespace relay {

bool gemm_tc_eligible(const GemmDesc &) { return false; }
relay_status_t launch_gemm_tc(const GemmDesc &, cudaStream_t) { return fail(RELAY_ERR_UNSUPPORTED, "tensor-core contraction not built"); }

}  // namespace relay
