// Chooses between the tensor-core and the SIMT contraction kernels.
#include "gemm.h"

namespace relay {

relay_status_t launch_gemm(const GemmDesc &g, cudaStream_t st)
{
    if (gemm_tc_eligible(g)) return launch_gemm_tc(g, st);
    return launch_gemm_simt(g, st);
}

}  // namespace relay
