// Accumulators of the SIMT contraction kernels.
//
// bf16 operands: a plain fp32 accumulator, products added in k order.
// fp32 operands: runs of products are summed in fp32 (exact products, one rounding per fused multiply-add, on a
// partial sum that stays small) and the run sums are added into an unevaluated pair of floats (hi + lo) with the
// error-free two-sum, so the total carries about 48 bits whatever the number of terms.  The fp64 pipe, far narrower
// than the fp32 one on this part, is not used in the loop.
#pragma once

namespace relay {

struct PairSum {
    float hi = 0.0f, lo = 0.0f;
    __device__ __forceinline__ void add(float p)
    {
        const float s = hi + p;
        const float bp = s - hi;
        lo += (hi - (s - bp)) + (p - bp);
        hi = s;
    }
    __device__ __forceinline__ double value() const { return (double)hi + (double)lo; }
};

}  // namespace relay
