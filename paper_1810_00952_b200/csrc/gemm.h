// One description for every contraction the groups need, so that the forward product, the
// input gradient and the weight gradient run without materialising a transpose:
//   C[m,n] = epilogue( sum_k A(m,k) * B(k,n) ),  A(m,k) = a[m*a_sm + k*a_sk],  B(k,n) = b[k*b_sk + n*b_sn]
// where exactly one stride of each operand is 1 (the other is its leading dimension).
#pragma once
#include "common.h"

namespace relay {

struct GemmDesc {
    int64_t M = 0, N = 0, K = 0;
    const void *a = nullptr; int64_t a_sm = 0, a_sk = 0;
    const void *b = nullptr; int64_t b_sk = 0, b_sn = 0;
    void *c = nullptr;       int64_t ldc = 0;      // C row-major, leading dimension ldc
    int32_t in_dtype = RELAY_F32;                   // dtype of A and B
    int32_t out_dtype = RELAY_F32;                  // dtype of C
    const void *bias = nullptr; int32_t bias_dtype = RELAY_F32;  // per column n, or nullptr
    int32_t act = RELAY_ACT_NONE;
    // > 0: the N columns are the pre-activations of an LSTM cell in four blocks of this many columns [ i | f | g | o ] and the
    // epilogue stores the activated gates (tanh for g, logistic for the others).  Only launch_gemm_tc2 implements it; the
    // caller checks gemm_tc_eligible && gemm_tc2_eligible first and calls it directly.
    int64_t gate_block = 0;
};

// Picks the tensor-core kernel when the description fits it, else the SIMT kernel (both on the
// GPU).  Enqueues on `st`.
relay_status_t launch_gemm(const GemmDesc &g, cudaStream_t st);

// the two tiers, callable directly
relay_status_t launch_gemm_simt(const GemmDesc &g, cudaStream_t st);
// fp32 problems large enough to give every SM a 128 x 64 tile (gemm_simt_big.cu); launch_gemm_simt picks it itself
bool gemm_simt_big_eligible(const GemmDesc &g);
relay_status_t launch_gemm_simt_big(const GemmDesc &g, cudaStream_t st);
bool gemm_tc_eligible(const GemmDesc &g);
relay_status_t launch_gemm_tc(const GemmDesc &g, cudaStream_t st);
// two-SM (cta_group::2) variant: 256 x 256 tiles computed by pairs of blocks
bool gemm_tc2_eligible(const GemmDesc &g, int sms);
relay_status_t launch_gemm_tc2(const GemmDesc &g, int sms, cudaStream_t st);

// dense anchor / gradient group of a problem that fits one thread block: a single launch each (dense_small.cu)
bool dense_small_eligible(int64_t M, int64_t K, int64_t N, int32_t dt);
relay_status_t launch_dense_small_fwd(int32_t dt, const void *x, const void *w, const void *bias, int32_t bias_dt, void *y, int64_t M, int64_t K,
                                      int64_t N, int act, cudaStream_t st);
relay_status_t launch_dense_small_grad(int32_t dt, const void *x, const void *w, const void *y, const void *dy, void *dx, void *dw, float *db,
                                       int64_t M, int64_t K, int64_t N, int act, cudaStream_t st);

}  // namespace relay
