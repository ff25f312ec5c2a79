// SIMT contraction kernel, sums in k order.  It is the fp32 path of the dense groups (tensor cores
// would round the operands to tf32) and the path for shapes the tensor-core kernel does not take.
// fp32 operands are accumulated in fp64 and rounded once on the store, so that results that suffer
// cancellation still meet the fp32 tolerance; bf16 operands are accumulated in fp32.
#include <type_traits>

#include "ewise_kernels.cuh"
#include "gemm.h"

namespace relay {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TIN, typename TOUT, bool FAST>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmDesc g)
{
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN + 1];
    const TIN *A = (const TIN *)g.a;
    const TIN *B = (const TIN *)g.b;
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int tm = (tid / 16) * 4, tn = (tid % 16) * 4;
    using Acc = typename std::conditional<sizeof(TIN) == 4, double, float>::type;
    Acc acc[4][4] = {};
    // loader index order follows the unit stride of each operand so that loads coalesce
    const bool a_k_fast = g.a_sk == 1, b_n_fast = g.b_sn == 1;
    for (int64_t k0 = 0; k0 < g.K; k0 += BK) {
        for (int e = tid; e < BM * BK; e += 256) {
            int mm = a_k_fast ? e / BK : e % BM, kk = a_k_fast ? e % BK : e / BM;
            int64_t m = m0 + mm, k = k0 + kk;
            As[kk][mm] = (m < g.M && k < g.K) ? to_f<TIN>(A[m * g.a_sm + k * g.a_sk]) : 0.0f;
        }
        for (int e = tid; e < BN * BK; e += 256) {
            int nn = b_n_fast ? e % BN : e / BK, kk = b_n_fast ? e / BN : e % BK;
            int64_t n = n0 + nn, k = k0 + kk;
            Bs[kk][nn] = (n < g.N && k < g.K) ? to_f<TIN>(B[k * g.b_sk + n * g.b_sn]) : 0.0f;
        }
        __syncthreads();
        // threads whose 4 x 4 outputs all lie outside the problem skip the arithmetic (a tiny M or N would
        // otherwise fill the fp64 pipe with products nobody stores)
        if (m0 + tm < g.M && n0 + tn < g.N)
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[kk][tm + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tn + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma((Acc)av[i], (Acc)bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    TOUT *C = (TOUT *)g.c;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int64_t m = m0 + tm + i;
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int64_t n = n0 + tn + j;
            if (n >= g.N) continue;
            Acc zz = acc[i][j];
            if (g.bias) zz += (Acc)(g.bias_dtype == RELAY_BF16 ? __bfloat162float(((const __nv_bfloat16 *)g.bias)[n]) : ((const float *)g.bias)[n]);
            const float z = (float)zz;
            float y = act_fwd<FAST>(z, g.act);
            if constexpr (sizeof(TOUT) == 2) C[m * g.ldc + n] = __float2bfloat16_rn(y);
            else C[m * g.ldc + n] = y;
        }
    }
}

relay_status_t launch_gemm_simt(const GemmDesc &g, cudaStream_t st)
{
    if (g.M == 0 || g.N == 0) return RELAY_OK;
    dim3 grid((unsigned)((g.M + BM - 1) / BM), (unsigned)((g.N + BN - 1) / BN));
    if (grid.y > 65535) return fail(RELAY_ERR_UNSUPPORTED, "SIMT contraction: N = %lld exceeds the grid limit", (long long)g.N);
    if (g.in_dtype == RELAY_F32 && g.out_dtype == RELAY_F32) gemm_simt_kernel<float, float, false><<<grid, 256, 0, st>>>(g);
    else if (g.in_dtype == RELAY_BF16 && g.out_dtype == RELAY_BF16) gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16, true><<<grid, 256, 0, st>>>(g);
    else if (g.in_dtype == RELAY_BF16 && g.out_dtype == RELAY_F32) gemm_simt_kernel<__nv_bfloat16, float, false><<<grid, 256, 0, st>>>(g);
    else return fail(RELAY_ERR_UNSUPPORTED, "SIMT contraction: %s -> %s has no instance", dtype_name(g.in_dtype), dtype_name(g.out_dtype));
    return check_launch("gemm_simt");
}

}  // namespace relay
