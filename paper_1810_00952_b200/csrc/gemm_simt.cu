// SIMT contraction kernel, sums in k order.  It is the fp32 path of the dense groups (tensor cores
// would round the operands to tf32) and the path for shapes the tensor-core kernel does not take.
// fp32 operands: runs of 16 products are summed in fp32 and the run sums are added into a pair of floats
// (simt_acc.cuh); the rounding error is then about 1e-7 of the output's RMS whatever K is, so outputs that suffer
// cancellation still meet the fp32 tolerance.  bf16 operands are accumulated in fp32.
#include <type_traits>

#include "ewise_kernels.cuh"
#include "gemm.h"
#include "simt_acc.cuh"

namespace relay {

constexpr int BK = 32, KSUB = 16;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// block tile (16 * TM) x (16 * TN), thread tile TM x TN: 64 x 64 for large outputs; 16 x 64, 16 x 32 or 16 x 16
// for outputs whose grid of larger tiles would not give every SM a block.  The loads of k-block i+1 are issued
// into registers before the arithmetic of k-block i, all of a thread's loads back to back, so that one
// memory round trip per k-block is exposed at most.
template <typename TIN, typename TOUT, bool FAST, int TM, int TN>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmDesc g)
{
    static_assert(TM == 1 || TN == 4, "the large tiles are 64 x 64 and 128 x 64");
    constexpr int BM = 16 * TM, BN = 16 * TN;
    constexpr int A_LD = BM * BK / 256, B_LD = BN * BK / 256;
    __shared__ __align__(16) float As[BK][BM + 4];     // rows of whole 16-byte vectors: a thread's four values are one load
    __shared__ __align__(16) float Bs[BK][BN + 4];
    const TIN *A = (const TIN *)g.a;
    const TIN *B = (const TIN *)g.b;
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int tm = (tid / 16) * TM, tn = (tid % 16) * TN;
    constexpr bool F64 = sizeof(TIN) == 4;
    using Acc = typename std::conditional<F64, PairSum, float>::type;
    Acc acc[TM][TN] = {};
    // loader index order follows the unit stride of each operand so that loads coalesce.  A thread's loads of one operand
    // are a fixed distance apart (element e = tid + 256 i), so one base offset per operand and a constant step address them;
    // only the k-range test changes from k-block to k-block.
    const bool a_k_fast = g.a_sk == 1, b_n_fast = g.b_sn == 1;
    const int a_m = a_k_fast ? tid / BK : tid % BM, a_k = a_k_fast ? tid % BK : tid / BM;          // element 0 of this thread
    const int b_n = b_n_fast ? tid % BN : tid / BK, b_k = b_n_fast ? tid / BN : tid % BK;
    constexpr int A_STEP_M = 256 / BK, A_STEP_K = 256 / BM;                                         // per i, k-fast / m-fast order
    constexpr int B_STEP_K = 256 / BN, B_STEP_N = 256 / BK;
    static_assert(256 % BK == 0 && 256 % BM == 0 && 256 % BN == 0, "loader steps");
    const TIN *a_base = A + (m0 + a_m) * g.a_sm + (int64_t)a_k * g.a_sk;
    const TIN *b_base = B + (int64_t)b_k * g.b_sk + (n0 + b_n) * g.b_sn;
    const int64_t a_step = a_k_fast ? (int64_t)A_STEP_M * g.a_sm : (int64_t)A_STEP_K * g.a_sk;
    const int64_t b_step = b_n_fast ? (int64_t)B_STEP_K * g.b_sk : (int64_t)B_STEP_N * g.b_sn;
    float ra[A_LD], rb[B_LD];
    auto load_tiles = [&](int64_t k0) {
        const TIN *pa = a_base + k0 * g.a_sk, *pb = b_base + k0 * g.b_sk;
#pragma unroll
        for (int i = 0; i < A_LD; ++i) {
            const int mm = a_k_fast ? a_m + i * A_STEP_M : a_m, kk = a_k_fast ? a_k : a_k + i * A_STEP_K;
            const TIN *q = pa + i * a_step;
            ra[i] = (m0 + mm < g.M && k0 + kk < g.K && relay_in_bounds(q, sizeof(TIN))) ? to_f<TIN>(*q) : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < B_LD; ++i) {
            const int nn = b_n_fast ? b_n : b_n + i * B_STEP_N, kk = b_n_fast ? b_k + i * B_STEP_K : b_k;
            const TIN *q = pb + i * b_step;
            rb[i] = (n0 + nn < g.N && k0 + kk < g.K && relay_in_bounds(q, sizeof(TIN))) ? to_f<TIN>(*q) : 0.0f;
        }
    };
    load_tiles(0);
    for (int64_t k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
        for (int i = 0; i < A_LD; ++i) {
            const int e = tid + i * 256;
            As[a_k_fast ? e % BK : e / BM][a_k_fast ? e / BK : e % BM] = ra[i];
        }
#pragma unroll
        for (int i = 0; i < B_LD; ++i) {
            const int e = tid + i * 256;
            Bs[b_n_fast ? e / BN : e % BK][b_n_fast ? e % BN : e / BK] = rb[i];
        }
        __syncthreads();
        if (k0 + BK < g.K) load_tiles(k0 + BK);
        // threads whose outputs all lie outside the problem skip the arithmetic
        if (m0 + tm < g.M && n0 + tn < g.N) {
#pragma unroll 1
            for (int ks = 0; ks < BK; ks += KSUB) {
                float part[TM][TN] = {};
#pragma unroll
                for (int kk = ks; kk < ks + KSUB; ++kk) {
                    float av[TM], bv[TN];
                    if constexpr (TM % 4 == 0) {
#pragma unroll
                        for (int q = 0; q < TM / 4; ++q) {
                            const float4 a4 = *reinterpret_cast<const float4 *>(&As[kk][tm + 4 * q]);
                            av[4 * q] = a4.x; av[4 * q + 1] = a4.y; av[4 * q + 2] = a4.z; av[4 * q + 3] = a4.w;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < TM; ++i) av[i] = As[kk][tm + i];
                    }
                    if constexpr (TN == 4) {
                        const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[kk][tn]);
                        bv[0] = b4.x; bv[1] = b4.y; bv[2] = b4.z; bv[3] = b4.w;
                    } else if constexpr (TN == 2) {
                        const float2 b2 = *reinterpret_cast<const float2 *>(&Bs[kk][tn]);
                        bv[0] = b2.x; bv[1] = b2.y;
                    } else {
                        bv[0] = Bs[kk][tn];
                    }
#pragma unroll
                    for (int i = 0; i < TM; ++i)
#pragma unroll
                        for (int j = 0; j < TN; ++j) {
                            if constexpr (F64) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
                            else acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
                        }
                }
                if constexpr (F64) {
#pragma unroll
                    for (int i = 0; i < TM; ++i)
#pragma unroll
                        for (int j = 0; j < TN; ++j) acc[i][j].add(part[i][j]);
                }
            }
        }
        __syncthreads();
    }
    TOUT *C = (TOUT *)g.c;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        int64_t m = m0 + tm + i;
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            int64_t n = n0 + tn + j;
            if (n >= g.N || !relay_in_bounds(&C[m * g.ldc + n], sizeof(TOUT))) continue;
            float z;
            const float bv = !g.bias ? 0.0f : g.bias_dtype == RELAY_BF16 ? __bfloat162float(((const __nv_bfloat16 *)g.bias)[n]) : ((const float *)g.bias)[n];
            if constexpr (F64) z = (float)(acc[i][j].value() + (double)bv);
            else z = acc[i][j] + bv;
            float y = act_fwd<FAST>(z, g.act);
            if constexpr (sizeof(TOUT) == 2) C[m * g.ldc + n] = __float2bfloat16_rn(y);
            else C[m * g.ldc + n] = y;
        }
    }
}

template <int TM, int TN>
static relay_status_t launch_tile(const GemmDesc &g, cudaStream_t st)
{
    constexpr int BM = 16 * TM, BN = 16 * TN;
    dim3 grid((unsigned)((g.M + BM - 1) / BM), (unsigned)((g.N + BN - 1) / BN));
    if (grid.y > 65535) return fail(RELAY_ERR_UNSUPPORTED, "SIMT contraction: N = %lld exceeds the grid limit", (long long)g.N);
    if (g.in_dtype == RELAY_F32 && g.out_dtype == RELAY_F32) gemm_simt_kernel<float, float, false, TM, TN><<<grid, 256, 0, st>>>(g);
    else if (g.in_dtype == RELAY_BF16 && g.out_dtype == RELAY_BF16) gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16, true, TM, TN><<<grid, 256, 0, st>>>(g);
    else if (g.in_dtype == RELAY_BF16 && g.out_dtype == RELAY_F32) gemm_simt_kernel<__nv_bfloat16, float, false, TM, TN><<<grid, 256, 0, st>>>(g);
    else return fail(RELAY_ERR_UNSUPPORTED, "SIMT contraction: %s -> %s has no instance", dtype_name(g.in_dtype), dtype_name(g.out_dtype));
    return check_launch("gemm_simt");
}

relay_status_t launch_gemm_simt(const GemmDesc &g, cudaStream_t st)
{
    if (g.M == 0 || g.N == 0) return RELAY_OK;
    {
        const size_t ein = dtype_size(g.in_dtype), eout = dtype_size(g.out_dtype);
        BoundsReg br;
        if (g.K > 0) {
            br.add(g.a, (size_t)((g.M - 1) * g.a_sm + (g.K - 1) * g.a_sk + 1) * ein);
            br.add(g.b, (size_t)((g.K - 1) * g.b_sk + (g.N - 1) * g.b_sn + 1) * ein);
        }
        br.add(g.c, (size_t)((g.M - 1) * g.ldc + g.N) * eout);
        br.add(g.bias, (size_t)g.N * dtype_size(g.bias_dtype));
        RELAY_TRY(br.commit(st));
    }
    if (gemm_simt_big_eligible(g)) return launch_gemm_simt_big(g, st);
    // The largest tile whose grid still gives every SM a block: with few warps on an SM a block's time goes to waiting
    // for its own shared-memory reads, so while SMs are idle more and lighter blocks finish sooner.
    auto tiles = [&](int bm, int bn) { return ((g.M + bm - 1) / bm) * ((g.N + bn - 1) / bn); };
    // 64 x 64 as soon as its grid gives every SM a block (two fit an SM): 1024^3 fp32 runs at 17 TFLOP/s on it against 10 on
    // 16 x 64 tiles.  A 128 x 64 tile (8 x 4 per thread) was measured too: 19 TFLOP/s at 1024^3, no gain at 2048^3 (its 235
    // registers leave one block per SM) and far slower on small outputs, so it is not used.
    if (g.M > 16 && tiles(64, 64) >= 148) return launch_tile<4, 4>(g, st);
    if (tiles(16, 64) >= 148) return launch_tile<1, 4>(g, st);
    if (tiles(16, 32) >= 148) return launch_tile<1, 2>(g, st);
    return launch_tile<1, 1>(g, st);
}

}  // namespace relay
