// SIMT contraction for LARGE fp32 problems: true fp32 fused multiply-adds (tensor cores would round the operands), the
// tier that the dense groups fall to when the operands are fp32 and the output is big enough to give every SM a
// 128 x 64 tile.  The small-tile kernel of gemm_simt.cu spends a third of its issue slots on loads, addressing and its
// accumulator pairs; here
//   * a thread owns 8 x 4 results (three 16-byte shared-memory reads per 32 multiply-adds),
//   * operand tiles go from global to shared memory by asynchronous 4-byte copies (any stride of either operand, zero fill
//     past the edges), three k-blocks deep, so no registers hold data in flight and one block-wide barrier per k-block
//     is enough,
//   * a k-block is 16 deep: its 16 products per result are summed in fp32 and the run sum is added to the result's running
//     total with a compensated addition (Kahan: the total's rounding error is carried in a second float and fed back), so
//     the error stays near one rounding of the result whatever K is, as with the pair sums of the small-tile kernel.
#include "ewise_kernels.cuh"
#include "gemm.h"

namespace relay {

namespace {

constexpr int BM = 128, BN = 64, BK = 16, STAGES = 3;
constexpr int TM = 8, TN = 4;
constexpr int A_PER = BM * BK / 256, B_PER = BN * BK / 256;      // elements a thread copies per k-block: 8 and 4

// 4 bytes global -> shared, asynchronously; `valid` false: nothing is read and the destination is zero-filled
__device__ __forceinline__ void cp_async_f32(float *dst_smem, const float *src, bool valid)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst_smem);
    const uint32_t n = valid ? 4u : 0u;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <bool FAST>
__global__ void __launch_bounds__(256, 1) gemm_simt_big_kernel(const GemmDesc g)
{
    __shared__ __align__(16) float As[STAGES][BK][BM + 4];
    __shared__ __align__(16) float Bs[STAGES][BK][BN + 4];
    const float *A = (const float *)g.a;
    const float *B = (const float *)g.b;
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int tm = (tid / 16) * TM, tn = (tid % 16) * TN;

    // loader: element e = tid + 256 i of a tile, index order following the operand's unit stride so that the copies coalesce
    const bool a_k_fast = g.a_sk == 1, b_n_fast = g.b_sn == 1;
    const int a_m = a_k_fast ? tid / BK : tid % BM, a_k = a_k_fast ? tid % BK : tid / BM;
    const int b_n = b_n_fast ? tid % BN : tid / BK, b_k = b_n_fast ? tid / BN : tid % BK;
    const int a_dm = a_k_fast ? 256 / BK : 0, a_dk = a_k_fast ? 0 : 256 / BM;        // step of (m, k) per i
    const int b_dn = b_n_fast ? 0 : 256 / BK, b_dk = b_n_fast ? 256 / BN : 0;
    const float *a_base = A + (m0 + a_m) * g.a_sm + (int64_t)a_k * g.a_sk;
    const float *b_base = B + (int64_t)b_k * g.b_sk + (n0 + b_n) * g.b_sn;
    const int64_t a_step = (int64_t)a_dm * g.a_sm + (int64_t)a_dk * g.a_sk;
    const int64_t b_step = (int64_t)b_dk * g.b_sk + (int64_t)b_dn * g.b_sn;
    auto copy_tiles = [&](int stage, int64_t k0) {
        const float *pa = a_base + k0 * g.a_sk, *pb = b_base + k0 * g.b_sk;
#pragma unroll
        for (int i = 0; i < A_PER; ++i) {
            const int mm = a_m + i * a_dm, kk = a_k + i * a_dk;
            const bool ok = m0 + mm < g.M && k0 + kk < g.K;
            cp_async_f32(&As[stage][kk][mm], ok ? pa + i * a_step : A, ok);
        }
#pragma unroll
        for (int i = 0; i < B_PER; ++i) {
            const int nn = b_n + i * b_dn, kk = b_k + i * b_dk;
            const bool ok = n0 + nn < g.N && k0 + kk < g.K;
            cp_async_f32(&Bs[stage][kk][nn], ok ? pb + i * b_step : B, ok);
        }
    };

    float sum[TM][TN], comp[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) { sum[i][j] = 0.0f; comp[i][j] = 0.0f; }

    const int n_kb = (int)((g.K + BK - 1) / BK);
    // two k-blocks in flight before the first is used
    copy_tiles(0, 0);
    cp_async_commit();
    if (n_kb > 1) copy_tiles(1, BK);
    cp_async_commit();
    for (int kb = 0; kb < n_kb; ++kb) {
        cp_async_wait<1>();                 // this thread's copies of k-block kb have landed ...
        __syncthreads();                    // ... and everybody's; everybody is also done with k-block kb - 1
        if (kb + 2 < n_kb) copy_tiles((kb + 2) % STAGES, (int64_t)(kb + 2) * BK);    // into the stage k-block kb - 1 used
        cp_async_commit();
        const int st = kb % STAGES;
        float part[TM][TN];
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) part[i][j] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4 *>(&As[st][kk][tm]);
            const float4 a1 = *reinterpret_cast<const float4 *>(&As[st][kk][tm + 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[st][kk][tn]);
            const float av[TM] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
        }
        // compensated addition of the run sums
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                const float y = part[i][j] - comp[i][j];
                const float t = sum[i][j] + y;
                comp[i][j] = (t - sum[i][j]) - y;
                sum[i][j] = t;
            }
    }
    cp_async_wait<0>();

    float *C = (float *)g.c;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t m = m0 + tm + i;
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int64_t n = n0 + tn + j;
            if (n >= g.N) continue;
            const float bv = !g.bias ? 0.0f : g.bias_dtype == RELAY_BF16 ? __bfloat162float(((const __nv_bfloat16 *)g.bias)[n]) : ((const float *)g.bias)[n];
            // the carried error is what the total still owes: sum - comp is the better value
            const float z = (float)(((double)sum[i][j] - (double)comp[i][j]) + (double)bv);
            C[m * g.ldc + n] = act_fwd<FAST>(z, g.act);
        }
    }
}

}  // namespace

bool gemm_simt_big_eligible(const GemmDesc &g)
{
#ifdef RELAY_BOUNDS_CHECK
    return false;                        // asynchronous copies do not pass through the checked access helpers
#endif
    if (g.in_dtype != RELAY_F32 || g.out_dtype != RELAY_F32) return false;
    if ((g.a_sk != 1 && g.a_sm != 1) || (g.b_sn != 1 && g.b_sk != 1)) return false;
    if (g.K < 1) return false;
    const int64_t tiles = ((g.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
    return tiles >= 120 && (g.N + BN - 1) / BN <= 65535;
}

relay_status_t launch_gemm_simt_big(const GemmDesc &g, cudaStream_t st)
{
    dim3 grid((unsigned)((g.M + BM - 1) / BM), (unsigned)((g.N + BN - 1) / BN));
    gemm_simt_big_kernel<false><<<grid, 256, 0, st>>>(g);
    return check_launch("gemm_simt_big");
}

}  // namespace relay
