// Dense anchor and its gradient group for problems that fit ONE thread block (the tiny fp32 layer of the first
// configuration): a single launch each.  All operands are brought into shared memory with every load in flight at
// once, then 256 threads compute the results straight from there: y = act(x w + b) forward; dZ = dy (.) act'(y),
// dx = dZ w^T, dw = x^T dZ, db = column sums of dZ for the gradient group, which otherwise takes five launches
// (dZ + column sums, finalize, two contractions) of which launch latency is nearly all the time.
// Sums run in k / n / m order as runs of 16 fp32 products whose run sums are added into a pair of floats
// (simt_acc.cuh), the accumulation of the general SIMT kernel.
#include "ewise_kernels.cuh"
#include "gemm.h"
#include "simt_acc.cuh"

namespace relay {

namespace {

template <typename T> __device__ __forceinline__ float ld_f(const T *p, int64_t i)
{
    if (!relay_in_bounds(p + i, sizeof(T))) return 0.0f;
    if constexpr (sizeof(T) == 2) return __bfloat162float(p[i]);
    else return p[i];
}
template <typename T> __device__ __forceinline__ void st_f(T *p, int64_t i, float v)
{
    if (!relay_in_bounds(p + i, sizeof(T))) return;
    if constexpr (sizeof(T) == 2) p[i] = __float2bfloat16_rn(v);
    else p[i] = v;
}

// Copies n elements of a 16-byte aligned global array into shared memory as floats, dst[perm(i)] = src[i], in two
// phases so that the loads of SEVERAL operands are in flight together: `begin` issues a thread's loads of the first
// 4 * 256 vectors (4096 fp32 elements, enough for every operand of the tiny layer), `end` stores them and copies whatever
// is left the plain way.  A kernel calls begin for all its operands, then end for all: one memory round trip in all.
template <typename T>
struct Stage {
    float4 v[4];
    __device__ __forceinline__ void begin(const T *__restrict__ src, int n)
    {
        if constexpr (sizeof(T) == 4) {
            const int n4 = n >> 2;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i4 = u * 256 + threadIdx.x;
                if (i4 < n4 && relay_in_bounds(reinterpret_cast<const float4 *>(src) + i4, 16)) v[u] = reinterpret_cast<const float4 *>(src)[i4];
                else v[u] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
        }
    }
    template <typename Perm>
    __device__ __forceinline__ void end(const T *__restrict__ src, float *dst, int n, Perm perm)
    {
        if constexpr (sizeof(T) == 4) {
            const int n4 = n >> 2;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i4 = u * 256 + threadIdx.x;
                if (i4 < n4) { dst[perm(4 * i4)] = v[u].x; dst[perm(4 * i4 + 1)] = v[u].y; dst[perm(4 * i4 + 2)] = v[u].z; dst[perm(4 * i4 + 3)] = v[u].w; }
            }
            for (int i4 = 4 * 256 + threadIdx.x; i4 < n4; i4 += 256) {
                float4 r = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                if (relay_in_bounds(reinterpret_cast<const float4 *>(src) + i4, 16)) r = reinterpret_cast<const float4 *>(src)[i4];
                dst[perm(4 * i4)] = r.x; dst[perm(4 * i4 + 1)] = r.y; dst[perm(4 * i4 + 2)] = r.z; dst[perm(4 * i4 + 3)] = r.w;
            }
            for (int i = 4 * n4 + threadIdx.x; i < n; i += 256) dst[perm(i)] = ld_f(src, i);
        } else {
            for (int i = threadIdx.x; i < n; i += 256) dst[perm(i)] = ld_f(src, i);
        }
    }
};

// sum over j < n of a[j * sa] * b[j * sb]
__device__ __forceinline__ float dot_runs(const float *a, int sa, const float *b, int sb, int n)
{
    PairSum acc;
    for (int j0 = 0; j0 < n; j0 += 16) {
        float part = 0.0f;
        const int j1 = min(n, j0 + 16);
        for (int j = j0; j < j1; ++j) part = fmaf(a[j * sa], b[j * sb], part);
        acc.add(part);
    }
    return (float)acc.value();
}

template <typename T, bool FAST>
__global__ void __launch_bounds__(256) dense_small_fwd_kernel(const T *__restrict__ x, const T *__restrict__ w, const void *__restrict__ bias, int bias_bf16,
                                                               T *__restrict__ y, int M, int K, int N, int act)
{
    extern __shared__ float sm[];
    float *xs = sm, *ws = sm + M * K;                 // xs[m][k], ws[k][n]
    pdl_wait();
    auto same = [](int i) { return i; };
    Stage<T> sx, sw;
    sx.begin(x, M * K);
    sw.begin(w, K * N);
    // the bias of this thread's first output travels with the operands
    float b0 = 0.0f;
    if (bias && (int)threadIdx.x < M * N) b0 = bias_bf16 ? ld_f((const __nv_bfloat16 *)bias, threadIdx.x % N) : ld_f((const float *)bias, threadIdx.x % N);
    sx.end(x, xs, M * K, same);
    sw.end(w, ws, K * N, same);
    __syncthreads();
    for (int o = threadIdx.x; o < M * N; o += 256) {
        const int m = o / N, n = o - m * N;
        float z = dot_runs(xs + m * K, 1, ws + n, N, K);
        if (bias) z += o == (int)threadIdx.x ? b0 : bias_bf16 ? ld_f((const __nv_bfloat16 *)bias, n) : ld_f((const float *)bias, n);
        st_f(y, o, act_fwd<FAST>(z, act));
    }
}

template <typename T>
__global__ void __launch_bounds__(256) dense_small_grad_kernel(const T *__restrict__ x, const T *__restrict__ w, const T *__restrict__ y,
                                                                const T *__restrict__ dy, T *__restrict__ dx, T *__restrict__ dw, float *__restrict__ db,
                                                                int M, int K, int N, int act)
{
    extern __shared__ float sm[];
    const int NP = N + 1;                               // padded rows of w: threads that differ in k hit different banks
    float *xs = sm, *ws = xs + M * K, *dz = ws + K * NP;   // xs[m][k], ws[k][n], dz[m][n]
    pdl_wait();
    float *ys = dz + M * N;                             // the saved output, until dZ is formed
    Stage<T> sx, sw, sdy, sy;
    sx.begin(x, M * K); sw.begin(w, K * N); sdy.begin(dy, M * N); sy.begin(y, M * N);
    sx.end(x, xs, M * K, [](int i) { return i; });
    sw.end(w, ws, K * N, [N, NP](int i) { return (i / N) * NP + i % N; });
    sdy.end(dy, dz, M * N, [](int i) { return i; });
    sy.end(y, ys, M * N, [](int i) { return i; });
    __syncthreads();
    for (int i = threadIdx.x; i < M * N; i += 256) {
        float v = dz[i] * act_grad_from_output(ys[i], act);
        if constexpr (sizeof(T) == 2) v = round_bf16(v);                  // dZ is a value of the operand type
        dz[i] = v;
    }
    __syncthreads();
    if (dx)
        for (int o = threadIdx.x; o < M * K; o += 256) {                  // dx[m,k] = sum_n dZ[m,n] w[k,n]
            const int m = o / K, k = o - m * K;
            st_f(dx, o, dot_runs(dz + m * N, 1, ws + k * NP, 1, N));
        }
    for (int o = threadIdx.x; o < K * N; o += 256) {                      // dw[k,n] = sum_m x[m,k] dZ[m,n]
        const int k = o / N, n = o - k * N;
        st_f(dw, o, dot_runs(xs + k, K, dz + n, N, M));
    }
    if (db)
        for (int n = threadIdx.x; n < N; n += 256) {                      // db[n] = sum_m dZ[m,n]
            PairSum acc;
            for (int m0 = 0; m0 < M; m0 += 16) {
                float part = 0.0f;
                for (int m = m0; m < min(M, m0 + 16); ++m) part += dz[m * N + n];
                acc.add(part);
            }
            if (relay_in_bounds(db + n, 4)) db[n] = (float)acc.value();
        }
}

}  // namespace

// one block does the whole problem when its operands fit the default shared memory and the work is a few hundred
// products per thread at most
bool dense_small_eligible(int64_t M, int64_t K, int64_t N, int32_t dt)
{
    if (dt != RELAY_F32 && dt != RELAY_BF16) return false;
    if (M < 1 || K < 1 || N < 1 || M * K * N > (1 << 17)) return false;
    return (M * K + K * (N + 1) + 2 * M * N) * 4 <= 44 * 1024;
}

relay_status_t launch_dense_small_fwd(int32_t dt, const void *x, const void *w, const void *bias, int32_t bias_dt, void *y, int64_t M, int64_t K,
                                      int64_t N, int act, cudaStream_t st)
{
    const size_t smem = (size_t)(M * K + K * N) * 4, es = dtype_size(dt);
    BoundsReg br;
    br.add(x, (size_t)M * K * es); br.add(w, (size_t)K * N * es); br.add(y, (size_t)M * N * es); br.add(bias, (size_t)N * dtype_size(bias_dt));
    RELAY_TRY(br.commit(st));
    if (dt == RELAY_F32)
        RELAY_CUDA(launch_pdl(dense_small_fwd_kernel<float, false>, dim3(1), dim3(256), smem, st, (const float *)x, (const float *)w, bias,
                              (int)(bias_dt == RELAY_BF16), (float *)y, (int)M, (int)K, (int)N, act));
    else
        RELAY_CUDA(launch_pdl(dense_small_fwd_kernel<__nv_bfloat16, true>, dim3(1), dim3(256), smem, st, (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w,
                              bias, (int)(bias_dt == RELAY_BF16), (__nv_bfloat16 *)y, (int)M, (int)K, (int)N, act));
    return check_launch("dense_small_fwd");
}

relay_status_t launch_dense_small_grad(int32_t dt, const void *x, const void *w, const void *y, const void *dy, void *dx, void *dw, float *db,
                                       int64_t M, int64_t K, int64_t N, int act, cudaStream_t st)
{
    const size_t smem = (size_t)(M * K + K * (N + 1) + 2 * M * N) * 4, es = dtype_size(dt);
    BoundsReg br;
    br.add(x, (size_t)M * K * es); br.add(w, (size_t)K * N * es); br.add(y, (size_t)M * N * es); br.add(dy, (size_t)M * N * es);
    br.add(dx, (size_t)M * K * es); br.add(dw, (size_t)K * N * es); br.add(db, (size_t)N * 4);
    RELAY_TRY(br.commit(st));
    if (dt == RELAY_F32)
        RELAY_CUDA(launch_pdl(dense_small_grad_kernel<float>, dim3(1), dim3(256), smem, st, (const float *)x, (const float *)w, (const float *)y,
                              (const float *)dy, (float *)dx, (float *)dw, db, (int)M, (int)K, (int)N, act));
    else
        RELAY_CUDA(launch_pdl(dense_small_grad_kernel<__nv_bfloat16>, dim3(1), dim3(256), smem, st, (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w,
                              (const __nv_bfloat16 *)y, (const __nv_bfloat16 *)dy, (__nv_bfloat16 *)dx, (__nv_bfloat16 *)dw, db, (int)M, (int)K, (int)N, act));
    return check_launch("dense_small_grad");
}

}  // namespace relay
