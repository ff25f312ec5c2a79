// Direct conv2d kernels (SIMT): one result element per thread, fp32 accumulation in a fixed
// loop order.  The fp32 instances sum short runs (one window, or 16 terms) in fp32 and add the run
// sums in fp64, so the rounding error does not grow with the number of terms.  They take every stride / padding / window size and both float types, and are
// the path for instances the implicit-GEMM tensor-core kernels do not cover.
#include "conv.h"
#include "ewise_kernels.cuh"

namespace relay {

template <typename T> __device__ __forceinline__ float ldf(const T *p, int64_t i)
{
    if constexpr (sizeof(T) == 2) return __bfloat162float(p[i]);
    else return p[i];
}
template <typename T> __device__ __forceinline__ void stf(T *p, int64_t i, float v)
{
    if constexpr (sizeof(T) == 2) p[i] = __float2bfloat16_rn(v);
    else p[i] = v;
}

template <typename T> constexpr bool kWideSum = sizeof(T) == 4;

template <typename T, bool FAST>
__global__ void __launch_bounds__(256) conv_fwd_direct_kernel(const ConvDims d, const T *__restrict__ x, const T *__restrict__ w,
                                                               const void *__restrict__ b, int b_dt, int act, T *__restrict__ y)
{
    const int64_t total = d.Nb * d.O * d.P * d.Q;
    for (int64_t lin = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; lin < total; lin += (int64_t)gridDim.x * blockDim.x) {
        int64_t q = lin % d.Q, t = lin / d.Q;
        int64_t p = t % d.P; t /= d.P;
        int64_t o = t % d.O, n = t / d.O;
        float acc = 0.0f;
        double wide = 0.0;
        for (int64_t c = 0; c < d.C; ++c) {
            for (int64_t r = 0; r < d.R; ++r) {
                int64_t i = p * d.stride - d.pad + r;
                if (i < 0 || i >= d.H) continue;
                for (int64_t s = 0; s < d.S; ++s) {
                    int64_t j = q * d.stride - d.pad + s;
                    if (j < 0 || j >= d.W) continue;
                    acc = fmaf(ldf(x, ((n * d.C + c) * d.H + i) * d.W + j), ldf(w, ((o * d.C + c) * d.R + r) * d.S + s), acc);
                }
            }
            if constexpr (kWideSum<T>) { wide += (double)acc; acc = 0.0f; }
        }
        if constexpr (kWideSum<T>) acc = (float)wide;
        if (b) acc += b_dt == RELAY_BF16 ? __bfloat162float(((const __nv_bfloat16 *)b)[o]) : ((const float *)b)[o];
        stf(y, lin, act_fwd<FAST>(acc, act));
    }
}

template <typename T>
__global__ void __launch_bounds__(256) conv_dx_direct_kernel(const ConvDims d, const T *__restrict__ dz, const T *__restrict__ w,
                                                              T *__restrict__ dx)
{
    const int64_t total = d.Nb * d.C * d.H * d.W;
    for (int64_t lin = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; lin < total; lin += (int64_t)gridDim.x * blockDim.x) {
        int64_t j = lin % d.W, t = lin / d.W;
        int64_t i = t % d.H; t /= d.H;
        int64_t c = t % d.C, n = t / d.C;
        float acc = 0.0f;
        double wide = 0.0;
        for (int64_t o = 0; o < d.O; ++o) {
            for (int64_t r = 0; r < d.R; ++r) {
                int64_t pn = i + d.pad - r;
                if (pn < 0 || pn % d.stride) continue;
                int64_t p = pn / d.stride;
                if (p >= d.P) continue;
                for (int64_t s = 0; s < d.S; ++s) {
                    int64_t qn = j + d.pad - s;
                    if (qn < 0 || qn % d.stride) continue;
                    int64_t q = qn / d.stride;
                    if (q >= d.Q) continue;
                    acc = fmaf(ldf(dz, ((n * d.O + o) * d.P + p) * d.Q + q), ldf(w, ((o * d.C + c) * d.R + r) * d.S + s), acc);
                }
            }
            if constexpr (kWideSum<T>) { wide += (double)acc; acc = 0.0f; }
        }
        if constexpr (kWideSum<T>) acc = (float)wide;
        stf(dx, lin, acc);
    }
}

// one warp per dw element: lanes stride over the (n, p, q) index space, fixed-order shuffle combine
template <typename T>
__global__ void __launch_bounds__(256) conv_dw_direct_kernel(const ConvDims d, const T *__restrict__ dz, const T *__restrict__ x,
                                                              T *__restrict__ dw)
{
    const int lane = threadIdx.x & 31;
    const int64_t e = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t total = d.O * d.C * d.R * d.S;
    if (e >= total) return;
    int64_t s = e % d.S, t = e / d.S;
    int64_t r = t % d.R; t /= d.R;
    int64_t c = t % d.C, o = t / d.C;
    const int64_t npq = d.Nb * d.P * d.Q;
    float acc = 0.0f;
    double wide = 0.0;
    int run = 0;
    for (int64_t l = lane; l < npq; l += 32) {
        int64_t q = l % d.Q, u = l / d.Q;
        int64_t p = u % d.P, n = u / d.P;
        int64_t i = p * d.stride - d.pad + r, j = q * d.stride - d.pad + s;
        if (i < 0 || i >= d.H || j < 0 || j >= d.W) continue;
        acc = fmaf(ldf(dz, ((n * d.O + o) * d.P + p) * d.Q + q), ldf(x, ((n * d.C + c) * d.H + i) * d.W + j), acc);
        if constexpr (kWideSum<T>) if (++run == 16) { wide += (double)acc; acc = 0.0f; run = 0; }
    }
    if constexpr (kWideSum<T>) {
        wide += (double)acc;
#pragma unroll
        for (int k = 16; k > 0; k >>= 1) wide += __shfl_xor_sync(0xffffffffu, wide, k);
        acc = (float)wide;
    } else {
#pragma unroll
        for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
    }
    if (lane == 0) stf(dw, e, acc);
}

// db[o] = sum over n, p, q of dz[n,o,p,q]: one block per channel, fixed-order combine
template <typename T>
__global__ void __launch_bounds__(256) conv_db_kernel(const ConvDims d, const T *__restrict__ dz, float *__restrict__ db)
{
    __shared__ float sm[8];
    const int64_t o = blockIdx.x, pq = d.P * d.Q;
    float acc = 0.0f;
    for (int64_t l = threadIdx.x; l < d.Nb * pq; l += blockDim.x) {
        int64_t n = l / pq, r = l % pq;
        acc += ldf(dz, (n * d.O + o) * pq + r);
    }
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.0f;
        for (int k = 0; k < 8; ++k) s += sm[k];
        db[o] = s;
    }
}

static unsigned grid_for(int64_t total)
{
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 32));
}

relay_status_t launch_conv_fwd_direct(const ConvDims &d, const void *x, const void *w, const void *b, int32_t b_dt, int act,
                                      void *y, cudaStream_t st)
{
    const int64_t total = d.Nb * d.O * d.P * d.Q;
    if (total == 0) return RELAY_OK;
    if (d.dt == RELAY_BF16)
        conv_fwd_direct_kernel<__nv_bfloat16, true><<<grid_for(total), 256, 0, st>>>(d, (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, b, b_dt, act, (__nv_bfloat16 *)y);
    else
        conv_fwd_direct_kernel<float, false><<<grid_for(total), 256, 0, st>>>(d, (const float *)x, (const float *)w, b, b_dt, act, (float *)y);
    return check_launch("conv_fwd_direct");
}

relay_status_t launch_conv_dx_direct(const ConvDims &d, const void *dz, const void *w, void *dx, cudaStream_t st)
{
    const int64_t total = d.Nb * d.C * d.H * d.W;
    if (total == 0) return RELAY_OK;
    if (d.dt == RELAY_BF16)
        conv_dx_direct_kernel<<<grid_for(total), 256, 0, st>>>(d, (const __nv_bfloat16 *)dz, (const __nv_bfloat16 *)w, (__nv_bfloat16 *)dx);
    else
        conv_dx_direct_kernel<<<grid_for(total), 256, 0, st>>>(d, (const float *)dz, (const float *)w, (float *)dx);
    return check_launch("conv_dx_direct");
}

relay_status_t launch_conv_dw_direct(const ConvDims &d, const void *dz, const void *x, void *dw, cudaStream_t st)
{
    const int64_t total = d.O * d.C * d.R * d.S;
    if (total == 0) return RELAY_OK;
    const unsigned grid = (unsigned)((total + 7) / 8);
    if (d.dt == RELAY_BF16)
        conv_dw_direct_kernel<<<grid, 256, 0, st>>>(d, (const __nv_bfloat16 *)dz, (const __nv_bfloat16 *)x, (__nv_bfloat16 *)dw);
    else
        conv_dw_direct_kernel<<<grid, 256, 0, st>>>(d, (const float *)dz, (const float *)x, (float *)dw);
    return check_launch("conv_dw_direct");
}

relay_status_t launch_conv_db(const ConvDims &d, const void *dz, float *db, cudaStream_t st)
{
    if (d.O == 0) return RELAY_OK;
    if (d.dt == RELAY_BF16) conv_db_kernel<<<(unsigned)d.O, 256, 0, st>>>(d, (const __nv_bfloat16 *)dz, db);
    else conv_db_kernel<<<(unsigned)d.O, 256, 0, st>>>(d, (const float *)dz, db);
    return check_launch("conv_db");
}

// ---- layout change (NCHW <-> NHWC): batched transpose through a 32 x 33 shared-memory tile --------------------
template <typename T>
__global__ void __launch_bounds__(256) layout_change_kernel(const T *__restrict__ in, T *__restrict__ out, int64_t R, int64_t S)
{
    __shared__ T tile[32][33];
    const int64_t b = blockIdx.z;
    const int64_t r0 = (int64_t)blockIdx.y * 32, s0 = (int64_t)blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const T *src = in + b * R * S;
    T *dst = out + b * R * S;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < R && s0 + tx < S) tile[i][tx] = src[(r0 + i) * S + s0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8)
        if (s0 + i < S && r0 + tx < R) dst[(s0 + i) * R + r0 + tx] = tile[tx][i];
}

relay_status_t launch_layout_change(int32_t dt, const void *in, void *out, int64_t batch, int64_t R, int64_t S, cudaStream_t st)
{
    if (batch == 0 || R == 0 || S == 0) return RELAY_OK;
    if (batch > 65535 || (R + 31) / 32 > 65535) return fail(RELAY_ERR_UNSUPPORTED, "layout change: extent exceeds the grid limit");
    dim3 grid((unsigned)((S + 31) / 32), (unsigned)((R + 31) / 32), (unsigned)batch);
    if (dtype_size(dt) == 2) layout_change_kernel<<<grid, 256, 0, st>>>((const uint16_t *)in, (uint16_t *)out, R, S);
    else layout_change_kernel<<<grid, 256, 0, st>>>((const uint32_t *)in, (uint32_t *)out, R, S);
    return check_launch("layout_change");
}

}  // namespace relay
