// Helpers of the general conv2d tier: the bias gradient and the layout change of layout-tagged tensors.
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

// db[o] = sum over n, p, q of dz[n,o,p,q]: one block of 32 warps per channel; warp w takes the images w, w + 32, ...,
// its lanes run along the contiguous pixels (four independent loads in flight per lane); fixed-order combine
template <typename T>
__global__ void __launch_bounds__(1024) conv_db_kernel(const ConvDims d, const T *__restrict__ dz, float *__restrict__ db)
{
    __shared__ float sm[32];
    const int64_t o = blockIdx.x, pq = d.P * d.Q;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
    for (int64_t n = warp; n < d.Nb; n += 32) {
        const T *row = dz + (n * d.O + o) * pq;
        int64_t r = lane;
        for (; r + 96 < pq; r += 128) {
            a0 += ldf(row, r); a1 += ldf(row, r + 32); a2 += ldf(row, r + 64); a3 += ldf(row, r + 96);
        }
        for (; r < pq; r += 32) a0 += ldf(row, r);
    }
    float acc = (a0 + a1) + (a2 + a3);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
    if (lane == 0) sm[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.0f;
        for (int k = 0; k < 32; ++k) s += sm[k];
        db[o] = s;
    }
}

relay_status_t launch_conv_db(const ConvDims &d, const void *dz, float *db, cudaStream_t st)
{
    if (d.O == 0) return RELAY_OK;
    if (d.dt == RELAY_BF16) conv_db_kernel<<<(unsigned)d.O, 1024, 0, st>>>(d, (const __nv_bfloat16 *)dz, db);
    else conv_db_kernel<<<(unsigned)d.O, 1024, 0, st>>>(d, (const float *)dz, db);
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
