// Max pooling of NCHW tensors and its gradient (Fig. 3 of the paper: relay.max_pool; Section 4.2).
// HBM-bound: x is read once and y / idx written once; the gradient reads idx and dy once and writes dx once.
#include <algorithm>

#include "common.h"
#include "ewise_kernels.cuh"

namespace relay {
namespace {

constexpr int kThreads = 256;

struct PoolDims {
    int64_t planes;           // N * C
    int H, W, P, Q, kh, kw, sh, sw;
};

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- any window: one thread per output ------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) max_pool_kernel(const T *__restrict__ x, T *__restrict__ y, int32_t *__restrict__ idx, PoolDims d)
{
    const int64_t total = d.planes * d.P * d.Q;
    pdl_wait();
    for (int64_t o = (int64_t)blockIdx.x * kThreads + threadIdx.x; o < total; o += (int64_t)gridDim.x * kThreads) {
        const int q = (int)(o % d.Q), p = (int)((o / d.Q) % d.P);
        const int64_t plane = o / ((int64_t)d.P * d.Q);
        const T *xp = x + plane * d.H * d.W;
        int best = (p * d.sh) * d.W + q * d.sw;
        float bv = to_f(xp[best]);
        for (int r = 0; r < d.kh; ++r)
            for (int s = 0; s < d.kw; ++s) {
                const int at = (p * d.sh + r) * d.W + (q * d.sw + s);
                const float v = to_f(xp[at]);
                if (v > bv) { bv = v; best = at; }          // strict: the first maximum wins
            }
        y[o] = from_f<T>(bv);
        if (idx) idx[o] = best;
    }
}

// one thread per input: sums dy over the windows that cover it and name it, in (p,q) order
template <typename T>
__global__ void __launch_bounds__(kThreads) max_pool_grad_kernel(const int32_t *__restrict__ idx, const T *__restrict__ dy, T *__restrict__ dx, PoolDims d)
{
    const int64_t total = d.planes * d.H * d.W;
    pdl_wait();
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const int w = (int)(i % d.W), h = (int)((i / d.W) % d.H);
        const int64_t plane = i / ((int64_t)d.H * d.W);
        const int at = h * d.W + w;
        // windows p with p*sh <= h < p*sh + kh
        const int p_lo = h >= d.kh ? (h - d.kh) / d.sh + 1 : 0, p_hi = min(h / d.sh, d.P - 1);
        const int q_lo = w >= d.kw ? (w - d.kw) / d.sw + 1 : 0, q_hi = min(w / d.sw, d.Q - 1);
        float acc = 0.0f;
        for (int p = p_lo; p <= p_hi; ++p)
            for (int q = q_lo; q <= q_hi; ++q) {
                const int64_t o = (plane * d.P + p) * d.Q + q;
                if (idx[o] == at) acc += to_f(dy[o]);
            }
        dx[i] = from_f<T>(acc);
    }
}

// ---- 2 x 2 windows, stride 2, rows of whole 8-element groups: 16-byte accesses ----------------------------
// One thread: 8 inputs of two rows -> 4 outputs.
template <typename T>
__device__ __forceinline__ void load8(const T *p, float (&f)[8])
{
    if constexpr (sizeof(T) == 2) {
        unpack(ld_stream(p), f);
    } else {
        float a[4], b[4];
        unpack(ld_stream(p), a);
        unpack(ld_stream(p + 4), b);
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[i] = a[i]; f[4 + i] = b[i]; }
    }
}
template <typename T>
__device__ __forceinline__ void store8(T *p, const float (&f)[8])
{
    if constexpr (sizeof(T) == 2) {
        st_stream(p, pack(f));
    } else {
        const float a[4] = {f[0], f[1], f[2], f[3]}, b[4] = {f[4], f[5], f[6], f[7]};
        st_stream(p, pack(a));
        st_stream(p + 4, pack(b));
    }
}

constexpr int kPer = 1;            // items a thread of the 2 x 2 kernels keeps in flight

template <typename T>
__global__ void __launch_bounds__(kThreads) max_pool_2x2_kernel(const T *__restrict__ x, T *__restrict__ y, int32_t *__restrict__ idx, PoolDims d)
{
    const int groups = d.W >> 3;                              // threads per output row; Q = 4 * groups
    const int64_t total = d.planes * d.P * groups;
    pdl_wait();
    for (int64_t t0 = (int64_t)blockIdx.x * (kThreads * kPer) + threadIdx.x; t0 < total; t0 += (int64_t)gridDim.x * (kThreads * kPer)) {
        float a[kPer][8], b[kPer][8];
        int base[kPer];
        int64_t o[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {                      // all loads first
            const int64_t t = t0 + (int64_t)u * kThreads;
            if (t < total) {
                const int g = (int)(t % groups), p = (int)((t / groups) % d.P);
                const int64_t plane = t / ((int64_t)groups * d.P);
                const T *r0 = x + (plane * d.H + 2 * p) * d.W + 8 * g;
                load8<T>(r0, a[u]);
                load8<T>(r0 + d.W, b[u]);
                base[u] = (2 * p) * d.W + 8 * g;
                o[u] = (plane * d.P + p) * d.Q + 4 * g;
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            if (t0 + (int64_t)u * kThreads < total) {
                float out[4];
                int where[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {                 // window order: (0,0) (0,1) (1,0) (1,1), first maximum wins
                    float bv = a[u][2 * j];
                    int at = base[u] + 2 * j;
                    if (a[u][2 * j + 1] > bv) { bv = a[u][2 * j + 1]; at = base[u] + 2 * j + 1; }
                    if (b[u][2 * j] > bv) { bv = b[u][2 * j]; at = base[u] + d.W + 2 * j; }
                    if (b[u][2 * j + 1] > bv) { bv = b[u][2 * j + 1]; at = base[u] + d.W + 2 * j + 1; }
                    out[j] = bv; where[j] = at;
                }
                if constexpr (sizeof(T) == 2) {
                    *reinterpret_cast<uint2 *>(y + o[u]) = make_uint2(pack2(out[0], out[1]), pack2(out[2], out[3]));
                } else {
                    st_stream(y + o[u], pack(out));
                }
                if (idx) st_stream(idx + o[u], make_uint4((uint32_t)where[0], (uint32_t)where[1], (uint32_t)where[2], (uint32_t)where[3]));
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads) max_pool_2x2_grad_kernel(const int32_t *__restrict__ idx, const T *__restrict__ dy, T *__restrict__ dx, PoolDims d)
{
    const int groups = d.W >> 3;
    const int64_t total = d.planes * d.P * groups;
    pdl_wait();
    for (int64_t t0 = (int64_t)blockIdx.x * (kThreads * kPer) + threadIdx.x; t0 < total; t0 += (int64_t)gridDim.x * (kThreads * kPer)) {
        uint4 wi[kPer];
        float g4[kPer][4];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {                      // all loads first
            const int64_t t = t0 + (int64_t)u * kThreads;
            if (t < total) {
                const int g = (int)(t % groups), p = (int)((t / groups) % d.P);
                const int64_t plane = t / ((int64_t)groups * d.P);
                const int64_t o = (plane * d.P + p) * d.Q + 4 * g;
                wi[u] = ld_stream(idx + o);
                if constexpr (sizeof(T) == 2) {
                    const uint2 v = *reinterpret_cast<const uint2 *>(dy + o);
                    g4[u][0] = __uint_as_float(v.x << 16); g4[u][1] = __uint_as_float(v.x & 0xffff0000u);
                    g4[u][2] = __uint_as_float(v.y << 16); g4[u][3] = __uint_as_float(v.y & 0xffff0000u);
                } else {
                    unpack(ld_stream(dy + o), g4[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const int64_t t = t0 + (int64_t)u * kThreads;
            if (t < total) {
                const int g = (int)(t % groups), p = (int)((t / groups) % d.P);
                const int64_t plane = t / ((int64_t)groups * d.P);
                const int where[4] = {(int)wi[u].x, (int)wi[u].y, (int)wi[u].z, (int)wi[u].w};
                const int base = (2 * p) * d.W + 8 * g;
                float a[8], b[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a[2 * j] = where[j] == base + 2 * j ? g4[u][j] : 0.0f;
                    a[2 * j + 1] = where[j] == base + 2 * j + 1 ? g4[u][j] : 0.0f;
                    b[2 * j] = where[j] == base + d.W + 2 * j ? g4[u][j] : 0.0f;
                    b[2 * j + 1] = where[j] == base + d.W + 2 * j + 1 ? g4[u][j] : 0.0f;
                }
                T *r0 = dx + (plane * d.H + 2 * p) * d.W + 8 * g;
                store8<T>(r0, a);
                store8<T>(r0 + d.W, b);
                if ((d.H & 1) && p == d.P - 1) {              // the last row of an odd plane lies in no window
                    const float z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    store8<T>(r0 + 2 * d.W, z);
                }
            }
        }
    }
}

relay_status_t check_pool(const relay_tensor_t *x, const relay_pool2d_attrs_t *at, PoolDims *d)
{
    RELAY_TRY(check_type(x, "x"));
    RELAY_TRY(check_rank(x, 4, "x"));
    if (!is_float(x->dtype)) return fail(RELAY_ERR_DTYPE, "x: base type %s, needs f32 or bf16", dtype_name(x->dtype));
    RELAY_TRY(check_layout(x, RELAY_NCHW, RELAY_ROWMAJOR, "x"));
    if (at->kh < 1 || at->kw < 1 || at->sh < 1 || at->sw < 1)
        return fail(RELAY_ERR_ATTR, "pooling window %dx%d stride %dx%d: every entry must be >= 1", at->kh, at->kw, at->sh, at->sw);
    if (at->kh > x->shape[2] || at->kw > x->shape[3])
        return fail(RELAY_ERR_ATTR, "pooling window %dx%d does not fit a %lldx%lld plane", at->kh, at->kw, (long long)x->shape[2],
                    (long long)x->shape[3]);
    if (x->shape[2] * x->shape[3] > 0x7fffffffLL) return fail(RELAY_ERR_UNSUPPORTED, "plane too large for i32 positions");
    d->planes = x->shape[0] * x->shape[1];
    d->H = (int)x->shape[2]; d->W = (int)x->shape[3];
    d->kh = at->kh; d->kw = at->kw; d->sh = at->sh; d->sw = at->sw;
    d->P = (d->H - d->kh) / d->sh + 1; d->Q = (d->W - d->kw) / d->sw + 1;
    return RELAY_OK;
}

bool fast_2x2(const PoolDims &d) { return d.kh == 2 && d.kw == 2 && d.sh == 2 && d.sw == 2 && d.W % 8 == 0; }

unsigned grid_for(int64_t items)
{
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>((items + kThreads - 1) / kThreads, 148 * 16));
}

}  // namespace
}  // namespace relay

using namespace relay;

extern "C" relay_status_t relay_infer_max_pool2d(const relay_tensor_t *x, const relay_pool2d_attrs_t *attrs, relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(out, "out"));
    PoolDims d{};
    RELAY_TRY(check_pool(x, attrs, &d));
    out->data = nullptr; out->dtype = x->dtype; out->rank = 4; out->layout = RELAY_NCHW;
    out->shape[0] = x->shape[0]; out->shape[1] = x->shape[1]; out->shape[2] = d.P; out->shape[3] = d.Q;
    out->shape[4] = out->shape[5] = 1;
    return RELAY_OK;
}

extern "C" relay_status_t relay_max_pool2d(const relay_tensor_t *x, const relay_pool2d_attrs_t *attrs, const relay_tensor_t *y,
                                           const relay_tensor_t *idx, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(y, "y"));
    PoolDims d{};
    RELAY_TRY(check_pool(x, attrs, &d));
    RELAY_TRY(check_type(y, "y"));
    RELAY_TRY(check_rank(y, 4, "y"));
    if (idx) { RELAY_TRY(check_type(idx, "idx")); RELAY_TRY(check_rank(idx, 4, "idx")); }
    RELAY_TRY(check_dtype(y, x->dtype, "y"));
    if (idx) RELAY_TRY(check_dtype(idx, RELAY_I32, "idx"));
    RELAY_TRY(check_layout(y, RELAY_NCHW, RELAY_ROWMAJOR, "y"));
    RELAY_TRY(check_shape(y, {x->shape[0], x->shape[1], (int64_t)d.P, (int64_t)d.Q}, "y"));
    if (idx) RELAY_TRY(check_shape(idx, {x->shape[0], x->shape[1], (int64_t)d.P, (int64_t)d.Q}, "idx"));
    RELAY_TRY(check_data(x, "x"));
    RELAY_TRY(check_data(y, "y"));
    if (idx) RELAY_TRY(check_data(idx, "idx"));
    const relay_tensor_t *outs[2] = {y, idx}, *ins[1] = {x};
    RELAY_TRY(check_no_overlap(outs, 2, ins, 1));
    if (numel(y) == 0) return RELAY_OK;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *ip = idx ? (int32_t *)idx->data : nullptr;
    if (fast_2x2(d)) {
        const unsigned grid = grid_for((d.planes * d.P * (d.W / 8) + kPer - 1) / kPer);
        if (x->dtype == RELAY_BF16) RELAY_CUDA(launch_pdl(max_pool_2x2_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st, (const __nv_bfloat16 *)x->data, (__nv_bfloat16 *)y->data, ip, d));
        else RELAY_CUDA(launch_pdl(max_pool_2x2_kernel<float>, dim3(grid), dim3(kThreads), 0, st, (const float *)x->data, (float *)y->data, ip, d));
    } else {
        const unsigned grid = grid_for(numel(y));
        if (x->dtype == RELAY_BF16) RELAY_CUDA(launch_pdl(max_pool_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st, (const __nv_bfloat16 *)x->data, (__nv_bfloat16 *)y->data, ip, d));
        else RELAY_CUDA(launch_pdl(max_pool_kernel<float>, dim3(grid), dim3(kThreads), 0, st, (const float *)x->data, (float *)y->data, ip, d));
    }
    return check_launch("max_pool2d");
}

extern "C" relay_status_t relay_max_pool2d_grad(const relay_tensor_t *idx, const relay_tensor_t *dy, const relay_pool2d_attrs_t *attrs,
                                                const relay_tensor_t *dx, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(idx, "idx"));
    RELAY_TRY(check_not_null(dy, "dy"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(dx, "dx"));
    PoolDims d{};
    RELAY_TRY(check_pool(dx, attrs, &d));                    // dx has the type of the pooled input
    RELAY_TRY(check_type(idx, "idx")); RELAY_TRY(check_type(dy, "dy"));
    RELAY_TRY(check_rank(idx, 4, "idx")); RELAY_TRY(check_rank(dy, 4, "dy"));
    RELAY_TRY(check_dtype(idx, RELAY_I32, "idx"));
    RELAY_TRY(check_dtype(dy, dx->dtype, "dy"));
    RELAY_TRY(check_layout(dy, RELAY_NCHW, RELAY_ROWMAJOR, "dy"));
    RELAY_TRY(check_shape(idx, {dx->shape[0], dx->shape[1], (int64_t)d.P, (int64_t)d.Q}, "idx"));
    RELAY_TRY(check_shape(dy, {dx->shape[0], dx->shape[1], (int64_t)d.P, (int64_t)d.Q}, "dy"));
    RELAY_TRY(check_data(idx, "idx")); RELAY_TRY(check_data(dy, "dy")); RELAY_TRY(check_data(dx, "dx"));
    const relay_tensor_t *outs[1] = {dx}, *ins[2] = {idx, dy};
    RELAY_TRY(check_no_overlap(outs, 1, ins, 2));
    if (numel(dx) == 0) return RELAY_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int32_t *ip = (const int32_t *)idx->data;
    if (fast_2x2(d)) {
        const unsigned grid = grid_for((d.planes * d.P * (d.W / 8) + kPer - 1) / kPer);
        if (dx->dtype == RELAY_BF16) RELAY_CUDA(launch_pdl(max_pool_2x2_grad_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st, ip, (const __nv_bfloat16 *)dy->data, (__nv_bfloat16 *)dx->data, d));
        else RELAY_CUDA(launch_pdl(max_pool_2x2_grad_kernel<float>, dim3(grid), dim3(kThreads), 0, st, ip, (const float *)dy->data, (float *)dx->data, d));
    } else {
        const unsigned grid = grid_for(numel(dx));
        if (dx->dtype == RELAY_BF16) RELAY_CUDA(launch_pdl(max_pool_grad_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st, ip, (const __nv_bfloat16 *)dy->data, (__nv_bfloat16 *)dx->data, d));
        else RELAY_CUDA(launch_pdl(max_pool_grad_kernel<float>, dim3(grid), dim3(kThreads), 0, st, ip, (const float *)dy->data, (float *)dx->data, d));
    }
    return check_launch("max_pool2d_grad");
}
