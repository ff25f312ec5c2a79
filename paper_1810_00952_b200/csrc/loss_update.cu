// Softmax cross-entropy loss, its gradient group, and the SGD parameter update (Fig. 3 of the paper:
// relay.softmax_cross_entropy, relay.update_model_params; Section 4.2 for the gradient group).
// All three are HBM-bound: every input element is read once, every output element written once.
#include <algorithm>

#include "common.h"
#include "ewise_kernels.cuh"

namespace relay {
namespace {

constexpr int kThreads = 256;
constexpr int kCache = 4;          // 16-byte vectors (or scalars) of a row that a thread keeps in registers

// V consecutive values of type TT as floats
template <typename TT, int V>
__device__ __forceinline__ void load_vals(const TT *p, float (&f)[V])
{
    if constexpr (V == 1) {
        if constexpr (sizeof(TT) == 2) f[0] = __bfloat162float(*p);
        else f[0] = *p;
    } else if constexpr (sizeof(TT) * V == 16) {
        unpack(ld_stream(p), f);
    } else {                        // f32 values beside a bf16 vector of 8
        static_assert(sizeof(TT) == 4 && V == 8, "unsupported vector shape");
        float a[4], b[4];
        unpack(ld_stream(p), a);
        unpack(ld_stream(p + 4), b);
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[i] = a[i]; f[4 + i] = b[i]; }
    }
}
template <typename T, int V>
__device__ __forceinline__ void store_vals(T *p, const float (&f)[V])
{
    if constexpr (V == 1) {
        if constexpr (sizeof(T) == 2) *p = __float2bfloat16_rn(f[0]);
        else *p = f[0];
    } else {
        st_stream(p, pack(f));
    }
}

// V consecutive values kept as loaded (packed), so that a cached bf16 vector costs 4 registers, not 8
template <typename TT, int V>
struct Raw {
    static constexpr int N = (sizeof(TT) * V + 15) / 16;
    uint4 q[N];
};
template <typename TT>
struct Raw<TT, 1> {
    float q[1];
};
template <typename TT, int V>
__device__ __forceinline__ void load_raw(const TT *p, Raw<TT, V> &r)
{
    if constexpr (V == 1) {
        load_vals<TT, 1>(p, r.q);
    } else {
#pragma unroll
        for (int i = 0; i < Raw<TT, V>::N; ++i) r.q[i] = ld_stream(reinterpret_cast<const uint4 *>(p) + i);
    }
}
template <typename TT, int V>
__device__ __forceinline__ void to_float(const Raw<TT, V> &r, float (&f)[V])
{
    if constexpr (V == 1) {
        f[0] = r.q[0];
    } else if constexpr (Raw<TT, V>::N == 1) {
        unpack(r.q[0], f);
    } else {
        float a[4], b[4];
        unpack(r.q[0], a);
        unpack(r.q[1], b);
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[i] = a[i]; f[4 + i] = b[i]; }
    }
}

template <bool FAST> __device__ __forceinline__ float exp_(float x) { return FAST ? __expf(x) : expf(x); }
template <bool FAST> __device__ __forceinline__ float log_(float x) { return FAST ? __logf(x) : logf(x); }

// largest of the V values of a packed vector
template <typename T, int V>
__device__ __forceinline__ float raw_max(const Raw<T, V> &r)
{
    if constexpr (V == 1) {
        return r.q[0];
    } else if constexpr (sizeof(T) == 2) {          // bf16 pairs: the maximum of bf16 values is exact in bf16
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&r.q[0]);
        const __nv_bfloat162 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
        return fmaxf(__low2float(m), __high2float(m));
    } else {
        float f[V];
        to_float<T, V>(r, f);
        float m = f[0];
#pragma unroll
        for (int j = 1; j < V; ++j) m = fmaxf(m, f[j]);
        return m;
    }
}

// Combines one value per thread over the TPR threads of a row; every thread gets the result.
// `slot` is a shared array of kThreads / 32 floats used by the block-wide form only.
template <int TPR, bool MAX>
__device__ __forceinline__ float row_combine(float v, float *slot)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = MAX ? fmaxf(v, o) : v + o;
    }
    if constexpr (TPR > 32) {
        if ((threadIdx.x & 31) == 0) slot[threadIdx.x >> 5] = v;
        __syncthreads();
        v = slot[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) v = MAX ? fmaxf(v, slot[w]) : v + slot[w];     // fixed order
    }
    return v;
}

// Sums of three values at once (one barrier for the three); `slot` holds 3 * kThreads / 32 floats.
template <int TPR>
__device__ __forceinline__ void row_sum3(float &a, float &b, float &c, float *slot)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, off);
        b += __shfl_xor_sync(0xffffffffu, b, off);
        c += __shfl_xor_sync(0xffffffffu, c, off);
    }
    if constexpr (TPR > 32) {
        constexpr int W = kThreads / 32;
        if ((threadIdx.x & 31) == 0) { slot[threadIdx.x >> 5] = a; slot[W + (threadIdx.x >> 5)] = b; slot[2 * W + (threadIdx.x >> 5)] = c; }
        __syncthreads();
        a = slot[0]; b = slot[W]; c = slot[2 * W];
#pragma unroll
        for (int w = 1; w < W; ++w) { a += slot[w]; b += slot[W + w]; c += slot[2 * W + w]; }     // fixed order
    }
}

// One row per TPR threads (a warp, or the whole block).  z and t are read once: the first kCache vectors
// of each thread stay packed in registers, and only rows longer than TPR * kCache vectors re-read the
// rest (from L2).  Phase A: row maximum m.  Phase B: s = sum exp(z - m), st = sum t, stz = sum t (z - m);
// loss = st log s - stz.  Phase C (gradient only): dz = dl (exp(z - m) st / s - t).
template <typename T, typename TT, int TPR, bool VEC, bool GRAD>
__global__ void __launch_bounds__(kThreads)
softmax_xent_kernel(const T *__restrict__ z, const TT *__restrict__ t, const float *__restrict__ dloss, float *__restrict__ loss,
                    T *__restrict__ dz, int64_t B, int64_t C)
{
    constexpr bool FAST = sizeof(T) == 2;
    constexpr int V = VEC ? VecN<T>::N : 1;
    constexpr int RPB = kThreads / TPR;
    __shared__ float slots[4][kThreads / 32];
    const int lane = threadIdx.x % TPR;
    const int64_t row = (int64_t)blockIdx.x * RPB + threadIdx.x / TPR;
    const bool live = row < B;
    const int64_t nvec = C / V;
    const int64_t rest0 = lane + (int64_t)kCache * TPR;
    pdl_wait();

    const T *zr = z + (live ? row : 0) * C;
    const TT *tr = t + (live ? row : 0) * C;
    Raw<T, V> zc[kCache];
    Raw<TT, V> tc[kCache];
    float m = -INFINITY;
    if (live) {
#pragma unroll
        for (int k = 0; k < kCache; ++k) {                  // all loads of the thread are issued before any use
            const int64_t vi = lane + (int64_t)k * TPR;
            if (vi < nvec) {
                load_raw<T, V>(zr + vi * V, zc[k]);
                load_raw<TT, V>(tr + vi * V, tc[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < kCache; ++k)
            if (lane + (int64_t)k * TPR < nvec) m = fmaxf(m, raw_max<T, V>(zc[k]));
        for (int64_t vi = rest0; vi < nvec; vi += TPR) {
            Raw<T, V> r;
            load_raw<T, V>(zr + vi * V, r);
            m = fmaxf(m, raw_max<T, V>(r));
        }
    }
    m = row_combine<TPR, true>(m, slots[0]);

    float s = 0.0f, st = 0.0f, stz = 0.0f;
    auto sums = [&](const float (&zz)[V], const float (&tt)[V]) {
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float d = zz[j] - m;
            s += exp_<FAST>(d);
            st += tt[j];
            stz = fmaf(tt[j], d, stz);
        }
    };
    if (live) {
#pragma unroll
        for (int k = 0; k < kCache; ++k) {
            if (lane + (int64_t)k * TPR < nvec) {
                float zz[V], tt[V];
                to_float<T, V>(zc[k], zz);
                to_float<TT, V>(tc[k], tt);
                sums(zz, tt);
            }
        }
        for (int64_t vi = rest0; vi < nvec; vi += TPR) {
            float zz[V], tt[V];
            load_vals<T, V>(zr + vi * V, zz);
            load_vals<TT, V>(tr + vi * V, tt);
            sums(zz, tt);
        }
    }
    row_sum3<TPR>(s, st, stz, slots[1]);
    if (!live) return;
    if (loss != nullptr && lane == 0) loss[row] = fmaf(st, log_<FAST>(s), -stz);     // sum t (log s - (z - m))
    if constexpr (GRAD) {
        const float dl = dloss[row];
        const float scale = dl * st / s;                                             // dl * sum t / sum exp
        T *dr = dz + row * C;
#pragma unroll
        for (int k = 0; k < kCache; ++k) {
            const int64_t vi = lane + (int64_t)k * TPR;
            if (vi < nvec) {
                float zz[V], tt[V], o[V];
                to_float<T, V>(zc[k], zz);
                to_float<TT, V>(tc[k], tt);
#pragma unroll
                for (int j = 0; j < V; ++j) o[j] = fmaf(scale, exp_<FAST>(zz[j] - m), -dl * tt[j]);
                store_vals<T, V>(dr + vi * V, o);
            }
        }
        for (int64_t vi = rest0; vi < nvec; vi += TPR) {
            float zz[V], tt[V], o[V];
            load_vals<T, V>(zr + vi * V, zz);
            load_vals<TT, V>(tr + vi * V, tt);
#pragma unroll
            for (int j = 0; j < V; ++j) o[j] = fmaf(scale, exp_<FAST>(zz[j] - m), -dl * tt[j]);
            store_vals<T, V>(dr + vi * V, o);
        }
    }
}

template <typename T, typename TT, bool GRAD>
relay_status_t launch_xent_typed(const void *z, const void *t, const float *dloss, float *loss, void *dz, int64_t B, int64_t C,
                                 cudaStream_t st)
{
    constexpr int V = VecN<T>::N;
    const bool vec = C % V == 0;
    const int64_t units = vec ? C / V : C;
    const bool warp_row = units <= 32 * kCache;              // the row fits the registers of one warp
    const int rpb = warp_row ? kThreads / 32 : 1;
    const dim3 grid((unsigned)((B + rpb - 1) / rpb)), block(kThreads);
#define XENT(TPR, VEC)                                                                                                          \
    RELAY_CUDA(launch_pdl(softmax_xent_kernel<T, TT, TPR, VEC, GRAD>, grid, block, 0, st, (const T *)z, (const TT *)t, dloss, loss, \
                          (T *)dz, B, C))
    if (warp_row && vec) XENT(32, true);
    else if (warp_row) XENT(32, false);
    else if (vec) XENT(kThreads, true);
    else XENT(kThreads, false);
#undef XENT
    return check_launch("softmax_xent");
}

template <bool GRAD>
relay_status_t launch_xent(int32_t zt, int32_t tt, const void *z, const void *t, const float *dloss, float *loss, void *dz,
                           int64_t B, int64_t C, cudaStream_t st)
{
    if (zt == RELAY_F32) return launch_xent_typed<float, float, GRAD>(z, t, dloss, loss, dz, B, C, st);
    if (tt == RELAY_BF16) return launch_xent_typed<__nv_bfloat16, __nv_bfloat16, GRAD>(z, t, dloss, loss, dz, B, C, st);
    return launch_xent_typed<__nv_bfloat16, float, GRAD>(z, t, dloss, loss, dz, B, C, st);
}

// ---- SGD: up to kSgdMax parameters per launch --------------------------------------------------------
constexpr int kSgdMax = 8;
constexpr int kSgdVecs = 4;        // 16-byte vectors of the parameter per thread
struct SgdTable {
    void *p[kSgdMax];
    const void *g[kSgdMax];
    long long n[kSgdMax];
    unsigned blk0[kSgdMax + 1];    // first block of each parameter
    int kind[kSgdMax];             // 0: f32 p, f32 g   1: bf16 p, bf16 g   2: bf16 p, f32 g
    int count;
    float lr;
};

template <typename PT, typename GT>
__device__ __forceinline__ void sgd_block(PT *__restrict__ p, const GT *__restrict__ g, long long n, unsigned blk, float lr)
{
    constexpr int V = VecN<PT>::N;
    const long long v0 = (long long)blk * (kThreads * kSgdVecs) + threadIdx.x;
    float pv[kSgdVecs][V], gv[kSgdVecs][V];
#pragma unroll
    for (int i = 0; i < kSgdVecs; ++i) {
        const long long e = (v0 + (long long)i * kThreads) * V;
        if (e + V <= n) {
            load_vals<PT, V>(p + e, pv[i]);
            load_vals<GT, V>(g + e, gv[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < kSgdVecs; ++i) {
        const long long e = (v0 + (long long)i * kThreads) * V;
        if (e + V <= n) {
#pragma unroll
            for (int j = 0; j < V; ++j) pv[i][j] = fmaf(-lr, gv[i][j], pv[i][j]);
            store_vals<PT, V>(p + e, pv[i]);
        } else {
            for (long long k = e; k < n; ++k) {                 // ragged end of the tensor: at most V - 1 elements
                float a[1], b[1];
                load_vals<PT, 1>(p + k, a);
                load_vals<GT, 1>(g + k, b);
                a[0] = fmaf(-lr, b[0], a[0]);
                store_vals<PT, 1>(p + k, a);
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) sgd_update_kernel(const __grid_constant__ SgdTable tb)
{
    int k = 0;
    while (k + 1 < tb.count && blockIdx.x >= tb.blk0[k + 1]) ++k;
    const unsigned blk = blockIdx.x - tb.blk0[k];
    pdl_wait();
    switch (tb.kind[k]) {
    case 0: sgd_block<float, float>((float *)tb.p[k], (const float *)tb.g[k], tb.n[k], blk, tb.lr); break;
    case 1: sgd_block<__nv_bfloat16, __nv_bfloat16>((__nv_bfloat16 *)tb.p[k], (const __nv_bfloat16 *)tb.g[k], tb.n[k], blk, tb.lr); break;
    default: sgd_block<__nv_bfloat16, float>((__nv_bfloat16 *)tb.p[k], (const float *)tb.g[k], tb.n[k], blk, tb.lr); break;
    }
}

// type relation of the loss on concrete descriptors
relay_status_t check_xent(const relay_tensor_t *z, const relay_tensor_t *t, int64_t *B, int64_t *C)
{
    RELAY_TRY(check_type(z, "scores"));
    RELAY_TRY(check_type(t, "targets"));
    RELAY_TRY(check_rank(z, 2, "scores"));
    RELAY_TRY(check_rank(t, 2, "targets"));
    if (!is_float(z->dtype)) return fail(RELAY_ERR_DTYPE, "scores: base type %s, needs f32 or bf16", dtype_name(z->dtype));
    if (t->dtype != z->dtype && t->dtype != RELAY_F32)
        return fail(RELAY_ERR_DTYPE, "targets: base type %s, needs %s or f32", dtype_name(t->dtype), dtype_name(z->dtype));
    RELAY_TRY(check_layout(z, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "scores"));
    RELAY_TRY(check_layout(t, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "targets"));
    RELAY_TRY(check_shape(t, {z->shape[0], z->shape[1]}, "targets"));
    if (z->shape[1] == 0) return fail(RELAY_ERR_SHAPE, "scores: a row without classes has no softmax");
    *B = z->shape[0]; *C = z->shape[1];
    return RELAY_OK;
}

relay_status_t check_vector_f32(const relay_tensor_t *v, int64_t n, const char *name)
{
    RELAY_TRY(check_type(v, name));
    RELAY_TRY(check_rank(v, 1, name));
    RELAY_TRY(check_dtype(v, RELAY_F32, name));
    RELAY_TRY(check_shape(v, {n}, name));
    return RELAY_OK;
}

}  // namespace
}  // namespace relay

using namespace relay;

extern "C" relay_status_t relay_infer_softmax_xent(const relay_tensor_t *scores, const relay_tensor_t *targets, relay_tensor_t *loss)
{
    clear_error();
    RELAY_TRY(check_not_null(scores, "scores"));
    RELAY_TRY(check_not_null(targets, "targets"));
    RELAY_TRY(check_not_null(loss, "loss"));
    int64_t B, C;
    RELAY_TRY(check_xent(scores, targets, &B, &C));
    loss->data = nullptr; loss->dtype = RELAY_F32; loss->rank = 1; loss->layout = RELAY_ROWMAJOR;
    for (int d = 0; d < 6; ++d) loss->shape[d] = d == 0 ? B : 1;
    return RELAY_OK;
}

extern "C" relay_status_t relay_softmax_xent(const relay_tensor_t *scores, const relay_tensor_t *targets, const relay_tensor_t *loss,
                                             void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(scores, "scores"));
    RELAY_TRY(check_not_null(targets, "targets"));
    RELAY_TRY(check_not_null(loss, "loss"));
    int64_t B, C;
    RELAY_TRY(check_xent(scores, targets, &B, &C));
    RELAY_TRY(check_vector_f32(loss, B, "loss"));
    RELAY_TRY(check_data(scores, "scores"));
    RELAY_TRY(check_data(targets, "targets"));
    RELAY_TRY(check_data(loss, "loss"));
    const relay_tensor_t *outs[1] = {loss}, *ins[2] = {scores, targets};
    RELAY_TRY(check_no_overlap(outs, 1, ins, 2));
    if (B == 0) return RELAY_OK;
    return launch_xent<false>(scores->dtype, targets->dtype, scores->data, targets->data, nullptr, (float *)loss->data, nullptr, B, C,
                              (cudaStream_t)stream);
}

extern "C" relay_status_t relay_softmax_xent_grad(const relay_tensor_t *scores, const relay_tensor_t *targets,
                                                  const relay_tensor_t *dloss, const relay_tensor_t *loss,
                                                  const relay_tensor_t *dscores, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(scores, "scores"));
    RELAY_TRY(check_not_null(targets, "targets"));
    RELAY_TRY(check_not_null(dloss, "dloss"));
    RELAY_TRY(check_not_null(dscores, "dscores"));
    int64_t B, C;
    RELAY_TRY(check_xent(scores, targets, &B, &C));
    RELAY_TRY(check_vector_f32(dloss, B, "dloss"));
    if (loss) RELAY_TRY(check_vector_f32(loss, B, "loss"));
    RELAY_TRY(check_type(dscores, "dscores"));
    RELAY_TRY(check_rank(dscores, 2, "dscores"));
    RELAY_TRY(check_dtype(dscores, scores->dtype, "dscores"));
    RELAY_TRY(check_layout(dscores, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "dscores"));
    RELAY_TRY(check_shape(dscores, {B, C}, "dscores"));
    const relay_tensor_t *ins[3] = {scores, targets, dloss}, *outs[2] = {dscores, loss};
    for (int i = 0; i < 3; ++i) RELAY_TRY(check_data(ins[i], "input"));
    for (int i = 0; i < 2; ++i) if (outs[i]) RELAY_TRY(check_data(outs[i], "output"));
    RELAY_TRY(check_no_overlap(outs, 2, ins, 3));
    if (B == 0) return RELAY_OK;
    return launch_xent<true>(scores->dtype, targets->dtype, scores->data, targets->data, (const float *)dloss->data,
                             loss ? (float *)loss->data : nullptr, dscores->data, B, C, (cudaStream_t)stream);
}

extern "C" relay_status_t relay_sgd_update(const relay_tensor_t *const *params, const relay_tensor_t *const *grads, int32_t n_params,
                                           float lr, void *stream)
{
    clear_error();
    if (n_params < 0) return fail(RELAY_ERR_ATTR, "n_params = %d", n_params);
    if (n_params == 0) return RELAY_OK;
    RELAY_TRY(check_not_null(params, "params"));
    RELAY_TRY(check_not_null(grads, "grads"));
    for (int k = 0; k < n_params; ++k) { RELAY_TRY(check_not_null(params[k], "params[k]")); RELAY_TRY(check_not_null(grads[k], "grads[k]")); }
    for (int k = 0; k < n_params; ++k) { RELAY_TRY(check_type(params[k], "params[k]")); RELAY_TRY(check_type(grads[k], "grads[k]")); }
    for (int k = 0; k < n_params; ++k) {
        const relay_tensor_t *p = params[k], *g = grads[k];
        if (g->rank != p->rank) return fail(RELAY_ERR_RANK, "grads[%d]: rank %d, parameter has rank %d", k, g->rank, p->rank);
    }
    for (int k = 0; k < n_params; ++k) {
        const relay_tensor_t *p = params[k], *g = grads[k];
        if (!is_float(p->dtype)) return fail(RELAY_ERR_DTYPE, "params[%d]: base type %s, needs f32 or bf16", k, dtype_name(p->dtype));
        if (g->dtype != p->dtype && g->dtype != RELAY_F32)
            return fail(RELAY_ERR_DTYPE, "grads[%d]: base type %s, needs %s or f32", k, dtype_name(g->dtype), dtype_name(p->dtype));
    }
    for (int k = 0; k < n_params; ++k)
        for (int d = 0; d < params[k]->rank; ++d)
            if (params[k]->shape[d] != grads[k]->shape[d])
                return fail(RELAY_ERR_SHAPE, "grads[%d]: axis %d has %lld entries, parameter has %lld", k, d, (long long)grads[k]->shape[d],
                            (long long)params[k]->shape[d]);
    for (int k = 0; k < n_params; ++k) { RELAY_TRY(check_data(params[k], "params[k]")); RELAY_TRY(check_data(grads[k], "grads[k]")); }
    // a parameter is read and written: it may overlap neither another parameter nor any gradient
    RELAY_TRY(check_no_overlap(params, n_params, grads, n_params));
    if (!(lr == lr)) return fail(RELAY_ERR_ATTR, "learning rate is NaN");

    cudaStream_t st = (cudaStream_t)stream;
    for (int first = 0; first < n_params; first += kSgdMax) {
        SgdTable tb{};
        tb.lr = lr;
        unsigned blocks = 0;
        for (int k = first; k < std::min(n_params, first + kSgdMax); ++k) {
            const relay_tensor_t *p = params[k], *g = grads[k];
            const long long n = numel(p);
            if (n == 0) continue;
            const int i = tb.count++;
            tb.p[i] = p->data; tb.g[i] = g->data; tb.n[i] = n;
            tb.kind[i] = p->dtype == RELAY_F32 ? 0 : g->dtype == RELAY_BF16 ? 1 : 2;
            const long long per_block = (long long)kThreads * kSgdVecs * (p->dtype == RELAY_F32 ? 4 : 8);
            const long long nb = (n + per_block - 1) / per_block;
            if (nb + blocks > 0x7fffffffLL) return fail(RELAY_ERR_UNSUPPORTED, "parameter set too large for one launch");
            tb.blk0[i] = blocks;
            blocks += (unsigned)nb;
            tb.blk0[i + 1] = blocks;
        }
        if (blocks == 0) continue;
        RELAY_CUDA(launch_pdl(sgd_update_kernel, dim3(blocks), dim3(kThreads), 0, st, tb));
        RELAY_TRY(check_launch("sgd_update"));
    }
    return RELAY_OK;
}
