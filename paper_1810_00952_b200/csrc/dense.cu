// Dense anchor with fused bias + activation, and its gradient group (host entry points).
#include "ewise_host.h"
#include "gemm.h"

namespace relay {

// scalar routes for shapes whose rows are not whole 16-byte vectors
template <typename T>
__global__ void act_grad_scalar_kernel(const T *__restrict__ dy, const T *__restrict__ y, T *__restrict__ dz, int64_t n, int act)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        float yv, dv;
        if constexpr (sizeof(T) == 2) { yv = __bfloat162float(y[i]); dv = __bfloat162float(dy[i]); }
        else { yv = y[i]; dv = dy[i]; }
        float g = act == RELAY_ACT_RELU ? (yv > 0.0f ? 1.0f : 0.0f)
                : act == RELAY_ACT_TANH ? 1.0f - yv * yv
                : act == RELAY_ACT_SIGMOID ? yv * (1.0f - yv) : 1.0f;
        if constexpr (sizeof(T) == 2) dz[i] = __float2bfloat16_rn(dv * g);
        else dz[i] = dv * g;
    }
}
template <typename T>
__global__ void colsum_scalar_kernel(const T *__restrict__ x, int64_t rows, int64_t cols, float *__restrict__ out)
{
    int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= cols) return;
    float s = 0.0f;
    for (int64_t r = 0; r < rows; ++r) {
        if constexpr (sizeof(T) == 2) s += __bfloat162float(x[r * cols + c]);
        else s += x[r * cols + c];
    }
    out[c] = s;
}

// dz = dy (.) act'(y) and db = column sums of dz, for any [rows, cols]
relay_status_t act_grad_any(int32_t dt, const void *dy, const void *y, void *dz, float *db, float *partials, int64_t rows,
                            int64_t cols, int act, cudaStream_t st)
{
    const int vec = dt == RELAY_BF16 ? 8 : 4;
    if (cols % vec == 0) return launch_act_grad(dt, dy, y, dz, db, partials, rows, cols, act, st);
    const int64_t n = rows * cols;
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((n + 255) / 256, 148 * 8));
    if (dt == RELAY_BF16) act_grad_scalar_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16 *)dy, (const __nv_bfloat16 *)y, (__nv_bfloat16 *)dz, n, act);
    else act_grad_scalar_kernel<<<grid, 256, 0, st>>>((const float *)dy, (const float *)y, (float *)dz, n, act);
    RELAY_TRY(check_launch("act_grad_scalar"));
    if (db) {
        const unsigned g2 = (unsigned)((cols + 127) / 128);
        if (dt == RELAY_BF16) colsum_scalar_kernel<<<g2, 128, 0, st>>>((const __nv_bfloat16 *)dz, rows, cols, db);
        else colsum_scalar_kernel<<<g2, 128, 0, st>>>((const float *)dz, rows, cols, db);
        RELAY_TRY(check_launch("colsum_scalar"));
    }
    return RELAY_OK;
}

// M counts the rows of all leading batch axes together: a batch of products with one weight matrix is one
// product over the stacked rows (Section 5.2: batching adds a leading axis to every tensor of the program)
struct DenseDims {
    int64_t M, K, N;
    int32_t dt;
    int rank;                         // of x, y, dy, dx
    int64_t xs[RELAY_MAX_RANK];       // x's shape;  ys: the same with N as last extent
    int64_t ys[RELAY_MAX_RANK];
};

// type relation of the dense anchor on concrete descriptors, in the documented check order
static relay_status_t check_dense(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b, DenseDims *d)
{
    relay_tensor_t yt;
    RELAY_TRY(relay_infer_dense(x, w, &yt));
    if (b) {
        RELAY_TRY(check_type(b, "b"));
        RELAY_TRY(check_rank(b, 1, "b"));
        if (b->dtype != x->dtype && b->dtype != RELAY_F32)
            return fail(RELAY_ERR_DTYPE, "b: base type %s, needs %s or f32", dtype_name(b->dtype), dtype_name(x->dtype));
        RELAY_TRY(check_shape(b, {w->shape[1]}, "b"));
    }
    d->rank = x->rank;
    d->M = 1;
    for (int i = 0; i < x->rank; ++i) { d->xs[i] = x->shape[i]; d->ys[i] = yt.shape[i]; if (i < x->rank - 1) d->M *= x->shape[i]; }
    d->K = x->shape[x->rank - 1]; d->N = w->shape[1]; d->dt = x->dtype;
    return RELAY_OK;
}

static size_t dense_grad_ws(const DenseDims &d, size_t *dz_bytes)
{
    *dz_bytes = align_up((size_t)d.M * d.N * dtype_size(d.dt), 256);
    const int vec = d.dt == RELAY_BF16 ? 8 : 4;
    size_t part = d.N % vec == 0 ? (size_t)colsum_slices(d.M, d.N, d.dt) * d.N * sizeof(float) : 0;
    return *dz_bytes + align_up(part, 256);
}

}  // namespace relay

using namespace relay;

extern "C" size_t relay_workspace_bytes_dense_act(const relay_tensor_t *, const relay_tensor_t *) { return 0; }

extern "C" size_t relay_workspace_bytes_dense_act_grad(const relay_tensor_t *x, const relay_tensor_t *w)
{
    DenseDims d{};
    if (!x || !w || check_dense(x, w, nullptr, &d) != RELAY_OK) return 0;
    size_t dzb;
    return dense_grad_ws(d, &dzb);
}

extern "C" relay_status_t relay_fused_dense_act(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b,
                                                int32_t act, const relay_tensor_t *y, void *ws, size_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(y, "y"));
    DenseDims d{};
    RELAY_TRY(check_dense(x, w, b, &d));
    RELAY_TRY(check_type(y, "y"));
    RELAY_TRY(check_rank(y, d.rank, "y"));
    RELAY_TRY(check_dtype(y, d.dt, "y"));
    RELAY_TRY(check_layout(y, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "y"));
    RELAY_TRY(check_shape_n(y, d.ys, d.rank, "y"));
    if (act < RELAY_ACT_NONE || act > RELAY_ACT_SIGMOID) return fail(RELAY_ERR_ATTR, "unknown activation %d", act);
    RELAY_TRY(check_data(x, "x"));
    RELAY_TRY(check_data(w, "w"));
    if (b) RELAY_TRY(check_data(b, "b"));
    RELAY_TRY(check_data(y, "y"));
    const relay_tensor_t *outs[1] = {y}, *ins[3] = {x, w, b};
    RELAY_TRY(check_no_overlap(outs, 1, ins, 3));
    if (dense_small_eligible(d.M, d.K, d.N, d.dt))
        return launch_dense_small_fwd(d.dt, x->data, w->data, b ? b->data : nullptr, b ? b->dtype : RELAY_F32, y->data, d.M, d.K, d.N, act,
                                      (cudaStream_t)stream);
    GemmDesc g;
    g.M = d.M; g.N = d.N; g.K = d.K;
    g.a = x->data; g.a_sm = d.K; g.a_sk = 1;
    g.b = w->data; g.b_sk = d.N; g.b_sn = 1;
    g.c = y->data; g.ldc = d.N;
    g.in_dtype = g.out_dtype = d.dt;
    g.bias = b ? b->data : nullptr; g.bias_dtype = b ? b->dtype : RELAY_F32;
    g.act = act;
    return launch_gemm(g, (cudaStream_t)stream);
}

extern "C" relay_status_t relay_fused_dense_act_grad(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *y,
                                                     const relay_tensor_t *dy, int32_t act, const relay_tensor_t *dx,
                                                     const relay_tensor_t *dw, const relay_tensor_t *db, void *ws, size_t ws_bytes,
                                                     void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(y, "y"));
    RELAY_TRY(check_not_null(dy, "dy"));
    RELAY_TRY(check_not_null(dw, "dw"));
    DenseDims d{};
    RELAY_TRY(check_dense(x, w, nullptr, &d));
    const relay_tensor_t *mn[2] = {y, dy};
    const char *mn_name[2] = {"y", "dy"};
    for (int i = 0; i < 2; ++i) { RELAY_TRY(check_type(mn[i], mn_name[i])); RELAY_TRY(check_rank(mn[i], d.rank, mn_name[i])); }
    if (dx) { RELAY_TRY(check_type(dx, "dx")); RELAY_TRY(check_rank(dx, d.rank, "dx")); }
    RELAY_TRY(check_type(dw, "dw")); RELAY_TRY(check_rank(dw, 2, "dw"));
    if (db) { RELAY_TRY(check_type(db, "db")); RELAY_TRY(check_rank(db, 1, "db")); }
    for (int i = 0; i < 2; ++i) RELAY_TRY(check_dtype(mn[i], d.dt, mn_name[i]));
    if (dx) RELAY_TRY(check_dtype(dx, d.dt, "dx"));
    RELAY_TRY(check_dtype(dw, d.dt, "dw"));
    if (db) RELAY_TRY(check_dtype(db, RELAY_F32, "db"));
    for (int i = 0; i < 2; ++i) RELAY_TRY(check_shape_n(mn[i], d.ys, d.rank, mn_name[i]));
    if (dx) RELAY_TRY(check_shape_n(dx, d.xs, d.rank, "dx"));
    RELAY_TRY(check_shape(dw, {d.K, d.N}, "dw"));
    if (db) RELAY_TRY(check_shape(db, {d.N}, "db"));
    if (act < RELAY_ACT_NONE || act > RELAY_ACT_SIGMOID) return fail(RELAY_ERR_ATTR, "unknown activation %d", act);
    const relay_tensor_t *ins[4] = {x, w, y, dy}, *outs[3] = {dx, dw, db};
    for (int i = 0; i < 4; ++i) RELAY_TRY(check_data(ins[i], "input"));
    for (int i = 0; i < 3; ++i) if (outs[i]) RELAY_TRY(check_data(outs[i], "output"));
    RELAY_TRY(check_no_overlap(outs, 3, ins, 4));
    size_t dz_bytes;
    const size_t need = dense_grad_ws(d, &dz_bytes);
    RELAY_TRY(check_workspace(ws, ws_bytes, need));
    cudaStream_t st = (cudaStream_t)stream;
    if (d.M == 0 || d.N == 0 || d.K == 0) {
        // empty contraction: every partial is the zero tensor of its type (Fig. 5 Type-Zero)
        if (dx && numel(dx)) RELAY_CUDA(cudaMemsetAsync(dx->data, 0, nbytes(dx), st));
        if (numel(dw)) RELAY_CUDA(cudaMemsetAsync(dw->data, 0, nbytes(dw), st));
        if (db && numel(db)) RELAY_CUDA(cudaMemsetAsync(db->data, 0, nbytes(db), st));
        return RELAY_OK;
    }

    if (dense_small_eligible(d.M, d.K, d.N, d.dt))
        return launch_dense_small_grad(d.dt, x->data, w->data, y->data, dy->data, dx ? dx->data : nullptr, dw->data, db ? (float *)db->data : nullptr,
                                       d.M, d.K, d.N, act, st);
    void *dz = ws;
    float *partials = (float *)((char *)ws + dz_bytes);
    RELAY_TRY(act_grad_any(d.dt, dy->data, y->data, dz, db ? (float *)db->data : nullptr, partials, d.M, d.N, act, st));

    GemmDesc g;
    g.in_dtype = g.out_dtype = d.dt;
    if (dx) {  // dx[m,k] = sum_n dZ[m,n] w[k,n]
        g.M = d.M; g.N = d.K; g.K = d.N;
        g.a = dz; g.a_sm = d.N; g.a_sk = 1;
        g.b = w->data; g.b_sk = 1; g.b_sn = d.N;
        g.c = dx->data; g.ldc = d.K;
        RELAY_TRY(launch_gemm(g, st));
    }
    // dw[k,n] = sum_m x[m,k] dZ[m,n]
    g.M = d.K; g.N = d.N; g.K = d.M;
    g.a = x->data; g.a_sm = 1; g.a_sk = d.K;
    g.b = dz; g.b_sk = d.N; g.b_sn = 1;
    g.c = dw->data; g.ldc = d.N;
    return launch_gemm(g, st);
}

// The contraction under the dense groups as a call of its own: c = act(op(a) op(b) + bias) with either operand read
// transposed where it lies (the forward product, dx = dZ w^T and dw = x^T dZ are its three forms).
extern "C" relay_status_t relay_contract_act(const relay_tensor_t *a, int32_t trans_a, const relay_tensor_t *b, int32_t trans_b,
                                             const relay_tensor_t *bias, int32_t act, const relay_tensor_t *c, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(a, "a"));
    RELAY_TRY(check_not_null(b, "b"));
    RELAY_TRY(check_not_null(c, "c"));
    const relay_tensor_t *t3[3] = {a, b, c};
    const char *names[3] = {"a", "b", "c"};
    for (int i = 0; i < 3; ++i) { RELAY_TRY(check_type(t3[i], names[i])); RELAY_TRY(check_rank(t3[i], 2, names[i])); }
    if (bias) { RELAY_TRY(check_type(bias, "bias")); RELAY_TRY(check_rank(bias, 1, "bias")); }
    if (!is_float(a->dtype)) return fail(RELAY_ERR_DTYPE, "a: base type %s, needs f32 or bf16", dtype_name(a->dtype));
    RELAY_TRY(check_dtype(b, a->dtype, "b"));
    if (c->dtype != a->dtype && c->dtype != RELAY_F32) return fail(RELAY_ERR_DTYPE, "c: base type %s, needs %s or f32", dtype_name(c->dtype), dtype_name(a->dtype));
    if (bias && bias->dtype != a->dtype && bias->dtype != RELAY_F32)
        return fail(RELAY_ERR_DTYPE, "bias: base type %s, needs %s or f32", dtype_name(bias->dtype), dtype_name(a->dtype));
    for (int i = 0; i < 3; ++i) RELAY_TRY(check_layout(t3[i], RELAY_ROWMAJOR, RELAY_ROWMAJOR, names[i]));
    const int64_t M = trans_a ? a->shape[1] : a->shape[0], K = trans_a ? a->shape[0] : a->shape[1];
    const int64_t Kb = trans_b ? b->shape[1] : b->shape[0], N = trans_b ? b->shape[0] : b->shape[1];
    if (K != Kb) return fail(RELAY_ERR_SHAPE, "contraction lengths differ: op(a) has %lld columns, op(b) has %lld rows", (long long)K, (long long)Kb);
    RELAY_TRY(check_shape(c, {M, N}, "c"));
    if (bias) RELAY_TRY(check_shape(bias, {N}, "bias"));
    if (act < RELAY_ACT_NONE || act > RELAY_ACT_SIGMOID) return fail(RELAY_ERR_ATTR, "unknown activation %d", act);
    RELAY_TRY(check_data(a, "a"));
    RELAY_TRY(check_data(b, "b"));
    if (bias) RELAY_TRY(check_data(bias, "bias"));
    RELAY_TRY(check_data(c, "c"));
    const relay_tensor_t *outs[1] = {c}, *ins[3] = {a, b, bias};
    RELAY_TRY(check_no_overlap(outs, 1, ins, 3));
    cudaStream_t st = (cudaStream_t)stream;
    if (M == 0 || N == 0) return RELAY_OK;
    if (K == 0 && !bias && act == RELAY_ACT_NONE) { RELAY_CUDA(cudaMemsetAsync(c->data, 0, nbytes(c), st)); return RELAY_OK; }
    GemmDesc g;
    g.M = M; g.N = N; g.K = K;
    g.a = a->data; g.a_sm = trans_a ? 1 : a->shape[1]; g.a_sk = trans_a ? a->shape[1] : 1;
    g.b = b->data; g.b_sk = trans_b ? 1 : b->shape[1]; g.b_sn = trans_b ? b->shape[1] : 1;
    g.c = c->data; g.ldc = N;
    g.in_dtype = a->dtype; g.out_dtype = c->dtype;
    g.bias = bias ? bias->data : nullptr; g.bias_dtype = bias ? bias->dtype : RELAY_F32;
    g.act = act;
    return launch_gemm(g, st);
}
