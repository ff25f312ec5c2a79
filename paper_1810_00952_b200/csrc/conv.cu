// conv2d anchor with fused per-channel bias + activation, and its gradient group (host entry
// points): type relation, workspace plan, choice of kernel tier.
#include "conv.h"
#include "ewise_host.h"

namespace relay {

static relay_status_t check_conv(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b,
                                 const relay_conv2d_attrs_t *attrs, ConvDims *d)
{
    relay_tensor_t yt;
    RELAY_TRY(relay_infer_conv2d(x, w, attrs, &yt));
    if (b) {
        RELAY_TRY(check_type(b, "b"));
        RELAY_TRY(check_rank(b, 1, "b"));
        if (b->dtype != x->dtype && b->dtype != RELAY_F32)
            return fail(RELAY_ERR_DTYPE, "b: base type %s, needs %s or f32", dtype_name(b->dtype), dtype_name(x->dtype));
        RELAY_TRY(check_shape(b, {w->shape[0]}, "b"));
    }
    d->nhwc = x->layout == RELAY_NHWC;
    d->Nb = x->shape[0];
    if (d->nhwc) { d->H = x->shape[1]; d->W = x->shape[2]; d->C = x->shape[3]; d->P = yt.shape[1]; d->Q = yt.shape[2]; }
    else { d->C = x->shape[1]; d->H = x->shape[2]; d->W = x->shape[3]; d->P = yt.shape[2]; d->Q = yt.shape[3]; }
    d->O = w->shape[0]; d->R = w->shape[2]; d->S = w->shape[3];
    d->stride = attrs->stride; d->pad = attrs->pad; d->dt = x->dtype;
    return RELAY_OK;
}

// the operator type's shape of an activation tensor with `ch` channels and an h x w plane, in x's layout
static relay_status_t check_act_shape(const ConvDims &d, const relay_tensor_t *t, int64_t ch, int64_t h, int64_t w, const char *name)
{
    RELAY_TRY(check_layout(t, d.nhwc ? RELAY_NHWC : RELAY_NCHW, d.nhwc ? RELAY_NHWC : RELAY_NCHW, name));
    if (d.nhwc) return check_shape(t, {d.Nb, h, w, ch}, name);
    return check_shape(t, {d.Nb, ch, h, w}, name);
}

// NHWC tensors are converted to the kernels' NCHW through the workspace (the layout change is part of the call)
static size_t x_bytes(const ConvDims &d) { return align_up((size_t)(d.Nb * d.C * d.H * d.W) * dtype_size(d.dt), 256); }
static size_t y_bytes(const ConvDims &d) { return align_up((size_t)(d.Nb * d.O * d.P * d.Q) * dtype_size(d.dt), 256); }

// 2-D view of a dense tensor of `total` elements whose rows are whole 16-byte vectors, if any
static void flat_view(int64_t total, int32_t dt, int64_t *rows, int64_t *cols)
{
    const int vec = dt == RELAY_BF16 ? 8 : 4;
    for (int64_t c : {4096, 2048, 1024, 512, 256, 128, 64, 32, 16, 8, 4})
        if (c % vec == 0 && total % c == 0) { *rows = total / c; *cols = c; return; }
    *rows = 1; *cols = total;
}

static size_t conv_grad_ws(const ConvDims &d, size_t *dz_bytes)
{
    *dz_bytes = align_up((size_t)(d.Nb * d.O * d.P * d.Q) * dtype_size(d.dt), 256);
    if (conv_tc_eligible(d)) return conv_tc_grad_workspace(d);   // the tensor-core tier keeps dZ in its own layout
    return *dz_bytes + conv_dw_partial_bytes(d);                 // dZ, then the split sums of the weight gradient
}

}  // namespace relay

using namespace relay;

extern "C" size_t relay_workspace_bytes_conv2d_act(const relay_tensor_t *x, const relay_tensor_t *w, const relay_conv2d_attrs_t *attrs)
{
    ConvDims d;
    if (!x || !w || !attrs || check_conv(x, w, nullptr, attrs, &d) != RELAY_OK) return 0;
    const size_t inner = conv_tc_eligible(d) ? conv_tc_fwd_workspace(d) : 0;
    if (!d.nhwc) return inner;
    return inner + y_bytes(d) + (conv_tc_eligible(d) ? 0 : x_bytes(d));     // y in NCHW; x too unless the kernel reads NHWC itself
}

extern "C" size_t relay_workspace_bytes_conv2d_act_grad(const relay_tensor_t *x, const relay_tensor_t *w,
                                                        const relay_conv2d_attrs_t *attrs)
{
    ConvDims d;
    if (!x || !w || !attrs || check_conv(x, w, nullptr, attrs, &d) != RELAY_OK) return 0;
    size_t dzb;
    const size_t inner = conv_grad_ws(d, &dzb);
    return d.nhwc ? inner + 2 * x_bytes(d) + 2 * y_bytes(d) : inner;       // x, dx, y, dy in NCHW
}

extern "C" relay_status_t relay_fused_conv2d_act(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b,
                                                 const relay_conv2d_attrs_t *attrs, int32_t act, const relay_tensor_t *y, void *ws,
                                                 size_t ws_bytes, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(y, "y"));
    ConvDims d;
    RELAY_TRY(check_conv(x, w, b, attrs, &d));
    RELAY_TRY(check_type(y, "y"));
    RELAY_TRY(check_rank(y, 4, "y"));
    RELAY_TRY(check_dtype(y, d.dt, "y"));
    RELAY_TRY(check_act_shape(d, y, d.O, d.P, d.Q, "y"));
    if (act < RELAY_ACT_NONE || act > RELAY_ACT_SIGMOID) return fail(RELAY_ERR_ATTR, "unknown activation %d", act);
    RELAY_TRY(check_data(x, "x"));
    RELAY_TRY(check_data(w, "w"));
    if (b) RELAY_TRY(check_data(b, "b"));
    RELAY_TRY(check_data(y, "y"));
    const relay_tensor_t *outs[1] = {y}, *ins[3] = {x, w, b};
    RELAY_TRY(check_no_overlap(outs, 1, ins, 3));
    cudaStream_t st = (cudaStream_t)stream;
    const bool tc = conv_tc_eligible(d);
    RELAY_TRY(check_workspace(ws, ws_bytes, relay_workspace_bytes_conv2d_act(x, w, attrs)));
    const void *bp = b ? b->data : nullptr;
    const int32_t b_dt = b ? b->dtype : RELAY_F32;
    if (!d.nhwc) {
        if (tc) return launch_conv_fwd_tc(d, x->data, false, w->data, bp, b_dt, act, y->data, ws, st);
        return launch_conv_fwd_direct(d, x->data, w->data, bp, b_dt, act, y->data, st);
    }
    // NHWC: the kernels write NCHW into the workspace, a layout change brings the result to y
    char *base = (char *)ws;
    void *y_nchw = base;
    if (tc) {
        // the tensor-core instance reads NHWC itself and, in its two-SM form, stores NHWC tiles
        return launch_conv_fwd_tc(d, x->data, true, w->data, bp, b_dt, act, y_nchw, base + y_bytes(d), st, y->data);
    } else {
        void *x_nchw = base + y_bytes(d);
        RELAY_TRY(launch_layout_change(d.dt, x->data, x_nchw, d.Nb, d.H * d.W, d.C, st));
        RELAY_TRY(launch_conv_fwd_direct(d, x_nchw, w->data, bp, b_dt, act, y_nchw, st));
    }
    return launch_layout_change(d.dt, y_nchw, y->data, d.Nb, d.O, d.P * d.Q, st);
}

extern "C" relay_status_t relay_fused_conv2d_act_grad(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *y,
                                                      const relay_tensor_t *dy, const relay_conv2d_attrs_t *attrs, int32_t act,
                                                      const relay_tensor_t *dx, const relay_tensor_t *dw, const relay_tensor_t *db,
                                                      void *ws, size_t ws_bytes, void *stream)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(y, "y"));
    RELAY_TRY(check_not_null(dy, "dy"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(dw, "dw"));
    ConvDims d;
    RELAY_TRY(check_conv(x, w, nullptr, attrs, &d));
    const relay_tensor_t *yy[2] = {y, dy};
    const char *yn[2] = {"y", "dy"};
    for (int i = 0; i < 2; ++i) { RELAY_TRY(check_type(yy[i], yn[i])); RELAY_TRY(check_rank(yy[i], 4, yn[i])); }
    if (dx) { RELAY_TRY(check_type(dx, "dx")); RELAY_TRY(check_rank(dx, 4, "dx")); }
    RELAY_TRY(check_type(dw, "dw")); RELAY_TRY(check_rank(dw, 4, "dw"));
    if (db) { RELAY_TRY(check_type(db, "db")); RELAY_TRY(check_rank(db, 1, "db")); }
    for (int i = 0; i < 2; ++i) RELAY_TRY(check_dtype(yy[i], d.dt, yn[i]));
    if (dx) RELAY_TRY(check_dtype(dx, d.dt, "dx"));
    RELAY_TRY(check_dtype(dw, d.dt, "dw"));
    if (db) RELAY_TRY(check_dtype(db, RELAY_F32, "db"));
    for (int i = 0; i < 2; ++i) RELAY_TRY(check_layout(yy[i], d.nhwc ? RELAY_NHWC : RELAY_NCHW, d.nhwc ? RELAY_NHWC : RELAY_NCHW, yn[i]));
    if (dx) RELAY_TRY(check_layout(dx, d.nhwc ? RELAY_NHWC : RELAY_NCHW, d.nhwc ? RELAY_NHWC : RELAY_NCHW, "dx"));
    RELAY_TRY(check_layout(dw, RELAY_OIHW, RELAY_OIHW, "dw"));
    for (int i = 0; i < 2; ++i) RELAY_TRY(check_act_shape(d, yy[i], d.O, d.P, d.Q, yn[i]));
    if (dx) RELAY_TRY(check_act_shape(d, dx, d.C, d.H, d.W, "dx"));
    RELAY_TRY(check_shape(dw, {d.O, d.C, d.R, d.S}, "dw"));
    if (db) RELAY_TRY(check_shape(db, {d.O}, "db"));
    if (act < RELAY_ACT_NONE || act > RELAY_ACT_SIGMOID) return fail(RELAY_ERR_ATTR, "unknown activation %d", act);
    const relay_tensor_t *ins[4] = {x, w, y, dy}, *outs[3] = {dx, dw, db};
    for (int i = 0; i < 4; ++i) RELAY_TRY(check_data(ins[i], "input"));
    for (int i = 0; i < 3; ++i) if (outs[i]) RELAY_TRY(check_data(outs[i], "output"));
    RELAY_TRY(check_no_overlap(outs, 3, ins, 4));
    size_t dz_bytes;
    conv_grad_ws(d, &dz_bytes);
    RELAY_TRY(check_workspace(ws, ws_bytes, relay_workspace_bytes_conv2d_act_grad(x, w, attrs)));
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t ny = d.Nb * d.O * d.P * d.Q;
    if (ny == 0 || d.C == 0) {
        if (dx && numel(dx)) RELAY_CUDA(cudaMemsetAsync(dx->data, 0, nbytes(dx), st));
        if (numel(dw)) RELAY_CUDA(cudaMemsetAsync(dw->data, 0, nbytes(dw), st));
        if (db && numel(db)) RELAY_CUDA(cudaMemsetAsync(db->data, 0, nbytes(db), st));
        return RELAY_OK;
    }
    // NHWC: x, y, dy go to NCHW copies in the workspace, dx comes back through one
    const void *xp = x->data, *yp = y->data, *dyp = dy->data;
    void *dxp = dx ? dx->data : nullptr;
    char *inner = (char *)ws;
    if (d.nhwc && conv_tc_eligible(d)) {
        // the tensor-core instance works on NHWC itself: no copies of x, y, dy; dx passes through an NCHW temporary only
        // where the one-SM kernel computes it
        char *base = (char *)ws;
        void *dx_nchw = base + x_bytes(d);
        float *partials = (float *)(base + 2 * x_bytes(d));            // at most N*H*W*O/8 bytes: fits the y-sized region
        inner = base + 2 * x_bytes(d) + 2 * y_bytes(d);
        return launch_conv_grad_tc(d, x->data, w->data, y->data, dy->data, act, dx ? dx_nchw : nullptr, dw->data,
                                   db ? (float *)db->data : nullptr, inner, st, true, partials, dx ? dx->data : nullptr);
    }
    if (d.nhwc) {
        char *base = (char *)ws;
        void *x_nchw = base, *dx_nchw = base + x_bytes(d), *y_nchw = base + 2 * x_bytes(d), *dy_nchw = base + 2 * x_bytes(d) + y_bytes(d);
        inner = base + 2 * x_bytes(d) + 2 * y_bytes(d);
        RELAY_TRY(launch_layout_change(d.dt, x->data, x_nchw, d.Nb, d.H * d.W, d.C, st));
        RELAY_TRY(launch_layout_change(d.dt, y->data, y_nchw, d.Nb, d.P * d.Q, d.O, st));
        RELAY_TRY(launch_layout_change(d.dt, dy->data, dy_nchw, d.Nb, d.P * d.Q, d.O, st));
        xp = x_nchw; yp = y_nchw; dyp = dy_nchw;
        if (dx) dxp = dx_nchw;
    }
    if (conv_tc_eligible(d)) {
        RELAY_TRY(launch_conv_grad_tc(d, xp, w->data, yp, dyp, act, dxp, dw->data, db ? (float *)db->data : nullptr, inner, st));
    } else {
        void *dz = inner;
        int64_t rows, cols;
        flat_view(ny, d.dt, &rows, &cols);
        RELAY_TRY(act_grad_any(d.dt, dyp, yp, dz, nullptr, nullptr, rows, cols, act, st));
        if (db) RELAY_TRY(launch_conv_db(d, dz, (float *)db->data, st));
        if (dx) RELAY_TRY(launch_conv_dx_direct(d, dz, w->data, dxp, st));
        RELAY_TRY(launch_conv_dw_direct(d, dz, xp, dw->data, (float *)(inner + dz_bytes), st));
    }
    if (d.nhwc && dx) RELAY_TRY(launch_layout_change(d.dt, dxp, dx->data, d.Nb, d.C, d.H * d.W, st));
    return RELAY_OK;
}
