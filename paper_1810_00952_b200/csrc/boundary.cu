// Host side of the boundary: status text, descriptor checks and the integer type relations
// (Fig. 4 kinding rules and Fig. 5 typing rules applied to concrete tensor descriptors).
#include <cstring>
#include <initializer_list>
#include <mutex>

#include "common.h"
#include "ewise_prog.h"
#include "tc_common.cuh"

namespace relay {

static thread_local char g_err[512] = "";
static int64_t g_launches = 0;
static std::mutex g_mu;

relay_status_t fail(relay_status_t st, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}
void clear_error() { g_err[0] = 0; }
void count_launch(int n) { __atomic_add_fetch(&g_launches, (int64_t)n, __ATOMIC_RELAXED); }

relay_status_t check_launch(const char *what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(RELAY_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
    count_launch();
    return RELAY_OK;
}

relay_status_t check_not_null(const void *p, const char *name)
{
    return p ? RELAY_OK : fail(RELAY_ERR_NULL, "%s is NULL", name);
}

relay_status_t check_type(const relay_tensor_t *t, const char *name)
{
    if (!t) return fail(RELAY_ERR_NULL, "%s is NULL", name);
    if (t->rank < 0 || t->rank > RELAY_MAX_RANK)
        return fail(RELAY_ERR_RANK, "%s: rank %d outside [0,%d]", name, t->rank, RELAY_MAX_RANK);
    if (dtype_size(t->dtype) == 0) return fail(RELAY_ERR_DTYPE, "%s: unknown base type %d", name, t->dtype);
    if (t->layout < RELAY_ROWMAJOR || t->layout > RELAY_OIHW)
        return fail(RELAY_ERR_LAYOUT, "%s: unknown layout %d", name, t->layout);
    for (int d = 0; d < t->rank; ++d)
        if (t->shape[d] < 0) return fail(RELAY_ERR_SHAPE, "%s: extent %lld of axis %d is not a natural number", name,
                                         (long long)t->shape[d], d);
    return RELAY_OK;
}

relay_status_t check_rank(const relay_tensor_t *t, int rank, const char *name)
{
    if (t->rank != rank) return fail(RELAY_ERR_RANK, "%s: rank %d, operator type needs rank %d", name, t->rank, rank);
    return RELAY_OK;
}

relay_status_t check_dtype(const relay_tensor_t *t, int32_t dt, const char *name)
{
    if (t->dtype != dt)
        return fail(RELAY_ERR_DTYPE, "%s: base type %s, operator type needs %s", name, dtype_name(t->dtype), dtype_name(dt));
    return RELAY_OK;
}

relay_status_t check_layout(const relay_tensor_t *t, int32_t a, int32_t b, const char *name)
{
    if (t->layout != a && t->layout != b) return fail(RELAY_ERR_LAYOUT, "%s: layout tag %d not accepted here", name, t->layout);
    return RELAY_OK;
}

relay_status_t check_shape(const relay_tensor_t *t, std::initializer_list<int64_t> want, const char *name)
{
    if ((size_t)t->rank != want.size())
        return fail(RELAY_ERR_RANK, "%s: rank %d, operator type needs rank %zu", name, t->rank, want.size());
    int d = 0;
    for (int64_t w : want) {
        if (t->shape[d] != w)
            return fail(RELAY_ERR_SHAPE, "%s: axis %d has extent %lld, operator type needs %lld", name, d,
                        (long long)t->shape[d], (long long)w);
        ++d;
    }
    return RELAY_OK;
}

relay_status_t check_shape_n(const relay_tensor_t *t, const int64_t *want, int rank, const char *name)
{
    if (t->rank != rank) return fail(RELAY_ERR_RANK, "%s: rank %d, operator type needs rank %d", name, t->rank, rank);
    for (int d = 0; d < rank; ++d)
        if (t->shape[d] != want[d])
            return fail(RELAY_ERR_SHAPE, "%s: axis %d has extent %lld, operator type needs %lld", name, d, (long long)t->shape[d],
                        (long long)want[d]);
    return RELAY_OK;
}

relay_status_t check_data(const relay_tensor_t *t, const char *name)
{
    if (numel(t) == 0) return RELAY_OK;
    if (!t->data) return fail(RELAY_ERR_NULL, "%s: data pointer is NULL", name);
    if (((uintptr_t)t->data & 15u) != 0) return fail(RELAY_ERR_ALIGN, "%s: data pointer not 16-byte aligned", name);
    return RELAY_OK;
}

relay_status_t check_workspace(const void *ws, size_t have, size_t need)
{
    if (need == 0) return RELAY_OK;
    if (!ws) return fail(RELAY_ERR_WORKSPACE, "workspace is NULL, %zu bytes needed", need);
    if (((uintptr_t)ws & 15u) != 0) return fail(RELAY_ERR_WORKSPACE, "workspace not 16-byte aligned");
    if (have < need) return fail(RELAY_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", have, need);
    return RELAY_OK;
}

relay_status_t check_no_overlap(const relay_tensor_t *const *outs, int n_out, const relay_tensor_t *const *ins, int n_in)
{
    for (int i = 0; i < n_out; ++i) {
        if (!outs[i] || numel(outs[i]) == 0) continue;
        Span a = span_of(outs[i]);
        for (int j = 0; j < n_in; ++j) {
            if (!ins[j] || numel(ins[j]) == 0) continue;
            Span b = span_of(ins[j]);
            if (a.lo < b.hi && b.lo < a.hi) return fail(RELAY_ERR_ATTR, "output %d overlaps input %d", i, j);
        }
        for (int j = i + 1; j < n_out; ++j) {
            if (!outs[j] || numel(outs[j]) == 0) continue;
            Span b = span_of(outs[j]);
            if (a.lo < b.hi && b.lo < a.hi) return fail(RELAY_ERR_ATTR, "output %d overlaps output %d", i, j);
        }
    }
    return RELAY_OK;
}

// [0]: the error word that kernels set; [1]: where relay_poll_status has it exchanged to.  One pair per device, shared by
// all streams: a poll reports (and clears) a time-out of any stream's kernel.
__device__ int g_error_word[2] = {0, 0};

__global__ void poll_exchange_kernel(int *word, int *result) { *result = atomicExch(word, 0); }

int *device_error_word()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    static int *addr[64] = {nullptr};
    std::lock_guard<std::mutex> lk(g_mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_error_word) != cudaSuccess) return nullptr;   // address of element [0]
        addr[dev] = (int *)p;
    }
    return addr[dev];
}

// waits on a barrier that nobody signals, for at most limit_cycles, then reports the time-out
__global__ void expire_wait_kernel(long long limit_cycles, int *err)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
        const long long t0 = clock64();
        bool done = false;
        while (!(done = tc::mbar_try_wait(&bar, 0)) && clock64() - t0 < limit_cycles) {}
        if (!done) atomicCAS(err, 0, tc::ERR_WAIT_STEP);
    }
}

static void fill_out(relay_tensor_t *out, int32_t dtype, int32_t layout, int rank, const int64_t *shape)
{
    std::memset(out, 0, sizeof(*out));
    out->data = nullptr;
    out->dtype = dtype;
    out->layout = layout;
    out->rank = rank;
    for (int d = 0; d < rank; ++d) out->shape[d] = shape[d];
}

}  // namespace relay

using namespace relay;

extern "C" {

const char *relay_last_error(void) { return g_err; }
int64_t relay_launch_count(void) { return __atomic_load_n(&g_launches, __ATOMIC_RELAXED); }
const char *relay_version(void) { return "relay_b200 0.1 (sm_100a)"; }

relay_status_t relay_poll_status(void *stream)
{
    clear_error();
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return fail(RELAY_ERR_CUDA, "stream reports: %s", cudaGetErrorString(e));
    int *w = device_error_word();
    if (!w) return fail(RELAY_ERR_CUDA, "no device error word (no CUDA device?)");
    // read and clear in one step (a kernel of another stream may set the word at any time): atomic exchange on the
    // device, result through a second word
    int v = 0;
    poll_exchange_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(w, w + 1);
    RELAY_TRY(check_launch("poll_exchange"));
    RELAY_CUDA(cudaMemcpyAsync(&v, w + 1, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    RELAY_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    if (v == kErrBounds) return fail(RELAY_ERR_CUDA, "a device-side bounds check failed: a kernel computed an address outside the call's tensors (the access was skipped)");
    if (v != 0) return fail(RELAY_ERR_TIMEOUT, "a bounded device-side wait expired (code %d)", v);
    return RELAY_OK;
}

#ifdef RELAY_BOUNDS_CHECK
__global__ void bounds_probe_kernel(const char *base) { (void)relay_in_bounds(base + 16, 16); }   // looks an address up; touches nothing
#endif

relay_status_t relay_debug_bounds_probe(void *stream)
{
    clear_error();
#ifdef RELAY_BOUNDS_CHECK
    int *w = device_error_word();
    if (!w) return fail(RELAY_ERR_CUDA, "no device error word (no CUDA device?)");
    BoundsReg br;
    br.add(w, 16);                         // a 16-byte range; the probe asks for the 16 bytes behind it
    RELAY_TRY(br.commit((cudaStream_t)stream));
    bounds_probe_kernel<<<1, 1, 0, (cudaStream_t)stream>>>((const char *)w);
    return check_launch("bounds_probe");
#else
    (void)stream;
    return fail(RELAY_ERR_UNSUPPORTED, "this build of the library carries no bounds checks");
#endif
}

relay_status_t relay_debug_expire_wait(int32_t limit_us, void *stream)
{
    clear_error();
    if (limit_us < 1 || limit_us > 1000000) return fail(RELAY_ERR_ATTR, "limit_us = %d outside [1, 1000000]", limit_us);
    int *w = device_error_word();
    if (!w) return fail(RELAY_ERR_CUDA, "no device error word (no CUDA device?)");
    int dev = 0, khz = 0;
    RELAY_CUDA(cudaGetDevice(&dev));
    RELAY_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    expire_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_us * (khz / 1000), w);
    return check_launch("expire_wait");
}

relay_status_t relay_infer_dense(const relay_tensor_t *x, const relay_tensor_t *w, relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(out, "out"));
    RELAY_TRY(check_type(x, "x"));
    RELAY_TRY(check_type(w, "w"));
    if (x->rank < 2) return fail(RELAY_ERR_RANK, "x: rank %d, operator type needs rank 2 or more (batch axes, M, K)", x->rank);
    RELAY_TRY(check_rank(w, 2, "w"));
    if (!is_float(x->dtype)) return fail(RELAY_ERR_DTYPE, "x: dense needs a float base type, got %s", dtype_name(x->dtype));
    RELAY_TRY(check_dtype(w, x->dtype, "w"));
    RELAY_TRY(check_layout(x, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "x"));
    RELAY_TRY(check_layout(w, RELAY_ROWMAJOR, RELAY_ROWMAJOR, "w"));
    const int r = x->rank;
    if (x->shape[r - 1] != w->shape[0])
        return fail(RELAY_ERR_SHAPE, "dense: x is (..,%lld,%lld) but w is (%lld,%lld): inner extents differ",
                    (long long)x->shape[r - 2], (long long)x->shape[r - 1], (long long)w->shape[0], (long long)w->shape[1]);
    int64_t s[RELAY_MAX_RANK];
    for (int d = 0; d < r - 1; ++d) s[d] = x->shape[d];
    s[r - 1] = w->shape[1];
    fill_out(out, x->dtype, RELAY_ROWMAJOR, r, s);
    return RELAY_OK;
}

relay_status_t relay_infer_conv2d(const relay_tensor_t *x, const relay_tensor_t *w, const relay_conv2d_attrs_t *attrs,
                                  relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w, "w"));
    RELAY_TRY(check_not_null(attrs, "attrs"));
    RELAY_TRY(check_not_null(out, "out"));
    RELAY_TRY(check_type(x, "x"));
    RELAY_TRY(check_type(w, "w"));
    RELAY_TRY(check_rank(x, 4, "x"));
    RELAY_TRY(check_rank(w, 4, "w"));
    if (!is_float(x->dtype)) return fail(RELAY_ERR_DTYPE, "x: conv2d needs a float base type, got %s", dtype_name(x->dtype));
    RELAY_TRY(check_dtype(w, x->dtype, "w"));
    RELAY_TRY(check_layout(x, RELAY_NCHW, RELAY_NHWC, "x"));
    RELAY_TRY(check_layout(w, RELAY_OIHW, RELAY_OIHW, "w"));
    const bool nhwc = x->layout == RELAY_NHWC;            // shape is (N,H,W,C) then: tensors are row-major in the order of `shape`
    const int64_t xc = nhwc ? x->shape[3] : x->shape[1];
    if (xc != w->shape[1])
        return fail(RELAY_ERR_SHAPE, "conv2d: x has %lld channels, w expects %lld", (long long)xc, (long long)w->shape[1]);
    if (attrs->stride < 1 || attrs->pad < 0) return fail(RELAY_ERR_ATTR, "conv2d: stride %d / pad %d invalid", attrs->stride, attrs->pad);
    if (attrs->dilation != 1 || attrs->groups != 1)
        return fail(RELAY_ERR_ATTR, "conv2d: dilation %d / groups %d: only 1 is defined here", attrs->dilation, attrs->groups);
    int64_t H = nhwc ? x->shape[1] : x->shape[2], W = nhwc ? x->shape[2] : x->shape[3], R = w->shape[2], S = w->shape[3];
    if (R < 1 || S < 1 || H + 2 * attrs->pad < R || W + 2 * attrs->pad < S)
        return fail(RELAY_ERR_SHAPE, "conv2d: %lldx%lld window does not fit the padded %lldx%lld image", (long long)R,
                    (long long)S, (long long)(H + 2 * attrs->pad), (long long)(W + 2 * attrs->pad));
    const int64_t P = (H + 2 * attrs->pad - R) / attrs->stride + 1, Q = (W + 2 * attrs->pad - S) / attrs->stride + 1;
    int64_t s[4] = {x->shape[0], w->shape[0], P, Q};
    if (nhwc) { s[1] = P; s[2] = Q; s[3] = w->shape[0]; }
    fill_out(out, x->dtype, nhwc ? RELAY_NHWC : RELAY_NCHW, 4, s);
    return RELAY_OK;
}

relay_status_t relay_infer_broadcast(const relay_tensor_t *a, const relay_tensor_t *b, relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(a, "a"));
    RELAY_TRY(check_not_null(b, "b"));
    RELAY_TRY(check_not_null(out, "out"));
    RELAY_TRY(check_type(a, "a"));
    RELAY_TRY(check_type(b, "b"));
    // the operator that follows the broadcast step needs one base type (Fig. 5, Type-Noncomp-BinaryOp)
    if (a->dtype != b->dtype) return fail(RELAY_ERR_DTYPE, "broadcast: base types %s and %s differ", dtype_name(a->dtype), dtype_name(b->dtype));
    int r = a->rank > b->rank ? a->rank : b->rank;
    int64_t s[RELAY_MAX_RANK];
    for (int d = 0; d < r; ++d) {
        int ia = d - (r - a->rank), ib = d - (r - b->rank);
        int64_t da = ia >= 0 ? a->shape[ia] : 1, db = ib >= 0 ? b->shape[ib] : 1;
        if (da == db) s[d] = da;
        else if (da == 1) s[d] = db;
        else if (db == 1) s[d] = da;
        else
            return fail(RELAY_ERR_SHAPE, "broadcast: extents %lld and %lld of right-aligned axis %d are neither equal nor 1",
                        (long long)da, (long long)db, d);
    }
    fill_out(out, a->dtype, a->layout, r, s);
    return RELAY_OK;
}

relay_status_t relay_infer_reduce(const relay_tensor_t *in, int32_t red_op, int32_t axes_mask, int32_t keepdims,
                                  relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(in, "in"));
    RELAY_TRY(check_not_null(out, "out"));
    RELAY_TRY(check_type(in, "in"));
    if (red_op < RELAY_RED_NONE || red_op > RELAY_RED_ARGMAX) return fail(RELAY_ERR_ATTR, "reduce: unknown reduction %d", red_op);
    if (red_op == RELAY_RED_NONE) {
        fill_out(out, in->dtype, in->layout, in->rank, in->shape);
        return RELAY_OK;
    }
    if (axes_mask < 0 || (axes_mask >> in->rank) != 0 || axes_mask == 0)
        return fail(RELAY_ERR_ATTR, "reduce: axes mask 0x%x names no axis or an axis outside rank %d", axes_mask, in->rank);
    int64_t s[RELAY_MAX_RANK];
    int r = 0;
    for (int d = 0; d < in->rank; ++d) {
        if (axes_mask >> d & 1) {
            if (in->shape[d] == 0) return fail(RELAY_ERR_SHAPE, "reduce: reduced axis %d is empty", d);
            if (keepdims) s[r++] = 1;
        } else
            s[r++] = in->shape[d];
    }
    fill_out(out, red_op == RELAY_RED_ARGMAX ? RELAY_I64 : RELAY_F32, RELAY_ROWMAJOR, r, s);
    return RELAY_OK;
}

relay_status_t relay_infer_stack(const relay_tensor_t *elem, int64_t m, relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(elem, "elem"));
    RELAY_TRY(check_not_null(out, "out"));
    RELAY_TRY(check_type(elem, "elem"));
    if (elem->rank + 1 > RELAY_MAX_RANK) return fail(RELAY_ERR_RANK, "stack: result rank %d exceeds %d", elem->rank + 1, RELAY_MAX_RANK);
    if (m < 1) return fail(RELAY_ERR_SHAPE, "stack: a tensor literal needs at least one element");
    int64_t s[RELAY_MAX_RANK];
    s[0] = m;
    for (int d = 0; d < elem->rank; ++d) s[d + 1] = elem->shape[d];
    fill_out(out, elem->dtype, RELAY_ROWMAJOR, elem->rank + 1, s);
    return RELAY_OK;
}

relay_status_t relay_infer_lstm(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                relay_tensor_t *h_all, relay_tensor_t *c_final)
{
    clear_error();
    RELAY_TRY(check_not_null(x, "x"));
    RELAY_TRY(check_not_null(w_ih, "w_ih"));
    RELAY_TRY(check_not_null(w_hh, "w_hh"));
    RELAY_TRY(check_not_null(h_all, "h_all"));
    RELAY_TRY(check_not_null(c_final, "c_final"));
    RELAY_TRY(check_type(x, "x"));
    RELAY_TRY(check_type(w_ih, "w_ih"));
    RELAY_TRY(check_type(w_hh, "w_hh"));
    RELAY_TRY(check_rank(x, 3, "x"));
    RELAY_TRY(check_rank(w_ih, 2, "w_ih"));
    RELAY_TRY(check_rank(w_hh, 2, "w_hh"));
    RELAY_TRY(check_dtype(x, RELAY_BF16, "x"));
    RELAY_TRY(check_dtype(w_ih, RELAY_BF16, "w_ih"));
    RELAY_TRY(check_dtype(w_hh, RELAY_BF16, "w_hh"));
    int64_t T = x->shape[0], B = x->shape[1], I = x->shape[2], H = w_hh->shape[0];
    if (w_ih->shape[0] != I) return fail(RELAY_ERR_SHAPE, "lstm: w_ih has %lld rows, x has input width %lld", (long long)w_ih->shape[0], (long long)I);
    if (w_ih->shape[1] != 4 * H || w_hh->shape[1] != 4 * H)
        return fail(RELAY_ERR_SHAPE, "lstm: gate axis must be 4H = %lld (w_ih has %lld, w_hh has %lld)", (long long)(4 * H),
                    (long long)w_ih->shape[1], (long long)w_hh->shape[1]);
    int64_t sh[3] = {T, B, H}, sc[2] = {B, H};
    fill_out(h_all, RELAY_F32, RELAY_ROWMAJOR, 3, sh);
    fill_out(c_final, RELAY_F32, RELAY_ROWMAJOR, 2, sc);
    return RELAY_OK;
}

relay_status_t relay_infer_ewise(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                 int32_t value, relay_tensor_t *out)
{
    clear_error();
    RELAY_TRY(check_not_null(out, "out"));
    TypedProgram tp;
    RELAY_TRY(type_program(prog, inputs, n_in, &tp));
    if (value < 0 || value >= tp.n_values) return fail(RELAY_ERR_ATTR, "value id %d outside [0,%d)", value, tp.n_values);
    fill_out(out, tp.dtype[value], RELAY_ROWMAJOR, tp.rank, tp.shape);
    return RELAY_OK;
}

}  // extern "C"
