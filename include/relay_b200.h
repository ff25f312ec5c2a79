/*
 * relay_b200.h -- C ABI of the fused primitive-operator groups that a Relay program executes.
 *
 * Background (Relay, arXiv 1810.00952).  Relay declares primitive operators as externally
 * implemented functions with a tensor type ("operator <GlobalId> : <Type>", Section 3, Fig. 1),
 * registers them with its runtime (Section 4.1) and instantiates them per concrete tensor
 * type, i.e. per base type and static shape (Section 5.1).  Every value is a tensor whose
 * type is Tensor(BaseType, Shape(d1..dn)) (Fig. 1; Fig. 4 rules BaseType-T, Shape-T,
 * Tensor-T).  This library is that operator layer for one B200 GPU: each entry point checks
 * the operand types against the operator's type relation on the host (Section 4.3: shapes live
 * in types, so the check needs no data), then enqueues hand-written sm_100a kernels.
 *
 * Common rules for every compute entry point
 *   - Tensors are dense and row-major in the order of `shape` (NCHW / OIHW are row-major over
 *     those four axes).  `data` is a DEVICE pointer aligned to 16 bytes.  The caller owns all
 *     buffers; the library allocates no device memory and keeps no pointer after return.
 *   - `ws` is caller-provided device scratch of `ws_bytes` bytes (16-byte aligned); the needed
 *     size comes from the matching relay_workspace_bytes_* query (0 means `ws` may be NULL).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls only enqueue
 *     work and return without synchronising.  Inputs are read-only; outputs must not overlap
 *     inputs or each other.
 *   - All descriptor errors are found before anything is launched and leave outputs untouched.
 *     Rules are checked in the order: null -> rank -> dtype -> layout -> shape -> attributes ->
 *     alignment/overlap -> workspace; the first failing rule decides the status.
 *     relay_last_error() returns a thread-local description of the last failure.
 *   - Kernels that wait on hardware barriers give up after a bounded number of polls and set a
 *     device-side error word instead of hanging; relay_poll_status() reads (and clears) it.
 *   - Stream capture: a compute entry point may be called while `stream` is being captured into a
 *     CUDA graph (it enqueues kernels on `stream` only, allocates nothing and does not synchronise),
 *     provided an entry point of the same kind was called once on this device before the capture
 *     (module loading and one-time address look-ups happen on first use).  The graph holds the
 *     pointers of the captured call: replaying it recomputes into the same buffers.
 *     relay_poll_status() synchronises and must stay outside a capture.
 */
#ifndef RELAY_B200_H_
#define RELAY_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RELAY_MAX_RANK 6
#define RELAY_MAX_INPUTS 8
#define RELAY_MAX_OUTPUTS 8
#define RELAY_MAX_INSTR 32

typedef enum {
    RELAY_OK = 0,
    RELAY_ERR_NULL = 1,        /* a required pointer is NULL */
    RELAY_ERR_RANK = 2,        /* rank outside what the operator's type allows */
    RELAY_ERR_SHAPE = 3,       /* shapes violate the operator's type relation */
    RELAY_ERR_DTYPE = 4,       /* base types violate the operator's type relation */
    RELAY_ERR_LAYOUT = 5,      /* layout tag not accepted by the operator */
    RELAY_ERR_ALIGN = 6,       /* data pointer not 16-byte aligned */
    RELAY_ERR_ATTR = 7,        /* bad attribute, malformed program, overlapping buffers */
    RELAY_ERR_UNSUPPORTED = 8, /* well-typed, but no kernel instance exists for it */
    RELAY_ERR_WORKSPACE = 9,   /* workspace missing, misaligned or too small */
    RELAY_ERR_CUDA = 10,       /* a CUDA runtime/driver call failed */
    RELAY_ERR_TIMEOUT = 11     /* a bounded device-side wait expired */
} relay_status_t;

/* Base types (Fig. 1 <BaseType>).  The paper's FloatType(width) carries only a width; the
 * 16-bit float here is bfloat16 (8 exponent, 7 fraction bits).  Bool is stored as one byte
 * holding 0 or 1. */
typedef enum { RELAY_F32 = 0, RELAY_BF16 = 1, RELAY_I32 = 2, RELAY_I64 = 3, RELAY_BOOL = 4 } relay_dtype_t;

typedef enum { RELAY_ROWMAJOR = 0, RELAY_NCHW = 1, RELAY_NHWC = 2, RELAY_OIHW = 3 } relay_layout_t;

typedef enum { RELAY_ACT_NONE = 0, RELAY_ACT_RELU = 1, RELAY_ACT_TANH = 2, RELAY_ACT_SIGMOID = 3 } relay_act_t;

/* A typed tensor value: Tensor(dtype, Shape(shape[0..rank))) plus its device address. */
typedef struct relay_tensor {
    void *data;
    int32_t dtype;  /* relay_dtype_t */
    int32_t rank;   /* 0..RELAY_MAX_RANK; rank 0 is a scalar (all values are tensors) */
    int64_t shape[RELAY_MAX_RANK];
    int32_t layout; /* relay_layout_t */
    int32_t reserved;
} relay_tensor_t;

/* ---------------------------------------------------------------------------------------------
 * Elementwise programs.  A fused elementwise group is a let-list (Fig. 1 "let") of at most
 * RELAY_MAX_INSTR instructions.  Value ids: 0..n_in-1 are the group's inputs, n_in+j is the
 * result of instruction j; an instruction may only name earlier values; unused operands are -1.
 * Opcodes are Fig. 1's BinOp / UnaryOp productions, the cast production, and the elementwise
 * library operators of Fig. 3.  Typing follows Fig. 5 after an explicit NumPy-style broadcast
 * of all inputs to one shape: arithmetic needs equal float base types and yields that type
 * (Type-Noncomp-BinaryOp, Type-UnaryOp); comparisons need equal base types and yield Bool
 * (Type-Comp-BinaryOp); select needs a Bool condition and equal branch types; cast yields the
 * named type; const is a literal of the named type.  `dtype` states the result type of each
 * instruction and is checked against these rules.
 * Arithmetic is carried out in fp32; a result whose type is bf16 is rounded to bf16 (nearest
 * even).  Integer types may appear only as sources or targets of cast.
 * ------------------------------------------------------------------------------------------- */
typedef enum {
    RELAY_OP_ADD = 0, RELAY_OP_SUB = 1, RELAY_OP_MUL = 2, RELAY_OP_DIV = 3,
    RELAY_OP_NEG = 4, RELAY_OP_SQ = 5,
    RELAY_OP_NE = 6, RELAY_OP_EQ = 7, RELAY_OP_LT = 8, RELAY_OP_LE = 9, RELAY_OP_GT = 10, RELAY_OP_GE = 11,
    RELAY_OP_SELECT = 12, /* a ? b : c */
    RELAY_OP_RELU = 13, RELAY_OP_TANH = 14, RELAY_OP_SIGMOID = 15,
    RELAY_OP_CAST = 16, RELAY_OP_CONST = 17, RELAY_OP_EXP = 18, RELAY_OP_LOG = 19,
    RELAY_OP_MAX = 20, RELAY_OP_MIN = 21,
    RELAY_OP_COUNT_ = 22
} relay_opcode_t;

typedef struct relay_instr {
    int32_t op;    /* relay_opcode_t */
    int32_t a, b, c;
    int32_t dtype; /* result type */
    int32_t reserved;
    double imm;    /* literal of RELAY_OP_CONST */
} relay_instr_t;

typedef struct relay_ewise_prog {
    int32_t n_instr;
    int32_t reserved;
    const relay_instr_t *instr; /* HOST pointer; read during the call only */
} relay_ewise_prog_t;

typedef enum { RELAY_RED_NONE = 0, RELAY_RED_SUM = 1, RELAY_RED_MAX = 2, RELAY_RED_MEAN = 3, RELAY_RED_ARGMAX = 4 } relay_reduce_op_t;

/* One result of a reduce group: program value `value`, reduced with `red_op` over the axes
 * whose bit is set in `axes_mask` (bit d = axis d of the broadcast shape).  RELAY_RED_NONE
 * returns the value unreduced.  With keepdims the reduced axes stay as extent 1. */
typedef struct relay_out_spec {
    int32_t value;
    int32_t red_op;    /* relay_reduce_op_t */
    int32_t axes_mask;
    int32_t keepdims;
} relay_out_spec_t;

typedef struct relay_conv2d_attrs {
    int32_t stride;   /* same in both spatial axes, >= 1 */
    int32_t pad;      /* zero padding on every side, >= 0 */
    int32_t dilation; /* must be 1 */
    int32_t groups;   /* must be 1 */
} relay_conv2d_attrs_t;

/* Pooling window (Fig. 3: relay.max_pool(x, ksize=[1,kh,kw,1], strides=[1,sh,sw,1])); no padding. */
typedef struct {
    int32_t kh, kw;   /* window extent, >= 1, not larger than the plane */
    int32_t sh, sw;   /* stride, >= 1 */
} relay_pool2d_attrs_t;

/* ---------------------------------------------------------------------------------------------
 * Type relations, host only (no GPU needed).  Each fills `out` (dtype, rank, shape, layout;
 * data = NULL) with the result type the operator's relation gives for the argument types,
 * the way Fig. 5 derives the type of an expression from the types of its parts.
 * ------------------------------------------------------------------------------------------- */

/* dense: Tensor(t,(M,K)) x Tensor(t,(K,N)) -> Tensor(t,(M,N)), t in {f32, bf16} (Fig. 3 relay.linear).
 * x may carry leading batch axes (Section 5.2: batching a program adds a leading axis to its tensors):
 * Tensor(t,(B1,..,Bk,M,K)) x Tensor(t,(K,N)) -> Tensor(t,(B1,..,Bk,M,N)), rank at most RELAY_MAX_RANK. */
relay_status_t relay_infer_dense(const relay_tensor_t *x, const relay_tensor_t *w, relay_tensor_t *out);

/* conv2d: x:(N,C,H,W) NCHW, w:(O,C,R,S) OIHW -> (N,O,P,Q) with P = floor((H+2p-R)/s)+1
 * (Fig. 3 relay.conv2d). */
relay_status_t relay_infer_conv2d(const relay_tensor_t *x, const relay_tensor_t *w,
                                  const relay_conv2d_attrs_t *attrs, relay_tensor_t *out);

/* NumPy-style broadcast of two shapes (the explicit step that precedes Fig. 5's same-shape
 * rules): right-align, each axis pair equal or one of them 1.  dtype/layout copied from a. */
relay_status_t relay_infer_broadcast(const relay_tensor_t *a, const relay_tensor_t *b, relay_tensor_t *out);

/* Type of value `value` of an elementwise program over the given inputs (Fig. 5 rules applied
 * instruction by instruction after broadcasting all inputs to one shape). */
relay_status_t relay_infer_ewise(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs,
                                 int32_t n_in, int32_t value, relay_tensor_t *out);

/* Reduction result: axes in axes_mask removed (or kept as 1).  out_dtype: f32 for sum/max/mean
 * of float input, i64 for argmax. */
relay_status_t relay_infer_reduce(const relay_tensor_t *in, int32_t red_op, int32_t axes_mask,
                                  int32_t keepdims, relay_tensor_t *out);

/* Tensor literal (Fig. 5 Type-Tensor-Literal): m tensors of type Tensor(b, Shape(d1..dn))
 * stack to Tensor(b, Shape(m, d1..dn)). */
relay_status_t relay_infer_stack(const relay_tensor_t *elem, int64_t m, relay_tensor_t *out);

/* LSTM sequence: x:(T,B,I), w_ih:(I,4H), w_hh:(H,4H) -> h_all:(T,B,H) f32, c_final:(B,H) f32. */
relay_status_t relay_infer_lstm(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                relay_tensor_t *h_all, relay_tensor_t *c_final);

/* ---------------------------------------------------------------------------------------------
 * Workspace queries, host only.  Return the scratch bytes the matching call needs for these
 * argument types (0 if the types are invalid; the call itself reports why).
 * ------------------------------------------------------------------------------------------- */
size_t relay_workspace_bytes_dense_act(const relay_tensor_t *x, const relay_tensor_t *w);
size_t relay_workspace_bytes_dense_act_grad(const relay_tensor_t *x, const relay_tensor_t *w);
size_t relay_workspace_bytes_conv2d_act(const relay_tensor_t *x, const relay_tensor_t *w,
                                        const relay_conv2d_attrs_t *attrs);
size_t relay_workspace_bytes_conv2d_act_grad(const relay_tensor_t *x, const relay_tensor_t *w,
                                             const relay_conv2d_attrs_t *attrs);
size_t relay_workspace_bytes_reduce(const relay_tensor_t *const *inputs, int32_t n_in,
                                    const relay_out_spec_t *specs, int32_t n_out);
size_t relay_workspace_bytes_lstm(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh);
size_t relay_workspace_bytes_lstm_grad(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh);

/* ---------------------------------------------------------------------------------------------
 * Compute entry points.
 * ------------------------------------------------------------------------------------------- */

/* Dense anchor fused with broadcast bias and elementwise activation (Fig. 3: relay.linear
 * followed by an elementwise operator; fusion of such chains is the optimisation Section 5.2
 * names):   y[m,n] = act( sum_k x[m,k] * w[k,n] + b[n] ).
 *   x:(M,K)  w:(K,N)  b:(N) or NULL  ->  y:(M,N); x, w, y share one dtype t in {f32, bf16};
 *   b has dtype t or f32.  f32 runs in true fp32 (FMA); bf16 multiplies bf16 and accumulates
 *   in fp32, rounding once on the store of y.
 *   x and y may carry the same leading batch axes, x:(B1,..,Bk,M,K) -> y:(B1,..,Bk,M,N): the batch
 *   elements share w and b, so the call is one product over the B1*..*Bk*M stacked rows. */
relay_status_t relay_fused_dense_act(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b,
                                     int32_t act, const relay_tensor_t *y, void *ws, size_t ws_bytes, void *stream);

/* Gradient group of the dense anchor (Section 4.2: reverse mode; `dy` is the partial of the
 * program's final scalar with respect to y, each returned tensor the partial with respect to
 * the argument of the same name; the pair (forward call, this call) is what `Grad` returns:
 * the original result bundled with all partials).
 *   dZ = dy (.) act'(y)  with act' taken from the SAVED forward output y:
 *        relu' = 1[y>0] (so relu'(0)=0), tanh' = 1-y^2, sigmoid' = y(1-y);
 *   dx[m,k] = sum_n dZ[m,n] w[k,n];   dw[k,n] = sum_m x[m,k] dZ[m,n];   db[n] = sum_m dZ[m,n].
 *   dx, db may be NULL (not wanted); dw is required.  dx, dw have dtype t; db is f32 (or t for
 *   t = f32).  Sums are deterministic (fixed order, no float atomics).
 *   With leading batch axes on x, y, dy and dx, m runs over all batch elements' rows: dw and db are
 *   summed over the batch (one weight, used by every element: its partials add up, Section 4.2). */
relay_status_t relay_fused_dense_act_grad(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *y,
                                          const relay_tensor_t *dy, int32_t act, const relay_tensor_t *dx,
                                          const relay_tensor_t *dw, const relay_tensor_t *db, void *ws,
                                          size_t ws_bytes, void *stream);

/* conv2d anchor (Fig. 3 relay.conv2d) as cross-correlation with zero padding, run as an
 * implicit GEMM and fused with per-channel bias and activation:
 *   y[n,o,p,q] = act( b[o] + sum_{c,r,s} x[n,c,p*st-pad+r,q*st-pad+s] * w[o,c,r,s] ).
 *   x:(N,C,H,W) NCHW  w:(O,C,R,S) OIHW  b:(O) or NULL  ->  y:(N,O,P,Q) NCHW.
 * Layout-tagged activations (Section 5.2 names layout change among the operator-level optimisations): x may
 * instead be tagged RELAY_NHWC with shape (N,H,W,C); then y is NHWC of shape (N,P,Q,O) (and in the gradient
 * group y, dy, dx are NHWC too); w stays OIHW.  Same values, other memory order: the call converts through
 * the workspace (the bf16 3x3 tensor-core instance reads an NHWC x as it is). */
relay_status_t relay_fused_conv2d_act(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *b,
                                      const relay_conv2d_attrs_t *attrs, int32_t act, const relay_tensor_t *y,
                                      void *ws, size_t ws_bytes, void *stream);

/* Gradient group of the conv2d anchor (Section 4.2), dZ = dy (.) act'(y) as above:
 *   dx[n,c,i,j]  = sum_{o,r,s} dZ[n,o,p,q] w[o,c,r,s]   over (p,q) with p*st-pad+r=i, q*st-pad+s=j
 *   dw[o,c,r,s]  = sum_{n,p,q} dZ[n,o,p,q] x[n,c,p*st-pad+r,q*st-pad+s]
 *   db[o]        = sum_{n,p,q} dZ[n,o,p,q]
 *   dx, db may be NULL; dw is required. */
relay_status_t relay_fused_conv2d_act_grad(const relay_tensor_t *x, const relay_tensor_t *w, const relay_tensor_t *y,
                                           const relay_tensor_t *dy, const relay_conv2d_attrs_t *attrs, int32_t act,
                                           const relay_tensor_t *dx, const relay_tensor_t *dw,
                                           const relay_tensor_t *db, void *ws, size_t ws_bytes, void *stream);

/* Fused broadcast-elementwise group (Fig. 1 BinOp/UnaryOp/cast; Fig. 5 typing; Section 5.2
 * operator fusion): evaluates `prog` at every index of the broadcast shape and stores the
 * values named in out_values[0..n_out) to outputs[k], whose type must equal the value's
 * inferred type (full broadcast shape). */
relay_status_t relay_fused_ewise(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                 const int32_t *out_values, const relay_tensor_t *const *outputs, int32_t n_out,
                                 void *ws, size_t ws_bytes, void *stream);

/* Fused elementwise + reduce group (Fig. 3 relay.argmax and the reduction inside
 * softmax_cross_entropy; the column sums a gradient program needs where a value was broadcast,
 * Section 5.2 "summing in the correct places"): evaluates `prog` (may have 0 instructions) and
 * for each spec stores the value unreduced or reduced.  sum/max/mean outputs are f32 (bf16
 * allowed for unreduced values per their type); argmax outputs are i64 positions inside the
 * reduced axes, the first maximum winning.  Reductions are deterministic. */
relay_status_t relay_fused_reduce(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                  const relay_out_spec_t *specs, const relay_tensor_t *const *outputs,
                                  int32_t n_out, void *ws, size_t ws_bytes, void *stream);

/* The same group as relay_fused_reduce, for callers that cannot allocate device memory (the paper
 * has no counterpart; this is a convenience of this library).  Some users of this ABI run where
 * cudaMalloc is not an option: inside a host framework whose memory pool they may not touch, in
 * a plug-in that is handed only its input and output buffers, or in a phase of a program where
 * allocation is forbidden.  They still pass inputs and outputs, but no workspace: the scratch for
 * the per-slice partial sums is a fixed array of RELAY_STATIC_SCRATCH_BYTES inside the library's
 * device image (each GPU that loads the library holds one copy until the process exits).
 *   - A group whose kernels would use more scratch than RELAY_STATIC_SCRATCH_BYTES is rejected
 *     with RELAY_ERR_WORKSPACE before anything is launched; use relay_fused_reduce then.  (What
 *     counts is what the group really uses, which is at most relay_workspace_bytes_reduce():
 *     a reduction over the last axis, for one, uses none and is never rejected.)
 *   - The call allocates nothing, on the device or through any allocating library routine.  That
 *     includes compiling a body for a program at run time: here a program uses a compiled body only
 *     if an earlier relay_fused_reduce / relay_fused_ewise call already compiled it, and runs on
 *     the library's built-in kernels otherwise (same results within the same tolerance).
 *   - The first call on each device looks up the array's device address (a one-time set-up with
 *     that device current); make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps whatever the last call left there.  A call
 *     overwrites every word it later reads, so no clearing is needed between calls; but two
 *     calls that overlap in time on the same GPU (different streams or threads) race on it --
 *     serialise them. */
#define RELAY_STATIC_SCRATCH_BYTES (8u << 20)
relay_status_t relay_fused_reduce_static_scratch(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs,
                                                 int32_t n_in, const relay_out_spec_t *specs,
                                                 const relay_tensor_t *const *outputs, int32_t n_out, void *stream);

/* LSTM cell applied over a sequence (a recursive program over time composed of the dense
 * anchor and elementwise gates; recursion is what Section 3.1 adds over dataflow graphs).
 * Gate blocks along the 4H axis are [ i | f | g | o ]:
 *   z = x_t w_ih + bf16(h) w_hh + b;  i,f,o = sigmoid(z_i,z_f,z_o);  g = tanh(z_g);
 *   c = f (.) c + i (.) g;  h = o (.) tanh(c)                      (c, h kept in f32)
 *   x:(T,B,I) bf16  w_ih:(I,4H) bf16  w_hh:(H,4H) bf16  b:(4H) f32  h0,c0:(B,H) f32
 *   -> h_all:(T,B,H) f32, c_final:(B,H) f32. */
relay_status_t relay_lstm_cell_seq(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                   const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                   const relay_tensor_t *h_all, const relay_tensor_t *c_final, void *ws,
                                   size_t ws_bytes, void *stream);

/* Gradient program of the LSTM sequence (Section 4.2: reverse mode through the recursion over time).
 * Given the saved forward result h_all and the partials dh_all:(T,B,H) f32 of the final scalar with respect
 * to every emitted h_t and dc_final:(B,H) f32 with respect to the final cell state (NULL = zero), for
 * t = T-1 .. 0:
 *   dh = dh_all[t] + dz_{t+1} w_hh^T;   do = dh (.) tanh(c_t);   dc = dc_next + dh (.) o (.) (1 - tanh(c_t)^2)
 *   di = dc (.) g;  df = dc (.) c_{t-1};  dg = dc (.) i;  dc_next = dc (.) f
 *   dz_t = bf16( [ di i(1-i) | df f(1-f) | dg (1-g^2) | do o(1-o) ] )      (the bf16 operand of four contractions)
 * and then  dx[t] = dz_t w_ih^T,  dw_ih = sum_t x_t^T dz_t,  dw_hh = sum_t bf16(h_{t-1})^T dz_t,
 * db = sum_t sum_rows dz_t,  dh0 = dz_0 w_hh^T,  dc0 = dc_next after t = 0.
 *   inputs as relay_lstm_cell_seq plus h_all (its output);  dx:(T,B,I) bf16 or NULL;  dw_ih:(I,4H) bf16;
 *   dw_hh:(H,4H) bf16;  db:(4H) f32 or NULL;  dh0, dc0:(B,H) f32 or NULL.
 * Gates and cell states are recomputed from x and h_all (nothing else is saved by the forward call).
 * `ws` must hold relay_workspace_bytes_lstm_grad() bytes. */
relay_status_t relay_lstm_cell_seq_grad(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                        const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                        const relay_tensor_t *h_all, const relay_tensor_t *dh_all, const relay_tensor_t *dc_final,
                                        const relay_tensor_t *dx, const relay_tensor_t *dw_ih, const relay_tensor_t *dw_hh,
                                        const relay_tensor_t *db, const relay_tensor_t *dh0, const relay_tensor_t *dc0, void *ws,
                                        size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Loss and parameter update: the two operators that close the training step of the LeNet listing
 * (Fig. 3: relay.softmax_cross_entropy(scores, y), relay.update_model_params(model, model_grad)).
 * ------------------------------------------------------------------------------------------- */

/* Softmax cross-entropy, one loss per row (the listing's loss is per sample; a batch adds the leading
 * axis, Section 5.2 "auto-batching"):
 *   p[i,j] = exp(z[i,j]) / sum_k exp(z[i,k]);   loss[i] = - sum_j t[i,j] log p[i,j]
 *   scores z:(B,C) t in {f32, bf16};  targets t:(B,C) of base type t or f32 (a Float tensor of the scores'
 *   shape, as in the listing: a one-hot row or any weighting of the classes);  loss:(B) f32.
 * Arithmetic in f32.  One pass over z and t; no workspace.  B = 0 is a no-op; C = 0 is RELAY_ERR_SHAPE.
 * Check order as everywhere: null, rank, dtype, layout, shape, alignment.  Device pointers; outputs may
 * not overlap inputs. */
relay_status_t relay_infer_softmax_xent(const relay_tensor_t *scores, const relay_tensor_t *targets, relay_tensor_t *loss);
relay_status_t relay_softmax_xent(const relay_tensor_t *scores, const relay_tensor_t *targets, const relay_tensor_t *loss,
                                  void *stream);

/* Gradient group of the loss (Section 4.2: returns the result together with the partial): given the partial
 * dloss:(B) f32 of the final scalar with respect to loss,
 *   dscores[i,j] = dloss[i] * ( p[i,j] * sum_k t[i,k] - t[i,j] )        dscores:(B,C) of the scores' type
 * and, if `loss` is not NULL, loss:(B) f32 as above, from the same pass over z and t. */
relay_status_t relay_softmax_xent_grad(const relay_tensor_t *scores, const relay_tensor_t *targets, const relay_tensor_t *dloss,
                                       const relay_tensor_t *loss, const relay_tensor_t *dscores, void *stream);

/* Max pooling of an NCHW tensor (Fig. 3 relay.max_pool), windows without padding:
 *   y[n,c,p,q]   = max_{r<kh, s<kw} x[n,c,p*sh+r, q*sw+s],   P = floor((H-kh)/sh)+1, Q = floor((W-kw)/sw)+1
 *   idx[n,c,p,q] = (p*sh+r)*W + (q*sw+s) of the first maximum in (r,s) row-major order   (i32, optional)
 *   x:(N,C,H,W) f32 or bf16, NCHW;  y:(N,C,P,Q) same base type;  idx:(N,C,P,Q) i32 or NULL.
 * y and idx are bit-exact functions of x.  H*W must fit an i32.  RELAY_ERR_ATTR for a window that is not
 * positive or does not fit the plane. */
relay_status_t relay_infer_max_pool2d(const relay_tensor_t *x, const relay_pool2d_attrs_t *attrs, relay_tensor_t *out);
relay_status_t relay_max_pool2d(const relay_tensor_t *x, const relay_pool2d_attrs_t *attrs, const relay_tensor_t *y,
                                const relay_tensor_t *idx, void *stream);

/* Gradient of max pooling (Section 4.2): each window adds its dy to the input that attained the maximum,
 * every other input gets zero:  dx[n,c,h,w] = sum over the windows (p,q) with idx[n,c,p,q] = h*W+w of dy[n,c,p,q],
 * summed in (p,q) order (deterministic; overlapping windows may name the same input).
 *   idx:(N,C,P,Q) i32 from the forward call;  dy:(N,C,P,Q);  dx:(N,C,H,W) of dy's base type, with the same
 *   attrs as the forward call (P and Q must be what they give for dx's H and W).
 * An idx entry outside its window contributes nothing. */
relay_status_t relay_max_pool2d_grad(const relay_tensor_t *idx, const relay_tensor_t *dy, const relay_pool2d_attrs_t *attrs,
                                     const relay_tensor_t *dx, void *stream);

/* Vanilla stochastic gradient descent on a set of parameters (Section 4.1: update_model_params is the one
 * place where the paper exposes mutation): for k < n_params, elementwise and IN PLACE,
 *   params[k] <- cast( params[k] - lr * grads[k] )
 *   params[k]: any rank <= 6, f32 or bf16;  grads[k]: same shape, the parameter's base type or f32.
 * Arithmetic in f32, one rounding to the parameter's type.  All tensors are updated by one launch per 8
 * parameters.  A parameter may not overlap any other parameter or gradient.  n_params = 0 is a no-op. */
relay_status_t relay_sgd_update(const relay_tensor_t *const *params, const relay_tensor_t *const *grads, int32_t n_params,
                                float lr, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Status helpers.
 * ------------------------------------------------------------------------------------------- */

/* Thread-local text describing the last non-OK status returned on this thread ("" if none). */
const char *relay_last_error(void);

/* The contraction that the dense groups are built from, as a primitive operator of its own (Fig. 3 relay.linear without
 * its hidden parameters; the adjoints that Section 4.2's reverse mode needs are the same product with one operand
 * transposed):   c[m,n] = act( sum_k A(m,k) * B(k,n) + bias[n] ),  A = a or a^T, B = b or b^T (trans_* != 0), the
 * transposed operand being READ in place, never materialised.
 *   a:(M,K) or (K,M)  b:(K,N) or (N,K)  bias:(N) or NULL  ->  c:(M,N); a and b share one dtype t in {f32, bf16};
 *   c has dtype t or f32 (the fp32 accumulator stored unrounded); bias has dtype t or f32.
 *   trans_a = trans_b = 0 is relay_fused_dense_act; (0,1) computes dx = dZ w^T and (1,0) dw = x^T dZ of its gradient
 *   group.  Device pointers, caller-owned; needs no workspace; K = 0 gives act(bias).  Errors as everywhere
 *   (null -> rank -> dtype -> layout -> shape -> attr -> alignment/overlap), detected before any launch. */
relay_status_t relay_contract_act(const relay_tensor_t *a, int32_t trans_a, const relay_tensor_t *b, int32_t trans_b,
                                  const relay_tensor_t *bias, int32_t act, const relay_tensor_t *c, void *stream);

/* Synchronises `stream`, then reads and clears (in one atomic step, enqueued on `stream`) the device-side error word
 * of the current device: RELAY_ERR_TIMEOUT if a bounded wait expired in any kernel since the last poll,
 * RELAY_ERR_CUDA if the stream reports an error, else RELAY_OK.  The word belongs to the device, not to a stream:
 * a poll also reports, and consumes, a time-out raised by work of another stream. */
relay_status_t relay_poll_status(void *stream);

/* Self-test of the time-out path (no counterpart in the paper): enqueues a one-block kernel that
 * waits, for at most `limit_us` microseconds (1..1000000), on a hardware barrier that nothing ever
 * signals, then gives up, records the time-out in the device error word and exits normally.  The next
 * relay_poll_status() therefore returns RELAY_ERR_TIMEOUT and clears the word; the context stays usable.
 * It shows a caller that an expired wait in any kernel of this library is reported rather than hung on. */
relay_status_t relay_debug_expire_wait(int32_t limit_us, void *stream);

/* Self-test of the bounds-check build (no counterpart in the paper).  The library can be built with
 * -DRELAY_BOUNDS_CHECK (librelay_b200_check.so): the memory-bound and SIMT kernels then look every global address they
 * compute up in the ranges of the call's tensors and workspace, skip an access that lies outside and record it in the
 * device error word, so that relay_poll_status() returns RELAY_ERR_CUDA ("bounds check failed") instead of the kernel
 * faulting.  This call registers one 16-byte range and has a kernel look up (not access) the address just behind it:
 * in the check build the next relay_poll_status() reports the failed check; in the ordinary build the call returns
 * RELAY_ERR_UNSUPPORTED. */
relay_status_t relay_debug_bounds_probe(void *stream);

/* Run-time compiled bodies (Section 4.1: an operator group is fused into ONE kernel generated for that group).  A fused
 * elementwise or elementwise + column-sum group over the collapsed 2-D view that has no pre-compiled body is written out
 * as the per-element body of a kernel, compiled for this GPU by the NVRTC library when that library can be loaded at run
 * time, cached for the life of the process (first call of a new program: some hundred milliseconds on the host), and
 * launched like any other kernel; without the library, in the bounds-check build, or when switched off here, the same
 * groups run on the library's in-kernel interpreter.  relay_debug_set_jit switches the compiled bodies on (non-zero,
 * the default) or off for the process and returns the previous setting; relay_debug_jit_compiled returns how many
 * bodies have been compiled so far, -1 when compiled bodies cannot be used in this process (no run-time compiler
 * library, no CUDA driver, the bounds-check build).  Neither touches the GPU. */
int32_t relay_debug_set_jit(int32_t enabled);
int32_t relay_debug_jit_compiled(void);
/* Host only (needs no GPU): generates the source of the body that would be compiled at run time for this group and
 * compiles it for sm_100a.  Returns 1 if it compiled (its text, NUL-terminated and cut to `cap` bytes, is copied to `src`
 * when that is not NULL), 0 if the group does not run on that tier, -1 without a run-time compiler, -2 if the source did
 * not compile (relay_last_error() has the compiler's messages), -3 if the group does not type-check. */
int32_t relay_debug_jit_compile(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                const relay_out_spec_t *specs, int32_t n_out, char *src, size_t cap);

/* Host-only view of how the two-SM contraction kernel cuts an M x N output (contraction length K) into work units
 * for `sms` SMs (no counterpart in the paper; touches no GPU): fills units[i] = row block (256 rows) |
 * first 128-column chunk << 12 | width in chunks << 24, in the order the kernel hands them to its SM pairs
 * (pair p takes units p, p + sms/2, ...).  Returns the number of units, -1 if the shape is too large for a list
 * (the kernel then follows its fixed scheme), -2 for bad arguments or max_units too small.  For tests of the plan. */
int32_t relay_debug_plan_units(int64_t M, int64_t N, int64_t K, int32_t sms, uint32_t *units, int32_t max_units);

/* relay_lstm_cell_seq with a per-phase cycle count of its dependent steps (no counterpart in the paper; same arguments and
 * results).  `cycles` is a DEVICE pointer to 8 int64 that one block of the persistent kernel fills with SM-clock cycle
 * counts summed over the T steps: [0] the whole step loop, [1] the epilogue warp waiting for the recurrent product,
 * [2] the epilogue (accumulator read, gates, publishing bf16(h_t)), [3] the loader waiting on the grid barrier for
 * h_{t-1} of all blocks, [4] the loader issuing the step's copies, [5] the MMA issuer waiting for the step's first
 * operand stage, [6] the issuer from there to the step's last commit, [7] T.  RELAY_ERR_UNSUPPORTED for shapes that run
 * one launch per step instead of the persistent kernel. */
relay_status_t relay_debug_lstm_phase_cycles(const relay_tensor_t *x, const relay_tensor_t *w_ih, const relay_tensor_t *w_hh,
                                             const relay_tensor_t *b, const relay_tensor_t *h0, const relay_tensor_t *c0,
                                             const relay_tensor_t *h_all, const relay_tensor_t *c_final, void *ws, size_t ws_bytes,
                                             int64_t *cycles, void *stream);

/* Host-only view of which kernel tier relay_fused_ewise / relay_fused_reduce would run a group on (no counterpart in the
 * paper; touches no GPU; arguments as for relay_fused_reduce, all-RELAY_RED_NONE specs describe a relay_fused_ewise call):
 * 0 a pre-compiled body, 1 the vectorised tier (16-byte accesses over the collapsed 2-D view: a body compiled at run
 * time where that is available, else the program interpreted on 16 elements at a time), 2 the scalar evaluator (any
 * rank, broadcast pattern, axes mask and base type), 3 the row-reduction kernel;
 * -1 if the group does not type-check (relay_last_error() says why).  For tests and for callers that want to know
 * whether a program takes the fast route. */
int32_t relay_debug_group_route(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                                const relay_out_spec_t *specs, int32_t n_out);

/* Number of kernels this library has launched on this process so far (monotonic counter). */
int64_t relay_launch_count(void);

/* Library version string. */
const char *relay_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RELAY_B200_H_ */
