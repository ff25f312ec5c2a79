/*
 * relay_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded fp64 evaluator of the primitive-operator groups a Relay
 * program executes (paper: Section 3 grammar, Fig. 1; Section 4.3 typing rules, Fig. 5;
 * Section 4.2 reverse-mode automatic differentiation).  It plays the role the paper gives its
 * interpreter: a reference used for differential testing (Section 5.1).  It is NOT a product
 * path: nothing outside the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it, and it shares no code with the CUDA library.
 *
 * Conventions
 *   - every tensor is a dense row-major array of double; values of narrower stored types
 *     (bf16, fp32) are held exactly;
 *   - all arithmetic is fp64; a value is rounded only where the program says "cast"
 *     (Fig. 1, production "( Type ) Expr") or where a result is stored in a declared dtype;
 *   - sums run in increasing index order of the contracted / reduced index;
 *   - parity status: every function below is pinned by tests/test_oracle_*.py (closed forms,
 *     brute force, finite differences, adjoint identities, independent second routes).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* dtype codes (same numbering as the C-ABI header; the table is restated here on purpose) */
enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_I32 = 2, ORC_I64 = 3, ORC_BOOL = 4, ORC_F64 = 5 };

/* activation codes */
enum { ORC_ACT_NONE = 0, ORC_ACT_RELU = 1, ORC_ACT_TANH = 2, ORC_ACT_SIGMOID = 3 };

/* elementwise opcodes: Fig. 1 BinOp / UnaryOp productions plus the library operators of the
 * LeNet listing (Fig. 3) that are elementwise */
enum {
    ORC_OP_ADD = 0, ORC_OP_SUB = 1, ORC_OP_MUL = 2, ORC_OP_DIV = 3,
    ORC_OP_NEG = 4, ORC_OP_SQ = 5,
    ORC_OP_NE = 6, ORC_OP_EQ = 7, ORC_OP_LT = 8, ORC_OP_LE = 9, ORC_OP_GT = 10, ORC_OP_GE = 11,
    ORC_OP_SELECT = 12, ORC_OP_RELU = 13, ORC_OP_TANH = 14, ORC_OP_SIGMOID = 15,
    ORC_OP_CAST = 16, ORC_OP_CONST = 17, ORC_OP_EXP = 18, ORC_OP_LOG = 19,
    ORC_OP_MAX = 20, ORC_OP_MIN = 21
};

/* reduction codes */
enum { ORC_RED_NONE = 0, ORC_RED_SUM = 1, ORC_RED_MAX = 2, ORC_RED_MEAN = 3, ORC_RED_ARGMAX = 4 };

#define ORC_MAX_RANK 6
#define ORC_MAX_VALUES 64

/* ------------------------------------------------------------------------------------------
 * Casts.  Round-to-nearest-even from fp64 straight to the target format (one rounding).
 * bf16 = 1 sign, 8 exponent, 7 stored fraction bits: 8 significant bits, exponent range of
 * binary32, gradual underflow kept.
 * ---------------------------------------------------------------------------------------- */
double orc_round_bf16(double v)
{
    if (v == 0.0 || !isfinite(v)) return v;
    int e;
    double m = frexp(v, &e);            /* v = m * 2^e with 0.5 <= |m| < 1 */
    int p = 8;                          /* significant bits kept */
    const int emin = -125;              /* smallest e of a normal binary32/bf16 number */
    if (e < emin) p -= (emin - e);      /* subnormal: fewer bits survive */
    if (p < 0) return copysign(0.0, v); /* below half the smallest subnormal */
    double r = nearbyint(ldexp(m, p));  /* ties to even in the default rounding mode */
    double out = ldexp(r, e - p);
    const double bf16_max = 3.3895313892515355e38; /* 0x7F7F */
    if (fabs(out) > bf16_max) return copysign(INFINITY, v);
    return out;
}

double orc_round_f32(double v)
{
    return (double)(float)v; /* IEEE conversion, round to nearest even */
}

double orc_cast(double v, int dtype)
{
    switch (dtype) {
    case ORC_F32:  return orc_round_f32(v);
    case ORC_BF16: return orc_round_bf16(v);
    case ORC_I32:
    case ORC_I64:  return trunc(v);
    case ORC_BOOL: return v != 0.0 ? 1.0 : 0.0;
    default:       return v;
    }
}

/* ------------------------------------------------------------------------------------------
 * Scalar library operators and their derivatives written from the saved output
 * (a gradient program consumes saved forward values).
 * ---------------------------------------------------------------------------------------- */
static double sigmoid_(double x) { return 1.0 / (1.0 + exp(-x)); }

double orc_act(double z, int act)
{
    switch (act) {
    case ORC_ACT_RELU:    return z > 0.0 ? z : 0.0;
    case ORC_ACT_TANH:    return tanh(z);
    case ORC_ACT_SIGMOID: return sigmoid_(z);
    default:              return z;
    }
}

/* d act / d z expressed through y = act(z) */
double orc_act_grad_from_output(double y, int act)
{
    switch (act) {
    case ORC_ACT_RELU:    return y > 0.0 ? 1.0 : 0.0;   /* relu'(0) = 0 */
    case ORC_ACT_TANH:    return 1.0 - y * y;
    case ORC_ACT_SIGMOID: return y * (1.0 - y);
    default:              return 1.0;
    }
}

/* ------------------------------------------------------------------------------------------
 * Elementwise program over broadcast inputs.
 *
 * The output has shape out_shape[rank].  Input i has shape in_shapes[i*rank .. i*rank+rank)
 * already right-aligned to the output rank (missing leading axes given as 1); an axis of
 * extent 1 in an input is replicated along the output axis (the explicit broadcast step that
 * precedes Fig. 5's same-shape rules).  Value ids: 0..n_in-1 are the inputs, n_in+j is the
 * result of instruction j (a let-list, Fig. 1 "let").  Returns 0, or a negative code for a
 * malformed program / illegal broadcast.
 * ---------------------------------------------------------------------------------------- */
static int eval_instr(int op, double x, double y, double z, double imm, int dt, double *r)
{
    switch (op) {
    case ORC_OP_ADD: *r = x + y; break;
    case ORC_OP_SUB: *r = x - y; break;
    case ORC_OP_MUL: *r = x * y; break;
    case ORC_OP_DIV: *r = x / y; break;
    case ORC_OP_NEG: *r = -x; break;
    case ORC_OP_SQ:  *r = x * x; break;
    case ORC_OP_NE:  *r = (x != y) ? 1.0 : 0.0; break;
    case ORC_OP_EQ:  *r = (x == y) ? 1.0 : 0.0; break;
    case ORC_OP_LT:  *r = (x <  y) ? 1.0 : 0.0; break;
    case ORC_OP_LE:  *r = (x <= y) ? 1.0 : 0.0; break;
    case ORC_OP_GT:  *r = (x >  y) ? 1.0 : 0.0; break;
    case ORC_OP_GE:  *r = (x >= y) ? 1.0 : 0.0; break;
    case ORC_OP_SELECT: *r = (x != 0.0) ? y : z; break;
    case ORC_OP_RELU: *r = x > 0.0 ? x : 0.0; break;
    case ORC_OP_TANH: *r = tanh(x); break;
    case ORC_OP_SIGMOID: *r = sigmoid_(x); break;
    case ORC_OP_CAST: *r = orc_cast(x, dt); break;
    case ORC_OP_CONST: *r = orc_cast(imm, dt); break;
    case ORC_OP_EXP: *r = exp(x); break;
    case ORC_OP_LOG: *r = log(x); break;
    case ORC_OP_MAX: *r = x > y ? x : y; break;
    case ORC_OP_MIN: *r = x < y ? x : y; break;
    default: return -1;
    }
    return 0;
}

static int check_program(int rank, const int64_t *out_shape, int n_in, const int64_t *in_shapes,
                         int n_instr, const int32_t *a, const int32_t *b, const int32_t *c,
                         int n_out, const int32_t *out_ids)
{
    if (rank < 0 || rank > ORC_MAX_RANK) return -2;
    if (n_in < 0 || n_instr < 0 || n_in + n_instr > ORC_MAX_VALUES) return -3;
    for (int i = 0; i < n_in; ++i)
        for (int d = 0; d < rank; ++d) {
            int64_t s = in_shapes[i * rank + d];
            if (s != out_shape[d] && s != 1) return -4; /* not broadcastable */
        }
    for (int j = 0; j < n_instr; ++j) {
        int lim = n_in + j; /* an instruction may only name earlier values */
        if (a[j] >= lim || b[j] >= lim || c[j] >= lim) return -5;
    }
    for (int k = 0; k < n_out; ++k)
        if (out_ids[k] < 0 || out_ids[k] >= n_in + n_instr) return -6;
    return 0;
}

/* evaluates all values of the program at one output multi-index */
static int eval_point(int rank, const int64_t *idx, int n_in, const double *const *in,
                      const int64_t *in_shapes, int n_instr, const int32_t *op, const int32_t *a,
                      const int32_t *b, const int32_t *c, const double *imm, const int32_t *dt,
                      double *vals)
{
    for (int i = 0; i < n_in; ++i) {
        int64_t off = 0;
        for (int d = 0; d < rank; ++d) {
            int64_t s = in_shapes[i * rank + d];
            int64_t id = (s == 1) ? 0 : idx[d];
            off = off * s + id;
        }
        vals[i] = in[i][off];
    }
    for (int j = 0; j < n_instr; ++j) {
        double x = a[j] >= 0 ? vals[a[j]] : 0.0;
        double y = b[j] >= 0 ? vals[b[j]] : 0.0;
        double z = c[j] >= 0 ? vals[c[j]] : 0.0;
        if (eval_instr(op[j], x, y, z, imm[j], dt[j], &vals[n_in + j]) != 0) return -1;
    }
    return 0;
}

int orc_ewise(int rank, const int64_t *out_shape, int n_in, const double *const *in,
              const int64_t *in_shapes, int n_instr, const int32_t *op, const int32_t *a,
              const int32_t *b, const int32_t *c, const double *imm, const int32_t *dt, int n_out,
              const int32_t *out_ids, double *const *out)
{
    int rc = check_program(rank, out_shape, n_in, in_shapes, n_instr, a, b, c, n_out, out_ids);
    if (rc) return rc;
    int64_t total = 1;
    for (int d = 0; d < rank; ++d) total *= out_shape[d];
    int64_t idx[ORC_MAX_RANK] = {0};
    double vals[ORC_MAX_VALUES];
    for (int64_t lin = 0; lin < total; ++lin) {
        int64_t rem = lin;
        for (int d = rank - 1; d >= 0; --d) { idx[d] = rem % out_shape[d]; rem /= out_shape[d]; }
        if (eval_point(rank, idx, n_in, in, in_shapes, n_instr, op, a, b, c, imm, dt, vals)) return -1;
        for (int k = 0; k < n_out; ++k) out[k][lin] = vals[out_ids[k]];
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Reduce group: the same elementwise program, then per output k either nothing
 * (ORC_RED_NONE: the value is returned unreduced) or a reduction over the axes whose bit is
 * set in axes_mask[k].  The reduced output is laid out row-major over the surviving axes
 * (keeping them as extent 1 does not change the layout).  Sums run in increasing index
 * order; argmax returns the row-major position inside the reduced axes of the FIRST maximum
 * (for a single axis: the lowest index along that axis).  out_dt[k] is the dtype the result
 * is stored in (applied once, after the reduction).
 * ---------------------------------------------------------------------------------------- */
int orc_reduce(int rank, const int64_t *out_shape, int n_in, const double *const *in,
               const int64_t *in_shapes, int n_instr, const int32_t *op, const int32_t *a,
               const int32_t *b, const int32_t *c, const double *imm, const int32_t *dt, int n_out,
               const int32_t *out_ids, const int32_t *red_op, const int32_t *axes_mask,
               const int32_t *out_dt, double *const *out)
{
    int rc = check_program(rank, out_shape, n_in, in_shapes, n_instr, a, b, c, n_out, out_ids);
    if (rc) return rc;
    int64_t total = 1;
    for (int d = 0; d < rank; ++d) total *= out_shape[d];

    int64_t kept_total[ORC_MAX_VALUES];
    int64_t red_count[ORC_MAX_VALUES];
    double *best[ORC_MAX_VALUES];
    if (n_out > ORC_MAX_VALUES) return -7;
    for (int k = 0; k < n_out; ++k) {
        best[k] = NULL;
        kept_total[k] = 1; red_count[k] = 1;
        for (int d = 0; d < rank; ++d) {
            if (axes_mask[k] & (1 << d)) red_count[k] *= out_shape[d];
            else kept_total[k] *= out_shape[d];
        }
        if (red_op[k] == ORC_RED_NONE) continue;
        if (red_count[k] == 0) return -8;
        for (int64_t i = 0; i < kept_total[k]; ++i)
            out[k][i] = (red_op[k] == ORC_RED_MAX) ? -INFINITY : 0.0;
        if (red_op[k] == ORC_RED_ARGMAX) {
            best[k] = (double *)malloc(sizeof(double) * (size_t)(kept_total[k] ? kept_total[k] : 1));
            for (int64_t i = 0; i < kept_total[k]; ++i) best[k][i] = -INFINITY;
        }
    }

    int64_t idx[ORC_MAX_RANK] = {0};
    double vals[ORC_MAX_VALUES];
    for (int64_t lin = 0; lin < total; ++lin) {
        int64_t rem = lin;
        for (int d = rank - 1; d >= 0; --d) { idx[d] = rem % out_shape[d]; rem /= out_shape[d]; }
        if (eval_point(rank, idx, n_in, in, in_shapes, n_instr, op, a, b, c, imm, dt, vals)) return -1;
        for (int k = 0; k < n_out; ++k) {
            double v = vals[out_ids[k]];
            if (red_op[k] == ORC_RED_NONE) { out[k][lin] = v; continue; }
            int64_t kept = 0, pos = 0; /* row-major positions over kept / reduced axes */
            for (int d = 0; d < rank; ++d) {
                if (axes_mask[k] & (1 << d)) pos = pos * out_shape[d] + idx[d];
                else kept = kept * out_shape[d] + idx[d];
            }
            switch (red_op[k]) {
            case ORC_RED_SUM:
            case ORC_RED_MEAN: out[k][kept] += v; break;
            case ORC_RED_MAX:  if (v > out[k][kept]) out[k][kept] = v; break;
            case ORC_RED_ARGMAX:
                if (v > best[k][kept]) { best[k][kept] = v; out[k][kept] = (double)pos; }
                break;
            default: return -9;
            }
        }
    }
    for (int k = 0; k < n_out; ++k) {
        if (red_op[k] == ORC_RED_NONE) continue;
        for (int64_t i = 0; i < kept_total[k]; ++i) {
            double v = out[k][i];
            if (red_op[k] == ORC_RED_MEAN) v /= (double)red_count[k];
            if (red_op[k] != ORC_RED_ARGMAX) v = orc_cast(v, out_dt[k]);
            out[k][i] = v;
        }
        free(best[k]);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Dense anchor with broadcast bias and activation (Fig. 3, relay.linear followed by an
 * elementwise operator):  y[m,n] = cast( act( sum_k x[m,k] * W[k,n] + b[n] ) ).
 * The k-sum of every element runs in increasing k; the loop nest is m,k,n so that the rows
 * of W are walked contiguously (it interleaves the sums of one output row, it does not
 * reorder any of them).
 * ---------------------------------------------------------------------------------------- */
int orc_dense_act(const double *x, const double *w, const double *b, int64_t M, int64_t K,
                  int64_t N, int act, int y_dtype, double *y)
{
    double *acc = (double *)malloc(sizeof(double) * (size_t)(N ? N : 1));
    if (!acc) return -1;
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) acc[n] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double xv = x[m * K + k];
            const double *wr = w + k * N;
            for (int64_t n = 0; n < N; ++n) acc[n] += xv * wr[n];
        }
        for (int64_t n = 0; n < N; ++n) {
            double z = acc[n] + (b ? b[n] : 0.0);
            y[m * N + n] = orc_cast(orc_act(z, act), y_dtype);
        }
    }
    free(acc);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Dense gradient group (Section 4.2: reverse mode; dy is the partial derivative of the final
 * scalar with respect to y; every partial starts from zero and contributions are summed):
 *   dZ = dy (.) act'(y)           (act' written through the saved output y)
 *   dx[m,k] = sum_n dZ[m,n] W[k,n]
 *   dW[k,n] = sum_m x[m,k] dZ[m,n]
 *   db[n]   = sum_m dZ[m,n]
 * dZ is itself a typed value: the elementwise product of two tensors of base type t has type t
 * (Fig. 5, Type-Noncomp-BinaryOp), so it is rounded to dz_dtype before the contractions consume it
 * (dz_dtype = fp64 code keeps it exact).
 * Any of dx, dw, db may be NULL (not requested).  Results are stored in the given dtypes.
 * ---------------------------------------------------------------------------------------- */
int orc_dense_act_grad(const double *x, const double *w, const double *y, const double *dy,
                       int64_t M, int64_t K, int64_t N, int act, int dz_dtype, int dx_dtype,
                       int dw_dtype, int db_dtype, double *dx, double *dw, double *db)
{
    double *dz = (double *)malloc(sizeof(double) * (size_t)(M * N ? M * N : 1));
    if (!dz) return -1;
    for (int64_t i = 0; i < M * N; ++i)
        dz[i] = orc_cast(dy[i] * orc_act_grad_from_output(y[i], act), dz_dtype);
    if (dx) {
        for (int64_t m = 0; m < M; ++m)
            for (int64_t k = 0; k < K; ++k) {
                double s = 0.0;
                for (int64_t n = 0; n < N; ++n) s += dz[m * N + n] * w[k * N + n];
                dx[m * K + k] = orc_cast(s, dx_dtype);
            }
    }
    if (dw) {
        for (int64_t i = 0; i < K * N; ++i) dw[i] = 0.0;
        for (int64_t m = 0; m < M; ++m)          /* m outermost: each dW[k,n] sums in m order */
            for (int64_t k = 0; k < K; ++k) {
                double xv = x[m * K + k];
                for (int64_t n = 0; n < N; ++n) dw[k * N + n] += xv * dz[m * N + n];
            }
        for (int64_t i = 0; i < K * N; ++i) dw[i] = orc_cast(dw[i], dw_dtype);
    }
    if (db) {
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int64_t m = 0; m < M; ++m) s += dz[m * N + n];
            db[n] = orc_cast(s, db_dtype);
        }
    }
    free(dz);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Softmax cross-entropy loss (Fig. 3, relay.softmax_cross_entropy(scores, y); y is a Float tensor
 * of the scores' shape, e.g. a one-hot row or any non-negative weighting of the classes).  Per row i
 * of z[B,C] and t[B,C]:
 *   p[i,j]  = exp(z[i,j]) / sum_k exp(z[i,k])
 *   loss[i] = - sum_j t[i,j] * log p[i,j]
 * written with log p[i,j] = (z[i,j] - m_i) - log sum_k exp(z[i,k] - m_i), m_i = max_k z[i,k]: the same
 * number, without overflow of exp.  Sums run in increasing j.  loss is stored in loss_dtype.
 * ---------------------------------------------------------------------------------------- */
int orc_softmax_xent(const double *z, const double *t, int64_t B, int64_t C, int loss_dtype, double *loss)
{
    if (C <= 0) return 1;
    for (int64_t i = 0; i < B; ++i) {
        const double *zr = z + i * C, *tr = t + i * C;
        double m = zr[0];
        for (int64_t j = 1; j < C; ++j) if (zr[j] > m) m = zr[j];
        double se = 0.0;
        for (int64_t j = 0; j < C; ++j) se += exp(zr[j] - m);
        double lse = log(se), l = 0.0;
        for (int64_t j = 0; j < C; ++j) l -= tr[j] * ((zr[j] - m) - lse);
        loss[i] = orc_cast(l, loss_dtype);
    }
    return 0;
}

/* Gradient group of the loss (Section 4.2: the upstream partial dloss[i] of the final scalar with respect
 * to loss[i] is given; the result is returned alongside the partial):
 *   dz[i,j] = dloss[i] * ( p[i,j] * sum_k t[i,k] - t[i,j] )
 * (the derivative of -sum_j t_j (z_j - logsumexp z) with respect to z_j).  Only the partial with respect
 * to the scores is produced; the targets are data.  loss may be NULL. */
int orc_softmax_xent_grad(const double *z, const double *t, const double *dloss, int64_t B, int64_t C,
                          int loss_dtype, int dz_dtype, double *loss, double *dz)
{
    if (C <= 0) return 1;
    if (loss && orc_softmax_xent(z, t, B, C, loss_dtype, loss)) return 1;
    for (int64_t i = 0; i < B; ++i) {
        const double *zr = z + i * C, *tr = t + i * C;
        double m = zr[0];
        for (int64_t j = 1; j < C; ++j) if (zr[j] > m) m = zr[j];
        double se = 0.0, st = 0.0;
        for (int64_t j = 0; j < C; ++j) se += exp(zr[j] - m);
        for (int64_t j = 0; j < C; ++j) st += tr[j];
        for (int64_t j = 0; j < C; ++j) {
            double pj = exp(zr[j] - m) / se;
            dz[i * C + j] = orc_cast(dloss[i] * (pj * st - tr[j]), dz_dtype);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Max pooling over windows of an NCHW tensor (Fig. 3, relay.max_pool(x, ksize, strides)), no padding:
 *   y[n,c,p,q]   = max_{r<kh, s<kw} x[n,c,p*sh+r, q*sw+s]
 *   idx[n,c,p,q] = (p*sh+r)*W + (q*sw+s) of the FIRST maximum in (r,s) row-major order
 * with P = floor((H-kh)/sh)+1, Q = floor((W-kw)/sw)+1.  idx may be NULL.  Returns 1 if a window does
 * not fit (kh > H or kw > W) or an attribute is not positive.
 * ---------------------------------------------------------------------------------------- */
int orc_max_pool2d(const double *x, int64_t Nb, int64_t C, int64_t H, int64_t W, int64_t kh, int64_t kw,
                   int64_t sh, int64_t sw, double *y, int32_t *idx)
{
    if (kh <= 0 || kw <= 0 || sh <= 0 || sw <= 0 || kh > H || kw > W) return 1;
    int64_t P = (H - kh) / sh + 1, Q = (W - kw) / sw + 1;
    for (int64_t nc = 0; nc < Nb * C; ++nc) {
        const double *xp = x + nc * H * W;
        for (int64_t p = 0; p < P; ++p)
            for (int64_t q = 0; q < Q; ++q) {
                int64_t best = (p * sh) * W + q * sw;
                for (int64_t r = 0; r < kh; ++r)
                    for (int64_t t = 0; t < kw; ++t) {
                        int64_t at = (p * sh + r) * W + (q * sw + t);
                        if (xp[at] > xp[best]) best = at;        /* strict: the first maximum wins */
                    }
                y[(nc * P + p) * Q + q] = xp[best];
                if (idx) idx[(nc * P + p) * Q + q] = (int32_t)best;
            }
    }
    return 0;
}

/* Gradient of max pooling (Section 4.2): the partial of every input starts at zero and each window adds
 * its dy to the input that attained the maximum (idx from the forward pass), windows visited in (p,q)
 * order:  dx[n,c,idx[n,c,p,q]] += dy[n,c,p,q].  Stored in dx_dtype. */
int orc_max_pool2d_grad(const int32_t *idx, const double *dy, int64_t Nb, int64_t C, int64_t H, int64_t W,
                        int64_t P, int64_t Q, int dx_dtype, double *dx)
{
    for (int64_t i = 0; i < Nb * C * H * W; ++i) dx[i] = 0.0;
    for (int64_t nc = 0; nc < Nb * C; ++nc)
        for (int64_t o = 0; o < P * Q; ++o) {
            int32_t at = idx[nc * P * Q + o];
            if (at < 0 || at >= H * W) return 1;
            dx[nc * H * W + at] += dy[nc * P * Q + o];
        }
    for (int64_t i = 0; i < Nb * C * H * W; ++i) dx[i] = orc_cast(dx[i], dx_dtype);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Parameter update (Section 4.1, relay.update_model_params: vanilla stochastic gradient descent, the one
 * place where the paper allows mutation):  p <- cast( p - lr * g ), elementwise, stored in p's dtype.
 * ---------------------------------------------------------------------------------------- */
void orc_sgd_update(const double *p, const double *g, int64_t n, double lr, int p_dtype, double *p_new)
{
    for (int64_t i = 0; i < n; ++i) p_new[i] = orc_cast(p[i] - lr * g[i], p_dtype);
}

/* ------------------------------------------------------------------------------------------
 * conv2d anchor (Fig. 3, relay.conv2d) as cross-correlation, NCHW input, OIHW weights, zero
 * padding, square stride, with per-channel bias and activation:
 *   y[n,o,p,q] = cast( act( b[o] + sum_{c,r,s} x[n,c,p*st-pad+r,q*st-pad+s] * Wt[o,c,r,s] ) )
 * Output extent P = floor((H + 2 pad - R) / st) + 1 (same for Q with W, S).
 * ---------------------------------------------------------------------------------------- */
int orc_conv2d_out_extent(int64_t in, int64_t k, int64_t stride, int64_t pad, int64_t *out)
{
    if (stride <= 0 || pad < 0 || k <= 0 || in + 2 * pad < k) return -1;
    *out = (in + 2 * pad - k) / stride + 1;
    return 0;
}

int orc_conv2d_act(const double *x, const double *wt, const double *b, int64_t Nb, int64_t C,
                   int64_t H, int64_t W, int64_t O, int64_t R, int64_t S, int64_t stride,
                   int64_t pad, int act, int y_dtype, double *y)
{
    int64_t P, Q;
    if (orc_conv2d_out_extent(H, R, stride, pad, &P) || orc_conv2d_out_extent(W, S, stride, pad, &Q))
        return -1;
    for (int64_t n = 0; n < Nb; ++n)
        for (int64_t o = 0; o < O; ++o)
            for (int64_t p = 0; p < P; ++p)
                for (int64_t q = 0; q < Q; ++q) {
                    double acc = 0.0;
                    for (int64_t c = 0; c < C; ++c)
                        for (int64_t r = 0; r < R; ++r) {
                            int64_t i = p * stride - pad + r;
                            if (i < 0 || i >= H) continue;
                            for (int64_t s = 0; s < S; ++s) {
                                int64_t j = q * stride - pad + s;
                                if (j < 0 || j >= W) continue;
                                acc += x[((n * C + c) * H + i) * W + j] *
                                       wt[((o * C + c) * R + r) * S + s];
                            }
                        }
                    double z = acc + (b ? b[o] : 0.0);
                    y[((n * O + o) * P + p) * Q + q] = orc_cast(orc_act(z, act), y_dtype);
                }
    return 0;
}

/* conv2d gradient group (Section 4.2):
 *   dZ = cast(dy (.) act'(y), dz_dtype)      (a typed value, as in the dense gradient group)
 *   dx[n,c,i,j]   = sum_{o,r,s} dZ[n,o,p,q] Wt[o,c,r,s]  over the (p,q) with p*st-pad+r = i, q*st-pad+s = j
 *   dWt[o,c,r,s]  = sum_{n,p,q} dZ[n,o,p,q] x[n,c,p*st-pad+r,q*st-pad+s]   (in-range taps only)
 *   db[o]         = sum_{n,p,q} dZ[n,o,p,q]
 */
int orc_conv2d_act_grad(const double *x, const double *wt, const double *y, const double *dy,
                        int64_t Nb, int64_t C, int64_t H, int64_t W, int64_t O, int64_t R,
                        int64_t S, int64_t stride, int64_t pad, int act, int dz_dtype, int dx_dtype,
                        int dw_dtype, int db_dtype, double *dx, double *dw, double *db)
{
    int64_t P, Q;
    if (orc_conv2d_out_extent(H, R, stride, pad, &P) || orc_conv2d_out_extent(W, S, stride, pad, &Q))
        return -1;
    int64_t ny = Nb * O * P * Q;
    double *dz = (double *)malloc(sizeof(double) * (size_t)(ny ? ny : 1));
    if (!dz) return -1;
    for (int64_t i = 0; i < ny; ++i)
        dz[i] = orc_cast(dy[i] * orc_act_grad_from_output(y[i], act), dz_dtype);
    if (dx) {
        for (int64_t n = 0; n < Nb; ++n)
            for (int64_t c = 0; c < C; ++c)
                for (int64_t i = 0; i < H; ++i)
                    for (int64_t j = 0; j < W; ++j) {
                        double acc = 0.0;
                        for (int64_t o = 0; o < O; ++o)
                            for (int64_t r = 0; r < R; ++r) {
                                int64_t pn = i + pad - r;
                                if (pn < 0 || pn % stride) continue;
                                int64_t p = pn / stride;
                                if (p >= P) continue;
                                for (int64_t s = 0; s < S; ++s) {
                                    int64_t qn = j + pad - s;
                                    if (qn < 0 || qn % stride) continue;
                                    int64_t q = qn / stride;
                                    if (q >= Q) continue;
                                    acc += dz[((n * O + o) * P + p) * Q + q] *
                                           wt[((o * C + c) * R + r) * S + s];
                                }
                            }
                        dx[((n * C + c) * H + i) * W + j] = orc_cast(acc, dx_dtype);
                    }
    }
    if (dw) {
        for (int64_t o = 0; o < O; ++o)
            for (int64_t c = 0; c < C; ++c)
                for (int64_t r = 0; r < R; ++r)
                    for (int64_t s = 0; s < S; ++s) {
                        double acc = 0.0;
                        for (int64_t n = 0; n < Nb; ++n)
                            for (int64_t p = 0; p < P; ++p) {
                                int64_t i = p * stride - pad + r;
                                if (i < 0 || i >= H) continue;
                                for (int64_t q = 0; q < Q; ++q) {
                                    int64_t j = q * stride - pad + s;
                                    if (j < 0 || j >= W) continue;
                                    acc += dz[((n * O + o) * P + p) * Q + q] *
                                           x[((n * C + c) * H + i) * W + j];
                                }
                            }
                        dw[((o * C + c) * R + r) * S + s] = orc_cast(acc, dw_dtype);
                    }
    }
    if (db) {
        for (int64_t o = 0; o < O; ++o) {
            double acc = 0.0;
            for (int64_t n = 0; n < Nb; ++n)
                for (int64_t p = 0; p < P; ++p)
                    for (int64_t q = 0; q < Q; ++q) acc += dz[((n * O + o) * P + p) * Q + q];
            db[o] = orc_cast(acc, db_dtype);
        }
    }
    free(dz);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * LSTM cell applied over a sequence (a recursive program over time built from the dense
 * anchor and elementwise operators).  Gate blocks along the 4H axis: [ i | f | g | o ].
 *   hq      = cast(h, rec_dtype)                        (the recurrent matmul's input dtype)
 *   z       = x_t W_ih + hq W_hh + b                    [B, 4H]
 *   i,f,o   = sigmoid(z_i), sigmoid(z_f), sigmoid(z_o);  g = tanh(z_g)
 *   c       = cast(f (.) c + i (.) g, state_dtype)
 *   h       = cast(o (.) tanh(c), state_dtype)
 * x: [T,B,I], W_ih: [I,4H], W_hh: [H,4H], b: [4H], h0,c0: [B,H] -> h_all: [T,B,H], c_final: [B,H]
 * ---------------------------------------------------------------------------------------- */
int orc_lstm_cell_seq(const double *x, const double *w_ih, const double *w_hh, const double *b,
                      const double *h0, const double *c0, int64_t T, int64_t B, int64_t I,
                      int64_t H, int rec_dtype, int state_dtype, double *h_all, double *c_final)
{
    int64_t G = 4 * H;
    double *z = (double *)malloc(sizeof(double) * (size_t)(G ? G : 1));
    double *h = (double *)malloc(sizeof(double) * (size_t)(B * H ? B * H : 1));
    double *c = (double *)malloc(sizeof(double) * (size_t)(B * H ? B * H : 1));
    double *hq = (double *)malloc(sizeof(double) * (size_t)(H ? H : 1));
    if (!z || !h || !c || !hq) { free(z); free(h); free(c); free(hq); return -1; }
    for (int64_t i = 0; i < B * H; ++i) { h[i] = h0[i]; c[i] = c0[i]; }
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t bi = 0; bi < B; ++bi) {
            const double *xt = x + (t * B + bi) * I;
            for (int64_t j = 0; j < H; ++j) hq[j] = orc_cast(h[bi * H + j], rec_dtype);
            for (int64_t g = 0; g < G; ++g) z[g] = 0.0;
            for (int64_t k = 0; k < I; ++k) {
                double xv = xt[k];
                const double *wr = w_ih + k * G;
                for (int64_t g = 0; g < G; ++g) z[g] += xv * wr[g];
            }
            for (int64_t k = 0; k < H; ++k) {
                double hv = hq[k];
                const double *wr = w_hh + k * G;
                for (int64_t g = 0; g < G; ++g) z[g] += hv * wr[g];
            }
            for (int64_t g = 0; g < G; ++g) z[g] += b[g];
            for (int64_t j = 0; j < H; ++j) {
                double ig = sigmoid_(z[j]);
                double fg = sigmoid_(z[H + j]);
                double gg = tanh(z[2 * H + j]);
                double og = sigmoid_(z[3 * H + j]);
                double cn = orc_cast(fg * c[bi * H + j] + ig * gg, state_dtype);
                double hn = orc_cast(og * tanh(cn), state_dtype);
                c[bi * H + j] = cn;
                h[bi * H + j] = hn;   /* rows are independent, so updating in place is safe */
                h_all[(t * B + bi) * H + j] = hn;
            }
        }
    }
    for (int64_t i = 0; i < B * H; ++i) c_final[i] = c[i];
    free(z); free(h); free(c); free(hq);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Gradient program of the LSTM sequence (Section 4.2, reverse mode through the recursion over time).
 * Given dh_all[T,B,H] (the partial of the final scalar with respect to every emitted h_t) and
 * dc_final[B,H] (with respect to the final cell state; NULL = zero), the forward values are recomputed
 * exactly as orc_lstm_cell_seq computes them and kept per step, then for t = T-1 .. 0:
 *   dh   = dh_all[t] + dh_next                 (h_t is used twice: emitted, and fed to step t+1)
 *   do   = dh (.) tanh(c_t);        dc = dc_next + dh (.) o (.) (1 - tanh(c_t)^2)
 *   di   = dc (.) g;   df = dc (.) c_{t-1};   dg = dc (.) i;   dc_next = dc (.) f
 *   dz   = cast( [ di i(1-i) | df f(1-f) | dg (1-g^2) | do o(1-o) ], dz_dtype )
 *   db  += dz;   dx[t] = dz W_ih^T;   dW_ih += x_t^T dz;   dW_hh += hq_t^T dz;   dh_next = dz W_hh^T
 * and finally dh0 = dh_next, dc0 = dc_next.  hq_t = cast(h_{t-1}, rec_dtype) is the recurrent matmul's
 * input; the cast is treated as the identity when differentiating.  dz is a typed value (the operand of
 * four contractions), hence its cast.  Every partial starts from zero.  Any output pointer may be NULL.
 * Results are stored as fp64 (the caller rounds if it wants a narrower type).
 * ---------------------------------------------------------------------------------------- */
int orc_lstm_cell_seq_grad(const double *x, const double *w_ih, const double *w_hh, const double *b,
                           const double *h0, const double *c0, const double *dh_all, const double *dc_final,
                           int64_t T, int64_t B, int64_t I, int64_t H, int rec_dtype, int state_dtype, int dz_dtype,
                           double *dx, double *dw_ih, double *dw_hh, double *db, double *dh0, double *dc0)
{
    int64_t G = 4 * H, BH = B * H, BG = B * G;
    size_t nbh = (size_t)(T * BH ? T * BH : 1), nbg = (size_t)(T * BG ? T * BG : 1);
    double *hq = (double *)malloc(sizeof(double) * nbh);      /* hq[t] = cast(h_{t-1}) */
    double *cs = (double *)malloc(sizeof(double) * (nbh + (size_t)(BH ? BH : 1)));   /* cs[0] = c0, cs[t+1] = c_t */
    double *gt = (double *)malloc(sizeof(double) * nbg);      /* activated gates [i|f|g|o] per step */
    double *h = (double *)malloc(sizeof(double) * (size_t)(BH ? BH : 1));
    double *z = (double *)malloc(sizeof(double) * (size_t)(G ? G : 1));
    double *dz = (double *)malloc(sizeof(double) * (size_t)(BG ? BG : 1));
    double *dhn = (double *)malloc(sizeof(double) * (size_t)(BH ? BH : 1));
    double *dcn = (double *)malloc(sizeof(double) * (size_t)(BH ? BH : 1));
    if (!hq || !cs || !gt || !h || !z || !dz || !dhn || !dcn) {
        free(hq); free(cs); free(gt); free(h); free(z); free(dz); free(dhn); free(dcn);
        return -1;
    }
    /* forward, as in orc_lstm_cell_seq, keeping what the reverse sweep reads */
    for (int64_t i = 0; i < BH; ++i) { h[i] = h0[i]; cs[i] = c0[i]; }
    for (int64_t t = 0; t < T; ++t)
        for (int64_t bi = 0; bi < B; ++bi) {
            double *hqr = hq + (t * B + bi) * H, *gr = gt + (t * B + bi) * G;
            for (int64_t j = 0; j < H; ++j) hqr[j] = orc_cast(h[bi * H + j], rec_dtype);
            for (int64_t g = 0; g < G; ++g) z[g] = 0.0;
            for (int64_t k = 0; k < I; ++k)
                for (int64_t g = 0; g < G; ++g) z[g] += x[(t * B + bi) * I + k] * w_ih[k * G + g];
            for (int64_t k = 0; k < H; ++k)
                for (int64_t g = 0; g < G; ++g) z[g] += hqr[k] * w_hh[k * G + g];
            for (int64_t g = 0; g < G; ++g) z[g] += b[g];
            for (int64_t j = 0; j < H; ++j) {
                gr[j] = sigmoid_(z[j]); gr[H + j] = sigmoid_(z[H + j]);
                gr[2 * H + j] = tanh(z[2 * H + j]); gr[3 * H + j] = sigmoid_(z[3 * H + j]);
                double cn = orc_cast(gr[H + j] * cs[t * BH + bi * H + j] + gr[j] * gr[2 * H + j], state_dtype);
                cs[(t + 1) * BH + bi * H + j] = cn;
                h[bi * H + j] = orc_cast(gr[3 * H + j] * tanh(cn), state_dtype);
            }
        }
    /* reverse sweep */
    if (dx) for (int64_t i = 0; i < T * B * I; ++i) dx[i] = 0.0;
    if (dw_ih) for (int64_t i = 0; i < I * G; ++i) dw_ih[i] = 0.0;
    if (dw_hh) for (int64_t i = 0; i < H * G; ++i) dw_hh[i] = 0.0;
    if (db) for (int64_t g = 0; g < G; ++g) db[g] = 0.0;
    for (int64_t i = 0; i < BH; ++i) { dhn[i] = 0.0; dcn[i] = dc_final ? dc_final[i] : 0.0; }
    for (int64_t t = T - 1; t >= 0; --t) {
        for (int64_t bi = 0; bi < B; ++bi) {
            const double *gr = gt + (t * B + bi) * G;
            for (int64_t j = 0; j < H; ++j) {
                double ig = gr[j], fg = gr[H + j], gg = gr[2 * H + j], og = gr[3 * H + j];
                double tc = tanh(cs[(t + 1) * BH + bi * H + j]);
                double dh = dh_all[(t * B + bi) * H + j] + dhn[bi * H + j];
                double d_o = dh * tc;
                double dc = dcn[bi * H + j] + dh * og * (1.0 - tc * tc);
                double d_i = dc * gg, d_f = dc * cs[t * BH + bi * H + j], d_g = dc * ig;
                dcn[bi * H + j] = dc * fg;
                double *dzr = dz + bi * G;
                dzr[j] = orc_cast(d_i * ig * (1.0 - ig), dz_dtype);
                dzr[H + j] = orc_cast(d_f * fg * (1.0 - fg), dz_dtype);
                dzr[2 * H + j] = orc_cast(d_g * (1.0 - gg * gg), dz_dtype);
                dzr[3 * H + j] = orc_cast(d_o * og * (1.0 - og), dz_dtype);
            }
        }
        for (int64_t bi = 0; bi < B; ++bi) {
            const double *dzr = dz + bi * G, *xr = x + (t * B + bi) * I, *hqr = hq + (t * B + bi) * H;
            if (db) for (int64_t g = 0; g < G; ++g) db[g] += dzr[g];
            for (int64_t k = 0; k < I; ++k) {
                if (dx) {
                    double s = 0.0;
                    for (int64_t g = 0; g < G; ++g) s += dzr[g] * w_ih[k * G + g];
                    dx[(t * B + bi) * I + k] = s;
                }
                if (dw_ih) for (int64_t g = 0; g < G; ++g) dw_ih[k * G + g] += xr[k] * dzr[g];
            }
            for (int64_t k = 0; k < H; ++k) {
                double s = 0.0;
                for (int64_t g = 0; g < G; ++g) s += dzr[g] * w_hh[k * G + g];
                dhn[bi * H + k] = s;
                if (dw_hh) for (int64_t g = 0; g < G; ++g) dw_hh[k * G + g] += hqr[k] * dzr[g];
            }
        }
    }
    if (dh0) for (int64_t i = 0; i < BH; ++i) dh0[i] = dhn[i];
    if (dc0) for (int64_t i = 0; i < BH; ++i) dc0[i] = dcn[i];
    free(hq); free(cs); free(gt); free(h); free(z); free(dz); free(dhn); free(dcn);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Integer type relations (Section 4.3: shapes live in types, so every output shape is a
 * function of the input shapes and attributes alone).
 * ---------------------------------------------------------------------------------------- */

/* NumPy-style broadcast of two shapes, right-aligned.  Returns the result rank, or -1 when an
 * axis pair is neither equal nor contains a 1. */
int orc_broadcast_shape(int ra, const int64_t *sa, int rb, const int64_t *sb, int64_t *out)
{
    int r = ra > rb ? ra : rb;
    for (int d = 0; d < r; ++d) {
        int ia = d - (r - ra), ib = d - (r - rb);
        int64_t da = ia >= 0 ? sa[ia] : 1;
        int64_t db = ib >= 0 ? sb[ib] : 1;
        if (da == db) out[d] = da;
        else if (da == 1) out[d] = db;
        else if (db == 1) out[d] = da;
        else return -1;
    }
    return r;
}

/* Shape of a reduction result: axes in `mask` removed, or kept as extent 1. */
int orc_reduce_shape(int rank, const int64_t *shape, int mask, int keepdims, int64_t *out)
{
    int r = 0;
    for (int d = 0; d < rank; ++d) {
        if (mask & (1 << d)) { if (keepdims) out[r++] = 1; }
        else out[r++] = shape[d];
    }
    return r;
}

/* cast of a whole array (used by the tests to model a stored tensor) */
void orc_cast_array(const double *in, int64_t n, int dtype, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_cast(in[i], dtype);
}
