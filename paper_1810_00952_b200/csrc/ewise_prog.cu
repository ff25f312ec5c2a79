// Type checking of elementwise programs (Fig. 5: Type-UnaryOp, Type-Noncomp-BinaryOp,
// Type-Comp-BinaryOp, literals, cast) preceded by the explicit broadcast step.
#include "ewise_prog.h"

namespace relay {

static int arity(int op)
{
    switch (op) {
    case RELAY_OP_ADD: case RELAY_OP_SUB: case RELAY_OP_MUL: case RELAY_OP_DIV:
    case RELAY_OP_NE: case RELAY_OP_EQ: case RELAY_OP_LT: case RELAY_OP_LE: case RELAY_OP_GT: case RELAY_OP_GE:
    case RELAY_OP_MAX: case RELAY_OP_MIN:
        return 2;
    case RELAY_OP_SELECT: return 3;
    case RELAY_OP_CONST: return 0;
    default: return 1;
    }
}

relay_status_t type_program(const relay_ewise_prog_t *prog, const relay_tensor_t *const *inputs, int32_t n_in,
                            TypedProgram *tp)
{
    RELAY_TRY(check_not_null(prog, "prog"));
    if (n_in < 0 || n_in > RELAY_MAX_INPUTS) return fail(RELAY_ERR_ATTR, "%d inputs, at most %d allowed", n_in, RELAY_MAX_INPUTS);
    if (n_in > 0) RELAY_TRY(check_not_null(inputs, "inputs"));
    if (prog->n_instr < 0 || prog->n_instr > RELAY_MAX_INSTR)
        return fail(RELAY_ERR_ATTR, "program has %d instructions, at most %d allowed", prog->n_instr, RELAY_MAX_INSTR);
    if (prog->n_instr > 0) RELAY_TRY(check_not_null(prog->instr, "prog->instr"));
    for (int i = 0; i < n_in; ++i) RELAY_TRY(check_not_null(inputs[i], "inputs[i]"));
    for (int i = 0; i < n_in; ++i) RELAY_TRY(check_type(inputs[i], "input"));

    tp->n_in = n_in;
    tp->n_instr = prog->n_instr;
    tp->n_values = n_in + prog->n_instr;
    for (int i = 0; i < n_in; ++i) tp->dtype[i] = inputs[i]->dtype;

    // instruction typing
    for (int j = 0; j < prog->n_instr; ++j) {
        const relay_instr_t &in = prog->instr[j];
        tp->instr[j] = in;
        if (in.op < 0 || in.op >= RELAY_OP_COUNT_) return fail(RELAY_ERR_ATTR, "instruction %d: unknown opcode %d", j, in.op);
        if (dtype_size(in.dtype) == 0) return fail(RELAY_ERR_DTYPE, "instruction %d: unknown result type %d", j, in.dtype);
        int ar = arity(in.op), lim = n_in + j;
        int src[3] = {in.a, in.b, in.c};
        for (int s = 0; s < 3; ++s) {
            if (s < ar) {
                if (src[s] < 0 || src[s] >= lim)
                    return fail(RELAY_ERR_ATTR, "instruction %d: operand %d names value %d, only 0..%d exist yet", j, s, src[s], lim - 1);
            } else if (src[s] != -1)
                return fail(RELAY_ERR_ATTR, "instruction %d: unused operand %d must be -1", j, s);
        }
        int32_t ta = ar > 0 ? tp->dtype[in.a] : -1, tb = ar > 1 ? tp->dtype[in.b] : -1, tc = ar > 2 ? tp->dtype[in.c] : -1;
        int32_t want;
        switch (in.op) {
        case RELAY_OP_ADD: case RELAY_OP_SUB: case RELAY_OP_MUL: case RELAY_OP_DIV: case RELAY_OP_MAX: case RELAY_OP_MIN:
            if (ta != tb) return fail(RELAY_ERR_DTYPE, "instruction %d: operand types %s and %s differ", j, dtype_name(ta), dtype_name(tb));
            if (!is_float(ta)) return fail(RELAY_ERR_DTYPE, "instruction %d: arithmetic on %s is not defined here", j, dtype_name(ta));
            want = ta;
            break;
        case RELAY_OP_NE: case RELAY_OP_EQ: case RELAY_OP_LT: case RELAY_OP_LE: case RELAY_OP_GT: case RELAY_OP_GE:
            if (ta != tb) return fail(RELAY_ERR_DTYPE, "instruction %d: operand types %s and %s differ", j, dtype_name(ta), dtype_name(tb));
            if (!is_float(ta) && ta != RELAY_BOOL) return fail(RELAY_ERR_DTYPE, "instruction %d: comparison of %s is not defined here", j, dtype_name(ta));
            want = RELAY_BOOL;
            break;
        case RELAY_OP_SELECT:
            if (ta != RELAY_BOOL) return fail(RELAY_ERR_DTYPE, "instruction %d: select condition has type %s, needs bool", j, dtype_name(ta));
            if (tb != tc) return fail(RELAY_ERR_DTYPE, "instruction %d: select branches have types %s and %s", j, dtype_name(tb), dtype_name(tc));
            want = tb;
            break;
        case RELAY_OP_CAST: case RELAY_OP_CONST:
            want = in.dtype;
            break;
        default:  // unary float operators
            if (!is_float(ta)) return fail(RELAY_ERR_DTYPE, "instruction %d: operator %d on %s is not defined here", j, in.op, dtype_name(ta));
            want = ta;
            break;
        }
        if (in.dtype != want)
            return fail(RELAY_ERR_DTYPE, "instruction %d: declared result type %s, the typing rule gives %s", j, dtype_name(in.dtype), dtype_name(want));
        tp->dtype[n_in + j] = want;
    }

    // broadcast of all inputs to one shape
    int r = 0;
    for (int i = 0; i < n_in; ++i) r = inputs[i]->rank > r ? inputs[i]->rank : r;
    tp->rank = r;
    for (int d = 0; d < r; ++d) tp->shape[d] = 1;
    for (int i = 0; i < n_in; ++i) {
        int off = r - inputs[i]->rank;
        for (int d = 0; d < r; ++d) {
            int64_t e = d >= off ? inputs[i]->shape[d - off] : 1;
            tp->in_shape[i][d] = e;
            if (e == tp->shape[d] || e == 1) continue;
            if (tp->shape[d] == 1) { tp->shape[d] = e; continue; }
            return fail(RELAY_ERR_SHAPE, "input %d: extent %lld of right-aligned axis %d does not broadcast against %lld", i,
                        (long long)e, d, (long long)tp->shape[d]);
        }
    }
    tp->total = 1;
    for (int d = 0; d < r; ++d) tp->total *= tp->shape[d];
    return RELAY_OK;
}

}  // namespace relay
