"""Pins for the oracle's casts, scalar operators, broadcasting, elementwise and reduce groups.

Each check ties the oracle to something other than itself: the bit-level definition of the
number formats, closed forms of the operators, NumPy's library routines on special cases, or
brute force on tiny inputs."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from relay_workloads import program as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------------
# casts (Fig. 1 cast production; bf16 = upper 16 bits of binary32, round to nearest even)
# ---------------------------------------------------------------------------------------------
def _bf16_by_bits(f32: np.ndarray) -> np.ndarray:
    """Independent route: integer arithmetic on the binary32 bit pattern."""
    u = f32.astype(np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def test_bf16_rounding_matches_bit_definition():
    rng = np.random.default_rng(1)
    v = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-3).astype(np.float32),
        (rng.standard_normal(2000) * 1e6).astype(np.float32),
        np.float32([0.0, -0.0, 1.0, -1.0, 2.0 ** -126, 2.0 ** -130, 2.0 ** -133, 3.0e38]),
    ])
    got = oracle.cast_array(v.astype(np.float64), oracle.BF16)
    want = _bf16_by_bits(v)
    assert np.array_equal(got, want)


def test_bf16_golden_values():
    # file: value -> expected, from the format definition (8 significant bits, ties to even)
    for line in open(os.path.join(GOLDEN, "bf16_rounding.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        v, want = (float.fromhex(t) if "0x" in t else float(t) for t in line.split())
        assert oracle.round_bf16(v) == want, line


def test_bf16_single_rounding_from_fp64():
    # 1 + 2^-8 + 2^-30 is above the tie, so it rounds up; via fp32 first it would be a tie -> down
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert oracle.round_bf16(v) == 1.0 + 2.0 ** -7
    assert oracle.round_bf16(-v) == -(1.0 + 2.0 ** -7)


def test_f32_cast_matches_ieee():
    rng = np.random.default_rng(2)
    v = rng.standard_normal(10000) * np.exp(rng.uniform(-20, 20, 10000))
    got = oracle.cast_array(v, oracle.F32)
    assert np.array_equal(got, v.astype(np.float32).astype(np.float64))


def test_int_bool_casts():
    v = np.array([-2.7, -0.2, 0.0, 0.9, 3.99])
    assert np.array_equal(oracle.cast_array(v, oracle.I32), [-2, -0.0, 0, 0, 3])
    assert np.array_equal(oracle.cast_array(v, oracle.BOOL), [1, 1, 0, 1, 1])


# ---------------------------------------------------------------------------------------------
# scalar operators: closed forms
# ---------------------------------------------------------------------------------------------
def test_activation_closed_forms():
    A = oracle
    assert A.act(0.0, A.ACT_TANH) == 0.0
    assert A.act(0.0, A.ACT_SIGMOID) == 0.5
    for x in np.linspace(-6, 6, 49):
        s, sm = A.act(x, A.ACT_SIGMOID), A.act(-x, A.ACT_SIGMOID)
        assert abs(s + sm - 1.0) < 1e-15
        assert abs(A.act(x, A.ACT_TANH) - (2 * A.act(2 * x, A.ACT_SIGMOID) - 1)) < 1e-15
        assert A.act(x, A.ACT_RELU) == max(x, 0.0)
        assert A.act(x, A.ACT_NONE) == x
        assert abs(A.act(x, A.ACT_TANH) - math.tanh(x)) < 1e-16


def test_activation_derivatives_against_central_differences():
    A = oracle
    h = 1e-6
    for code in (A.ACT_NONE, A.ACT_RELU, A.ACT_TANH, A.ACT_SIGMOID):
        for z in np.linspace(-3, 3, 25):
            if code == A.ACT_RELU and abs(z) < 1e-3:
                continue
            fd = (A.act(z + h, code) - A.act(z - h, code)) / (2 * h)
            an = A.act_grad_from_output(A.act(z, code), code)
            assert abs(fd - an) < 1e-9
    assert A.act_grad_from_output(0.0, A.ACT_RELU) == 0.0          # relu'(0) = 0
    assert set(A.act_grad_from_output(v, A.ACT_RELU) for v in (-1.0, 0.0, 2.0)) == {0.0, 1.0}


# ---------------------------------------------------------------------------------------------
# broadcasting: brute force over all shape pairs of rank <= 3 with extents in {1,2,3}
# ---------------------------------------------------------------------------------------------
def _all_shapes(max_rank=3, dims=(1, 2, 3)):
    for r in range(max_rank + 1):
        yield from itertools.product(dims, repeat=r)


def _replicate(a, shape):
    """Materialise the broadcast by explicit index arithmetic (no numpy broadcasting)."""
    out = np.empty(shape)
    off = len(shape) - a.ndim
    for idx in itertools.product(*[range(s) for s in shape]):
        src = tuple(0 if a.shape[d] == 1 else idx[d + off] for d in range(a.ndim))
        out[idx] = a[src]
    return out


def test_broadcast_rule_brute_force():
    rng = np.random.default_rng(3)
    add = P.Program([P.F32, P.F32])
    r = add.add(0, 1)
    n_legal = n_illegal = 0
    for sa in _all_shapes():
        for sb in _all_shapes():
            # the rule, restated: right-align; each axis pair equal or one of them 1
            ra, rb = sa[::-1], sb[::-1]
            legal, res = True, []
            for d in range(max(len(ra), len(rb))):
                x = ra[d] if d < len(ra) else 1
                y = rb[d] if d < len(rb) else 1
                if x != y and x != 1 and y != 1:
                    legal = False
                res.append(max(x, y))
            want = tuple(res[::-1]) if legal else None
            assert oracle.broadcast_shape(sa, sb) == want
            if not legal:
                n_illegal += 1
                with pytest.raises(ValueError):
                    oracle.ewise(add.arrays(), [np.zeros(sa), np.zeros(sb)], [r])
                continue
            n_legal += 1
            assert want == np.broadcast_shapes(sa, sb)
            a, b = rng.standard_normal(sa), rng.standard_normal(sb)
            (got,) = oracle.ewise(add.arrays(), [a, b], [r])
            assert got.shape == want
            assert np.array_equal(got, _replicate(a, want) + _replicate(b, want))
    assert n_legal > 500 and n_illegal > 500


def test_tensor_literal_stacking_rule():
    # Fig. 5 Type-Tensor-Literal: m tensors of Shape(d1..dn) stack to Shape(m, d1..dn)
    for m in (1, 2, 5):
        for s in [(), (3,), (2, 4)]:
            stacked = np.stack([np.zeros(s)] * m)
            assert stacked.shape == (m,) + s


# ---------------------------------------------------------------------------------------------
# elementwise opcodes against NumPy on random arrays (Fig. 1 BinOp/UnaryOp, Fig. 5 result types)
# ---------------------------------------------------------------------------------------------
def test_every_opcode_against_numpy():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((5, 7))
    y = rng.standard_normal((5, 7))
    y[0, :3] = x[0, :3]  # some equal elements for the comparisons
    cases = {
        "add": (lambda p: p.add(0, 1), x + y), "sub": (lambda p: p.sub(0, 1), x - y),
        "mul": (lambda p: p.mul(0, 1), x * y), "div": (lambda p: p.div(0, 1), x / y),
        "neg": (lambda p: p.neg(0), -x), "sq": (lambda p: p.sq(0), x * x),
        "ne": (lambda p: p.cmp(P.OP_NE, 0, 1), x != y), "eq": (lambda p: p.cmp(P.OP_EQ, 0, 1), x == y),
        "lt": (lambda p: p.cmp(P.OP_LT, 0, 1), x < y), "le": (lambda p: p.cmp(P.OP_LE, 0, 1), x <= y),
        "gt": (lambda p: p.cmp(P.OP_GT, 0, 1), x > y), "ge": (lambda p: p.cmp(P.OP_GE, 0, 1), x >= y),
        "select": (lambda p: p.select(p.cmp(P.OP_GT, 0, 1), 0, 1), np.where(x > y, x, y)),
        "relu": (lambda p: p.relu(0), np.maximum(x, 0)), "tanh": (lambda p: p.tanh(0), np.tanh(x)),
        "sigmoid": (lambda p: p.sigmoid(0), 1 / (1 + np.exp(-x))),
        "exp": (lambda p: p.exp(0), np.exp(x)), "log": (lambda p: p.log(p.sq(0)), np.log(x * x)),
        "max": (lambda p: p.max(0, 1), np.maximum(x, y)), "min": (lambda p: p.min(0, 1), np.minimum(x, y)),
        "const": (lambda p: p.add(0, p.const(2.5)), x + 2.5),
        "cast": (lambda p: p.cast(0, P.BF16), _bf16_by_bits(x.astype(np.float32))),
    }
    xs = x.astype(np.float32).astype(np.float64)  # the cast case needs fp32-exact inputs
    for name, (build, want) in cases.items():
        p = P.Program([5, 5])  # 5 = fp64 "no rounding" code of the oracle
        out = build(p)
        a0 = xs if name == "cast" else x
        (got,) = oracle.ewise(p.arrays(), [a0, y], [out])
        np.testing.assert_allclose(got, np.asarray(want, dtype=np.float64), rtol=1e-15, atol=0, err_msg=name)
        if name in ("ne", "eq", "lt", "le", "gt", "ge"):
            assert set(np.unique(got)) <= {0.0, 1.0}
            assert p.dtype_of(out) == P.BOOL        # Type-Comp-BinaryOp
        if name in ("neg", "sq", "add"):
            assert p.dtype_of(out) == p.dtype_of(0)  # Type-UnaryOp / Type-Noncomp-BinaryOp


def test_program_rejects_forward_references():
    p = P.Program([P.F32])
    p.emit(P.OP_ADD, 0, 5)  # names a value that does not exist yet
    with pytest.raises(ValueError):
        oracle.ewise(p.arrays(), [np.zeros(3)], [1])


def test_cfg2_forward_program_against_numpy():
    rng = np.random.default_rng(5)
    x = oracle.cast_array(rng.standard_normal((6, 10)), oracle.BF16)
    a = oracle.cast_array(rng.uniform(0.5, 1.5, 10), oracle.BF16)
    b = oracle.cast_array(rng.standard_normal((1, 10)) * 0.1, oracle.BF16)
    prog, outs = P.tanh_affine_residual_fwd(P.BF16)
    (got,) = oracle.ewise(prog.arrays(), [x, a, b], outs)
    want = np.tanh(a[None, :] * x + b) + x
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
    assert np.all(np.abs(got - want) <= 0.5 * ulp + 1e-15)     # one rounding to bf16, nothing else
    assert np.array_equal(got, _bf16_by_bits(got.astype(np.float32)))  # results are bf16 values


def test_cfg2_gradient_program_against_finite_differences():
    """The gradient group's program (dx with fan-out of x, da, db as column sums) is checked
    against central differences of L = sum(dout * out) through the FORWARD program."""
    rng = np.random.default_rng(6)
    R, C = 5, 4
    x = rng.standard_normal((R, C)); a = rng.uniform(0.5, 1.5, C); b = rng.standard_normal((1, C)) * 0.1
    dout = rng.standard_normal((R, C))
    F64 = 5
    fwd, fo = P.tanh_affine_residual_fwd(F64, F64)
    grd, (dx_id, dae_id, dbe_id) = P.tanh_affine_residual_grad(F64, F64)

    def loss(x_, a_, b_):
        (o,) = oracle.ewise(fwd.arrays(), [x_, a_, b_], fo)
        return float(np.sum(dout * o))

    dx, da, db = oracle.reduce(grd.arrays(), [dout, x, a, b], [
        (dx_id, oracle.RED_NONE, (), False, F64),
        (dae_id, oracle.RED_SUM, (0,), False, F64),
        (dbe_id, oracle.RED_SUM, (0,), True, F64)])
    assert dx.shape == (R, C) and da.shape == (C,) and db.shape == (1, C)
    h = 1e-5
    for arr, grad in ((x, dx), (a, da), (b, db)):
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + h; lp = loss(x, a, b)
            arr[idx] = keep - h; lm = loss(x, a, b)
            arr[idx] = keep
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(fd)), (idx, fd, grad[idx])
    # invariants of this group: a*s+1 lies in [1, 2.5) for a in (0.5, 1.5)
    assert np.all(np.sign(dx) == np.sign(dout))
    assert np.all(np.abs(dx) >= np.abs(dout) - 1e-15) and np.all(np.abs(dx) <= 2.5 * np.abs(dout))


def test_sigmoid_product_relu_programs_against_numpy_and_finite_differences():
    """The second pair of benchmark programs (out = sigmoid(x*y) + relu(z), z constant down the rows): the forward program
    against its closed form, the gradient program (dx, dy unreduced, dz as a column sum) against central differences of
    L = sum(dout * out) through the forward program, away from the kink of relu."""
    rng = np.random.default_rng(16)
    R, C = 5, 4
    x, y = rng.standard_normal((R, C)), rng.standard_normal((R, C))
    z = rng.standard_normal(C); z[np.abs(z) < 1e-2] = 0.5
    dout = rng.standard_normal((R, C))
    F64 = 5
    fwd, fo = P.sigmoid_product_relu_fwd(F64, F64)
    grd, (dx_id, dy_id, dz_id) = P.sigmoid_product_relu_grad(F64, F64)
    (o,) = oracle.ewise(fwd.arrays(), [x, y, z], fo)
    assert np.allclose(o, 1.0 / (1.0 + np.exp(-x * y)) + np.maximum(z, 0.0)[None, :], rtol=0, atol=1e-15)

    def loss(x_, y_, z_):
        (o_,) = oracle.ewise(fwd.arrays(), [x_, y_, z_], fo)
        return float(np.sum(dout * o_))

    dx, dy, dz = oracle.reduce(grd.arrays(), [dout, x, y, z], [
        (dx_id, oracle.RED_NONE, (), False, F64), (dy_id, oracle.RED_NONE, (), False, F64), (dz_id, oracle.RED_SUM, (0,), False, F64)])
    assert dx.shape == (R, C) and dy.shape == (R, C) and dz.shape == (C,)
    h = 1e-5
    for arr, grad in ((x, dx), (y, dy), (z, dz)):
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + h; lp = loss(x, y, z)
            arr[idx] = keep - h; lm = loss(x, y, z)
            arr[idx] = keep
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(fd)), (idx, fd, grad[idx])
    assert np.all(dz[z < 0] == 0.0)                       # relu'(z) = 0 below the kink


# ---------------------------------------------------------------------------------------------
# reduce group
# ---------------------------------------------------------------------------------------------
def _ident(dt=5):
    p = P.Program([dt])
    return p, 0


def test_reduce_closed_forms():
    p, v = _ident()
    ones = np.ones((7, 5, 3))
    for axes in [(0,), (1,), (2,), (0, 2), (0, 1, 2)]:
        (s,) = oracle.reduce(p.arrays(), [ones], [(v, oracle.RED_SUM, axes, False, 5)])
        cnt = int(np.prod([ones.shape[a] for a in axes]))
        assert np.all(s == cnt)
        (m,) = oracle.reduce(p.arrays(), [ones * 2.5], [(v, oracle.RED_MEAN, axes, True, 5)])
        assert np.all(m == 2.5)
        assert m.shape == tuple(1 if d in axes else ones.shape[d] for d in range(3))


def test_reduce_against_numpy_all_axis_subsets():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((4, 6, 5))
    p, v = _ident()
    for r in range(1, 4):
        for axes in itertools.combinations(range(3), r):
            for keep in (False, True):
                s, mx, mean = oracle.reduce(p.arrays(), [x], [
                    (v, oracle.RED_SUM, axes, keep, 5), (v, oracle.RED_MAX, axes, keep, 5),
                    (v, oracle.RED_MEAN, axes, keep, 5)])
                np.testing.assert_allclose(s, x.sum(axis=axes, keepdims=keep), rtol=1e-14)
                assert np.array_equal(mx, x.max(axis=axes, keepdims=keep))
                np.testing.assert_allclose(mean, x.mean(axis=axes, keepdims=keep), rtol=1e-14)
                assert s.shape == oracle.reduce_shape(x.shape, axes, keep)


def test_argmax_first_maximum_and_integer_result():
    p, v = _ident()
    x = np.array([[1.0, 3.0, 3.0, 2.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -2.0, -0.5, -0.5]])
    (am,) = oracle.reduce(p.arrays(), [x], [(v, oracle.RED_ARGMAX, (1,), False, P.I64)])
    assert am.dtype == np.int64 and am.tolist() == [1, 0, 2]      # ties -> lowest index
    (am0,) = oracle.reduce(p.arrays(), [x], [(v, oracle.RED_ARGMAX, (0,), False, P.I64)])
    assert am0.tolist() == np.argmax(x, axis=0).tolist()
    rng = np.random.default_rng(8)
    y = rng.integers(0, 4, size=(9, 11)).astype(np.float64)       # many ties
    for ax in (0, 1):
        (g,) = oracle.reduce(p.arrays(), [y], [(v, oracle.RED_ARGMAX, (ax,), False, P.I64)])
        assert np.array_equal(g, np.argmax(y, axis=ax))            # numpy also returns the first


def test_reduce_with_prologue_and_unreduced_output():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((8, 5)); w = rng.standard_normal((5,))
    p = P.Program([5, 5])
    prod = p.mul(0, 1)
    sq = p.sq(prod)
    full, colsum, rowmax = oracle.reduce(p.arrays(), [x, w], [
        (prod, oracle.RED_NONE, (), False, 5), (sq, oracle.RED_SUM, (0,), False, 5),
        (prod, oracle.RED_MAX, (1,), True, 5)])
    assert np.array_equal(full, x * w)
    np.testing.assert_allclose(colsum, ((x * w) ** 2).sum(0), rtol=1e-14)
    assert np.array_equal(rowmax, (x * w).max(1, keepdims=True))


def test_reduce_output_dtype_rounds_once_after_the_sum():
    p, v = _ident()
    x = np.full((1000, 1), 1.0 + 2.0 ** -20)       # every partial sum would round in fp32
    (s32,) = oracle.reduce(p.arrays(), [x], [(v, oracle.RED_SUM, (0,), False, P.F32)])
    assert s32[0] == float(np.float32(1000.0 * (1.0 + 2.0 ** -20)))
