"""GPU parity: programs without a pre-compiled body on the vectorised tier -- once as bodies compiled at run time, once on
the in-kernel interpreter -- and integer-typed values on the scalar evaluator, against the CPU oracle through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I
from relay_workloads import program as P

from parity import Guarded, assert_bf16, assert_f32, to_np, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TDT = {P.BF16: torch.bfloat16, P.F32: torch.float32, P.BOOL: torch.uint8}
VEC = 1


@pytest.fixture(autouse=True, params=["compiled", "interpreted"])
def tier(request):
    """Every test of this file runs twice: with the run-time compiled bodies and with them switched off."""
    if request.param == "compiled" and B.relay_debug_jit_compiled() < 0:
        pytest.skip("no run-time compiler library on this machine")
    before = B.relay_debug_set_jit(request.param == "compiled")
    yield request.param
    B.relay_debug_set_jit(before)


def rnd(shape, tdt, seed, scale=1.0):
    return (torch.randn(*shape, generator=torch.Generator().manual_seed(seed)) * scale).to(tdt)


def run_ewise(p, ins, out_ids, expect_route=VEC):
    shape = torch.broadcast_shapes(*[tuple(t.shape) for t in ins])
    assert B.relay_debug_group_route(p.arrays(), ins, [(v, B.RED_NONE, 0, 0) for v in out_ids]) == expect_route
    outs = [Guarded(shape, TDT[p.dtype_of(v)], DEV) for v in out_ids]
    B.relay_fused_ewise(p.arrays(), [t.to(DEV) for t in ins], out_ids, [o.t for o in outs])
    torch.cuda.synchronize()
    B.relay_poll_status()
    want = oracle.ewise(p.arrays(), [t.double().numpy() for t in ins], out_ids)
    return [o.check() for o in outs], want


@pytest.mark.parametrize("rows,cols", [(1, 8), (7, 264), (37, 520), (70, 1032), (9, 256), (300, 136)])
@pytest.mark.parametrize("code", [P.BF16, P.F32])
def test_every_opcode_full_rowvector_and_scalar_operands(rows, cols, code):
    """Every operator, each as its own group, over a full-shape x, a y that is constant down the rows and a scalar k, at
    shapes with ragged last tiles in both directions (one block and several, a single row, fewer than 8 rows)."""
    tdt = TDT[code]
    x, y, k = rnd((rows, cols), tdt, 1), rnd((cols,), tdt, 2), torch.tensor(0.75).to(tdt)
    y[: min(4, cols)] = x[0, : min(4, cols)]                         # equal operands for the comparisons
    chk = assert_f32 if code == P.F32 else assert_bf16
    builds = {
        "add": lambda p, a, b, c: p.add(a, b), "sub": lambda p, a, b, c: p.sub(a, c), "mul": lambda p, a, b, c: p.mul(a, b),
        "div": lambda p, a, b, c: p.div(a, p.add(p.sq(b), p.const(1.0))), "neg": lambda p, a, b, c: p.neg(a), "sq": lambda p, a, b, c: p.sq(b),
        "relu": lambda p, a, b, c: p.relu(a), "tanh": lambda p, a, b, c: p.tanh(p.mul(a, c)), "sigmoid": lambda p, a, b, c: p.sigmoid(a),
        "exp": lambda p, a, b, c: p.exp(a), "log": lambda p, a, b, c: p.log(p.add(p.sq(a), p.const(0.5))),
        "max": lambda p, a, b, c: p.max(a, b), "min": lambda p, a, b, c: p.min(a, c),
        "select": lambda p, a, b, c: p.select(p.cmp(P.OP_GT, a, b), a, c),
    }
    for name, build in builds.items():
        p = P.Program([code] * 3)
        a, b, c = (p.cast(i, P.F32) for i in range(3))
        v = p.cast(build(p, a, b, c), code)
        (got,), (want,) = run_ewise(p, [x, y, k], [v])
        if code == P.BF16:
            q = P.Program([code] * 3); a, b, c = (q.cast(i, 5) for i in range(3))       # fp64 values before the storage rounding
            v64 = build(q, a, b, c)
            (want,) = oracle.ewise(q.arrays(), [t.double().numpy() for t in (x, y, k)], [v64])
        chk(got, want, what=name)
    for op in (P.OP_NE, P.OP_EQ, P.OP_LT, P.OP_LE, P.OP_GT, P.OP_GE):                    # Bool results: bit-exact
        p = P.Program([code] * 3); v = p.cmp(op, 0, 1)
        (got,), (want,) = run_ewise(p, [x, y, k], [v])
        assert np.array_equal(got.cpu().numpy(), want.astype(np.uint8)), op


def test_values_of_type_bf16_are_rounded_after_every_operator():
    """Arithmetic written directly on bf16 values (no cast to f32): Fig. 5 gives every intermediate the type bf16, so it
    holds a bf16 number.  The oracle is given the same expression with that rounding written out as casts; the results
    then agree to the last bit except where a rounding decision falls within the fp32-vs-fp64 difference of an operand."""
    x, y = rnd((50, 264), torch.bfloat16, 3), rnd((50, 264), torch.bfloat16, 4)
    p = P.Program([P.BF16, P.BF16])
    v = p.add(p.mul(0, 1), p.sq(p.sub(0, 1)))
    q = P.Program([P.BF16, P.BF16])
    r = lambda e: q.cast(q.cast(e, P.BF16), 5)            # a bf16 number, carried on in fp64
    a, b = q.cast(0, 5), q.cast(1, 5)
    vq = r(q.add(r(q.mul(a, b)), r(q.sq(r(q.sub(a, b))))))
    (got,), _ = run_ewise(p, [x, y], [v])
    (want,) = oracle.ewise(q.arrays(), [x.double().numpy(), y.double().numpy()], [vq])
    assert_bf16(got, want, what="bf16 chain")
    assert float((to_np(got) == want).mean()) > 0.99


@pytest.mark.parametrize("code", [P.BF16, P.F32])
def test_several_results_shared_subexpressions_and_type_changing_casts(code):
    tdt = TDT[code]
    x, y = rnd((33, 776), tdt, 5), rnd((1, 776), tdt, 6)
    p = P.Program([code, code])
    a, b = p.cast(0, P.F32), p.cast(1, P.F32)
    s = p.sigmoid(p.mul(a, b))                       # used three times
    o1 = p.cast(p.mul(s, p.sub(p.const(1.0), s)), code)
    o2 = p.add(s, a)                                 # stays f32
    o3 = p.cmp(P.OP_GT, s, p.const(0.5))             # Bool
    o4 = p.cast(p.cast(p.mul(a, a), P.BF16), P.F32)  # rounded to bf16, stored as f32
    got, want = run_ewise(p, [x, y], [o1, o2, o3, o4])
    chk = assert_f32 if code == P.F32 else (lambda g, o, what: assert_bf16(g, o, stored_bf16=False, what=what))
    if code == P.F32:
        assert_f32(got[0], want[0], what="o1")
    else:
        assert_bf16(got[0], want[0], what="o1")
    chk(got[1], want[1], what="o2")
    sg = 1 / (1 + np.exp(-(x.double().numpy() * y.double().numpy())))
    clear = np.abs(sg - 0.5) > 1e-2                  # away from the threshold the comparison is decided alike
    assert np.array_equal(got[2].cpu().numpy()[clear], want[2].astype(np.uint8)[clear])
    assert_bf16(got[3], want[3], what="o4")


@pytest.mark.parametrize("rows,cols,code", [(8192 // 16, 512, P.BF16), (130, 264, P.F32), (5, 8, P.BF16), (1000, 1288, P.BF16)])
def test_gradient_group_with_unreduced_results_and_column_sums(rows, cols, code):
    """sigmoid(x*y) + relu(z) with z constant down the rows: dx and dy unreduced, dz summed over the rows (and its mean
    with keepdims), in one pass."""
    tdt = TDT[code]
    d, x, y, z = rnd((rows, cols), tdt, 7), rnd((rows, cols), tdt, 8), rnd((rows, cols), tdt, 9), rnd((cols,), tdt, 10)
    g, ids = P.sigmoid_product_relu_grad(code)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_NONE, 0, 0), (ids[2], B.RED_SUM, 1, 0), (ids[2], B.RED_MEAN, 1, 1)]
    ins = [d, x, y, z]
    assert B.relay_debug_group_route(g.arrays(), ins, specs) == VEC
    outs = [Guarded((rows, cols), tdt, DEV), Guarded((rows, cols), tdt, DEV), Guarded((cols,), torch.float32, DEV), Guarded((1, cols), torch.float32, DEV)]
    ws = workspace(B.relay_workspace_bytes_reduce(ins, specs), DEV)
    for _ in range(2):
        B.relay_fused_reduce(g.arrays(), [t.to(DEV) for t in ins], specs, [o.t for o in outs], ws)
    torch.cuda.synchronize()
    B.relay_poll_status()
    g64, i64 = P.sigmoid_product_relu_grad(5, 5)              # fp64 values before the storage rounding
    ospecs = [(i64[0], 0, (), False, 5), (i64[1], 0, (), False, 5), (i64[2], 1, (0,), False, 5), (i64[2], 3, (0,), True, 5)]
    want = oracle.reduce(g64.arrays(), [t.double().numpy() for t in ins], ospecs)
    if code == P.F32:
        for o, w, n in zip(outs, want, ("dx", "dy", "dz", "mean")):
            assert_f32(o.check(), w, what=n)
    else:
        assert_bf16(outs[0].check(), want[0], what="dx"); assert_bf16(outs[1].check(), want[1], what="dy")
        assert_bf16(outs[2].check(), want[2], stored_bf16=False, what="dz"); assert_bf16(outs[3].check(), want[3], stored_bf16=False, what="mean")


def test_full_size_programs_sampled_columns():
    """The two benchmark programs that run on the vectorised evaluator, at 8192 x 8192 bf16 in the launch shape the
    benchmark times: the oracle recomputes whole columns, at least one in every 256-column block of the grid, so the
    column sum of dz is covered; the outputs are screened for unwritten elements."""
    rows = cols = 8192
    t = I.cfg2_ewise()
    x, y, d = t["x"], t["dout"], I.normal(2, 5, (rows, cols), 1.0, torch.bfloat16)
    z = I.normal(2, 6, (cols,), 1.0, torch.bfloat16)
    rng = np.random.default_rng(31)
    sel = np.unique(np.concatenate([[0, 7, 8, 255, 256, 8191], np.arange(0, cols, 256) + rng.integers(0, 256, 32)]))
    f, fo = P.sigmoid_product_relu_fwd(P.BF16)
    out = Guarded((rows, cols), torch.bfloat16, DEV)
    xd, yd, dd, zd = (v.to(DEV) for v in (x, y, d, z))
    assert B.relay_debug_group_route(f.arrays(), [xd, yd, zd], [(fo[0], B.RED_NONE, 0, 0)]) == VEC
    B.relay_fused_ewise(f.arrays(), [xd, yd, zd], fo, [out.t])
    f64, fo64 = P.sigmoid_product_relu_fwd(5, 5)
    (want,) = oracle.ewise(f64.arrays(), [I.as_f64(x[:, sel]), I.as_f64(y[:, sel]), I.as_f64(z[sel])], fo64)
    assert_bf16(out.check()[:, sel], want, what="fwd")
    g, ids = P.sigmoid_product_relu_grad(P.BF16)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_NONE, 0, 0), (ids[2], B.RED_SUM, 1, 0)]
    outs = [Guarded((rows, cols), torch.bfloat16, DEV), Guarded((rows, cols), torch.bfloat16, DEV), Guarded((cols,), torch.float32, DEV)]
    ws = workspace(B.relay_workspace_bytes_reduce([dd, xd, yd, zd], specs), DEV)
    B.relay_fused_reduce(g.arrays(), [dd, xd, yd, zd], specs, [o.t for o in outs], ws)
    torch.cuda.synchronize()
    B.relay_poll_status()
    g64, i64 = P.sigmoid_product_relu_grad(5, 5)
    wdx, wdy, wdz = oracle.reduce(g64.arrays(), [I.as_f64(d[:, sel]), I.as_f64(x[:, sel]), I.as_f64(y[:, sel]), I.as_f64(z[sel])],
                                  [(i64[0], 0, (), False, 5), (i64[1], 0, (), False, 5), (i64[2], 1, (0,), False, 5)])
    assert_bf16(outs[0].check()[:, sel], wdx, what="dx"); assert_bf16(outs[1].check()[:, sel], wdy, what="dy")
    assert_bf16(outs[2].check()[sel], wdz, stored_bf16=False, what="dz")


def test_integer_values_are_exact_beyond_24_bits():
    """IntType values (cast sources and targets, select branches, literals) keep every bit: 32-bit values above 2^24 and
    64-bit values above 2^32 pass through casts unchanged; float -> int truncates toward zero; int -> float rounds once."""
    rng = np.random.default_rng(37)
    a32 = torch.from_numpy(np.concatenate([[20000001, -20000001, 2**31 - 1, -2**31 + 1, 0, 16777217], rng.integers(-2**31, 2**31, 250)]).astype(np.int32)).reshape(8, 32)
    a64 = torch.from_numpy(np.concatenate([[2**40 + 1, -(2**40) - 1, 2**52 + 1, 9007199254740991, 0, 20000001], rng.integers(-2**52, 2**52, 250)]).astype(np.int64)).reshape(8, 32)
    f = (torch.randn(8, 32, generator=torch.Generator().manual_seed(2)) * 1e6)
    f[0, :4] = torch.tensor([2.9, -2.9, 16777216.0, -0.5])
    p = P.Program([P.I32, P.I64, P.F32])
    w = p.cast(0, P.I64)                                 # widen
    back = p.cast(w, P.I32)                              # and narrow again
    pick = p.select(p.cmp(P.OP_GT, 2, p.const(0.0)), w, 1)   # Int branches
    as_f = p.cast(0, P.F32)                              # one rounding
    as_b = p.cast(1, P.BF16)
    tr = p.cast(2, P.I64)                                # truncation toward zero
    tr32 = p.cast(2, P.I32)
    nz = p.cast(0, P.BOOL)
    lit = p.select(p.cast(0, P.BOOL), p.const(20000001, P.I32), 0)
    ids = [w, back, pick, as_f, as_b, tr, tr32, nz, lit]
    dts = [torch.int64, torch.int32, torch.int64, torch.float32, torch.bfloat16, torch.int64, torch.int32, torch.uint8, torch.int32]
    assert B.relay_debug_group_route(p.arrays(), [a32, a64, f], [(v, B.RED_NONE, 0, 0) for v in ids[:8]]) == 2
    outs = [Guarded((8, 32), dt, DEV) for dt in dts[:8]]
    B.relay_fused_ewise(p.arrays(), [a32.to(DEV), a64.to(DEV), f.to(DEV)], ids[:8], [o.t for o in outs])
    o9 = Guarded((8, 32), dts[8], DEV)
    B.relay_fused_ewise(p.arrays(), [a32.to(DEV), a64.to(DEV), f.to(DEV)], ids[8:], [o9.t])
    torch.cuda.synchronize()
    want = oracle.ewise(p.arrays(), [a32.double().numpy(), a64.double().numpy(), f.double().numpy()], ids)
    for o, wv, dt, name in zip(outs + [o9], want, dts, ("widen", "narrow", "select", "to f32", "to bf16", "trunc i64", "trunc i32", "to bool", "literal")):
        got = o.check().cpu()
        if dt in (torch.int64, torch.int32, torch.uint8):
            assert np.array_equal(got.numpy().astype(np.int64), wv.astype(np.int64)), name
        else:
            assert np.array_equal(got.double().numpy(), wv), name      # one rounding to nearest even on both sides


def test_a_body_is_compiled_once_per_program_and_only_when_switched_on(tier):
    x, y = rnd((64, 264), torch.float32, 5), rnd((264,), torch.float32, 6)
    p = P.Program([P.F32, P.F32]); v = p.add(p.mul(0, p.const(1.0 + 2.0 ** -20)), p.tanh(1))      # a program no other test uses
    n0 = B.relay_debug_jit_compiled()
    for _ in range(2):
        (got,), (want,) = run_ewise(p, [x, y], [v])
        assert_f32(got, want, "out")
    n1 = B.relay_debug_jit_compiled()
    if tier == "compiled":
        assert n1 == n0 + 1                         # the second call found it in the cache
        x2 = rnd((7, 520), torch.float32, 8)        # another shape: same body, same kernel
        run_ewise(p, [x2, rnd((520,), torch.float32, 9)], [v])
        assert B.relay_debug_jit_compiled() == n1
    else:
        assert n1 == n0 or n0 < 0


def test_a_program_beyond_the_interpreters_limits(tier):
    """More values alive at once than the interpreter has temporaries for: a compiled body where the compiler is present, the
    scalar evaluator otherwise -- the same results either way."""
    x = rnd((37, 264), torch.float32, 11, 0.5)
    p = P.Program([P.F32]); vals = [p.exp(0)]
    for i in range(7):
        vals.append(p.tanh(p.add(vals[-1], vals[0])))
    acc = vals[0]
    for t in vals[1:]:
        acc = p.mul(acc, t)
    total = p.add(acc, p.add(vals[1], p.add(vals[2], p.add(vals[3], p.add(vals[4], p.add(vals[5], p.add(vals[6], vals[7])))))))
    (got,), (want,) = run_ewise(p, [x], [total], expect_route=VEC if tier == "compiled" else 2)
    assert_f32(got, want, "total")
