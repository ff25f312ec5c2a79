"""GPU parity: fused broadcast-elementwise and elementwise+reduce groups against the CPU oracle,
through the C-ABI, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I
from relay_workloads import program as P

from parity import Guarded, assert_bf16, assert_f32, rms, to_np, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TDT = {P.BF16: torch.bfloat16, P.F32: torch.float32}


def _fwd(t, storage, rows, cols):
    prog, outs = P.tanh_affine_residual_fwd(storage)
    x, a, b = (t[k].to(DEV) for k in ("x", "a", "b"))
    out = Guarded((rows, cols), TDT[storage], DEV)
    B.relay_fused_ewise(prog.arrays(), [x, a, b], outs, [out.t])
    torch.cuda.synchronize()
    return prog, outs, out.check()


# several column slabs, several row slices, ragged row tail; cols % 8 != 0 takes the generic evaluator
@pytest.mark.parametrize("rows,cols", [(1, 8), (333, 2048), (77, 520), (64, 1000), (5, 3), (300, 264)])
@pytest.mark.parametrize("storage", [P.BF16, P.F32])
def test_tanh_affine_residual_forward(rows, cols, storage):
    t = I.cfg2_ewise(rows, cols, dtype=TDT[storage])
    prog, outs, got = _fwd(t, storage, rows, cols)
    oprog, oouts = P.tanh_affine_residual_fwd(5, 5)     # oracle: fp64 values before storage rounding
    (want,) = oracle.ewise(oprog.arrays(), [I.as_f64(t[k]) for k in ("x", "a", "b")], oouts)
    (assert_bf16 if storage == P.BF16 else assert_f32)(got, want, what=f"fwd {rows}x{cols}")


def _grad(t, storage, a_shape=None):
    prog, (dx_id, da_id, db_id) = P.tanh_affine_residual_grad(storage)
    d, x, a, b = (t[k].to(DEV) for k in ("dout", "x", "a", "b"))
    if a_shape is not None:
        a = a.reshape(a_shape)
    rows, cols = x.shape
    specs = [(dx_id, B.RED_NONE, 0, 0), (da_id, B.RED_SUM, 1, 0), (db_id, B.RED_SUM, 1, 1)]
    dx = Guarded((rows, cols), TDT[storage], DEV)
    da = Guarded((cols,), torch.float32, DEV)
    db = Guarded((1, cols), torch.float32, DEV)
    ws = workspace(B.relay_workspace_bytes_reduce([d, x, a, b], specs), DEV)
    B.relay_fused_reduce(prog.arrays(), [d, x, a, b], specs, [dx.t, da.t, db.t], ws)
    torch.cuda.synchronize()
    return dx.check(), da.check(), db.check()


def _grad_oracle(t):
    prog, (dx_id, da_id, db_id) = P.tanh_affine_residual_grad(5, 5)
    return oracle.reduce(prog.arrays(), [I.as_f64(t[k]) for k in ("dout", "x", "a", "b")],
                         [(dx_id, oracle.RED_NONE, (), False, 5), (da_id, oracle.RED_SUM, (0,), False, 5),
                          (db_id, oracle.RED_SUM, (0,), True, 5)])


@pytest.mark.parametrize("rows,cols", [(1, 8), (333, 2048), (1000, 264), (64, 1000), (7, 5)])
@pytest.mark.parametrize("storage", [P.BF16, P.F32])
def test_tanh_affine_residual_gradient_group(rows, cols, storage):
    t = I.cfg2_ewise(rows, cols, dtype=TDT[storage])
    dx, da, db = _grad(t, storage)
    odx, oda, odb = _grad_oracle(t)
    if storage == P.BF16:
        assert_bf16(dx, odx, what="dx")
        assert_bf16(da, oda, stored_bf16=False, what="da")
        assert_bf16(db, odb, stored_bf16=False, what="db")
    else:
        for g, o, n in ((dx, odx, "dx"), (da, oda, "da"), (db, odb, "db")):
            assert_f32(g, o, what=n)
    # invariants of this group: a*s+1 in [1, 2.5)
    gx, d = to_np(dx), I.as_f64(t["dout"])
    assert np.all(np.sign(gx) == np.sign(d)) and np.all(np.abs(gx) <= 2.5 * np.abs(d) * (1 + 2.0 ** -7))


def test_gradient_group_is_deterministic_and_generic_route_agrees():
    t = I.cfg2_ewise(517, 1024)
    r1 = _grad(t, P.BF16)
    r2 = _grad(t, P.BF16)
    for u, v in zip(r1, r2):
        assert torch.equal(u, v)                       # fixed summation order: bit-identical reruns
    r3 = _grad(t, P.BF16, a_shape=(1, 1024))            # same program, same result types ...
    assert torch.equal(r1[0], r3[0])
    odx, oda, odb = _grad_oracle(t)
    assert_bf16(r3[1], oda, stored_bf16=False)


def test_every_opcode_generic_evaluator_with_broadcasting():
    rng = np.random.default_rng(40)
    x = torch.from_numpy(rng.standard_normal((6, 1, 33))).float()
    y = torch.from_numpy(rng.standard_normal((5, 33))).float()
    y[0, :4] = x[0, 0, :4]
    builds = {
        "add": lambda p: p.add(0, 1), "sub": lambda p: p.sub(0, 1), "mul": lambda p: p.mul(0, 1),
        "div": lambda p: p.div(0, p.add(p.sq(1), p.const(1.0))), "neg": lambda p: p.neg(0), "sq": lambda p: p.sq(1),
        "relu": lambda p: p.relu(0), "tanh": lambda p: p.tanh(0), "sigmoid": lambda p: p.sigmoid(1),
        "exp": lambda p: p.exp(0), "log": lambda p: p.log(p.add(p.sq(0), p.const(0.5))),
        "max": lambda p: p.max(0, 1), "min": lambda p: p.min(0, 1),
        "select": lambda p: p.select(p.cmp(P.OP_GT, 0, 1), 0, 1),
        "cast_bf16": lambda p: p.cast(p.mul(0, 1), P.BF16),
    }
    for name, build in builds.items():
        p = P.Program([P.F32, P.F32]); v = build(p)
        dt = p.dtype_of(v)
        out = Guarded((6, 5, 33), TDT.get(dt, torch.float32), DEV)
        B.relay_fused_ewise(p.arrays(), [x.to(DEV), y.to(DEV)], [v], [out.t])
        (want,) = oracle.ewise(p.arrays(), [x.double().numpy(), y.double().numpy()], [v])
        if dt == P.BF16:
            q = P.Program([P.F32, P.F32]); u = q.mul(0, 1)
            (unrounded,) = oracle.ewise(q.arrays(), [x.double().numpy(), y.double().numpy()], [u])
            assert_bf16(out.check(), unrounded, what=name)
        else:
            assert_f32(out.check(), want, what=name)
    for op in (P.OP_NE, P.OP_EQ, P.OP_LT, P.OP_LE, P.OP_GT, P.OP_GE):   # Bool results: bit-exact
        p = P.Program([P.F32, P.F32]); v = p.cmp(op, 0, 1)
        out = Guarded((6, 5, 33), torch.uint8, DEV)
        B.relay_fused_ewise(p.arrays(), [x.to(DEV), y.to(DEV)], [v], [out.t])
        (want,) = oracle.ewise(p.arrays(), [x.double().numpy(), y.double().numpy()], [v])
        assert np.array_equal(out.check().cpu().numpy(), want.astype(np.uint8)), op


def test_multi_output_scalar_and_rank0_inputs():
    p = P.Program([P.F32, P.F32])
    s = p.add(0, 1); m = p.mul(s, 1)
    x = torch.randn(4, 9, generator=torch.Generator().manual_seed(1)); k = torch.tensor(1.5)
    o1, o2 = Guarded((4, 9), torch.float32, DEV), Guarded((4, 9), torch.float32, DEV)
    B.relay_fused_ewise(p.arrays(), [x.to(DEV), k.to(DEV)], [s, m], [o1.t, o2.t])
    w1, w2 = oracle.ewise(p.arrays(), [x.double().numpy(), k.double().numpy()], [s, m])
    assert_f32(o1.check(), w1); assert_f32(o2.check(), w2)


RED = {B.RED_SUM: "sum", B.RED_MAX: "max", B.RED_MEAN: "mean"}


@pytest.mark.parametrize("shape,axes", [((300, 512), (0,)), ((300, 512), (1,)), ((37, 29), (0,)), ((37, 29), (1,)),
                                         ((5, 6, 64), (0, 1)), ((5, 6, 64), (2,)), ((5, 6, 7), (0, 2)), ((4, 3, 5, 6), (1, 3)),
                                         ((3000,), (0,)), ((2, 4096), (0, 1)), ((1100, 4872), (0,))])
@pytest.mark.parametrize("tdt", [torch.bfloat16, torch.float32])
def test_standalone_reduce_all_routes(shape, axes, tdt):
    g = torch.Generator().manual_seed(7)
    x = torch.randn(*shape, generator=g).to(tdt)
    mask = sum(1 << a for a in axes)
    ident = P.Program([P.BF16 if tdt == torch.bfloat16 else P.F32])
    xo = x.double().numpy()
    for red, name in RED.items():
        for keep in (False, True):
            oshape = oracle.reduce_shape(shape, axes, keep)
            out = Guarded(oshape, torch.float32, DEV)
            specs = [(0, red, mask, int(keep))]
            ws = workspace(B.relay_workspace_bytes_reduce([x], specs), DEV)
            B.relay_fused_reduce(None, [x.to(DEV)], specs, [out.t], ws)
            (want,) = oracle.reduce(ident.arrays(), [xo], [(0, red, axes, keep, 5)])
            if tdt == torch.bfloat16 and red != B.RED_MAX:
                assert_bf16(out.check(), want, stored_bf16=False, what=f"{name} {shape} {axes}")
            else:
                assert_f32(out.check(), want, what=f"{name} {shape} {axes}")


@pytest.mark.parametrize("shape,axis", [((64, 4096), 1), ((64, 4096), 0), ((9, 11), 1), ((9, 11), 0), ((6, 5, 40), 1), ((1, 24), 1)])
def test_argmax_bit_exact_with_ties(shape, axis):
    g = torch.Generator().manual_seed(11)
    for tdt in (torch.float32, torch.bfloat16):
        x = torch.randint(0, 5, shape, generator=g).to(tdt)      # many ties: the lowest index must win
        oshape = oracle.reduce_shape(shape, (axis,), False)
        out = Guarded(oshape, torch.int64, DEV)
        B.relay_fused_reduce(None, [x.to(DEV)], [(0, B.RED_ARGMAX, 1 << axis, 0)], [out.t], None)
        ident = P.Program([P.F32])
        (want,) = oracle.reduce(ident.arrays(), [x.double().numpy()], [(0, oracle.RED_ARGMAX, (axis,), False, P.I64)])
        assert np.array_equal(out.check().cpu().numpy(), want)


def test_standalone_reductions_full_size_all_results():
    """The standalone reductions at the size and in the launch shape the benchmark times (8192 x 8192 bf16): sum, max and
    argmax over the last axis and the sum over axis 0, EVERY result against the oracle.  Ties are planted for the argmax:
    in every row the maximum is written to several columns (two of them inside one 16-byte vector, others in the strips
    of other lanes), and in some rows to column 0 and the last column; the lowest index must win, bit for bit."""
    t = I.cfg2_ewise()
    x = t["x"].clone()
    rng = np.random.default_rng(29)
    top = float(x.max()) + 1.0
    for r in range(8192):
        c = np.sort(rng.choice(8192, 4, replace=False))
        x[r, c] = top
        x[r, min(int(c[0]) + 1, 8191)] = top                  # a neighbour in the same (or the next) vector
    x[5, 0] = top; x[6, 8191] = top; x[7] = top               # first column, a late column, a constant row
    xd = x.to(DEV)
    ident = P.Program([P.BF16])
    outs = dict(sum1=Guarded((8192,), torch.float32, DEV), max1=Guarded((8192,), torch.float32, DEV),
                arg1=Guarded((8192,), torch.int64, DEV), sum0=Guarded((8192,), torch.float32, DEV))
    specs = dict(sum1=(0, B.RED_SUM, 2, 0), max1=(0, B.RED_MAX, 2, 0), arg1=(0, B.RED_ARGMAX, 2, 0), sum0=(0, B.RED_SUM, 1, 0))
    for k, sp in specs.items():
        ws = workspace(B.relay_workspace_bytes_reduce([xd], [sp]), DEV)
        B.relay_fused_reduce(None, [xd], [sp], [outs[k].t], ws)
    torch.cuda.synchronize()
    xo = x.double().numpy()
    w_sum1, w_max1, w_arg1, w_sum0 = oracle.reduce(ident.arrays(), [xo], [(0, oracle.RED_SUM, (1,), False, 5), (0, oracle.RED_MAX, (1,), False, 5),
                                                                          (0, oracle.RED_ARGMAX, (1,), False, P.I64), (0, oracle.RED_SUM, (0,), False, 5)])
    assert np.array_equal(outs["arg1"].check().cpu().numpy(), w_arg1)
    assert np.array_equal(to_np(outs["max1"].check()), w_max1)              # a maximum is one of the inputs: exact
    assert_bf16(outs["sum1"].check(), w_sum1, stored_bf16=False, what="sum over the last axis")
    assert_bf16(outs["sum0"].check(), w_sum0, stored_bf16=False, what="sum over axis 0")
    assert int(w_arg1[7]) == 0 and int(w_arg1[5]) == 0


@pytest.mark.parametrize("shape,axes", [((1024, 2048), (0, 1)), ((3, 700, 301), (1, 2)), ((2, 517, 1031), (0, 1, 2)), ((262144, 2), (0,))])
def test_few_results_over_a_long_extent_are_split_over_blocks(shape, axes):
    """A reduction with a handful of results over a long reduced extent (a sum over all axes, say) is cut into runs that
    separate blocks reduce and a second pass combines in run order: sum, mean, max and argmax (ties: the lowest position
    wins across runs too), with and without a program in front, and a sum whose terms nearly cancel."""
    g = torch.Generator().manual_seed(23)
    x = torch.randn(*shape, generator=g)
    mask = sum(1 << a for a in axes)
    ident, sqp = P.Program([P.F32]), P.Program([P.F32])
    sq = sqp.sq(0)
    xo = x.double().numpy()
    oshape = oracle.reduce_shape(shape, axes, False)
    for red in (B.RED_SUM, B.RED_MEAN, B.RED_MAX):
        for prog, val in ((None, 0), (sqp, sq)):
            out = Guarded(oshape, torch.float32, DEV)
            specs = [(val, red, mask, 0)]
            B.relay_fused_reduce(prog.arrays() if prog else None, [x.to(DEV)], specs, [out.t],
                                 workspace(B.relay_workspace_bytes_reduce([x], specs), DEV))
            (want,) = oracle.reduce((prog or ident).arrays(), [xo], [(val, red, axes, False, 5)])
            if red == B.RED_MAX and prog is None:
                assert np.array_equal(to_np(out.check()), want)
            elif prog is None and red != B.RED_MAX:
                # a sum of zero-mean terms: bounded against the size of the terms, not of the (cancelled) result
                n_red = int(np.prod([shape[a] for a in axes]))
                scale = 1.0 if red == B.RED_SUM else 1.0 / n_red
                assert np.all(np.abs(to_np(out.check()) - want) <= 1e-6 * scale * np.sqrt(n_red) * 8)
            else:
                assert_f32(out.check(), want, what=f"{red} {shape} {axes}")
    xt = torch.randint(0, 7, shape, generator=g).float()          # many ties, in every run
    out = Guarded(oshape, torch.int64, DEV)
    specs = [(0, B.RED_ARGMAX, mask, 0)]
    B.relay_fused_reduce(None, [xt.to(DEV)], specs, [out.t], workspace(B.relay_workspace_bytes_reduce([xt], specs), DEV))
    (want,) = oracle.reduce(ident.arrays(), [xt.double().numpy()], [(0, oracle.RED_ARGMAX, axes, False, P.I64)])
    assert np.array_equal(out.check().cpu().numpy(), want)
    B.relay_poll_status()


def test_reduce_with_prologue_and_unreduced_output_generic():
    g = torch.Generator().manual_seed(13)
    x, w = torch.randn(40, 24, generator=g), torch.randn(24, generator=g)
    p = P.Program([P.F32, P.F32]); prod = p.mul(0, 1); sq = p.sq(prod)
    o_full, o_col, o_row = Guarded((40, 24), torch.float32, DEV), Guarded((24,), torch.float32, DEV), Guarded((40, 1), torch.float32, DEV)
    specs = [(prod, B.RED_NONE, 0, 0), (sq, B.RED_SUM, 1, 0), (prod, B.RED_MAX, 2, 1)]
    B.relay_fused_reduce(p.arrays(), [x.to(DEV), w.to(DEV)], specs, [o_full.t, o_col.t, o_row.t], None)
    wf, wc, wr = oracle.reduce(p.arrays(), [x.double().numpy(), w.double().numpy()],
                               [(prod, 0, (), False, 5), (sq, 1, (0,), False, 5), (prod, 2, (1,), True, 5)])
    assert_f32(o_full.check(), wf); assert_f32(o_col.check(), wc); assert_f32(o_row.check(), wr)


def test_descriptor_errors_launch_nothing_and_leave_outputs_untouched():
    prog, outs = P.tanh_affine_residual_fwd(P.BF16)
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device=DEV); a = torch.zeros(64, dtype=torch.bfloat16, device=DEV)
    b = torch.zeros(1, 64, dtype=torch.bfloat16, device=DEV)
    out = torch.full((16, 64), 3.0, dtype=torch.bfloat16, device=DEV)
    n0 = B.relay_launch_count()
    cases = [([x, a[:63].contiguous(), b], out, "ERR_SHAPE"),
             ([x, a, b], torch.empty(16, 64, dtype=torch.float32, device=DEV), "ERR_DTYPE"),
             ([x, a, b], torch.empty(16, 32, dtype=torch.bfloat16, device=DEV), "ERR_SHAPE"),
             ([x, a, b], x, "ERR_ATTR"),                                        # output aliases an input
             ([x, a, b], out.view(-1)[1:1 + 15 * 64].view(15, 64), "ERR_SHAPE")]
    for ins, o, status in cases:
        with pytest.raises(B.RelayError) as e:
            B.relay_fused_ewise(prog.arrays(), ins, outs, [o])
        assert e.value.status_name == status, str(e.value)
    mis = torch.empty(16 * 64 + 8, dtype=torch.bfloat16, device=DEV)[1:1 + 16 * 64].view(16, 64)   # 2-byte offset
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_ewise(prog.arrays(), [x, a, b], outs, [mis])
    assert e.value.status_name == "ERR_ALIGN"
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((out == 3.0).all())
    # workspace too small for the gradient group
    gp, ids = P.tanh_affine_residual_grad(P.BF16)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_SUM, 1, 0), (ids[2], B.RED_SUM, 1, 1)]
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_reduce(gp.arrays(), [x, x, a, b], specs,
                             [torch.empty_like(x), torch.empty(64, device=DEV), torch.empty(1, 64, device=DEV)], None)
    assert e.value.status_name in ("ERR_WORKSPACE", "ERR_ATTR")


def test_empty_tensors_are_accepted():
    p = P.Program([P.F32]); v = p.relu(0)
    x = torch.empty(0, 8, device=DEV); out = torch.empty(0, 8, device=DEV)
    B.relay_fused_ewise(p.arrays(), [x], [v], [out])


def test_full_size_forward_and_gradient_sampled_columns():
    """Configuration 2 at full size (8192 x 8192, bf16) in the launch shape the benchmark times;
    the oracle recomputes whole columns (all 8192 rows each, so column sums are covered): at least one in
    every 256-column slab of the launch grid, the slab edges, and random ones."""
    t = I.cfg2_ewise()
    prog, outs, got = _fwd(t, P.BF16, 8192, 8192)
    dx, da, db = _grad(t, P.BF16)
    rng = np.random.default_rng(3)
    cols = np.unique(np.concatenate([[0, 7, 8, 255, 256, 8191], np.arange(0, 8192, 256) + rng.integers(0, 256, 32),
                                     rng.integers(0, 8192, 16)]))
    assert len(np.unique(cols // 256)) == 32
    sub = {k: t[k][..., cols] for k in ("x", "a", "b", "dout")}
    fp, fo = P.tanh_affine_residual_fwd(5, 5)
    (want,) = oracle.ewise(fp.arrays(), [I.as_f64(sub[k]) for k in ("x", "a", "b")], fo)
    assert_bf16(got[:, cols], want, what="fwd")
    odx, oda, odb = _grad_oracle(sub)
    assert_bf16(dx[:, cols], odx, what="dx")
    assert_bf16(da[cols], oda, stored_bf16=False, what="da")
    assert_bf16(db[:, cols], odb, stored_bf16=False, what="db")
    # properties over the whole output
    gx, d = dx.float(), t["dout"].to(DEV).float()
    assert bool((torch.sign(gx) == torch.sign(d)).all()) and bool((gx.abs() <= 2.5 * d.abs() * (1 + 2.0 ** -7)).all())
    assert bool(((got.float() - t["x"].to(DEV).float()).abs() <= 1.0 + 2.0 ** -5).all())   # |tanh| <= 1
