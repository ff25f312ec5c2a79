"""Host-side: which kernel tier a fused group is planned for (no GPU: descriptors are not dereferenced)."""
import pytest
import torch

from paper_1810_00952_b200 import binding as B
from relay_workloads import program as P

BF, F32 = torch.bfloat16, torch.float32
PRE, VEC, SCALAR, ROW = 0, 1, 2, 3


def route(prog, inputs, specs):
    return B.relay_debug_group_route(prog.arrays() if prog is not None else None, inputs, specs)


def test_benchmark_groups_take_their_pre_compiled_bodies():
    x, a, b = torch.empty(64, 512, dtype=BF), torch.empty(512, dtype=BF), torch.empty(1, 512, dtype=BF)
    p, outs = P.tanh_affine_residual_fwd(P.BF16)
    assert route(p, [x, a, b], [(outs[0], B.RED_NONE, 0, 0)]) == PRE
    g, ids = P.tanh_affine_residual_grad(P.BF16)
    assert route(g, [x, x, a, b], [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_SUM, 1, 0), (ids[2], B.RED_SUM, 1, 1)]) == PRE
    assert route(None, [x], [(0, B.RED_SUM, 1, 0)]) == PRE and route(None, [x], [(0, B.RED_ARGMAX, 2, 0)]) == ROW


@pytest.mark.parametrize("tdt,code", [(BF, P.BF16), (F32, P.F32)])
def test_other_programs_over_a_2d_view_take_the_vectorised_evaluator(tdt, code):
    x, y, z = torch.empty(64, 512, dtype=tdt), torch.empty(64, 512, dtype=tdt), torch.empty(512, dtype=tdt)
    p, outs = P.sigmoid_product_relu_fwd(code)
    assert route(p, [x, y, z], [(outs[0], B.RED_NONE, 0, 0)]) == VEC
    g, ids = P.sigmoid_product_relu_grad(code)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_NONE, 0, 0), (ids[2], B.RED_SUM, 1, 0)]
    assert route(g, [x, x, y, z], specs) == VEC
    # the same tanh-affine expression with a full-shape `a` has no pre-compiled instance
    p2, o2 = P.tanh_affine_residual_fwd(code)
    assert route(p2, [x, y, z.reshape(1, 512)], [(o2[0], B.RED_NONE, 0, 0)]) == VEC
    # a scalar operand, a Bool result, a rank-3 tensor collapsing to [rows, cols]
    q = P.Program([code, code]); m = q.cmp(P.OP_GT, q.mul(0, 1), 0)
    assert route(q, [torch.empty(4, 16, 64, dtype=tdt), torch.empty((), dtype=tdt)], [(m, B.RED_NONE, 0, 0)]) == VEC


def test_what_the_vectorised_evaluator_does_not_take_runs_on_the_scalar_one():
    x = torch.empty(6, 33, dtype=F32)                                   # rows are not whole 16-byte vectors
    p = P.Program([P.F32]); v = p.tanh(0)
    assert route(p, [x], [(v, B.RED_NONE, 0, 0)]) == SCALAR
    xi = torch.empty(8, 64, dtype=torch.int32)                          # integer values
    p = P.Program([P.I32]); v = p.cast(0, P.I64)
    assert route(p, [xi], [(v, B.RED_NONE, 0, 0)]) == SCALAR
    x3, col = torch.empty(4, 8, 64, dtype=F32), torch.empty(8, 1, dtype=F32)   # broadcast along the middle axis only
    p = P.Program([P.F32, P.F32]); v = p.add(0, 1)
    assert route(p, [x3, col], [(v, B.RED_NONE, 0, 0)]) == SCALAR
    p = P.Program([P.F32]); v = p.sq(0)                                 # max over rows is no column sum
    assert route(p, [torch.empty(8, 64, dtype=F32)], [(v, B.RED_MAX, 1, 0)]) == SCALAR
    # an expression with more values alive at once than the interpreter has temporaries for: compiled at run time where a
    # compiler library is present (a generated body has no such limit), on the scalar evaluator otherwise
    p = P.Program([P.F32]); vals = [p.exp(0)]
    for i in range(7):
        vals.append(p.tanh(p.add(vals[-1], vals[0])))
    acc = vals[0]
    for t in vals[1:]:
        acc = p.mul(acc, t)
    total = p.add(acc, p.add(vals[1], p.add(vals[2], p.add(vals[3], p.add(vals[4], p.add(vals[5], p.add(vals[6], vals[7])))))))
    specs = [(total, B.RED_NONE, 0, 0)]
    have_compiler = B.relay_debug_jit_compiled() >= 0
    assert route(p, [torch.empty(8, 64, dtype=F32)], specs) == (VEC if have_compiler else SCALAR)
    before = B.relay_debug_set_jit(False)
    try:
        assert route(p, [torch.empty(8, 64, dtype=F32)], specs) == SCALAR
    finally:
        B.relay_debug_set_jit(before)


def test_ill_typed_groups_are_reported():
    p = P.Program([P.F32, P.BF16]); v = p.emit(P.OP_ADD, 0, 1, dtype=P.F32)
    with pytest.raises(B.RelayError):
        route(p, [torch.empty(8, 8), torch.empty(8, 8, dtype=BF)], [(v, B.RED_NONE, 0, 0)])
