"""Host-side: the bodies generated for run-time compilation are well-formed CUDA for sm_100a (no GPU: the source is generated and
compiled, nothing is loaded or launched).  What the compiled bodies compute is checked against the oracle in the GPU tests."""
import pytest
import torch

from paper_1810_00952_b200 import binding as B
from relay_workloads import program as P

BF, F32 = torch.bfloat16, torch.float32
def compile_group(prog, inputs, specs, want_source=False):
    return B.relay_debug_jit_compile(prog.arrays() if prog is not None else None, inputs, specs, want_source)


def _no_compiler():
    p = P.Program([P.F32]); v = p.neg(0)
    return compile_group(p, [torch.empty(8, 64)], [(v, B.RED_NONE, 0, 0)]) == -1


pytestmark = pytest.mark.skipif(_no_compiler(), reason="no run-time compiler library on this machine")


@pytest.mark.parametrize("tdt,code", [(BF, P.BF16), (F32, P.F32)])
def test_benchmark_programs_compile(tdt, code):
    x, y, z = torch.empty(64, 512, dtype=tdt), torch.empty(64, 512, dtype=tdt), torch.empty(512, dtype=tdt)
    p, outs = P.sigmoid_product_relu_fwd(code)
    r, src = compile_group(p, [x, y, z], [(outs[0], B.RED_NONE, 0, 0)], want_source=True)
    assert r == 1
    # one kernel; the row-constant operand is read once per thread, outside the loop over rows
    assert src.count("__global__") == 1 and "relay_jit_kernel" in src
    assert src.index("float f2[") < src.index("for (i64 r = r0 + ty")
    g, ids = P.sigmoid_product_relu_grad(code)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_NONE, 0, 0), (ids[2], B.RED_SUM, 1, 0)]
    r, src = compile_group(g, [x, x, y, z], specs, want_source=True)
    assert r == 1 and "acc2[e] +=" in src and "A.partial[2]" in src and "__shared__" in src


def test_every_operator_and_result_type_compiles():
    for tdt, code in ((BF, P.BF16), (F32, P.F32)):
        x, y, s = torch.empty(8, 4, 64, dtype=tdt), torch.empty(64, dtype=tdt), torch.empty((), dtype=tdt)
        # arithmetic and transcendental operators; a result in the storage type, one in f32, a mean and a sum over the rows
        p = P.Program([code, code, code])
        a = p.cast(0, P.F32); b = p.cast(1, P.F32); c = p.cast(2, P.F32)
        vals = [p.add(a, b), p.sub(a, c), p.div(a, p.add(p.sq(b), p.const(1.5, P.F32))), p.neg(a), p.tanh(a), p.sigmoid(b),
                p.exp(p.mul(a, p.const(0.125, P.F32))), p.log(p.add(p.sq(a), p.const(1.0, P.F32)))]
        acc = vals[0]
        for v in vals[1:]:
            acc = p.add(acc, v)
        out = p.cast(acc, code)
        assert compile_group(p, [x, y, s], [(out, B.RED_NONE, 0, 0), (acc, B.RED_NONE, 0, 0)]) == 1
        assert compile_group(p, [x, y, s], [(out, B.RED_NONE, 0, 0), (acc, B.RED_MEAN, 3, 0), (vals[2], B.RED_SUM, 3, 1)]) == 1
        # comparisons, selection, max / min / relu, Bool results stored as bytes, arithmetic typed in the storage type
        q = P.Program([code, code, code])
        m = q.cmp(P.OP_GE, 0, 1)
        sel = q.select(m, q.max(0, 2), q.min(q.relu(1), q.mul(0, 1)))
        outs = [sel, m, q.cmp(P.OP_NE, 0, 2), q.cmp(P.OP_EQ, 0, 1), q.cmp(P.OP_LT, 0, 1), q.cmp(P.OP_LE, 0, 1), q.cmp(P.OP_GT, 0, 2),
                q.cast(q.cmp(P.OP_LT, 0, 1), code)]
        assert compile_group(q, [x, y, s], [(o, B.RED_NONE, 0, 0) for o in outs]) == 1


def test_groups_outside_the_tier_are_not_compiled():
    p = P.Program([P.F32]); v = p.tanh(0)
    assert compile_group(p, [torch.empty(6, 33, dtype=F32)], [(v, B.RED_NONE, 0, 0)]) == 0          # rows are not whole vectors
    p = P.Program([P.I32]); v = p.cast(0, P.I64)
    assert compile_group(p, [torch.empty(8, 64, dtype=torch.int32)], [(v, B.RED_NONE, 0, 0)]) == 0   # integer values
    p = P.Program([P.F32]); v = p.sq(0)
    assert compile_group(p, [torch.empty(8, 64, dtype=F32)], [(v, B.RED_MAX, 1, 0)]) == 0            # no column sum
