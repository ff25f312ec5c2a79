"""The allocation-free variant of the reduce group against the ordinary entry point.

Some callers of this library may not allocate device memory (they live inside another
framework's memory pool, or are handed only their input and output buffers).  For them
relay_fused_reduce_static_scratch keeps the partial sums in an array built into the library
instead of a caller-provided workspace.  This file is collected last on purpose."""
import pytest
import torch

from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I
from relay_workloads import program as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _outputs(rows, cols):
    return [torch.full((rows, cols), 9.0, dtype=torch.bfloat16, device=DEV), torch.full((cols,), 9.0, device=DEV),
            torch.full((1, cols), 9.0, device=DEV)]


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    prog, ids = P.tanh_affine_residual_grad(P.BF16)
    specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_SUM, 1, 0), (ids[2], B.RED_SUM, 1, 1)]
    # calls in a row on the shared array: a larger one after a smaller one, then a smaller one again (fewer row slices
    # than the array still holds from the call before: stale partials must not be read)
    for call, (rows, cols) in enumerate([(517, 1024), (2048, 4096), (96, 1024)]):
        t = I.cfg2_ewise(rows, cols, salt=call)
        ins = [t[k].to(DEV) for k in ("dout", "x", "a", "b")]
        need = B.relay_workspace_bytes_reduce(ins, specs)
        assert 0 < need <= B.STATIC_SCRATCH_BYTES
        ws = torch.empty(need, dtype=torch.uint8, device=DEV)
        want = _outputs(rows, cols)
        B.relay_fused_reduce(prog.arrays(), ins, specs, want, ws)
        got = _outputs(rows, cols)
        B.relay_fused_reduce_static_scratch(prog.arrays(), ins, specs, got)
        torch.cuda.synchronize()
        for g, w, name in zip(got, want, ("dx", "da", "db")):
            # same kernels, same summation order: the tests' bf16 tolerance holds with room to spare
            assert torch.allclose(g.float(), w.float(), rtol=0, atol=1e-2 * float(w.float().pow(2).mean().sqrt())), name
            assert torch.equal(g, w), name
    # a plain column sum through the same entry point
    x = torch.randn(300, 512, device=DEV)
    got, want = torch.empty(512, device=DEV), torch.empty(512, device=DEV)
    sp = [(0, B.RED_SUM, 1, 0)]
    B.relay_fused_reduce(None, [x], sp, [want], torch.empty(B.relay_workspace_bytes_reduce([x], sp), dtype=torch.uint8, device=DEV))
    B.relay_fused_reduce_static_scratch(None, [x], sp, [got])
    torch.cuda.synchronize()
    assert torch.equal(got, want)


def test_static_scratch_rejects_groups_beyond_its_size():
    x = torch.zeros(8192, 2048, dtype=torch.bfloat16, device=DEV)
    sp = [(0, B.RED_SUM, 1, 0)] * 8                       # eight column sums at once: 9.7 MB of partials
    assert B.relay_workspace_bytes_reduce([x], sp) > B.STATIC_SCRATCH_BYTES
    outs = [torch.full((2048,), 5.0, device=DEV) for _ in range(8)]
    n0 = B.relay_launch_count()
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_reduce_static_scratch(None, [x], sp, outs)
    assert e.value.status_name == "ERR_WORKSPACE" and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and all(bool((o == 5.0).all()) for o in outs)


def test_static_scratch_takes_groups_that_use_less_than_their_bound():
    """What decides is the scratch a group's kernels really use: a reduction over the last axis uses none, so it is taken even
    where the program-independent bound of relay_workspace_bytes_reduce lies beyond the built-in array."""
    x = torch.randn(16, 2_400_000, device=DEV).to(torch.bfloat16)
    sp = [(0, B.RED_SUM, 2, 0)]
    assert B.relay_workspace_bytes_reduce([x], sp) > B.STATIC_SCRATCH_BYTES
    got, want = torch.full((16,), 9.0, device=DEV), torch.full((16,), 9.0, device=DEV)
    B.relay_fused_reduce(None, [x], sp, [want], torch.empty(B.relay_workspace_bytes_reduce([x], sp), dtype=torch.uint8, device=DEV))
    B.relay_fused_reduce_static_scratch(None, [x], sp, [got])
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    assert torch.allclose(got, x.float().sum(1), rtol=1e-3, atol=1.0)


def test_static_scratch_compiles_nothing():
    """Compiling a body at run time allocates, so this entry point never does it: a program without a pre-compiled body
    runs on the built-in kernels until relay_fused_reduce has compiled it, and gives the same sums either way."""
    x = torch.randn(300, 512, device=DEV)
    p = P.Program([P.F32]); v = p.tanh(p.sq(0))
    sp = [(v, B.RED_SUM, 1, 0)]
    n0 = B.relay_debug_jit_compiled()
    a, b, c = (torch.full((512,), 9.0, device=DEV) for _ in range(3))
    B.relay_fused_reduce_static_scratch(p.arrays(), [x], sp, [a])
    assert B.relay_debug_jit_compiled() == n0
    B.relay_fused_reduce(p.arrays(), [x], sp, [b], torch.empty(B.relay_workspace_bytes_reduce([x], sp), dtype=torch.uint8, device=DEV))
    B.relay_fused_reduce_static_scratch(p.arrays(), [x], sp, [c])
    torch.cuda.synchronize()
    assert torch.equal(b, c)
    want = torch.tanh(x.double() ** 2).sum(0)
    for got in (a, b):
        assert float((got.double() - want).abs().max()) <= 1e-4 * float(want.abs().max())
