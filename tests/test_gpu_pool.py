"""GPU parity: max pooling and its gradient against the CPU oracle (values and positions bit-exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I

from parity import Guarded, assert_bf16, assert_f32, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
F32, BF16 = torch.float32, torch.bfloat16


def run_pool(x, k, want_idx=True):
    kh, kw, sh, sw = k
    N, C, H, W = x.shape
    P, Q = (H - kh) // sh + 1, (W - kw) // sw + 1
    y = Guarded((N, C, P, Q), x.dtype, DEV)
    idx = Guarded((N, C, P, Q), torch.int32, DEV) if want_idx else None
    B.relay_max_pool2d(x.to(DEV), kh, kw, sh, sw, y.t, idx.t if idx else None)
    torch.cuda.synchronize()
    return y.check(), (idx.check() if idx else None)


def run_grad(idx, dy, k, H, W):
    N, C = dy.shape[:2]
    dx = Guarded((N, C, H, W), dy.dtype, DEV)
    B.relay_max_pool2d_grad(idx.to(DEV), dy.to(DEV), *k, dx.t)
    torch.cuda.synchronize()
    return dx.check()


CASES = [((2, 20, 24, 24), (2, 2, 2, 2)),      # LeNet's first pooling layer
         ((3, 50, 8, 8), (2, 2, 2, 2)),        # its second one
         ((2, 3, 7, 16), (2, 2, 2, 2)),        # odd height on the 16-byte route
         ((2, 3, 9, 10), (2, 2, 2, 2)),        # rows that are not whole vectors
         ((1, 4, 12, 12), (3, 3, 1, 1)),       # overlapping windows
         ((2, 2, 11, 9), (3, 2, 2, 1)),
         ((1, 2, 6, 6), (6, 6, 1, 1)),         # one window per plane
         ((1, 1, 5, 5), (1, 1, 1, 1)),         # identity
         ((2, 2, 13, 17), (2, 3, 3, 2))]


@pytest.mark.parametrize("shape,k", CASES)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("levels", [0, 3])
def test_pool_and_gradient(shape, k, dt, levels):
    x = I.pool_input(*shape, dtype=dt, levels=levels, salt=shape[2] * 7 + k[0])
    y, idx = run_pool(x, k)
    oy, oidx = oracle.max_pool2d(I.as_f64(x), *k)
    assert np.array_equal(to_np(y), oy)                           # a maximum is one of the inputs: exact
    assert np.array_equal(idx.cpu().numpy(), oidx)                # first maximum wins, bit-exact positions
    y2, none = run_pool(x, k, want_idx=False)
    assert none is None and torch.equal(y, y2)
    dy = I.normal(8, 1, tuple(y.shape), 1.0, dt, salt=shape[3])
    dx = run_grad(idx, dy, k, shape[2], shape[3])
    odx = oracle.max_pool2d_grad(oidx, I.as_f64(dy), shape[2], shape[3])
    if k[2] >= k[0] and k[3] >= k[1]:                             # disjoint windows: dx is a placement of dy, exact
        assert np.array_equal(to_np(dx), odx)
    elif dt == F32:
        assert_f32(dx, odx, what="dx")
    else:
        assert_bf16(dx, odx, what="dx")


def test_gradient_ignores_positions_outside_their_window_and_rejections():
    x = I.pool_input(1, 2, 8, 8, dtype=F32)
    y, idx = run_pool(x, (2, 2, 2, 2))
    bad = idx.clone(); bad[0, 0, 0, 0] = 63                       # names an input of another window
    dy = torch.ones_like(y)
    dx = run_grad(bad, dy, (2, 2, 2, 2), 8, 8)
    assert float(dx.sum()) == dy.numel() - 1 and float(dx[0, 0, 7, 7]) == (1.0 if int(idx[0, 0, 3, 3]) == 63 else 0.0)
    xd = x.to(DEV)
    out = torch.full((1, 2, 4, 4), 5.0, device=DEV)
    n0 = B.relay_launch_count()
    for fn, status in [(lambda: B.relay_max_pool2d(xd, 9, 2, 1, 1, out), "ERR_ATTR"),
                       (lambda: B.relay_max_pool2d(xd, 2, 2, 0, 2, out), "ERR_ATTR"),
                       (lambda: B.relay_max_pool2d(xd, 2, 2, 2, 2, out.bfloat16()), "ERR_DTYPE"),
                       (lambda: B.relay_max_pool2d(xd, 2, 2, 2, 2, torch.zeros(1, 2, 4, 3, device=DEV)), "ERR_SHAPE"),
                       (lambda: B.relay_max_pool2d(xd, 2, 2, 2, 2, out, torch.zeros(1, 2, 4, 4, device=DEV)), "ERR_DTYPE"),
                       (lambda: B.relay_max_pool2d(xd.view(2, 8, 8), 2, 2, 2, 2, out), "ERR_RANK"),
                       (lambda: B.relay_max_pool2d_grad(idx.to(DEV), out.bfloat16(), 2, 2, 2, 2, torch.empty_like(xd)), "ERR_DTYPE"),
                       (lambda: B.relay_max_pool2d_grad(idx.to(DEV), out, 2, 2, 1, 1, torch.empty_like(xd)), "ERR_SHAPE")]:
        with pytest.raises(B.RelayError) as e:
            fn()
        assert e.value.status_name == status, str(e.value)
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((out == 5.0).all())


def test_full_size_pool_sampled_planes():
    """32 x 256 x 56 x 56 bf16 (the activation of the conv configuration), 2 x 2 windows, stride 2."""
    x = I.pool_input()
    k = (2, 2, 2, 2)
    y, idx = run_pool(x, k)
    dy = I.normal(8, 1, tuple(y.shape), 1.0, BF16)
    dx = run_grad(idx, dy, k, 56, 56)
    rng = np.random.default_rng(2)
    for n, c in [(0, 0), (31, 255)] + [tuple(v) for v in rng.integers(0, [32, 256], (6, 2))]:
        oy, oidx = oracle.max_pool2d(I.as_f64(x[n:n + 1, c:c + 1]), *k)
        assert np.array_equal(to_np(y[n:n + 1, c:c + 1]), oy) and np.array_equal(idx[n:n + 1, c:c + 1].cpu().numpy(), oidx)
        odx = oracle.max_pool2d_grad(oidx, I.as_f64(dy[n:n + 1, c:c + 1]), 56, 56)
        assert np.array_equal(to_np(dx[n:n + 1, c:c + 1]), odx)
    # properties that hold for the whole tensor: every position lies in its window; dx conserves dy per plane
    pos = idx.long()
    p = torch.arange(28, device=DEV).view(1, 1, 28, 1); q = torch.arange(28, device=DEV).view(1, 1, 1, 28)
    h, w = pos // 56, pos % 56
    assert bool(((h >= 2 * p) & (h < 2 * p + 2) & (w >= 2 * q) & (w < 2 * q + 2)).all())
    assert torch.equal(torch.gather(x.to(DEV).view(32, 256, -1), 2, pos.view(32, 256, -1)).view_as(y), y)
    assert int((dx != 0).sum()) <= dy.numel()
