"""GPU parity: softmax cross-entropy loss, its gradient group and the SGD parameter update against the CPU
oracle, through the C ABI."""
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


def run_loss(t):
    z, tg = t["scores"].to(DEV), t["targets"].to(DEV)
    loss = Guarded((z.shape[0],), F32, DEV)
    B.relay_softmax_xent(z, tg, loss.t)
    torch.cuda.synchronize()
    return loss.check()


def run_grad(t, want_loss=True):
    z, tg, dl = t["scores"].to(DEV), t["targets"].to(DEV), t["dloss"].to(DEV)
    loss = Guarded((z.shape[0],), F32, DEV) if want_loss else None
    dz = Guarded(tuple(z.shape), z.dtype, DEV)
    B.relay_softmax_xent_grad(z, tg, dl, loss.t if loss else None, dz.t)
    torch.cuda.synchronize()
    return (loss.check() if loss else None), dz.check()


# rows per warp or per block, whole 16-byte vectors or not, rows longer than the register cache
SHAPES = [(1, 1), (7, 10), (64, 1000), (33, 37), (16, 1024), (300, 512), (9, 8200), (5, 5003), (3, 40000)]


@pytest.mark.parametrize("Bn,C", SHAPES)
@pytest.mark.parametrize("dt,tdt", [(F32, F32), (BF16, BF16), (BF16, F32)])
@pytest.mark.parametrize("one_hot", [False, True])
def test_loss_and_gradient_group(Bn, C, dt, tdt, one_hot):
    t = I.loss_batch(Bn, C, dt, tdt, one_hot=one_hot, salt=Bn * 131 + C)
    zo, to_, dlo = (I.as_f64(t[k]) for k in ("scores", "targets", "dloss"))
    want_loss, want_dz = oracle.softmax_xent_grad(zo, to_, dlo)
    loss = run_loss(t)
    loss2, dz = run_grad(t)
    assert torch.equal(loss, loss2)                     # the same arithmetic in both entry points
    if dt == F32:
        assert_f32(loss, want_loss, what="loss"); assert_f32(dz, want_dz, what="dscores")
    else:
        assert_bf16(loss, want_loss, stored_bf16=False, what="loss"); assert_bf16(dz, want_dz, what="dscores")
    _, dz_only = run_grad(t, want_loss=False)
    assert torch.equal(dz, dz_only)


def test_large_scores_do_not_overflow_and_constant_rows_give_log_c():
    z = torch.tensor([[1000.0, 0.0, -1000.0], [-50.0, -50.0, -50.0], [80.0, 90.0, 100.0]])
    tg = torch.tensor([[0.0, 1.0, 0.0], [1.0, 0.0, 0.0], [0.0, 0.0, 1.0]])
    t = dict(scores=z, targets=tg, dloss=torch.ones(3))
    loss, dz = run_grad(t)
    want_loss, want_dz = oracle.softmax_xent_grad(z.double().numpy(), tg.double().numpy(), np.ones(3))
    assert_f32(loss, want_loss, what="loss"); assert_f32(dz, want_dz, what="dscores")
    assert abs(float(loss[1]) - np.log(3)) < 1e-6 and abs(float(loss[0]) - 1000.0) < 1e-3


def test_empty_batch_and_rejections_leave_outputs_untouched():
    z0 = torch.zeros(0, 5, device=DEV); l0 = torch.zeros(0, device=DEV)
    B.relay_softmax_xent(z0, z0.clone(), l0)
    z = torch.zeros(4, 8, device=DEV); tg = torch.zeros(4, 8, device=DEV)
    loss = torch.full((4,), 5.0, device=DEV); dz = torch.full((4, 8), 5.0, device=DEV); dl = torch.ones(4, device=DEV)
    n0 = B.relay_launch_count()
    cases = [(lambda: B.relay_softmax_xent(z, tg.bfloat16(), loss), "ERR_DTYPE"),
             (lambda: B.relay_softmax_xent(z, tg[:, :7].contiguous(), loss), "ERR_SHAPE"),
             (lambda: B.relay_softmax_xent(z, tg, torch.zeros(5, device=DEV)), "ERR_SHAPE"),
             (lambda: B.relay_softmax_xent(z, tg, loss.double().float().bfloat16()), "ERR_DTYPE"),
             (lambda: B.relay_softmax_xent_grad(z, tg, dl, loss, dz.bfloat16()), "ERR_DTYPE"),
             (lambda: B.relay_softmax_xent_grad(z, tg, dl[:3].contiguous(), loss, dz), "ERR_SHAPE"),
             (lambda: B.relay_softmax_xent_grad(z, tg, dl, loss, z), "ERR_ATTR"),          # output aliases an input
             (lambda: B.relay_softmax_xent(z.view(4, 8, 1), tg, loss), "ERR_RANK")]
    for fn, status in cases:
        with pytest.raises(B.RelayError) as e:
            fn()
        assert e.value.status_name == status, str(e.value)
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((loss == 5.0).all()) and bool((dz == 5.0).all())


def test_full_size_loss_group_sampled_rows():
    """8192 x 8192 bf16 scores and targets (the size the benchmark times); the oracle recomputes sampled rows."""
    t = I.loss_batch(8192, 8192, BF16)
    loss, dz = run_grad(t)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, 1, 255, 256, 8191], rng.integers(0, 8192, 27)]))
    zo, to_, dlo = (I.as_f64(t[k][rows]) for k in ("scores", "targets", "dloss"))
    want_loss, want_dz = oracle.softmax_xent_grad(zo, to_, dlo)
    assert_bf16(loss[rows], want_loss, stored_bf16=False, what="loss"); assert_bf16(dz[rows], want_dz, what="dscores")
    assert bool(torch.isfinite(loss).all()) and bool(torch.isfinite(dz.float()).all())
    # every row of the partial sums to zero (sum_j p_j = 1) up to the bf16 rounding of its 8192 entries
    # (each entry is off by at most half a bf16 step, 2^-9 relative) and the fp32 arithmetic before it
    d = dz.double()
    assert bool((d.sum(dim=1).abs() <= d.abs().sum(dim=1) * (2.0 ** -9 + 1e-5)).all())


# ---- SGD ------------------------------------------------------------------------------------------------
def sgd_case(shapes, dt, gdt, lr, salt=0):
    ps, gs = I.param_set(shapes, dt, gdt, salt)
    dev_p = [Guarded(tuple(p.shape), dt, DEV) for p in ps]
    for g, p in zip(dev_p, ps):
        g.t.copy_(p)
    dev_g = [g.to(DEV) for g in gs]
    g_before = [g.clone() for g in dev_g]
    B.relay_sgd_update([g.t for g in dev_p], dev_g, lr)
    torch.cuda.synchronize()
    code = oracle.F32 if dt == F32 else oracle.BF16
    for k, (p, g) in enumerate(zip(ps, gs)):
        got = dev_p[k].check()
        exact = oracle.sgd_update(I.as_f64(p), I.as_f64(g), lr, oracle.F64)
        if dt == F32:
            assert_f32(got, exact, what=f"param {k}")
        else:
            assert_bf16(got, exact, what=f"param {k}")
            # one rounding from an fp32 value: at most one bf16 step away from the oracle's stored value
            stored = oracle.sgd_update(I.as_f64(p), I.as_f64(g), lr, code)
            assert np.all(np.abs(to_np(got) - stored) <= 2.0 ** (np.floor(np.log2(np.maximum(np.abs(stored), 1e-30))) - 7) * 1.0001)
        assert torch.equal(dev_g[k], g_before[k])              # gradients are inputs


LR = float(np.float32(0.01))


@pytest.mark.parametrize("dt,gdt", [(F32, F32), (BF16, BF16), (BF16, F32)])
def test_sgd_update_mixed_shapes_one_launch(dt, gdt):
    sgd_case([(64, 32), (32,), (5, 3, 3, 7), (1,), (), (8191,), (1024, 1030)], dt, gdt, LR)


def test_sgd_update_more_parameters_than_one_launch_takes_and_empty_tensors():
    n0 = B.relay_launch_count()
    sgd_case([(17,), (0, 4), (256, 40)] + [(33 + i,) for i in range(9)], BF16, F32, LR, salt=1)
    assert B.relay_launch_count() - n0 == 2                    # 12 parameters: 8 + 4
    sgd_case([(0,)], F32, F32, LR)                               # nothing to launch


def test_sgd_update_zero_rate_keeps_parameters_bit_exact_and_rejections():
    ps, gs = I.param_set([(100, 9)], BF16, BF16)
    p, g = ps[0].to(DEV), gs[0].to(DEV)
    B.relay_sgd_update([p], [g], 0.0)
    torch.cuda.synchronize()
    assert torch.equal(p.cpu(), ps[0])
    n0 = B.relay_launch_count()
    for fn, status in [(lambda: B.relay_sgd_update([p], [g[:50].contiguous()], LR), "ERR_SHAPE"),
                       (lambda: B.relay_sgd_update([p.float()], [g], LR), "ERR_DTYPE"),
                       (lambda: B.relay_sgd_update([p], [p], LR), "ERR_ATTR"),
                       (lambda: B.relay_sgd_update([p, p], [g, g.clone()], LR), "ERR_ATTR"),
                       (lambda: B.relay_sgd_update([p], [g], float("nan")), "ERR_ATTR")]:
        with pytest.raises(B.RelayError) as e:
            fn()
        assert e.value.status_name == status, str(e.value)
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and torch.equal(p.cpu(), ps[0])


def test_full_size_sgd_update_of_three_weight_matrices():
    """The three 4096 x 4096 bf16 weight matrices of the MLP configuration with their gradients, one launch."""
    ps, gs = I.param_set([(4096, 4096)] * 3, BF16, BF16, salt=5)
    dev_p, dev_g = [p.to(DEV) for p in ps], [g.to(DEV) for g in gs]
    n0 = B.relay_launch_count()
    B.relay_sgd_update(dev_p, dev_g, LR)
    torch.cuda.synchronize()
    assert B.relay_launch_count() - n0 == 1
    rng = np.random.default_rng(1)
    for k in range(3):
        idx = np.unique(np.concatenate([[0, 1, 4095, 4096 * 4096 - 1], rng.integers(0, 4096 * 4096, 20000)]))
        got = dev_p[k].view(-1)[torch.from_numpy(idx).to(DEV)]
        want = oracle.sgd_update(I.as_f64(ps[k]).reshape(-1)[idx], I.as_f64(gs[k]).reshape(-1)[idx], LR, oracle.F64)
        assert_bf16(got, want, what=f"w{k}")
